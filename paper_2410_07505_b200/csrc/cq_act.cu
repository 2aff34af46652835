// CrossQuant activation quantizer: absmax pass, scale vectors, quantize pass (sm_100a).
//
// Pass 1 reads X once and produces partial row maxima (one per row and column strip) and partial
// column maxima (one per column and row block) of the 15-bit magnitudes; the scale-vector kernel
// finishes both reductions, so no atomics and no zero-initialisation are needed and the result does
// not depend on scheduling.  Pass 2 re-reads X (from L2 where it still lives there: it walks the
// row blocks in the opposite order), forms s_ij = a_i * b_j in registers and emits codes, the
// dequantized matrix and the number of zero codes.
#include <math.h>

#include <initializer_list>

#include "cq_common.cuh"
#include "cq_host.h"

namespace cq {

// ============================================================================ pass 1: absmax
// Grid: x = column strip (blockDim.x vectors of 8 columns), y = row block of R rows.
// ATOMIC = false: partial maxima to rowpart[T][nstrips] and colpart[nrb][I8*8] (16-bit magnitudes).
// ATOMIC = true : order-independent atomic max on the float bit patterns of t / c (pre-zeroed).
template <bool ATOMIC, int DT>
__global__ void __launch_bounds__(kThreads)
k1_absmax(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8, int R, int nstrips,
          uint16_t* __restrict__ rowpart, uint4* __restrict__ colpart,
          float* __restrict__ t, float* __restrict__ c) {
    __shared__ uint16_t s_row[kThreads / 32][kMaxRowsPerCta];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * R;
    const int rows = static_cast<int>(min(static_cast<int64_t>(R), T - r0));
    const uint4* p = X + r0 * ld8 + v;
    uint4 cm = make_uint4(0, 0, 0, 0);

    for (int r = 0; r < rows; r += 4) {
        uint4 w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            w[u] = make_uint4(0, 0, 0, 0);
            if (active && r + u < rows) w[u] = ld_nc(p + u * ld8);
        }
        p += 4 * ld8;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            uint4 m = w[u];
            m.x &= 0x7FFF7FFFu; m.y &= 0x7FFF7FFFu; m.z &= 0x7FFF7FFFu; m.w &= 0x7FFF7FFFu;
            cm.x = max_u16x2(cm.x, m.x); cm.y = max_u16x2(cm.y, m.y);
            cm.z = max_u16x2(cm.z, m.z); cm.w = max_u16x2(cm.w, m.w);
            uint32_t mm = max_u16x2(max_u16x2(m.x, m.y), max_u16x2(m.z, m.w));
            uint32_t m16 = max(mm & 0xFFFFu, mm >> 16);
            uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, m16);
            if (lane == 0 && r + u < rows) s_row[warp][r + u] = static_cast<uint16_t>(wm);
        }
    }

    if (active) {
        if constexpr (ATOMIC) {
            if (c != nullptr) {
                uint32_t words[4] = {cm.x, cm.y, cm.z, cm.w};
                unsigned int* cu = reinterpret_cast<unsigned int*>(c) + static_cast<int64_t>(v) * 8;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint32_t lo = words[k] & 0xFFFFu, hi = words[k] >> 16;
                    if (lo) atomicMax(cu + 2 * k, __float_as_uint(cvt16<DT>(static_cast<uint16_t>(lo))));
                    if (hi) atomicMax(cu + 2 * k + 1, __float_as_uint(cvt16<DT>(static_cast<uint16_t>(hi))));
                }
            }
        } else {
            colpart[static_cast<int64_t>(blockIdx.y) * I8 + v] = cm;
        }
    }
    __syncthreads();
    const int nwarps = (blockDim.x + 31) >> 5;
    for (int k = tid; k < rows; k += blockDim.x) {
        uint32_t m = 0;
        for (int wdx = 0; wdx < nwarps; ++wdx) m = max(m, static_cast<uint32_t>(s_row[wdx][k]));
        if constexpr (ATOMIC) {
            if (t != nullptr && m)
                atomicMax(reinterpret_cast<unsigned int*>(t) + r0 + k,
                          __float_as_uint(cvt16<DT>(static_cast<uint16_t>(m))));
        } else {
            rowpart[(r0 + k) * nstrips + blockIdx.x] = static_cast<uint16_t>(m);
        }
    }
}

// General shapes / alignments: one column per thread, scalar loads, atomic combine (t, c pre-zeroed).
template <int DT>
__global__ void __launch_bounds__(kThreads)
g1_absmax(const uint16_t* __restrict__ X, int64_t T, int64_t I, int64_t ld, int R,
          float* __restrict__ t, float* __restrict__ c) {
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const bool active = j < I;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * R;
    const int64_t r1 = min(T, r0 + R);
    uint32_t cm = 0;
    for (int64_t r = r0; r < r1; ++r) {
        uint32_t m = active ? (X[r * ld + j] & 0x7FFFu) : 0u;
        cm = max(cm, m);
        uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, m);
        if ((threadIdx.x & 31) == 0 && t != nullptr && wm)
            atomicMax(reinterpret_cast<unsigned int*>(t) + r, __float_as_uint(cvt16<DT>(static_cast<uint16_t>(wm))));
    }
    if (active && c != nullptr && cm)
        atomicMax(reinterpret_cast<unsigned int*>(c) + j, __float_as_uint(cvt16<DT>(static_cast<uint16_t>(cm))));
}

// ============================================================================ scale vectors
// One thread per row (first T threads) or per column (next I threads).  Finishes the reductions of
// pass 1 (from_partials) or takes t, c as given, then
//   a_i = fl32(pow(t_i, alpha) / qmax), b_j = fl32(pow(c_j, 1 - alpha)) in fp64, with alpha in {0, 1}
//   special-cased so that they reduce exactly to per-column / per-token quantization,
// plus the reciprocals the quantize pass uses for its candidate codes.
template <int DT>
__global__ void __launch_bounds__(kThreads)
k2_scales(int64_t T, int64_t I, int nstrips, int nrb, int64_t colpart_ld,
          const uint16_t* __restrict__ rowpart, const uint16_t* __restrict__ colpart,
          const float* __restrict__ t_in, const float* __restrict__ c_in,
          double alpha, int qmax,
          float* __restrict__ t_out, float* __restrict__ c_out,
          float* __restrict__ a, float* __restrict__ b, float* __restrict__ ra, float* __restrict__ rb,
          unsigned long long* __restrict__ zero_count) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx == 0 && zero_count != nullptr) *zero_count = 0ull;
    const float qmaxf = static_cast<float>(qmax);
    if (idx < T) {
        float ti;
        if (rowpart != nullptr) {
            uint32_t m = 0;
            for (int s = 0; s < nstrips; ++s) m = max(m, static_cast<uint32_t>(rowpart[idx * nstrips + s]));
            ti = cvt16<DT>(static_cast<uint16_t>(m));
        } else {
            ti = t_in[idx];
        }
        if (t_out != nullptr) t_out[idx] = ti;
        float ai;
        if (alpha == 1.0) ai = __fdiv_rn(ti, qmaxf);
        else if (alpha == 0.0) ai = 1.0f;
        else ai = static_cast<float>(pow(static_cast<double>(ti), alpha) / static_cast<double>(qmax));
        a[idx] = ai;
        ra[idx] = __fdiv_rn(1.0f, ai);
    } else if (idx - T < I) {
        const int64_t j = idx - T;
        float cj;
        if (colpart != nullptr) {
            uint32_t m = 0;
            for (int rbk = 0; rbk < nrb; ++rbk) m = max(m, static_cast<uint32_t>(colpart[rbk * colpart_ld + j]));
            cj = cvt16<DT>(static_cast<uint16_t>(m));
        } else {
            cj = c_in[j];
        }
        if (c_out != nullptr) c_out[j] = cj;
        float bj;
        if (alpha == 1.0) bj = 1.0f;
        else if (alpha == 0.0) bj = __fdiv_rn(cj, qmaxf);
        else bj = static_cast<float>(pow(static_cast<double>(cj), 1.0 - alpha));
        b[j] = bj;
        rb[j] = __fdiv_rn(1.0f, bj);
    }
}

// ============================================================================ pass 2: quantize
// Same tiling as pass 1; row blocks are visited in descending order.  Per thread and row: one
// 128-bit load of 8 elements, s = a_i b_j, candidate code through the reciprocal product, exact
// IEEE division only for the rare elements the residual test cannot decide.
// DEQ: 0 none, 1 same 16-bit type as X, 2 fp32.
template <int DT, int BITS, int DEQ, bool CODES, bool COUNT>
__global__ void __launch_bounds__(kThreads, 3)
k3_quantize(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8, int R,
            const float* __restrict__ a, const float* __restrict__ ra,
            const float* __restrict__ b, const float* __restrict__ rb,
            void* __restrict__ codes, void* __restrict__ deq,
            unsigned long long* __restrict__ zero_count) {
    constexpr float qmaxf = static_cast<float>((1 << (BITS - 1)) - 1);
    const int tid = threadIdx.x;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const int64_t rblk = static_cast<int64_t>(gridDim.y - 1 - blockIdx.y);
    const int64_t r0 = rblk * R;
    const int rows = static_cast<int>(min(static_cast<int64_t>(R), T - r0));
    unsigned int zeros = 0;

    if (active) {
        float bj[8], rbj[8];
        {
            const float4* bp = reinterpret_cast<const float4*>(b) + static_cast<int64_t>(v) * 2;
            const float4* rp = reinterpret_cast<const float4*>(rb) + static_cast<int64_t>(v) * 2;
            float4 b0 = __ldg(bp), b1 = __ldg(bp + 1), q0 = __ldg(rp), q1 = __ldg(rp + 1);
            bj[0] = b0.x; bj[1] = b0.y; bj[2] = b0.z; bj[3] = b0.w;
            bj[4] = b1.x; bj[5] = b1.y; bj[6] = b1.z; bj[7] = b1.w;
            rbj[0] = q0.x; rbj[1] = q0.y; rbj[2] = q0.z; rbj[3] = q0.w;
            rbj[4] = q1.x; rbj[5] = q1.y; rbj[6] = q1.z; rbj[7] = q1.w;
        }
        const uint4* p = X + r0 * ld8 + v;
        for (int r = 0; r < rows; r += 4) {
            uint4 w[4];
            float ar[4], rar[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (r + u < rows) {
                    w[u] = ld_stream(p + u * ld8);
                    ar[u] = __ldg(a + r0 + r + u);
                    rar[u] = __ldg(ra + r0 + r + u);
                }
            }
            p += 4 * ld8;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (r + u >= rows) break;
                const int64_t row = r0 + r + u;
                const uint32_t words[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
                float x[8], y[8];
                unsigned int bad = 0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float2 f = unpack16x2<DT>(words[k]);
                    x[2 * k] = f.x; x[2 * k + 1] = f.y;
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    bool ok;
                    y[e] = quant_candidate(x[e], __fmul_rn(ar[u], bj[e]), __fmul_rn(rar[u], rbj[e]), qmaxf, ok);
                    bad |= (ok ? 0u : 1u) << e;
                }
                if (bad) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if ((bad >> e) & 1u) y[e] = quant_exact(x[e], __fmul_rn(ar[u], bj[e]), qmaxf);
                }
                const int64_t vec = row * I8 + v;
                if constexpr (BITS == 8) {
                    uint32_t c0 = pack_int8x4(y[0], y[1], y[2], y[3]);
                    uint32_t c1 = pack_int8x4(y[4], y[5], y[6], y[7]);
                    if constexpr (COUNT) zeros += zero_bytes(c0) + zero_bytes(c1);
                    if constexpr (CODES) st_stream(reinterpret_cast<uint2*>(codes) + vec, make_uint2(c0, c1));
                } else {
                    uint32_t c0 = pack_int4x8(y);
                    if constexpr (COUNT) zeros += zero_nibbles(c0);
                    if constexpr (CODES) st_stream(reinterpret_cast<uint32_t*>(codes) + vec, c0);
                }
                if constexpr (DEQ != 0) {
                    float d[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) d[e] = __fmul_rn(code_as_float(y[e]), __fmul_rn(ar[u], bj[e]));
                    if constexpr (DEQ == 1) {
                        uint4 o;
                        o.x = pack16x2<DT>(d[0], d[1]); o.y = pack16x2<DT>(d[2], d[3]);
                        o.z = pack16x2<DT>(d[4], d[5]); o.w = pack16x2<DT>(d[6], d[7]);
                        st_stream(reinterpret_cast<uint4*>(deq) + vec, o);
                    } else {
                        float4* o = reinterpret_cast<float4*>(deq) + vec * 2;
                        st_stream(o, make_float4(d[0], d[1], d[2], d[3]));
                        st_stream(o + 1, make_float4(d[4], d[5], d[6], d[7]));
                    }
                }
            }
        }
    }
    if constexpr (COUNT) cta_count_add(zeros, zero_count);
}

// General shapes / alignments: one thread per pair of adjacent columns.
template <int DT>
__global__ void __launch_bounds__(kThreads)
g3_quantize(const uint16_t* __restrict__ X, int64_t T, int64_t I, int64_t ld, int bits,
            const float* __restrict__ a, const float* __restrict__ b,
            void* __restrict__ codes, void* __restrict__ deq, int deq_dt,
            unsigned long long* __restrict__ zero_count) {
    const float qmaxf = static_cast<float>((1 << (bits - 1)) - 1);
    const int64_t pairs = (I + 1) / 2;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    unsigned int zeros = 0;
    if (idx < T * pairs) {
        const int64_t i = idx / pairs, j0 = (idx % pairs) * 2;
        int q[2] = {0, 0};
        for (int e = 0; e < 2; ++e) {
            const int64_t j = j0 + e;
            if (j >= I) break;
            float x = cvt16<DT>(X[i * ld + j]);
            float s = __fmul_rn(a[i], b[j]);
            float y = quant_exact(x, s, qmaxf);
            q[e] = code_as_int(y);
            zeros += (q[e] == 0);
            float d = __fmul_rn(static_cast<float>(q[e]), s);
            if (deq != nullptr) {
                if (deq_dt == CQ_F32) reinterpret_cast<float*>(deq)[i * I + j] = d;
                else reinterpret_cast<uint16_t*>(deq)[i * I + j] = pack16<DT>(d);
            }
            if (codes != nullptr && bits == 8) reinterpret_cast<int8_t*>(codes)[i * I + j] = static_cast<int8_t>(q[e]);
        }
        if (codes != nullptr && bits == 4)
            reinterpret_cast<uint8_t*>(codes)[i * (I / 2) + j0 / 2] =
                static_cast<uint8_t>((q[0] & 0xF) | ((q[1] & 0xF) << 4));
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
}

// ============================================================================ host side
static int g_tune_k1_rows = 0;
static int g_tune_k3_rows = 0;
static cudaEvent_t g_ev_before = nullptr, g_ev_after = nullptr;

static inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

Plan make_plan(int64_t T, int64_t I) {
    Plan p{};
    p.I8 = static_cast<int>((I + 7) / 8);
    if (p.I8 <= kThreads) {
        p.W = p.I8 > 0 ? round_up(p.I8, 32) : 32;
    } else {
        int64_t best = -1;
        for (int w = kThreads; w >= 128; w -= 32) {
            int64_t cost = static_cast<int64_t>((p.I8 + w - 1) / w) * w;
            if (best < 0 || cost < best) { best = cost; p.W = w; }
        }
    }
    p.nstrips = p.I8 > 0 ? (p.I8 + p.W - 1) / p.W : 1;
    // pass 1: about one resident wave (8 CTAs of 256 threads per SM, 148 SMs)
    int r1 = g_tune_k1_rows > 0 ? g_tune_k1_rows
                                : static_cast<int>((T * p.nstrips + 1183) / 1184);
    r1 = round_up(r1 < 16 ? 16 : r1, 4);
    p.R1 = r1 > kMaxRowsPerCta ? kMaxRowsPerCta : r1;
    p.nrb1 = static_cast<int>(T > 0 ? (T + p.R1 - 1) / p.R1 : 1);
    int r3 = g_tune_k3_rows > 0 ? g_tune_k3_rows : 16;
    r3 = round_up(r3, 4);
    p.R3 = r3 > 4096 ? 4096 : r3;
    p.nrb3 = static_cast<int>(T > 0 ? (T + p.R3 - 1) / p.R3 : 1);

    auto carve = [&](size_t bytes) { size_t off = p.total; p.total += (bytes + 255) / 256 * 256; return off; };
    p.total = 0;
    p.off_t = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_c = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    p.off_a = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_b = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    p.off_ra = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_rb = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    // sized for the finest pass-1 tiling the tuning knob can select (16 rows per CTA)
    size_t max_nrb = static_cast<size_t>((T + 15) / 16 + 1);
    p.off_rowpart = carve(sizeof(uint16_t) * static_cast<size_t>(T) * p.nstrips);
    p.off_colpart = carve(sizeof(uint16_t) * max_nrb * static_cast<size_t>(p.I8) * 8);
    return p;
}

static bool aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }

int check_matrix(const void* X, int dtype, int64_t T, int64_t I, int64_t ld) {
    if (T < 0 || I < 0 || ld < I) return CQ_ERR_SHAPE;
    if (T > (int64_t(1) << 31) - 1 - kMaxRowsPerCta || I > (int64_t(1) << 31) - 64) return CQ_ERR_SHAPE;
    if (dtype != CQ_F16 && dtype != CQ_BF16) return CQ_ERR_DTYPE;
    if (T > 0 && I > 0) {
        if (X == nullptr) return CQ_ERR_NULL;
        if (!aligned(X, 2)) return CQ_ERR_ALIGN;
    }
    return CQ_OK;
}

static bool fast_input(const void* X, int64_t I, int64_t ld) {
    return aligned(X, 16) && (I % 8 == 0) && (ld % 8 == 0);
}

static int launch_status() { return cudaGetLastError() == cudaSuccess ? CQ_OK : CQ_ERR_CUDA; }

// pass 1 with atomics into pre-zeroed t / c (either may be null)
static int absmax_atomic(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t, float* c,
                         cudaStream_t st) {
    if (t != nullptr && cudaMemsetAsync(t, 0, sizeof(float) * T, st) != cudaSuccess) return CQ_ERR_CUDA;
    if (c != nullptr && cudaMemsetAsync(c, 0, sizeof(float) * I, st) != cudaSuccess) return CQ_ERR_CUDA;
    if (T == 0 || I == 0) return CQ_OK;
    Plan p = make_plan(T, I);
    if (fast_input(X, I, ld)) {
        dim3 grid(p.nstrips, p.nrb1);
        if (dtype == CQ_F16)
            k1_absmax<true, CQ_F16><<<grid, p.W, 0, st>>>(static_cast<const uint4*>(X), T, p.I8, ld / 8, p.R1,
                                                            p.nstrips, nullptr, nullptr, t, c);
        else
            k1_absmax<true, CQ_BF16><<<grid, p.W, 0, st>>>(static_cast<const uint4*>(X), T, p.I8, ld / 8, p.R1,
                                                             p.nstrips, nullptr, nullptr, t, c);
    } else {
        const int R = 64;
        dim3 grid(static_cast<unsigned>((I + kThreads - 1) / kThreads), static_cast<unsigned>((T + R - 1) / R));
        if (dtype == CQ_F16)
            g1_absmax<CQ_F16><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, R, t, c);
        else
            g1_absmax<CQ_BF16><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, R, t, c);
    }
    return launch_status();
}

template <int DT, int BITS, int DEQ>
static void launch_k3(bool has_codes, bool has_count, dim3 grid, int W, cudaStream_t st, const uint4* X, int64_t T,
                      int I8, int64_t ld8, int R, const float* a, const float* ra, const float* b, const float* rb,
                      void* codes, void* deq, unsigned long long* zc) {
    if (has_codes) {
        if (has_count) k3_quantize<DT, BITS, DEQ, true, true><<<grid, W, 0, st>>>(X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
        else k3_quantize<DT, BITS, DEQ, true, false><<<grid, W, 0, st>>>(X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
    } else {
        if (has_count) k3_quantize<DT, BITS, DEQ, false, true><<<grid, W, 0, st>>>(X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
        else k3_quantize<DT, BITS, DEQ, false, false><<<grid, W, 0, st>>>(X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
    }
}

template <int DT, int BITS>
static void launch_k3_deq(int deq_mode, bool has_codes, bool has_count, dim3 grid, int W, cudaStream_t st,
                          const uint4* X, int64_t T, int I8, int64_t ld8, int R, const float* a, const float* ra,
                          const float* b, const float* rb, void* codes, void* deq, unsigned long long* zc) {
    if (deq_mode == 0) launch_k3<DT, BITS, 0>(has_codes, has_count, grid, W, st, X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
    else if (deq_mode == 1) launch_k3<DT, BITS, 1>(has_codes, has_count, grid, W, st, X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
    else launch_k3<DT, BITS, 2>(has_codes, has_count, grid, W, st, X, T, I8, ld8, R, a, ra, b, rb, codes, deq, zc);
}

// Shared body of cq_quantize_act and cq_kernel_count_x.  t_given/c_given: skip pass 1.
int quantize_act_impl(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                      const float* t_given, const float* c_given,
                      float* t, float* c, float* row_scale, float* col_scale,
                      void* codes, void* deq, int deq_dtype, unsigned long long* zero_count,
                      void* workspace, size_t ws_bytes, cudaStream_t st) {
    int rc = check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (!(alpha >= 0.0 && alpha <= 1.0)) return CQ_ERR_ALPHA;
    if (deq != nullptr && deq_dtype != dtype && deq_dtype != CQ_F32) return CQ_ERR_DTYPE;
    if (bits == 4 && (I % 2) != 0) return CQ_ERR_ALIGN;
    if (deq != nullptr && !aligned(deq, deq_dtype == CQ_F32 ? 4 : 2)) return CQ_ERR_ALIGN;
    if (zero_count != nullptr && !aligned(zero_count, 8)) return CQ_ERR_ALIGN;
    for (const float* f : {static_cast<const float*>(t), static_cast<const float*>(c),
                           static_cast<const float*>(row_scale), static_cast<const float*>(col_scale),
                           t_given, c_given})
        if (f != nullptr && !aligned(f, 4)) return CQ_ERR_ALIGN;
    if (T == 0 || I == 0) {
        if (zero_count != nullptr && cudaMemsetAsync(zero_count, 0, sizeof(unsigned long long), st) != cudaSuccess)
            return CQ_ERR_CUDA;
        return CQ_OK;
    }
    Plan p = make_plan(T, I);
    if (workspace == nullptr || !aligned(workspace, 256) || ws_bytes < p.total) return CQ_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    // Vectors the caller did not ask for live in the workspace.  The fast quantize pass reads b / rb
    // as whole float4 pairs, so col_scale must be 16-byte aligned to be used in place.
    const bool given = t_given != nullptr && c_given != nullptr;
    float* t_dev = t != nullptr ? t : reinterpret_cast<float*>(ws + p.off_t);
    float* c_dev = c != nullptr ? c : reinterpret_cast<float*>(ws + p.off_c);
    float* a_dev = row_scale != nullptr ? row_scale : reinterpret_cast<float*>(ws + p.off_a);
    const bool b_in_place = col_scale != nullptr && aligned(col_scale, 16);
    float* b_dev = b_in_place ? col_scale : reinterpret_cast<float*>(ws + p.off_b);
    float* ra_dev = reinterpret_cast<float*>(ws + p.off_ra);
    float* rb_dev = reinterpret_cast<float*>(ws + p.off_rb);
    uint16_t* rowpart = reinterpret_cast<uint16_t*>(ws + p.off_rowpart);
    uint16_t* colpart = reinterpret_cast<uint16_t*>(ws + p.off_colpart);
    const int qmax = (1 << (bits - 1)) - 1;

    const bool fast_in = fast_input(X, I, ld);
    const bool fast_out = (codes == nullptr || aligned(codes, bits == 8 ? 8 : 4)) &&
                          (deq == nullptr || aligned(deq, 16));
    const int64_t n2 = T + I;
    const unsigned k2_blocks = static_cast<unsigned>((n2 + kThreads - 1) / kThreads);

    // ---- pass 1 + scale vectors
    if (given) {
        if (dtype == CQ_F16)
            k2_scales<CQ_F16><<<k2_blocks, kThreads, 0, st>>>(T, I, 0, 0, 0, nullptr, nullptr, t_given, c_given, alpha,
                                                              qmax, t, c, a_dev, b_dev, ra_dev, rb_dev, zero_count);
        else
            k2_scales<CQ_BF16><<<k2_blocks, kThreads, 0, st>>>(T, I, 0, 0, 0, nullptr, nullptr, t_given, c_given, alpha,
                                                               qmax, t, c, a_dev, b_dev, ra_dev, rb_dev, zero_count);
    } else if (fast_in) {
        dim3 grid(p.nstrips, p.nrb1);
        const int64_t cp_ld = static_cast<int64_t>(p.I8) * 8;
        if (dtype == CQ_F16) {
            k1_absmax<false, CQ_F16><<<grid, p.W, 0, st>>>(static_cast<const uint4*>(X), T, p.I8, ld / 8, p.R1, p.nstrips,
                                                             rowpart, reinterpret_cast<uint4*>(colpart), nullptr, nullptr);
            k2_scales<CQ_F16><<<k2_blocks, kThreads, 0, st>>>(T, I, p.nstrips, p.nrb1, cp_ld, rowpart, colpart, nullptr,
                                                              nullptr, alpha, qmax, t_dev, c_dev, a_dev, b_dev, ra_dev,
                                                              rb_dev, zero_count);
        } else {
            k1_absmax<false, CQ_BF16><<<grid, p.W, 0, st>>>(static_cast<const uint4*>(X), T, p.I8, ld / 8, p.R1, p.nstrips,
                                                              rowpart, reinterpret_cast<uint4*>(colpart), nullptr, nullptr);
            k2_scales<CQ_BF16><<<k2_blocks, kThreads, 0, st>>>(T, I, p.nstrips, p.nrb1, cp_ld, rowpart, colpart, nullptr,
                                                               nullptr, alpha, qmax, t_dev, c_dev, a_dev, b_dev, ra_dev,
                                                               rb_dev, zero_count);
        }
    } else {
        rc = absmax_atomic(X, dtype, T, I, ld, t_dev, c_dev, st);
        if (rc != CQ_OK) return rc;
        if (dtype == CQ_F16)
            k2_scales<CQ_F16><<<k2_blocks, kThreads, 0, st>>>(T, I, 0, 0, 0, nullptr, nullptr, t_dev, c_dev, alpha, qmax,
                                                              nullptr, nullptr, a_dev, b_dev, ra_dev, rb_dev, zero_count);
        else
            k2_scales<CQ_BF16><<<k2_blocks, kThreads, 0, st>>>(T, I, 0, 0, 0, nullptr, nullptr, t_dev, c_dev, alpha, qmax,
                                                               nullptr, nullptr, a_dev, b_dev, ra_dev, rb_dev, zero_count);
    }
    if ((rc = launch_status()) != CQ_OK) return rc;

    // ---- pass 2
    const bool any_out = codes != nullptr || deq != nullptr || zero_count != nullptr;
    if (any_out) {
        const bool timed = g_ev_before != nullptr && g_ev_after != nullptr;
        if (timed) cudaEventRecord(g_ev_before, st);
        if (fast_in && fast_out) {
            dim3 grid(p.nstrips, p.nrb3);
            const int deq_mode = deq == nullptr ? 0 : (deq_dtype == CQ_F32 ? 2 : 1);
            const uint4* Xv = static_cast<const uint4*>(X);
            const bool hc = codes != nullptr, hz = zero_count != nullptr;
            if (dtype == CQ_F16) {
                if (bits == 8) launch_k3_deq<CQ_F16, 8>(deq_mode, hc, hz, grid, p.W, st, Xv, T, p.I8, ld / 8, p.R3, a_dev, ra_dev, b_dev, rb_dev, codes, deq, zero_count);
                else launch_k3_deq<CQ_F16, 4>(deq_mode, hc, hz, grid, p.W, st, Xv, T, p.I8, ld / 8, p.R3, a_dev, ra_dev, b_dev, rb_dev, codes, deq, zero_count);
            } else {
                if (bits == 8) launch_k3_deq<CQ_BF16, 8>(deq_mode, hc, hz, grid, p.W, st, Xv, T, p.I8, ld / 8, p.R3, a_dev, ra_dev, b_dev, rb_dev, codes, deq, zero_count);
                else launch_k3_deq<CQ_BF16, 4>(deq_mode, hc, hz, grid, p.W, st, Xv, T, p.I8, ld / 8, p.R3, a_dev, ra_dev, b_dev, rb_dev, codes, deq, zero_count);
            }
        } else {
            const int64_t n = T * ((I + 1) / 2);
            const unsigned blocks = static_cast<unsigned>((n + kThreads - 1) / kThreads);
            if (dtype == CQ_F16)
                g3_quantize<CQ_F16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, bits, a_dev, b_dev,
                                                                 codes, deq, deq_dtype, zero_count);
            else
                g3_quantize<CQ_BF16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, bits, a_dev, b_dev,
                                                                  codes, deq, deq_dtype, zero_count);
        }
        if (timed) cudaEventRecord(g_ev_after, st);
        if ((rc = launch_status()) != CQ_OK) return rc;
    }
    if (col_scale != nullptr && !b_in_place) {
        if (cudaMemcpyAsync(col_scale, b_dev, sizeof(float) * I, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return CQ_ERR_CUDA;
    }
    return CQ_OK;
}

}  // namespace cq

// ============================================================================ C ABI
extern "C" {

int cq_version(void) { return 100; }

const char* cq_status_string(int status) {
    switch (status) {
        case CQ_OK: return "ok";
        case CQ_ERR_NULL: return "a required pointer is NULL";
        case CQ_ERR_SHAPE: return "bad shape (negative size, ld < columns, or too large)";
        case CQ_ERR_DTYPE: return "dtype not valid for this argument";
        case CQ_ERR_BITS: return "bits must be 4 or 8";
        case CQ_ERR_ALPHA: return "alpha must lie in [0, 1]";
        case CQ_ERR_ALIGN: return "misaligned pointer, or odd number of columns with INT4";
        case CQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CQ_ERR_CUDA: return "CUDA runtime error at launch";
        default: return "unknown status";
    }
}

int cq_set_tuning(const char* key, int value) {
    if (key == nullptr) return CQ_ERR_NULL;
    if (value > cq::kMaxRowsPerCta * 32) return CQ_ERR_SHAPE;
    const char* k1 = "k1_rows"; const char* k3 = "k3_rows";
    auto eq = [](const char* x, const char* y) { while (*x && *x == *y) { ++x; ++y; } return *x == *y; };
    if (eq(key, k1)) { cq::g_tune_k1_rows = value > 0 ? value : 0; return CQ_OK; }
    if (eq(key, k3)) { cq::g_tune_k3_rows = value > 0 ? value : 0; return CQ_OK; }
    return CQ_ERR_SHAPE;
}

int cq_set_timing_events(void* before_quantize_pass, void* after_quantize_pass) {
    cq::g_ev_before = static_cast<cudaEvent_t>(before_quantize_pass);
    cq::g_ev_after = static_cast<cudaEvent_t>(after_quantize_pass);
    return CQ_OK;
}

size_t cq_workspace_bytes(int64_t T, int64_t I) {
    if (T < 0 || I < 0) return 0;
    return cq::make_plan(T, I).total + 256;
}

int cq_absmax_rows(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t, void* stream) {
    int rc = cq::check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (t == nullptr && T > 0) return CQ_ERR_NULL;
    return cq::absmax_atomic(X, dtype, T, I, ld, t, nullptr, static_cast<cudaStream_t>(stream));
}

int cq_absmax_cols(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* c, void* stream) {
    int rc = cq::check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (c == nullptr && I > 0) return CQ_ERR_NULL;
    return cq::absmax_atomic(X, dtype, T, I, ld, nullptr, c, static_cast<cudaStream_t>(stream));
}

int cq_absmax_rows_cols(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t, float* c, void* stream) {
    int rc = cq::check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if ((t == nullptr && T > 0) || (c == nullptr && I > 0)) return CQ_ERR_NULL;
    return cq::absmax_atomic(X, dtype, T, I, ld, t, c, static_cast<cudaStream_t>(stream));
}

int cq_quantize_act(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                    float* t, float* c, float* row_scale, float* col_scale,
                    void* codes, void* deq, int deq_dtype, unsigned long long* zero_count,
                    void* workspace, size_t workspace_bytes, void* stream) {
    return cq::quantize_act_impl(X, dtype, T, I, ld, alpha, bits, nullptr, nullptr, t, c, row_scale, col_scale,
                                 codes, deq, deq_dtype, zero_count, workspace, workspace_bytes,
                                 static_cast<cudaStream_t>(stream));
}

int cq_kernel_count_x(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                      const float* t, const float* c, unsigned long long* count,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (count == nullptr) return CQ_ERR_NULL;
    if (T > 0 && I > 0 && (t == nullptr || c == nullptr)) return CQ_ERR_NULL;
    return cq::quantize_act_impl(X, dtype, T, I, ld, alpha, bits, t, c, nullptr, nullptr, nullptr, nullptr,
                                 nullptr, nullptr, dtype, count, workspace, workspace_bytes,
                                 static_cast<cudaStream_t>(stream));
}

size_t cq_host_scratch_bytes(int64_t T, int64_t I, int bits, int want_codes, int want_deq, int deq_dtype) {
    if (T < 0 || I < 0 || (bits != 4 && bits != 8)) return 0;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    size_t n = static_cast<size_t>(T) * static_cast<size_t>(I);
    size_t total = up(n * 2) + up(cq_workspace_bytes(T, I)) + 2 * up(sizeof(float) * T) + 2 * up(sizeof(float) * I) + 256;
    if (want_codes) total += up(bits == 8 ? n : n / 2);
    if (want_deq) total += up(n * (deq_dtype == CQ_F32 ? 4 : 2));
    return total + 256;
}

int cq_quantize_act_host(const void* X_host, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                         float* t_host, float* c_host, float* row_scale_host, float* col_scale_host,
                         void* codes_host, void* deq_host, int deq_dtype, unsigned long long* zero_count_host,
                         void* device_scratch, size_t scratch_bytes, void* stream) {
    int rc = cq::check_matrix(X_host, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (!(alpha >= 0.0 && alpha <= 1.0)) return CQ_ERR_ALPHA;
    if (deq_host != nullptr && deq_dtype != dtype && deq_dtype != CQ_F32) return CQ_ERR_DTYPE;
    if (bits == 4 && (I % 2) != 0) return CQ_ERR_ALIGN;
    const size_t need = cq_host_scratch_bytes(T, I, bits, codes_host != nullptr, deq_host != nullptr, deq_dtype);
    if (device_scratch == nullptr || (reinterpret_cast<uintptr_t>(device_scratch) % 256) != 0 || scratch_bytes < need)
        return CQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t n = static_cast<size_t>(T) * static_cast<size_t>(I);
    char* base = static_cast<char*>(device_scratch);
    size_t off = 0;
    auto carve = [&](size_t bytes) { char* q = base + off; off += up(bytes); return q; };
    void* Xd = carve(n * 2);
    const size_t ws_bytes = cq_workspace_bytes(T, I);
    void* ws = carve(ws_bytes);
    float* td = reinterpret_cast<float*>(carve(sizeof(float) * T));
    float* ad = reinterpret_cast<float*>(carve(sizeof(float) * T));
    float* cd = reinterpret_cast<float*>(carve(sizeof(float) * I));
    float* bd = reinterpret_cast<float*>(carve(sizeof(float) * I));
    unsigned long long* zd = reinterpret_cast<unsigned long long*>(carve(256));
    const size_t code_bytes = bits == 8 ? n : n / 2;
    const size_t deq_bytes = n * (deq_dtype == CQ_F32 ? 4 : 2);
    void* codes_d = codes_host != nullptr ? carve(code_bytes) : nullptr;
    void* deq_d = deq_host != nullptr ? carve(deq_bytes) : nullptr;

    if (n > 0) {
        cudaError_t e = (ld == I)
            ? cudaMemcpyAsync(Xd, X_host, n * 2, cudaMemcpyHostToDevice, st)
            : cudaMemcpy2DAsync(Xd, static_cast<size_t>(I) * 2, X_host, static_cast<size_t>(ld) * 2,
                                static_cast<size_t>(I) * 2, static_cast<size_t>(T), cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return CQ_ERR_CUDA;
    }
    rc = cq::quantize_act_impl(Xd, dtype, T, I, I, alpha, bits, nullptr, nullptr, td, cd, ad, bd, codes_d, deq_d,
                               deq_dtype, zd, ws, ws_bytes, st);
    if (rc != CQ_OK) return rc;
    auto back = [&](void* dst, const void* src, size_t bytes) {
        if (dst == nullptr || bytes == 0) return true;
        return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };
    bool ok = true;
    if (n > 0) {
        ok = ok && back(t_host, td, sizeof(float) * T) && back(c_host, cd, sizeof(float) * I);
        ok = ok && back(row_scale_host, ad, sizeof(float) * T) && back(col_scale_host, bd, sizeof(float) * I);
        ok = ok && back(codes_host, codes_d, code_bytes) && back(deq_host, deq_d, deq_bytes);
    }
    ok = ok && back(zero_count_host, zd, sizeof(unsigned long long));
    return ok ? CQ_OK : CQ_ERR_CUDA;
}

}  // extern "C"
