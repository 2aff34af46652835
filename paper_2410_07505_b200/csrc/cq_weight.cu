// Per-channel weight quantizer (Eq. 2), dequantization from stored codes and the zero-code count
// (Definition 1) for sm_100a.
#include "cq_common.cuh"
#include "cq_host.h"

namespace cq {

constexpr int kMaxSmemRowBytes = 221184;   // 216 KB of the 227 KB a CTA may use: C <= 110,592

// ============================================================================ weight rows
// One CTA per stored row.  The row is read from HBM once into shared memory while its absolute
// maximum is reduced; each thread later quantizes exactly the vectors it staged itself.
// BULK (long rows, of which only a few CTAs fit on an SM): the row arrives through one asynchronous bulk
// copy issued by thread 0, so the whole row is in flight at once instead of four vectors per thread.
__device__ unsigned int g_weight_stage_fault = 0;   // set if the bounded wait on a row copy ever gave up

#ifndef CQ_K4_BULK_MIN_BYTES
#define CQ_K4_BULK_MIN_BYTES (32 * 1024)
#endif
#ifndef CQ_K4_MIN_CTAS
#define CQ_K4_MIN_CTAS 6
#endif

template <int DT, int BITS, int DEQ, bool CODES, bool BULK>
__global__ void __launch_bounds__(kThreads, BULK ? 1 : CQ_K4_MIN_CTAS)
k4_weight_rows(const uint4* __restrict__ W, int C8, int64_t ld8,
               void* __restrict__ codes, float* __restrict__ scale, void* __restrict__ deq,
               unsigned long long* __restrict__ zero_count) {
    extern __shared__ uint4 s_vec[];
    __shared__ uint32_t s_max[kThreads / 32];
    constexpr float qmaxf = static_cast<float>((1 << (BITS - 1)) - 1);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = blockIdx.x;
    const uint4* p = W + row * ld8;

    uint32_t mm = 0;
    if constexpr (BULK) {
        __shared__ uint64_t s_bar;
        if (tid == 0) {
            mbar_init(&s_bar, 1);
            mbar_init_fence();
        }
        __syncthreads();
        if (tid == 0) {
            mbar_expect_tx(&s_bar, static_cast<uint32_t>(C8) * 16u);
            bulk_load(s_vec, p, static_cast<uint32_t>(C8) * 16u, &s_bar);
        }
        if (!mbar_wait(&s_bar, 0u)) atomicExch(&g_weight_stage_fault, 1u);
#pragma unroll 4
        for (int v = tid; v < C8; v += kThreads) {
            const uint4 w = s_vec[v];
            mm = max_u16x2(mm, max_u16x2(max_u16x2(w.x & 0x7FFF7FFFu, w.y & 0x7FFF7FFFu),
                                         max_u16x2(w.z & 0x7FFF7FFFu, w.w & 0x7FFF7FFFu)));
        }
    } else {
#pragma unroll 4
        for (int v = tid; v < C8; v += kThreads) {
            uint4 w = ld_stream(p + v);
            s_vec[v] = w;
            mm = max_u16x2(mm, max_u16x2(max_u16x2(w.x & 0x7FFF7FFFu, w.y & 0x7FFF7FFFu),
                                         max_u16x2(w.z & 0x7FFF7FFFu, w.w & 0x7FFF7FFFu)));
        }
    }
    uint32_t m16 = __reduce_max_sync(0xFFFFFFFFu, max(mm & 0xFFFFu, mm >> 16));
    if (lane == 0) s_max[warp] = m16;
    __syncthreads();
    m16 = 0;
#pragma unroll
    for (int k = 0; k < kThreads / 32; ++k) m16 = max(m16, s_max[k]);
    const float d = __fdiv_rn(cvt16<DT>(static_cast<uint16_t>(m16)), qmaxf);
    const float rd = guarded_rcp(d);
    if (tid == 0 && scale != nullptr) scale[row] = d;

    const float2 d2s = make_float2(d, d), nm2 = make_float2(-kMagic, -kMagic);
    const bool scale_ok = rd == rd;                   // false: d outside [2^-40, 2^40] (NaN marker)
    unsigned int zeros = 0;
    for (int v = tid; v < C8; v += kThreads) {
        const uint4 w = s_vec[v];
        float2 y2[4];
        if (scale_ok) exact_codes_uniform_row8<DT>(w, d, rd, y2);
        else exact_codes_uniform_slow<DT, BITS>(w, d, y2);                // extreme scale: the whole row, never mixed
        const int64_t vec = row * C8 + v;
        if constexpr (BITS == 8) {
            const uint32_t c0 = pack_int8x4(y2[0].x, y2[0].y, y2[1].x, y2[1].y);
            const uint32_t c1 = pack_int8x4(y2[2].x, y2[2].y, y2[3].x, y2[3].y);
            zeros += zero_bytes(c0) + zero_bytes(c1);
            if constexpr (CODES) st_stream(reinterpret_cast<uint2*>(codes) + vec, make_uint2(c0, c1));
        } else {
            const uint32_t c0 = pack_int4x8(y2);
            zeros += zero_nibbles(c0);
            if constexpr (CODES) st_stream(reinterpret_cast<uint32_t*>(codes) + vec, c0);
        }
        if constexpr (DEQ != 0) {
            float2 dq[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) dq[k] = __fmul2_rn(__fadd2_rn(y2[k], nm2), d2s);
            if constexpr (DEQ == 1) {
                uint4 o;
                o.x = pack16x2<DT>(dq[0].x, dq[0].y); o.y = pack16x2<DT>(dq[1].x, dq[1].y);
                o.z = pack16x2<DT>(dq[2].x, dq[2].y); o.w = pack16x2<DT>(dq[3].x, dq[3].y);
                st_stream(reinterpret_cast<uint4*>(deq) + vec, o);
            } else {
                float4* o = reinterpret_cast<float4*>(deq) + vec * 2;
                st_stream(o, make_float4(dq[0].x, dq[0].y, dq[1].x, dq[1].y));
                st_stream(o + 1, make_float4(dq[2].x, dq[2].y, dq[3].x, dq[3].y));
            }
        }
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
}

// General shapes / alignments / very long rows: one CTA per row, scalar accesses, two reads.
template <int DT>
__global__ void __launch_bounds__(kThreads)
g4_weight_rows(const uint16_t* __restrict__ W, int64_t C, int64_t ld, int bits,
               void* __restrict__ codes, float* __restrict__ scale, void* __restrict__ deq, int deq_dt,
               unsigned long long* __restrict__ zero_count) {
    __shared__ uint32_t s_max[kThreads / 32];
    const float qmaxf = static_cast<float>((1 << (bits - 1)) - 1);
    const int tid = threadIdx.x;
    const int64_t row = blockIdx.x;
    const uint16_t* p = W + row * ld;
    uint32_t m = 0;
    for (int64_t k = tid; k < C; k += kThreads) m = max(m, static_cast<uint32_t>(p[k] & 0x7FFFu));
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((tid & 31) == 0) s_max[tid >> 5] = m;
    __syncthreads();
    m = 0;
    for (int k = 0; k < kThreads / 32; ++k) m = max(m, s_max[k]);
    const float d = __fdiv_rn(cvt16<DT>(static_cast<uint16_t>(m)), qmaxf);
    if (tid == 0 && scale != nullptr) scale[row] = d;
    unsigned int zeros = 0;
    const int64_t pairs = (C + 1) / 2;
    for (int64_t pr = tid; pr < pairs; pr += kThreads) {
        int q[2] = {0, 0};
        for (int e = 0; e < 2; ++e) {
            const int64_t k = 2 * pr + e;
            if (k >= C) break;
            float y = quant_exact(cvt16<DT>(p[k]), d, qmaxf);
            q[e] = code_as_int(y);
            zeros += (q[e] == 0);
            float dq = __fmul_rn(static_cast<float>(q[e]), d);
            if (deq != nullptr) {
                if (deq_dt == CQ_F32) reinterpret_cast<float*>(deq)[row * C + k] = dq;
                else reinterpret_cast<uint16_t*>(deq)[row * C + k] = pack16<DT>(dq);
            }
            if (codes != nullptr && bits == 8) reinterpret_cast<int8_t*>(codes)[row * C + k] = static_cast<int8_t>(q[e]);
        }
        if (codes != nullptr && bits == 4)
            reinterpret_cast<uint8_t*>(codes)[row * (C / 2) + pr] = static_cast<uint8_t>((q[0] & 0xF) | ((q[1] & 0xF) << 4));
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
}

// ============================================================================ dequantize
// Block = (W vector columns of 8 codes) x (256 / W row groups), W = 256 or, for narrower matrices, the power of two that
// covers the row; grid x = blocks of W vector columns, grid y = blocks of row groups of kDeqRows rows (looped when there
// are more than the grid may have).  A thread keeps the scale factors of its eight columns and handles the same
// vector column in kDeqRows consecutive rows: all its code loads are issued before the first is used.
// ODT: CQ_F16 / CQ_BF16 / CQ_F32.
constexpr int kDeqRows = 4;

// NARROW: rows shorter than 256 vectors, several row groups per block (the group then differs from thread to thread;
// with one group per block its row scales and addresses stay uniform across the block, which halves the registers).
template <int BITS, int ODT, bool NARROW>
__global__ void __launch_bounds__(kThreads)
k5_dequantize(const void* __restrict__ codes, int64_t T, int I8, const float* __restrict__ a,
              const float* __restrict__ b, void* __restrict__ out) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= I8) return;
    const int g0 = NARROW ? blockIdx.y * blockDim.y + threadIdx.y : blockIdx.y;          // at most 65535 * 256
    const int gstep = NARROW ? gridDim.y * blockDim.y : gridDim.y;
    const float4 b0 = __ldg(reinterpret_cast<const float4*>(b) + 2 * v);
    const float4 b1 = __ldg(reinterpret_cast<const float4*>(b) + 2 * v + 1);
    const float bj[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    const int64_t ngroups = (T + kDeqRows - 1) / kDeqRows;
#pragma unroll 1
    for (int64_t g = g0; g < ngroups; g += gstep) {
        const int64_t r0 = g * kDeqRows;
        uint2 w8[kDeqRows];
        uint32_t w4[kDeqRows];
        float ai[kDeqRows];
#pragma unroll
        for (int u = 0; u < kDeqRows; ++u) {
            const int64_t row = r0 + u < T ? r0 + u : T - 1;          // rows past the end re-read the last one, store nothing
            const int64_t idx = row * I8 + v;
            if constexpr (BITS == 8) w8[u] = __ldcs(reinterpret_cast<const uint2*>(codes) + idx);
            else w4[u] = __ldcs(reinterpret_cast<const uint32_t*>(codes) + idx);
            ai[u] = __ldg(a + row);
        }
#pragma unroll
        for (int u = 0; u < kDeqRows; ++u) {
            if (r0 + u >= T) break;
            const int64_t idx = (r0 + u) * I8 + v;
            int q[8];
            if constexpr (BITS == 8) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    q[e] = static_cast<int8_t>((w8[u].x >> (8 * e)) & 0xFF);
                    q[4 + e] = static_cast<int8_t>((w8[u].y >> (8 * e)) & 0xFF);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) q[e] = (static_cast<int>(w4[u] << (28 - 4 * e))) >> 28;
            }
            float d[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) d[e] = __fmul_rn(static_cast<float>(q[e]), __fmul_rn(ai[u], bj[e]));
            if constexpr (ODT == CQ_F32) {
                float4* o = reinterpret_cast<float4*>(out) + idx * 2;
                st_stream(o, make_float4(d[0], d[1], d[2], d[3]));
                st_stream(o + 1, make_float4(d[4], d[5], d[6], d[7]));
            } else {
                uint4 o;
                o.x = pack16x2<ODT>(d[0], d[1]); o.y = pack16x2<ODT>(d[2], d[3]);
                o.z = pack16x2<ODT>(d[4], d[5]); o.w = pack16x2<ODT>(d[6], d[7]);
                st_stream(reinterpret_cast<uint4*>(out) + idx, o);
            }
        }
    }
}

// General shapes / alignments: one thread per pair of adjacent columns.
__global__ void __launch_bounds__(kThreads)
g5_dequantize(const void* __restrict__ codes, int bits, int64_t T, int64_t I, const float* __restrict__ a,
              const float* __restrict__ b, void* __restrict__ out, int out_dt) {
    const int64_t pairs = (I + 1) / 2;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= T * pairs) return;
    const int64_t i = idx / pairs, j0 = (idx % pairs) * 2;
    for (int e = 0; e < 2; ++e) {
        const int64_t j = j0 + e;
        if (j >= I) break;
        int q;
        if (bits == 8) {
            q = reinterpret_cast<const int8_t*>(codes)[i * I + j];
        } else {
            uint32_t byte = reinterpret_cast<const uint8_t*>(codes)[i * (I / 2) + j0 / 2];
            q = (static_cast<int>((e ? (byte >> 4) : byte) << 28)) >> 28;
        }
        float d = __fmul_rn(static_cast<float>(q), __fmul_rn(a[i], b[j]));
        if (out_dt == CQ_F32) reinterpret_cast<float*>(out)[i * I + j] = d;
        else if (out_dt == CQ_BF16) reinterpret_cast<uint16_t*>(out)[i * I + j] = pack16<CQ_BF16>(d);
        else reinterpret_cast<uint16_t*>(out)[i * I + j] = pack16<CQ_F16>(d);
    }
}

// ============================================================================ zero-code count
// `body` aligned 16-byte vectors starting `head` bytes into the buffer, plus head and tail bytes.
__global__ void __launch_bounds__(kThreads)
k6_count_zero_codes(const uint8_t* __restrict__ codes, int bits, int64_t head, int64_t body, int64_t tail,
                    unsigned long long* __restrict__ count) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    unsigned int zeros = 0;
    const uint4* vec = reinterpret_cast<const uint4*>(codes + head);
    auto count16 = [bits](const uint4& w) -> unsigned int {
        if (bits == 8) return zero_bytes(w.x) + zero_bytes(w.y) + zero_bytes(w.z) + zero_bytes(w.w);
        return zero_nibbles(w.x) + zero_nibbles(w.y) + zero_nibbles(w.z) + zero_nibbles(w.w);
    };
    // four independent 16-byte loads per thread and round, all issued before the first is used
    int64_t k = idx;
    for (; k + 3 * stride < body; k += 4 * stride) {
        const uint4 w0 = __ldcs(vec + k), w1 = __ldcs(vec + k + stride), w2 = __ldcs(vec + k + 2 * stride),
                    w3 = __ldcs(vec + k + 3 * stride);
        zeros += count16(w0) + count16(w1) + count16(w2) + count16(w3);
    }
    for (; k < body; k += stride) zeros += count16(__ldcs(vec + k));
    auto byte_zeros = [bits](uint8_t v) -> unsigned int {
        if (bits == 8) return v == 0;
        return ((v & 0xF) == 0) + ((v >> 4) == 0);
    };
    if (idx < head) zeros += byte_zeros(codes[idx]);
    if (idx < tail) zeros += byte_zeros(codes[head + body * 16 + idx]);
    cta_count_add(zeros, count);
}

static bool aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }

template <int DT, int BITS, int DEQ, bool CODES>
static int launch_k4(int64_t R, int C8, int64_t ld8, const void* W, void* codes, float* scale, void* deq,
                     unsigned long long* zc, cudaStream_t st) {
    const size_t smem = static_cast<size_t>(C8) * 16;
    // rows of 32 KB or more leave room for at most seven CTAs per SM: those take the bulk-copy variant
    const bool bulk = smem >= CQ_K4_BULK_MIN_BYTES && !tuning_no_stage();
    auto kern = bulk ? k4_weight_rows<DT, BITS, DEQ, CODES, true> : k4_weight_rows<DT, BITS, DEQ, CODES, false>;
    static thread_local LaunchMemo memo[2];          // raises the dynamic shared-memory limit once per row length
    if (smem > 48 * 1024 && resident_ctas(kern, kThreads, smem, kMaxSmemRowBytes, memo[bulk ? 1 : 0]) < 1) return CQ_ERR_CUDA;
    kern<<<static_cast<unsigned>(R), kThreads, smem, st>>>(static_cast<const uint4*>(W), C8, ld8, codes, scale, deq, zc);
    return launch_status();
}

template <int DT, int BITS>
static int launch_k4_out(int deq_mode, bool has_codes, int64_t R, int C8, int64_t ld8, const void* W, void* codes,
                         float* scale, void* deq, unsigned long long* zc, cudaStream_t st) {
    if (has_codes) {
        if (deq_mode == 0) return launch_k4<DT, BITS, 0, true>(R, C8, ld8, W, codes, scale, deq, zc, st);
        if (deq_mode == 1) return launch_k4<DT, BITS, 1, true>(R, C8, ld8, W, codes, scale, deq, zc, st);
        return launch_k4<DT, BITS, 2, true>(R, C8, ld8, W, codes, scale, deq, zc, st);
    }
    if (deq_mode == 0) return launch_k4<DT, BITS, 0, false>(R, C8, ld8, W, codes, scale, deq, zc, st);
    if (deq_mode == 1) return launch_k4<DT, BITS, 1, false>(R, C8, ld8, W, codes, scale, deq, zc, st);
    return launch_k4<DT, BITS, 2, false>(R, C8, ld8, W, codes, scale, deq, zc, st);
}

int weight_stage_fault(unsigned int* fault_host) {
    return cudaMemcpyFromSymbol(fault_host, g_weight_stage_fault, sizeof(unsigned int)) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

}  // namespace cq

extern "C" {

int cq_quantize_weight_per_channel(const void* W, int dtype, int64_t R, int64_t C, int64_t ld, int bits,
                                   void* codes, float* scale, void* deq, int deq_dtype,
                                   unsigned long long* zero_count, void* stream) {
    using namespace cq;
    int rc = check_matrix(W, dtype, R, C, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (deq != nullptr && deq_dtype != dtype && deq_dtype != CQ_F32) return CQ_ERR_DTYPE;
    if (bits == 4 && (C % 2) != 0) return CQ_ERR_ALIGN;
    if (deq != nullptr && !aligned(deq, deq_dtype == CQ_F32 ? 4 : 2)) return CQ_ERR_ALIGN;
    if (scale != nullptr && !aligned(scale, 4)) return CQ_ERR_ALIGN;
    if (zero_count != nullptr && !aligned(zero_count, 8)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (zero_count != nullptr && cudaMemsetAsync(zero_count, 0, sizeof(unsigned long long), st) != cudaSuccess)
        return CQ_ERR_CUDA;
    if (R == 0 || C == 0) return CQ_OK;
    const bool fast = aligned(W, 16) && (C % 8 == 0) && (ld % 8 == 0) && (C * 2 <= kMaxSmemRowBytes) &&
                      (codes == nullptr || aligned(codes, bits == 8 ? 8 : 4)) && (deq == nullptr || aligned(deq, 16));
    if (fast) {
        const int C8 = static_cast<int>(C / 8);
        const int deq_mode = deq == nullptr ? 0 : (deq_dtype == CQ_F32 ? 2 : 1);
        const bool hc = codes != nullptr;
        if (dtype == CQ_F16) {
            if (bits == 8) return launch_k4_out<CQ_F16, 8>(deq_mode, hc, R, C8, ld / 8, W, codes, scale, deq, zero_count, st);
            return launch_k4_out<CQ_F16, 4>(deq_mode, hc, R, C8, ld / 8, W, codes, scale, deq, zero_count, st);
        }
        if (bits == 8) return launch_k4_out<CQ_BF16, 8>(deq_mode, hc, R, C8, ld / 8, W, codes, scale, deq, zero_count, st);
        return launch_k4_out<CQ_BF16, 4>(deq_mode, hc, R, C8, ld / 8, W, codes, scale, deq, zero_count, st);
    }
    if (dtype == CQ_F16)
        g4_weight_rows<CQ_F16><<<static_cast<unsigned>(R), kThreads, 0, st>>>(static_cast<const uint16_t*>(W), C, ld, bits,
                                                                             codes, scale, deq, deq_dtype, zero_count);
    else
        g4_weight_rows<CQ_BF16><<<static_cast<unsigned>(R), kThreads, 0, st>>>(static_cast<const uint16_t*>(W), C, ld, bits,
                                                                              codes, scale, deq, deq_dtype, zero_count);
    return launch_status();
}

int cq_dequantize(const void* codes, int bits, int64_t T, int64_t I, const float* row_scale, const float* col_scale,
                  void* out, int out_dtype, void* stream) {
    using namespace cq;
    if (T < 0 || I < 0 || T > (int64_t(1) << 31) - 256 || I > (int64_t(1) << 31) - 64) return CQ_ERR_SHAPE;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (out_dtype != CQ_F16 && out_dtype != CQ_BF16 && out_dtype != CQ_F32) return CQ_ERR_DTYPE;
    if (bits == 4 && (I % 2) != 0) return CQ_ERR_ALIGN;
    if (T == 0 || I == 0) return CQ_OK;
    if (codes == nullptr || row_scale == nullptr || col_scale == nullptr || out == nullptr) return CQ_ERR_NULL;
    if (!aligned(row_scale, 4) || !aligned(col_scale, 4) || !aligned(out, out_dtype == CQ_F32 ? 4 : 2)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool fast = (I % 8 == 0) && aligned(codes, bits == 8 ? 8 : 4) && aligned(col_scale, 16) && aligned(out, 16);
    if (fast) {
        const int I8 = static_cast<int>(I / 8);
        const int64_t ngroups = (T + kDeqRows - 1) / kDeqRows;
        int W = kThreads;
        while (W / 2 >= I8 && W > 1) W /= 2;
        const dim3 threads(static_cast<unsigned>(W), static_cast<unsigned>(kThreads / W));
        const int64_t gblocks = (ngroups + threads.y - 1) / threads.y;
        const dim3 blocks(static_cast<unsigned>((I8 + W - 1) / W), static_cast<unsigned>(gblocks < 65535 ? gblocks : 65535));
#define CQ_K5(B, O)                                                                                        \
    do {                                                                                                   \
        if (W < kThreads) k5_dequantize<B, O, true><<<blocks, threads, 0, st>>>(codes, T, I8, row_scale, col_scale, out);  \
        else k5_dequantize<B, O, false><<<blocks, threads, 0, st>>>(codes, T, I8, row_scale, col_scale, out);             \
    } while (0)
        if (bits == 8) {
            if (out_dtype == CQ_F16) CQ_K5(8, CQ_F16); else if (out_dtype == CQ_BF16) CQ_K5(8, CQ_BF16); else CQ_K5(8, CQ_F32);
        } else {
            if (out_dtype == CQ_F16) CQ_K5(4, CQ_F16); else if (out_dtype == CQ_BF16) CQ_K5(4, CQ_BF16); else CQ_K5(4, CQ_F32);
        }
#undef CQ_K5
    } else {
        const int64_t n = T * ((I + 1) / 2);
        const unsigned blocks = static_cast<unsigned>((n + kThreads - 1) / kThreads);
        g5_dequantize<<<blocks, kThreads, 0, st>>>(codes, bits, T, I, row_scale, col_scale, out, out_dtype);
    }
    return launch_status();
}

int cq_kernel_count(const void* codes, int bits, int64_t T, int64_t I, unsigned long long* count, void* stream) {
    using namespace cq;
    if (T < 0 || I < 0) return CQ_ERR_SHAPE;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (bits == 4 && (I % 2) != 0) return CQ_ERR_ALIGN;
    if (count == nullptr) return CQ_ERR_NULL;
    if (!aligned(count, 8)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(count, 0, sizeof(unsigned long long), st) != cudaSuccess) return CQ_ERR_CUDA;
    if (T == 0 || I == 0) return CQ_OK;
    if (codes == nullptr) return CQ_ERR_NULL;
    const int64_t nbytes = bits == 8 ? T * I : T * (I / 2);
    int64_t head = static_cast<int64_t>((16 - (reinterpret_cast<uintptr_t>(codes) & 15)) & 15);
    if (head > nbytes) head = nbytes;
    const int64_t body = (nbytes - head) / 16;
    const int64_t tail = nbytes - head - body * 16;
    int64_t blocks = (body + kThreads - 1) / kThreads;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 16) blocks = 148 * 16;
    k6_count_zero_codes<<<static_cast<unsigned>(blocks), kThreads, 0, st>>>(static_cast<const uint8_t*>(codes), bits, head,
                                                                             body, tail, count);
    return launch_status();
}

}  // extern "C"
