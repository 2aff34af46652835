// CrossQuant activation quantizer: absmax pass, scale vectors, quantize pass (sm_100a).
//
// Pass 1 reads X once and produces partial row maxima (one per row and column strip) and partial
// column maxima (one per column and resident CTA) of the 15-bit magnitudes; a small second kernel
// finishes both reductions and writes t, c and the scale vectors, so no atomics or zero-initialised
// buffers are involved and the result does not depend on scheduling.  Pass 2 re-reads X (walking the
// rows in the opposite order; the rows arrive through a shared-memory ring filled by asynchronous bulk
// copies), forms s_ij = a_i * b_j in registers and emits codes, the dequantized matrix and the number
// of zero codes.
#include <cooperative_groups.h>
#include <math.h>

#include <atomic>
#include <initializer_list>
#include <mutex>

#include "cq_common.cuh"
#include "cq_host.h"
#include "cq_passes.cuh"

#ifndef CQ_K3_MIN_CTAS
#define CQ_K3_MIN_CTAS 2
#endif
#ifndef CQ_STAGES
#define CQ_STAGES 4
#endif

namespace cq {

// ============================================================================ pass 1: absmax
// Grid: x = column strip (blockDim.x vectors of 8 columns), y = one of Y resident CTAs per strip.
// CTA y walks the row groups (kG1 rows each) y, y+Y, y+2Y, ...  Each of its row slots is re-loaded
// for the next group as soon as it has been consumed, so kG1 128-bit loads per thread stay in flight.  Threads past the last column re-read the last vector and rows past the end
// re-read the last row: duplicates do not change a maximum.
// ATOMIC = false: partial maxima to rowpart[T][nstrips] and colpart[Y][I8*8] (16-bit magnitudes).
// ATOMIC = true : order-independent atomic max on the float bit patterns of t / c (pre-zeroed).
#ifndef CQ_K1_GROUP_ROWS
#define CQ_K1_GROUP_ROWS 4
#endif
constexpr int kG1 = CQ_K1_GROUP_ROWS; // rows per group of pass 1
constexpr int kChunkGroups = 32;     // row maxima are flushed to global memory every 32 groups

template <bool ATOMIC, int DT>
__global__ void __launch_bounds__(kThreads)
k1_absmax(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8, int nstrips,
          uint16_t* __restrict__ rowpart, uint4* __restrict__ colpart,
          float* __restrict__ t, float* __restrict__ c) {
    __shared__ uint16_t s_row[kThreads / 32][kChunkGroups * kG1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const int64_t nfull = T / kG1;
    const int64_t ngroups = (T + kG1 - 1) / kG1;
    const int64_t Y = gridDim.y;
    const uint4* xp = X + (active ? v : I8 - 1);
    const int64_t step = kG1 * Y * ld8;
    uint4 cm = make_uint4(0, 0, 0, 0);
    // The quantize pass may be scheduled onto SMs as this grid drains; it waits for this grid to
    // complete (griddepcontrol.wait) before it touches anything written here.
    asm volatile("griddepcontrol.launch_dependents;");

    auto reduce_row = [&](const uint4& w, int slot) {
        uint4 m = w;
        m.x &= 0x7FFF7FFFu; m.y &= 0x7FFF7FFFu; m.z &= 0x7FFF7FFFu; m.w &= 0x7FFF7FFFu;
        cm.x = max_u16x2(cm.x, m.x); cm.y = max_u16x2(cm.y, m.y);
        cm.z = max_u16x2(cm.z, m.z); cm.w = max_u16x2(cm.w, m.w);
        const uint32_t mm = max_u16x2(max_u16x2(m.x, m.y), max_u16x2(m.z, m.w));
        const uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, max(mm & 0xFFFFu, mm >> 16));
        if (lane == 0) s_row[warp][slot] = static_cast<uint16_t>(wm);
    };
    auto flush_rows = [&](int64_t chunk_g0, int lg) {
        __syncthreads();
        const int nwarps = (blockDim.x + 31) >> 5;
        for (int k = tid; k < lg * kG1; k += blockDim.x) {
            const int64_t row = (chunk_g0 + static_cast<int64_t>(k / kG1) * Y) * kG1 + (k % kG1);
            if (row < T) {
                uint32_t m = 0;
                for (int wdx = 0; wdx < nwarps; ++wdx) m = max(m, static_cast<uint32_t>(s_row[wdx][k]));
                if constexpr (ATOMIC) {
                    if (t != nullptr && m)
                        atomicMax(reinterpret_cast<unsigned int*>(t) + row,
                                  __float_as_uint(cvt16<DT>(static_cast<uint16_t>(m))));
                } else {
                    rowpart[row * nstrips + blockIdx.x] = static_cast<uint16_t>(m);
                }
            }
        }
        __syncthreads();
    };

    int64_t g = blockIdx.y;
    int64_t chunk_g0 = g;
    int lg = 0;
    const uint4* p = xp + g * kG1 * ld8;
    uint4 w[kG1];
    if (g < nfull) {
#pragma unroll
        for (int u = 0; u < kG1; ++u) w[u] = ld_nc(p + u * ld8);
    }
    for (; g < ngroups; g += Y) {
        if (g < nfull) {
            const bool has_next = g + Y < nfull;
            const uint4* pn = p + step;
#pragma unroll
            for (int u = 0; u < kG1; ++u) {
                const uint4 cur = w[u];
                if (has_next) w[u] = ld_nc(pn + u * ld8);
                reduce_row(cur, lg * kG1 + u);
            }
            p = pn;
        } else {                                   // the ragged last group: rows past T re-read row T-1
#pragma unroll
            for (int u = 0; u < kG1; ++u) {
                const int64_t row = min(g * kG1 + u, T - 1);
                reduce_row(ld_nc(xp + row * ld8), lg * kG1 + u);
            }
        }
        if (++lg == kChunkGroups) {
            flush_rows(chunk_g0, lg);
            lg = 0;
            chunk_g0 = g + Y;
        }
    }
    if (lg > 0) flush_rows(chunk_g0, lg);

    if constexpr (ATOMIC) {
        // The CTAs of a thread-block cluster (up to 8 along y: the same columns, different rows) first combine their
        // column maxima through distributed shared memory; only the cluster's first CTA goes to memory, which cuts the
        // atomics on every column by the cluster size (they were what this variant spent most of its time on).
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        const unsigned members = cluster.num_blocks();
        if (members > 1) {
            __shared__ uint4 s_cm[kThreads];
            s_cm[tid] = cm;
            cluster.sync();
            if (cluster.block_rank() == 0) {
                for (unsigned r = 1; r < members; ++r) {
                    const uint4 o = cluster.map_shared_rank(s_cm, r)[tid];
                    cm.x = max_u16x2(cm.x, o.x); cm.y = max_u16x2(cm.y, o.y);
                    cm.z = max_u16x2(cm.z, o.z); cm.w = max_u16x2(cm.w, o.w);
                }
            }
            cluster.sync();                              // nobody's shared memory goes away while it is being read
            if (cluster.block_rank() != 0) return;
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
                    // the plain read only skips atomics that could not raise the stored maximum
                    const unsigned int flo = __float_as_uint(cvt16<DT>(static_cast<uint16_t>(lo)));
                    const unsigned int fhi = __float_as_uint(cvt16<DT>(static_cast<uint16_t>(hi)));
                    if (flo > __ldcg(cu + 2 * k)) atomicMax(cu + 2 * k, flo);
                    if (fhi > __ldcg(cu + 2 * k + 1)) atomicMax(cu + 2 * k + 1, fhi);
                }
            }
        } else {
            colpart[static_cast<int64_t>(blockIdx.y) * I8 + v] = cm;
        }
    }
}

// Zeroes the two absmax vectors (the identity of the atomic maxima) in one launch.  Either pointer may be null.
// (Letting the absmax kernel overlap it as a programmatic dependent gained 1.5 us on 16-42 MB matrices and lost 7 us
// on 235 MB, so the two are ordinary, ordered launches.)
__global__ void __launch_bounds__(kThreads)
k0_zero_vectors(float* __restrict__ t, int64_t T, float* __restrict__ c, int64_t I) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t k = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; k < T + I; k += stride) {
        if (k < T) { if (t != nullptr) t[k] = 0.0f; }
        else if (c != nullptr) c[k - T] = 0.0f;
    }
}

// General shapes / alignments: one column per thread, scalar loads, atomic combine (t, c pre-zeroed).
template <int DT>
__global__ void __launch_bounds__(kThreads)
g1_absmax(const uint16_t* __restrict__ X, int64_t T, int64_t I, int64_t ld, int R, unsigned col_blocks,
          float* __restrict__ t, float* __restrict__ c) {
    // one-dimensional grid (row blocks x column blocks fit in 2^31 - 1, not in the 65,535 of the other dimensions)
    const int64_t j = static_cast<int64_t>(blockIdx.x % col_blocks) * blockDim.x + threadIdx.x;
    const bool active = j < I;
    const int64_t r0 = static_cast<int64_t>(blockIdx.x / col_blocks) * R;
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
// From the partial maxima of pass 1: one block of the scale-vector step (cq_passes.cuh) per CTA.
template <int DT>
__global__ void __launch_bounds__(kThreads)
k2_scales_from_partials(int64_t T, int64_t I, int I8, int nstrips, int Y, int col_ctas,
                        const uint16_t* __restrict__ rowpart, const uint4* __restrict__ colpart,
                        double alpha, int qmax,
                        float* __restrict__ t_out, float* __restrict__ c_out,
                        float* __restrict__ a, float* __restrict__ b, float* __restrict__ ra, float* __restrict__ rb,
                        unsigned long long* __restrict__ zero_count) {
    __shared__ uint4 s_part[kK2Groups][kK2Cols];
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0 && threadIdx.x == 0 && zero_count != nullptr) *zero_count = 0ull;
    scales_block<DT>(static_cast<int>(blockIdx.x), T, I, I8, nstrips, Y, col_ctas, rowpart, colpart, alpha, qmax,
                     t_out, c_out, a, b, ra, rb, s_part);
}

// From finished t, c (the general path, and callers that supply the absmax vectors): one thread
// per row (first T threads) or per column (next I threads).
__global__ void __launch_bounds__(kThreads)
k2_scales_from_vectors(int64_t T, int64_t I, const float* __restrict__ t_in, const float* __restrict__ c_in,
                       double alpha, int qmax,
                       float* __restrict__ a, float* __restrict__ b, float* __restrict__ ra, float* __restrict__ rb,
                       unsigned long long* __restrict__ zero_count) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx == 0 && zero_count != nullptr) *zero_count = 0ull;
    if (idx < T) {
        float ai, rai;
        row_scale_of(t_in[idx], alpha, qmax, ai, rai);
        a[idx] = ai;
        ra[idx] = rai;
    } else if (idx - T < I) {
        const int64_t j = idx - T;
        float bj, rbj;
        col_scale_of(c_in[j], alpha, qmax, bj, rbj);
        b[j] = bj;
        rb[j] = rbj;
    }
}

// An empty matrix (no rows or no columns) still has scale vectors in its non-empty dimension: those of the
// supplied maxima, or of 0 (the maximum over nothing) where none are supplied.  Every pointer may be null.
__global__ void __launch_bounds__(kThreads)
k2_scales_of_empty(int64_t T, int64_t I, const float* __restrict__ t_in, const float* __restrict__ c_in,
                   double alpha, int qmax, float* __restrict__ a, float* __restrict__ b) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    float f, r;
    if (idx < T) {
        if (a != nullptr) { row_scale_of(t_in != nullptr ? t_in[idx] : 0.0f, alpha, qmax, f, r); a[idx] = f; }
    } else if (idx - T < I) {
        if (b != nullptr) { col_scale_of(c_in != nullptr ? c_in[idx - T] : 0.0f, alpha, qmax, f, r); b[idx - T] = f; }
    }
}

// acc_j = max(acc_j, v_j): combines the maxima of row blocks of one matrix (magnitudes, so never NaN-ordered
// surprises: fmaxf of two non-negative floats).
__global__ void __launch_bounds__(kThreads)
k_vector_max(float* acc, const float* v, int64_t n) {
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j < n) acc[j] = fmaxf(acc[j], v[j]);
}

// ============================================================================ pass 2: quantize
// Same strip / resident-CTA layout and rolling four-row prefetch as pass 1.  Full row groups are
// walked from the last one backwards (the rows pass 1 touched last are the likeliest to be still in
// L2) unless `forward` is set; a ragged last group (T not a multiple of 4) is done first by CTA y = 0.
// Lanes past the last column compute on the last vector and store nothing.
// DEQ: 0 none, 1 same 16-bit type as X, 2 fp32.
// STAGED: the rows are brought into a ring of shared-memory stages by asynchronous bulk copies
// (kStages groups of four rows per CTA, issued by thread 0 one group ahead of the ring's free slot), so
// the bytes in flight per SM are set by the ring (up to 3 x 16 KB per CTA) instead of by registers.
constexpr int kStages = CQ_STAGES;
__device__ unsigned int g_stage_fault = 0;      // set if a bounded wait on a stage ever gave up

// MODE 0: rows straight into registers; MODE 2 / 3: staged, compiled for 2 / 3 resident CTAs per SM
// (two are faster when X streams from HBM, three when it is served by L2).
template <int DT, int BITS, int DEQ, bool CODES, bool COUNT, int MODE>
__global__ void __launch_bounds__(kThreads, MODE == 0 ? CQ_K3_MIN_CTAS : MODE)
k3_quantize(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8,
            const float* __restrict__ a, const float* __restrict__ ra,
            const float* __restrict__ b, const float* __restrict__ rb,
            void* __restrict__ codes, void* __restrict__ deq,
            unsigned long long* __restrict__ zero_count, int forward) {
    constexpr bool STAGED = MODE != 0;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ uint64_t s_full[kStages];
    __shared__ int s_abort;                      // a wait on a row copy gave up: the CTA stops issuing and leaves
    const int tid = threadIdx.x, lane = tid & 31;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const bool warp_active = (v - lane) < I8;
    const int vv = active ? v : I8 - 1;
    const int64_t nfull = T >> 2;
    const int64_t Y = gridDim.y;
    unsigned int zeros = 0;

    // ---- staged: ring geometry, barriers and the first copies.  X is an input of the whole call, not a product of
    // the preceding kernel, so the ring is filled while that kernel (the scale vectors) is still running.
    uint4* stage = reinterpret_cast<uint4*>(s_dyn);                   // [kStages][4 rows][blockDim.x]
    const int Wv = blockDim.x;
    const int strip0 = blockIdx.x * Wv;
    const uint32_t seg_bytes = static_cast<uint32_t>(min(Wv, I8 - strip0)) * 16u;
    const int64_t first = blockIdx.y;
    const int64_t mine = (STAGED && first < nfull) ? (nfull - first + Y - 1) / Y : 0;      // groups of this CTA
    auto group_at = [&](int64_t k) { const int64_t pos = first + k * Y; return forward ? pos : nfull - 1 - pos; };
    auto issue = [&](int64_t k) {                                     // thread 0 only
        if (k >= mine) return;
        const int st = static_cast<int>(k % kStages);
        const uint4* src = X + (group_at(k) << 2) * ld8 + strip0;
        mbar_expect_tx(&s_full[st], 4u * seg_bytes);
#pragma unroll
        for (int u = 0; u < 4; ++u) bulk_load(stage + (st * 4 + u) * Wv, src + u * ld8, seg_bytes, &s_full[st]);
    };
    if constexpr (STAGED) {
        if (tid == 0) {
            s_abort = 0;
#pragma unroll
            for (int st = 0; st < kStages; ++st) mbar_init(&s_full[st], 1);
            mbar_init_fence();
            for (int k = 0; k < kStages - 1; ++k) issue(k);
        }
        __syncthreads();
    }

    // Everything else this kernel reads is produced by the preceding kernel of the stream.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp_active || STAGED) {
        const ColumnScales cs = load_column_scales(b, rb, vv);
        const uint4* xp = X + vv;
        // lanes 0-3 fetch a_i of a group's four rows, lanes 4-7 the reciprocals (rows clamped to T-1)
        auto load_scales = [&](int64_t g) {
            const int64_t row = min((g << 2) + (lane & 3), T - 1);
            return lane < 8 ? __ldg((lane < 4 ? a : ra) + row) : 0.0f;
        };
        auto do_row = [&](const uint4& x, float au, float rau, int vec) {
            quantize_store_row8<DT, BITS, DEQ, CODES, COUNT>(x, au, rau, cs, active, vec, codes, deq, zeros);
        };

        if ((T & 3) != 0 && blockIdx.y == 0 && warp_active) {          // ragged last group
            const float arv = load_scales(nfull);
            for (int u = 0; u < static_cast<int>(T & 3); ++u) {
                const int64_t row = (nfull << 2) + u;
                do_row(ld_stream(xp + row * ld8), __shfl_sync(0xFFFFFFFFu, arv, u), __shfl_sync(0xFFFFFFFFu, arv, 4 + u),
                       static_cast<int>(row * I8 + vv));
            }
        }

        if constexpr (STAGED) {
            int64_t k = 0;
            for (; k < mine; ++k) {
                const int64_t g = group_at(k);
                const float arv = load_scales(g);
                __syncthreads();                                          // everybody is done with group k-1: its stage is free
                if (s_abort) break;
                if (tid == 0) issue(k + kStages - 1);
                const int st = static_cast<int>(k % kStages);
                if (!mbar_wait(&s_full[st], static_cast<uint32_t>((k / kStages) & 1))) {
                    atomicExch(&g_stage_fault, 1u);
                    s_abort = 1;                                          // seen by everybody after the next barrier
                }
                if (warp_active) {
                    const int vec = static_cast<int>((g << 2) * I8 + vv);
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        do_row(stage[(st * 4 + u) * Wv + tid], __shfl_sync(0xFFFFFFFFu, arv, u),
                               __shfl_sync(0xFFFFFFFFu, arv, 4 + u), vec + u * I8);
                }
            }
            if (k < mine && tid == 0) {
                // Abandoned: nothing more is issued; the copies still in flight (groups k .. k + kStages - 2) get one
                // more bounded wait each so that none of them lands in shared memory the next CTA already owns.
                for (int64_t kk = k; kk < min(mine, k + kStages - 1); ++kk)
                    mbar_wait(&s_full[kk % kStages], static_cast<uint32_t>((kk / kStages) & 1));
            }
        }

        int64_t pos = blockIdx.y;
        if (!STAGED && pos < nfull) {
            const int64_t dgroups = forward ? Y : -Y;
            int64_t g = forward ? pos : nfull - 1 - pos;
            const int64_t xstep = 4 * dgroups * ld8;
            const int ostep = static_cast<int>(4 * dgroups * I8);
            const uint4* p = xp + (g << 2) * ld8;
            int vec = static_cast<int>((g << 2) * I8 + vv);
            uint4 w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) w[u] = ld_stream(p + u * ld8);
            float arv = load_scales(g);
            for (; pos < nfull; pos += Y) {
                const bool has_next = pos + Y < nfull;
                const uint4* pn = p + xstep;
                float arvn = 0.0f;
                if (has_next) arvn = load_scales(g + dgroups);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint4 cur = w[u];
                    if (has_next) w[u] = ld_stream(pn + u * ld8);
                    do_row(cur, __shfl_sync(0xFFFFFFFFu, arv, u), __shfl_sync(0xFFFFFFFFu, arv, 4 + u), vec + u * I8);
                }
                p = pn;
                vec += ostep;
                g += dgroups;
                arv = arvn;
            }
        }
        if (!active) zeros = 0;
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
// Process-wide measurement settings (cq_set_tuning, cq_set_timing_events).  They never change a result; each is
// read once per call, atomically, so a call sees one consistent value even if another thread sets it meanwhile.
static std::atomic<int> g_tune_k1_ctas{0};      // resident CTAs per SM assumed for pass 1 (0 = ask the runtime)
static std::atomic<int> g_tune_k3_ctas{0};      // the same for pass 2
static std::atomic<int> g_tune_k3_forward{0};   // walk pass 2 in ascending row order
static std::atomic<int> g_tune_no_pdl{0};       // launch pass 2 without programmatic dependent launch
static std::atomic<int> g_tune_no_small{0};     // never take the single-launch path for small matrices
static std::atomic<int> g_tune_no_stage{0};     // pass 2 loads rows straight into registers instead of staging them
struct TimingEvents { cudaEvent_t before = nullptr, after = nullptr; };
static TimingEvents g_events;                   // both or neither, under g_events_mutex
static std::mutex g_events_mutex;
static TimingEvents timing_events() {
    std::lock_guard<std::mutex> lock(g_events_mutex);
    return g_events;
}

static inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// Upper bound on the CTAs per column strip of pass 1 (= rows of the column-partial buffer): keeps
// that buffer at 4 MiB or less whatever the device.
static int y_cap(int I8) {
    int64_t cap = (int64_t(4) << 20) / (static_cast<int64_t>(I8 > 0 ? I8 : 1) * 16);
    if (cap < 8) cap = 8;
    if (cap > 2048) cap = 2048;
    return static_cast<int>(cap);
}

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
    p.ngroups = (T + 3) / 4;
    p.ycap = y_cap(p.I8);

    auto carve = [&](size_t bytes) { size_t off = p.total; p.total += (bytes + 255) / 256 * 256; return off; };
    p.total = 0;
    p.off_t = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_c = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    p.off_a = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_b = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    p.off_ra = carve(sizeof(float) * static_cast<size_t>(T));
    p.off_rb = carve(sizeof(float) * static_cast<size_t>(p.I8) * 8);
    p.off_rowpart = carve(sizeof(uint16_t) * static_cast<size_t>(T) * p.nstrips);
    const int64_t ymax = p.ngroups < p.ycap ? (p.ngroups > 0 ? p.ngroups : 1) : p.ycap;
    p.off_colpart = carve(sizeof(uint16_t) * static_cast<size_t>(ymax) * static_cast<size_t>(p.I8) * 8);
    return p;
}

static bool aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }
constexpr int64_t kMaxGridX = (int64_t(1) << 31) - 1;      // most blocks a one-dimensional grid may have

int check_matrix(const void* X, int dtype, int64_t T, int64_t I, int64_t ld) {
    if (T < 0 || I < 0 || ld < I) return CQ_ERR_SHAPE;
    if (T > (int64_t(1) << 31) - 1024 || I > (int64_t(1) << 31) - 64) return CQ_ERR_SHAPE;
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

int launch_status() { return cudaGetLastError() == cudaSuccess ? CQ_OK : CQ_ERR_CUDA; }

int sm_count() {
    static int known[64] = {};                       // per device; 0 = not asked yet (a benign race: same value)
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev >= 0 && dev < 64 && known[dev] > 0) return known[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    if (dev >= 0 && dev < 64) known[dev] = n;
    return n;
}

// CTAs per column strip so that the whole grid is resident at once: floor(SMs * CTAs/SM / strips).
template <typename Kernel>
static int resident_y(Kernel kern, int W, int nstrips, int64_t ngroups, int tuned_ctas_per_sm, int cap, LaunchMemo& memo) {
    int per_sm = tuned_ctas_per_sm;
    if (per_sm <= 0) per_sm = resident_ctas(kern, W, 0, 0, memo);
    if (per_sm < 1) per_sm = 1;
    int64_t y = static_cast<int64_t>(sm_count()) * per_sm / nstrips;
    if (y > ngroups) y = ngroups;
    if (cap > 0 && y > cap) y = cap;
    if (y > 65535) y = 65535;
    if (y < 1) y = 1;
    return static_cast<int>(y);
}

template <bool ATOMIC, int DT>
static int launch_k1(const Plan& p, const void* X, int64_t T, int64_t ld, uint16_t* rowpart, uint16_t* colpart,
                     float* t, float* c, cudaStream_t st) {
    auto kern = k1_absmax<ATOMIC, DT>;
    static thread_local LaunchMemo memo;
    int Y = resident_y(kern, p.W, p.nstrips, (p.ngroups * 4 + kG1 - 1) / kG1, g_tune_k1_ctas.load(), ATOMIC ? 0 : p.ycap, memo);
    if constexpr (ATOMIC) {
        // clusters of up to 8 CTAs along y (a portable size); the grid's y extent becomes a multiple of the cluster's
        int cy = 8;
        while (cy > 1 && Y < cy) cy >>= 1;
        Y = Y / cy * cy;
        if (cy > 1) {
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 1;
            attr[0].val.clusterDim.y = static_cast<unsigned>(cy);
            attr[0].val.clusterDim.z = 1;
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3(p.nstrips, Y);
            cfg.blockDim = dim3(p.W);
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, kern, static_cast<const uint4*>(X), T, p.I8, ld / 8, p.nstrips, rowpart,
                                   reinterpret_cast<uint4*>(colpart), t, c) == cudaSuccess)
                return Y;
            cudaGetLastError();                          // refused as a cluster launch: an ordinary one does the same work
        }
    }
    kern<<<dim3(p.nstrips, Y), p.W, 0, st>>>(static_cast<const uint4*>(X), T, p.I8, ld / 8, p.nstrips, rowpart,
                                             reinterpret_cast<uint4*>(colpart), t, c);
    return Y;
}

// pass 1 with atomics into pre-zeroed t / c (either may be null)
static int absmax_atomic(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t, float* c,
                         cudaStream_t st) {
    {
        const int64_t n = (t != nullptr ? T : 0) + (c != nullptr ? I : 0);
        if (n > 0) {
            int64_t blocks = (T + I + kThreads - 1) / kThreads;
            if (blocks > 2 * sm_count()) blocks = 2 * sm_count();
            k0_zero_vectors<<<static_cast<unsigned>(blocks), kThreads, 0, st>>>(t, T, c, I);
        }
    }
    if (T == 0 || I == 0) return launch_status();
    Plan p = make_plan(T, I);
    if (fast_input(X, I, ld)) {
        if (dtype == CQ_F16) launch_k1<true, CQ_F16>(p, X, T, ld, nullptr, nullptr, t, c, st);
        else launch_k1<true, CQ_BF16>(p, X, T, ld, nullptr, nullptr, t, c, st);
    } else {
        const int R = 64;
        const int64_t col_blocks = (I + kThreads - 1) / kThreads, row_blocks = (T + R - 1) / R;
        if (col_blocks * row_blocks > kMaxGridX) return CQ_ERR_SHAPE;
        const unsigned grid = static_cast<unsigned>(col_blocks * row_blocks), cb = static_cast<unsigned>(col_blocks);
        if (dtype == CQ_F16)
            g1_absmax<CQ_F16><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, R, cb, t, c);
        else
            g1_absmax<CQ_BF16><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, R, cb, t, c);
    }
    return launch_status();
}

// Programmatic dependent launch: the kernel's CTAs may become resident while the previous kernel of
// the stream drains; the kernel itself waits (griddepcontrol.wait) before reading what that one wrote.
template <typename... KArgs, typename... Args>
static void launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_tune_no_pdl ? 0 : 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

struct K3Args {
    const uint4* X; int64_t T; int I8; int64_t ld8;
    const float *a, *ra, *b, *rb;
    void* codes; void* deq; unsigned long long* zc;
};

template <int DT, int BITS, int DEQ, bool CODES, bool COUNT, int MODE>
static bool launch_k3_staged(const Plan& p, const K3Args& k, cudaStream_t st) {
    auto kern = k3_quantize<DT, BITS, DEQ, CODES, COUNT, MODE>;
    const size_t smem = static_cast<size_t>(kStages) * 4 * p.W * 16;
    static thread_local LaunchMemo memo;
    const int per_sm = resident_ctas(kern, p.W, smem, static_cast<size_t>(kStages) * 4 * kThreads * 16, memo);
    if (per_sm < 1) return false;
    int64_t y = static_cast<int64_t>(sm_count()) * per_sm / p.nstrips;
    if (y > p.ngroups) y = p.ngroups;
    if (y > 65535) y = 65535;
    if (y < 1) y = 1;
    launch_dependent(kern, dim3(p.nstrips, static_cast<unsigned>(y)), dim3(p.W), smem, st, k.X, k.T, k.I8, k.ld8, k.a, k.ra,
                     k.b, k.rb, k.codes, k.deq, k.zc, g_tune_k3_forward.load());
    return true;
}

template <int DT, int BITS, int DEQ, bool CODES, bool COUNT>
static void launch_k3_one(const Plan& p, const K3Args& k, cudaStream_t st) {
    if (!g_tune_no_stage) {
        // matrices that stream from HBM run two CTAs per SM, those L2 can hold run three (INT8; with INT4
        // codes the two-CTA build is the faster one at every size measured)
        const int64_t bytes = k.T * k.ld8 * 16;
        int mode = (bytes > (int64_t(120) << 20) || BITS == 4) ? 2 : 3;
        const int tuned = g_tune_k3_ctas;
        if (tuned == 2 || tuned == 3) mode = tuned;
        const bool ok = mode == 2 ? launch_k3_staged<DT, BITS, DEQ, CODES, COUNT, 2>(p, k, st)
                                  : launch_k3_staged<DT, BITS, DEQ, CODES, COUNT, 3>(p, k, st);
        if (ok) return;
    }
    auto kern = k3_quantize<DT, BITS, DEQ, CODES, COUNT, 0>;
    static thread_local LaunchMemo memo;
    const int Y = resident_y(kern, p.W, p.nstrips, p.ngroups, g_tune_k3_ctas.load(), 0, memo);
    launch_dependent(kern, dim3(p.nstrips, Y), dim3(p.W), 0, st, k.X, k.T, k.I8, k.ld8, k.a, k.ra, k.b, k.rb, k.codes,
                     k.deq, k.zc, g_tune_k3_forward.load());
}

template <int DT, int BITS, int DEQ>
static void launch_k3_flags(const Plan& p, const K3Args& k, cudaStream_t st) {
    const bool hc = k.codes != nullptr, hz = k.zc != nullptr;
    if (hc && hz) launch_k3_one<DT, BITS, DEQ, true, true>(p, k, st);
    else if (hc) launch_k3_one<DT, BITS, DEQ, true, false>(p, k, st);
    else if (hz) launch_k3_one<DT, BITS, DEQ, false, true>(p, k, st);
    else launch_k3_one<DT, BITS, DEQ, false, false>(p, k, st);
}

template <int DT, int BITS>
static void launch_k3_deq(const Plan& p, const K3Args& k, int deq_mode, cudaStream_t st) {
    if (deq_mode == 0) launch_k3_flags<DT, BITS, 0>(p, k, st);
    else if (deq_mode == 1) launch_k3_flags<DT, BITS, 1>(p, k, st);
    else launch_k3_flags<DT, BITS, 2>(p, k, st);
}

bool tuning_no_pdl() { return g_tune_no_pdl != 0; }
bool tuning_no_stage() { return g_tune_no_stage != 0; }

// Scale vectors and their reciprocals into the workspace from finished t, c (for the diagnostics
// kernels); *to_zero, if given, is cleared by the same launch.
int scales_from_vectors(int64_t T, int64_t I, const float* t, const float* c, double alpha, int bits,
                        void* workspace, size_t ws_bytes, unsigned long long* to_zero, cudaStream_t st) {
    const Plan p = make_plan(T, I);
    if (workspace == nullptr || !aligned(workspace, 256) || ws_bytes < p.total) return CQ_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    const unsigned blocks = static_cast<unsigned>((T + I + kThreads - 1) / kThreads);
    k2_scales_from_vectors<<<blocks, kThreads, 0, st>>>(T, I, t, c, alpha, (1 << (bits - 1)) - 1,
                                                        reinterpret_cast<float*>(ws + p.off_a), reinterpret_cast<float*>(ws + p.off_b),
                                                        reinterpret_cast<float*>(ws + p.off_ra), reinterpret_cast<float*>(ws + p.off_rb),
                                                        to_zero);
    return launch_status();
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
    if (bits == 4 && (I % 2) != 0 && codes != nullptr) return CQ_ERR_ALIGN;      // packed codes need whole bytes
    if (deq != nullptr && !aligned(deq, deq_dtype == CQ_F32 ? 4 : 2)) return CQ_ERR_ALIGN;
    if (zero_count != nullptr && !aligned(zero_count, 8)) return CQ_ERR_ALIGN;
    for (const float* f : {static_cast<const float*>(t), static_cast<const float*>(c),
                           static_cast<const float*>(row_scale), static_cast<const float*>(col_scale),
                           t_given, c_given})
        if (f != nullptr && !aligned(f, 4)) return CQ_ERR_ALIGN;
    if (T == 0 || I == 0) {
        // Nothing to quantize, but the vectors of the non-empty dimension are still results: maxima over nothing
        // are 0 (a row block without rows must contribute zeros to the combined column maxima).
        if (zero_count != nullptr && cudaMemsetAsync(zero_count, 0, sizeof(unsigned long long), st) != cudaSuccess)
            return CQ_ERR_CUDA;
        if (t != nullptr && T > 0 && cudaMemsetAsync(t, 0, sizeof(float) * T, st) != cudaSuccess) return CQ_ERR_CUDA;
        if (c != nullptr && I > 0 && cudaMemsetAsync(c, 0, sizeof(float) * I, st) != cudaSuccess) return CQ_ERR_CUDA;
        float* a_out = T > 0 ? row_scale : nullptr;
        float* b_out = I > 0 ? col_scale : nullptr;
        if (a_out != nullptr || b_out != nullptr) {
            const unsigned blocks = static_cast<unsigned>((T + I + kThreads - 1) / kThreads);
            k2_scales_of_empty<<<blocks, kThreads, 0, st>>>(T, I, t_given, c_given, alpha, (1 << (bits - 1)) - 1, a_out, b_out);
            return launch_status();
        }
        return CQ_OK;
    }
    Plan p = make_plan(T, I);
    if (workspace == nullptr || !aligned(workspace, 256) || ws_bytes < p.total) return CQ_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    // Vectors the caller did not ask for live in the workspace.  The fast quantize pass reads b / rb
    // as whole float4 pairs, so col_scale must be 16-byte aligned to be used in place.
    const bool given = t_given != nullptr && c_given != nullptr;
    float* t_dev = t != nullptr ? t : reinterpret_cast<float*>(ws + p.off_t);
    const bool c_in_place = c != nullptr;
    float* c_dev = c_in_place ? c : reinterpret_cast<float*>(ws + p.off_c);
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
                          (deq == nullptr || aligned(deq, 16)) &&
                          T * static_cast<int64_t>(p.I8) < (int64_t(1) << 31);     // 32-bit vector indices
    const unsigned k2v_blocks = static_cast<unsigned>((T + I + kThreads - 1) / kThreads);

    // ---- small matrices: everything in one launch of one thread-block cluster
    const TimingEvents ev = timing_events();
    const bool timed = ev.before != nullptr && ev.after != nullptr;
    if (!given && fast_in && fast_out && !g_tune_no_small && !timed &&
        (codes != nullptr || deq != nullptr || zero_count != nullptr)) {      // (callers without outputs want the workspace vectors)
        const SmallArgs sa{X, dtype, T, p.I8, ld / 8, p.W, p.nstrips, alpha, bits, t_dev, c_dev, a_dev, b_dev,
                           codes, deq, deq == nullptr ? 0 : (deq_dtype == CQ_F32 ? 2 : 1), zero_count};
        if (launch_small(sa, st)) {
            if ((rc = launch_status()) != CQ_OK) return rc;
            if (col_scale != nullptr && !b_in_place &&
                cudaMemcpyAsync(col_scale, b_dev, sizeof(float) * I, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return CQ_ERR_CUDA;
            return CQ_OK;
        }
    }

    // ---- pass 1 + scale vectors
    if (given) {
        k2_scales_from_vectors<<<k2v_blocks, kThreads, 0, st>>>(T, I, t_given, c_given, alpha, qmax, a_dev, b_dev,
                                                                ra_dev, rb_dev, zero_count);
    } else if (fast_in) {
        const int col_ctas = (p.I8 + kK2Cols - 1) / kK2Cols;
        const unsigned blocks = static_cast<unsigned>(col_ctas + (T + kThreads - 1) / kThreads);
        const uint4* cp4 = reinterpret_cast<const uint4*>(colpart);
        if (dtype == CQ_F16) {
            const int Y = launch_k1<false, CQ_F16>(p, X, T, ld, rowpart, colpart, nullptr, nullptr, st);
            launch_dependent(k2_scales_from_partials<CQ_F16>, dim3(blocks), dim3(kThreads), 0, st, T, I, p.I8, p.nstrips, Y,
                             col_ctas, static_cast<const uint16_t*>(rowpart), cp4, alpha, qmax, t_dev, c_dev, a_dev, b_dev,
                             ra_dev, rb_dev, zero_count);
        } else {
            const int Y = launch_k1<false, CQ_BF16>(p, X, T, ld, rowpart, colpart, nullptr, nullptr, st);
            launch_dependent(k2_scales_from_partials<CQ_BF16>, dim3(blocks), dim3(kThreads), 0, st, T, I, p.I8, p.nstrips, Y,
                             col_ctas, static_cast<const uint16_t*>(rowpart), cp4, alpha, qmax, t_dev, c_dev, a_dev, b_dev,
                             ra_dev, rb_dev, zero_count);
        }
    } else {
        rc = absmax_atomic(X, dtype, T, I, ld, t_dev, c_dev, st);
        if (rc != CQ_OK) return rc;
        k2_scales_from_vectors<<<k2v_blocks, kThreads, 0, st>>>(T, I, t_dev, c_dev, alpha, qmax, a_dev, b_dev, ra_dev,
                                                                rb_dev, zero_count);
    }
    if ((rc = launch_status()) != CQ_OK) return rc;

    // ---- pass 2
    const bool any_out = codes != nullptr || deq != nullptr || zero_count != nullptr;
    if (any_out) {
        if (timed) cudaEventRecord(ev.before, st);
        if (fast_in && fast_out) {
            const int deq_mode = deq == nullptr ? 0 : (deq_dtype == CQ_F32 ? 2 : 1);
            const K3Args k{static_cast<const uint4*>(X), T, p.I8, ld / 8, a_dev, ra_dev, b_dev, rb_dev, codes, deq, zero_count};
            if (dtype == CQ_F16) {
                if (bits == 8) launch_k3_deq<CQ_F16, 8>(p, k, deq_mode, st);
                else launch_k3_deq<CQ_F16, 4>(p, k, deq_mode, st);
            } else {
                if (bits == 8) launch_k3_deq<CQ_BF16, 8>(p, k, deq_mode, st);
                else launch_k3_deq<CQ_BF16, 4>(p, k, deq_mode, st);
            }
        } else {
            const int64_t n = T * ((I + 1) / 2);
            if ((n + kThreads - 1) / kThreads > kMaxGridX) return CQ_ERR_SHAPE;
            const unsigned blocks = static_cast<unsigned>((n + kThreads - 1) / kThreads);
            if (dtype == CQ_F16)
                g3_quantize<CQ_F16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, bits, a_dev, b_dev,
                                                                 codes, deq, deq_dtype, zero_count);
            else
                g3_quantize<CQ_BF16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(X), T, I, ld, bits, a_dev, b_dev,
                                                                  codes, deq, deq_dtype, zero_count);
        }
        if (timed) cudaEventRecord(ev.after, st);
        if ((rc = launch_status()) != CQ_OK) return rc;
    }
    if (c != nullptr && !c_in_place && !given) {
        if (cudaMemcpyAsync(c, c_dev, sizeof(float) * I, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return CQ_ERR_CUDA;
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
        case CQ_ERR_TOO_LARGE: return "matrix needs more scratch than the built-in no-allocation buffer holds";
        default: return "unknown status";
    }
}

int cq_set_tuning(const char* key, int value) {
    if (key == nullptr) return CQ_ERR_NULL;
    auto eq = [](const char* x, const char* y) { while (*x && *x == *y) { ++x; ++y; } return *x == *y; };
    const int v = value > 0 ? value : 0;
    if (v > 64) return CQ_ERR_SHAPE;
    if (eq(key, "k1_ctas_per_sm")) { cq::g_tune_k1_ctas = v; return CQ_OK; }
    if (eq(key, "k3_ctas_per_sm")) { cq::g_tune_k3_ctas = v; return CQ_OK; }
    if (eq(key, "k3_forward")) { cq::g_tune_k3_forward = v ? 1 : 0; return CQ_OK; }
    if (eq(key, "no_pdl")) { cq::g_tune_no_pdl = v ? 1 : 0; return CQ_OK; }
    if (eq(key, "no_stage")) { cq::g_tune_no_stage = v ? 1 : 0; return CQ_OK; }
    if (eq(key, "no_small")) { cq::g_tune_no_small = v ? 1 : 0; return CQ_OK; }
    return CQ_ERR_SHAPE;
}

int cq_stage_fault(unsigned int* fault_host) {
    if (fault_host == nullptr) return CQ_ERR_NULL;
    unsigned int quantize_pass = 0, diagnostics = 0, weights = 0, small = 0;
    if (cudaMemcpyFromSymbol(&quantize_pass, cq::g_stage_fault, sizeof(unsigned int)) != cudaSuccess) return CQ_ERR_CUDA;
    int rc = cq::diag_stage_fault(&diagnostics);
    if (rc == CQ_OK) rc = cq::weight_stage_fault(&weights);
    if (rc == CQ_OK) rc = cq::small_stage_fault(&small);
    if (rc != CQ_OK) return rc;
    *fault_host = quantize_pass | diagnostics | weights | small;
    return CQ_OK;
}

int cq_set_timing_events(void* before_quantize_pass, void* after_quantize_pass) {
    std::lock_guard<std::mutex> lock(cq::g_events_mutex);
    const bool both = before_quantize_pass != nullptr && after_quantize_pass != nullptr;
    cq::g_events.before = both ? static_cast<cudaEvent_t>(before_quantize_pass) : nullptr;
    cq::g_events.after = both ? static_cast<cudaEvent_t>(after_quantize_pass) : nullptr;
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

int cq_vector_max(float* acc, const float* v, int64_t n, void* stream) {
    if (n < 0) return CQ_ERR_SHAPE;
    if (n == 0) return CQ_OK;
    if (acc == nullptr || v == nullptr) return CQ_ERR_NULL;
    if (!cq::aligned(acc, 4) || !cq::aligned(v, 4)) return CQ_ERR_ALIGN;
    const unsigned blocks = static_cast<unsigned>((n + cq::kThreads - 1) / cq::kThreads);
    cq::k_vector_max<<<blocks, cq::kThreads, 0, static_cast<cudaStream_t>(stream)>>>(acc, v, n);
    return cq::launch_status();
}

int cq_quantize_act_given(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                          const float* t, const float* c, float* row_scale, float* col_scale,
                          void* codes, void* deq, int deq_dtype, unsigned long long* zero_count,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (T > 0 && I > 0 && (t == nullptr || c == nullptr)) return CQ_ERR_NULL;
    return cq::quantize_act_impl(X, dtype, T, I, ld, alpha, bits, t, c, nullptr, nullptr, row_scale, col_scale,
                                 codes, deq, deq_dtype, zero_count, workspace, workspace_bytes,
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
