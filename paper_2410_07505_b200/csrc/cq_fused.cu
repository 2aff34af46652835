// CrossQuant of an activation matrix that the chip can hold (up to roughly the size of L2) in ONE cooperative launch.
//
// The three-launch path pays two kernel boundaries and reads X twice from wherever it lives.  Here a grid of
// co-resident CTAs (two per SM) does all three steps of Section 4.2 with two grid-wide barriers in between:
//   phase 1  every CTA brings its row groups of one column strip into a shared-memory ring by asynchronous bulk
//            copies and reduces the partial row / column maxima; the last `S` groups stay in the ring
//   barrier  (all partial maxima are in global memory)
//   scales   the blocks of the scale-vector step are dealt round-robin to the CTAs (t, c, a, b, 1/a, 1/b)
//   barrier  (all scale factors are in global memory)
//   phase 2  every CTA walks its groups backwards: the groups still in its ring are quantized straight from shared
//            memory, the earlier ones are fetched again (from L2) into the slots that become free
// With X up to ~28 MB every group is still on chip in phase 2, so X is read from memory exactly once.
// The barriers spin on a counter in the caller's workspace with a bounded number of polls (a wait that gives up
// raises a flag and lets the CTA run on to the end: the kernel cannot hang); the launch is cooperative, so the
// driver guarantees that all CTAs are resident.  Arithmetic and results are those of the three-launch path.
#include <atomic>
#include <chrono>

#include "cq_common.cuh"
#include "cq_host.h"
#include "cq_passes.cuh"

namespace cq {

constexpr int kFusedMaxSlots = 16;                 // ring slots (groups of four rows) per CTA, at most
constexpr int kFusedChunk = 32;                    // row maxima are flushed to global memory every 32 groups
__device__ unsigned int g_fused_fault = 0;         // 1: a wait on a row copy gave up, 2: a grid barrier gave up

// Barrier state in the caller's workspace (contents undefined on entry).  `owner` holds the call's nonce once CTA 0
// has cleared the counters; the other CTAs arrive only after they have seen it, and the last CTA to leave the kernel
// clears it again (so a replay of the same launch, with the same nonce, starts clean).
struct FusedSync {
    unsigned long long owner;
    unsigned int arrived[2];
    unsigned int departed;
};

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned int* p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// Grid-wide barrier number `which` (0 or 1).  Called by every thread of every CTA.  Bounded: ~2^22 polls with a short
// sleep in between (about a second); a CTA that gives up raises the flag and goes on.
__device__ __forceinline__ void grid_barrier(FusedSync* sync, int which, unsigned long long nonce, unsigned int n_ctas) {
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = true;
        if (which == 0) {
            ok = false;
            for (uint32_t polls = 0; polls < (1u << 22); ++polls) {
                if (ld_acquire_u64(&sync->owner) == nonce) { ok = true; break; }
                __nanosleep(32);
            }
        }
        if (ok) {
            __threadfence();
            red_release_add(&sync->arrived[which], 1u);
            ok = false;
            for (uint32_t polls = 0; polls < (1u << 22); ++polls) {
                if (ld_acquire_u32(&sync->arrived[which]) >= n_ctas) { ok = true; break; }
                __nanosleep(32);
            }
        }
        if (!ok) atomicExch(&g_fused_fault, 2u);
        __threadfence();
    }
    __syncthreads();
}

// Grid: nstrips * Yc CTAs of W threads; CTA n owns column strip n % nstrips and the row groups y, y + Yc, ... with
// y = n / nstrips (groups of four rows; the last one may be ragged).  S ring slots of 4 x W vectors each.
template <int DT, int BITS, int DEQ, bool CODES, bool COUNT>
__global__ void __launch_bounds__(kThreads, 2)
k_fused(const uint4* __restrict__ X, int64_t T, int64_t I, int I8, int64_t ld8, int nstrips, int Yc, int S,
        double alpha, uint16_t* __restrict__ rowpart, uint4* __restrict__ colpart,
        float* __restrict__ t_out, float* __restrict__ c_out,
        float* __restrict__ a, float* __restrict__ b, float* __restrict__ ra, float* __restrict__ rb,
        void* __restrict__ codes, void* __restrict__ deq, unsigned long long* __restrict__ zero_count,
        FusedSync* __restrict__ sync, unsigned long long nonce) {
    constexpr int qmax = (1 << (BITS - 1)) - 1;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ uint64_t s_full[kFusedMaxSlots];
    __shared__ uint16_t s_row[kThreads / 32][kFusedChunk * 4];
    __shared__ uint4 s_part[kK2Groups][kK2Cols];
    __shared__ int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, Wv = blockDim.x;
    const int sx = static_cast<int>(blockIdx.x) % nstrips, y = static_cast<int>(blockIdx.x) / nstrips;
    const int v = sx * Wv + tid;
    const bool active = v < I8;
    const bool warp_active = (v - lane) < I8;
    const int vv = active ? v : I8 - 1;
    const int strip0 = sx * Wv;
    const uint32_t seg_bytes = static_cast<uint32_t>(min(Wv, I8 - strip0)) * 16u;
    const int64_t ngroups = (T + 3) >> 2;
    const int mine = y < ngroups ? static_cast<int>((ngroups - y + Yc - 1) / Yc) : 0;     // groups of this CTA
    uint4* stage = reinterpret_cast<uint4*>(s_dyn);                                        // [S][4 rows][Wv]
    auto group_at = [&](int k) { return static_cast<int64_t>(y) + static_cast<int64_t>(k) * Yc; };
    auto rows_in = [&](int64_t g) { const int64_t left = T - (g << 2); return left < 4 ? static_cast<int>(left) : 4; };
    auto issue = [&](int k) {                                          // thread 0 only; group k goes to slot k % S
        const int st = k % S;
        const int64_t g = group_at(k);
        const int nr = rows_in(g);
        const uint4* src = X + (g << 2) * ld8 + strip0;
        mbar_expect_tx(&s_full[st], static_cast<uint32_t>(nr) * seg_bytes);
        for (int u = 0; u < nr; ++u) bulk_load(stage + (st * 4 + u) * Wv, src + u * ld8, seg_bytes, &s_full[st]);
    };

    if (tid == 0) {
        s_abort = 0;
        for (int st = 0; st < S; ++st) mbar_init(&s_full[st], 1);
        mbar_init_fence();
        for (int k = 0; k < min(S, mine); ++k) issue(k);
        if (blockIdx.x == 0) {                                          // this call owns the barrier words from here on
            sync->arrived[0] = 0u;
            sync->arrived[1] = 0u;
            sync->departed = 0u;
            __threadfence();
            st_release_u64(&sync->owner, nonce);
        }
    }
    __syncthreads();

    // ---------------------------------------------------------------- phase 1: partial maxima
    {
        uint4 cm = make_uint4(0, 0, 0, 0);
        const int nwarps = Wv >> 5;
        auto flush_rows = [&](int k0, int count) {                      // groups k0 .. k0 + count - 1 of this CTA
            __syncthreads();
            for (int q = tid; q < count * 4; q += Wv) {
                const int64_t row = (group_at(k0 + (q >> 2)) << 2) + (q & 3);
                if (row < T) {
                    uint32_t m = 0;
                    for (int wdx = 0; wdx < nwarps; ++wdx) m = max(m, static_cast<uint32_t>(s_row[wdx][q]));
                    rowpart[row * nstrips + sx] = static_cast<uint16_t>(m);
                }
            }
            __syncthreads();
        };
        int k0 = 0;
        for (int k = 0; k < mine; ++k) {
            const int st = k % S;
            if (!s_abort && !mbar_wait(&s_full[st], static_cast<uint32_t>((k / S) & 1))) {
                atomicExch(&g_fused_fault, 1u);
                s_abort = 1;
            }
            const int nr = rows_in(group_at(k));
            const int lg = k - k0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint4 m = (active && u < nr) ? stage[(st * 4 + u) * Wv + tid] : make_uint4(0, 0, 0, 0);
                m.x &= 0x7FFF7FFFu; m.y &= 0x7FFF7FFFu; m.z &= 0x7FFF7FFFu; m.w &= 0x7FFF7FFFu;
                cm.x = max_u16x2(cm.x, m.x); cm.y = max_u16x2(cm.y, m.y);
                cm.z = max_u16x2(cm.z, m.z); cm.w = max_u16x2(cm.w, m.w);
                const uint32_t mm = max_u16x2(max_u16x2(m.x, m.y), max_u16x2(m.z, m.w));
                const uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, max(mm & 0xFFFFu, mm >> 16));
                if (lane == 0) s_row[warp][lg * 4 + u] = static_cast<uint16_t>(wm);
            }
            if (k + S < mine) {                                         // the slot is needed again in this phase
                __syncthreads();
                if (tid == 0 && !s_abort) issue(k + S);
            }
            if (lg + 1 == kFusedChunk) {
                flush_rows(k0, kFusedChunk);
                k0 = k + 1;
            }
        }
        if (mine > k0) flush_rows(k0, mine - k0);
        if (active) colpart[static_cast<int64_t>(y) * I8 + v] = cm;
    }

    grid_barrier(sync, 0, nonce, gridDim.x);

    // ---------------------------------------------------------------- scale vectors
    {
        const int col_ctas = (I8 + kK2Cols - 1) / kK2Cols;
        const int blocks = col_ctas + static_cast<int>((T + kThreads - 1) / kThreads);
        if (blockIdx.x == 0 && tid == 0 && zero_count != nullptr) *zero_count = 0ull;
        for (int vb = blockIdx.x; vb < blocks; vb += gridDim.x)
            scales_block<DT>(vb, T, I, I8, nstrips, Yc, col_ctas, rowpart, colpart, alpha, qmax, t_out, c_out, a, b, ra, rb,
                             s_part);
    }

    grid_barrier(sync, 1, nonce, gridDim.x);

    // ---------------------------------------------------------------- phase 2: quantize, last group first
    unsigned int zeros = 0;
    {
        const ColumnScales cs = load_column_scales(b, rb, vv);
        for (int p = 0; p < mine; ++p) {
            const int k = mine - 1 - p;
            const int st = k % S;
            const int64_t g = group_at(k);
            // lanes 0-3 fetch a_i of the group's rows, lanes 4-7 the reciprocals (rows clamped to T-1)
            const int64_t srow = min((g << 2) + (lane & 3), T - 1);
            const float arv = lane < 8 ? __ldcg((lane < 4 ? a : ra) + srow) : 0.0f;
            if (p >= S) {
                // fetched again in this phase: fill number (fills of this slot in phase 1) + p / S - 1 of its barrier
                const int fills1 = (mine - st + S - 1) / S;
                if (!s_abort && !mbar_wait(&s_full[st], static_cast<uint32_t>((fills1 + p / S - 1) & 1))) {
                    atomicExch(&g_fused_fault, 1u);
                    s_abort = 1;
                }
            }
            const int nr = rows_in(g);
            if (warp_active) {
                const int64_t vec = (g << 2) * I8 + vv;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (u < nr)
                        quantize_store_row8<DT, BITS, DEQ, CODES, COUNT>(stage[(st * 4 + u) * Wv + tid],
                                                                         __shfl_sync(0xFFFFFFFFu, arv, u),
                                                                         __shfl_sync(0xFFFFFFFFu, arv, 4 + u), cs, active,
                                                                         vec + static_cast<int64_t>(u) * I8, codes, deq, zeros);
                }
            }
            if (k >= S) {                                               // the slot takes group k - S
                __syncthreads();
                if (tid == 0 && !s_abort) issue(k - S);
            }
        }
        if (!active) zeros = 0;
    }
    if constexpr (COUNT) cta_count_add(zeros, zero_count);

    // the last CTA to leave hands the barrier words back
    if (tid == 0) {
        const unsigned int before = atomicAdd(&sync->departed, 1u);
        if (before + 1u == gridDim.x) st_release_u64(&sync->owner, 0ull);
    }
}

// ============================================================================ host side
static std::atomic<unsigned long long> g_nonce{
    0x9E3779B97F4A7C15ull ^ static_cast<unsigned long long>(std::chrono::steady_clock::now().time_since_epoch().count())};

template <int DT, int BITS, int DEQ, bool CODES, bool COUNT>
static bool launch_fused_typed(const FusedArgs& f, cudaStream_t st) {
    auto kern = k_fused<DT, BITS, DEQ, CODES, COUNT>;
    constexpr size_t kBudget = 104 * 1024;                      // dynamic shared memory per CTA that leaves room for two CTAs per SM
    const size_t slot_bytes = static_cast<size_t>(4) * f.W * 16;
    const int64_t ngroups = (f.T + 3) / 4;
    static thread_local LaunchMemo memo;
    // slots: as many as fit, but no more than the groups a CTA can get when every SM holds two CTAs
    int S = static_cast<int>(kBudget / slot_bytes);
    if (S > kFusedMaxSlots) S = kFusedMaxSlots;
    const int64_t ctas_guess = static_cast<int64_t>(sm_count()) * 2 / f.nstrips;
    if (ctas_guess < 1) return false;
    const int64_t per_cta = (ngroups + ctas_guess - 1) / ctas_guess;
    if (S > per_cta) S = static_cast<int>(per_cta < 1 ? 1 : per_cta);
    if (S < 2 && per_cta > 1) return false;
    const size_t smem = slot_bytes * S;
    const int per_sm = resident_ctas(kern, f.W, smem, kBudget, memo);
    if (per_sm < 1) return false;
    int64_t Yc = static_cast<int64_t>(sm_count()) * per_sm / f.nstrips;
    if (Yc > ngroups) Yc = ngroups;
    if (Yc > f.ymax) Yc = f.ymax;
    if (Yc < 1) return false;
    unsigned long long nonce = g_nonce.fetch_add(1, std::memory_order_relaxed) + 1;
    if (nonce == 0) nonce = g_nonce.fetch_add(1, std::memory_order_relaxed) + 1;

    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(f.nstrips * Yc));
    cfg.blockDim = dim3(static_cast<unsigned>(f.W));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<const uint4*>(f.X), f.T, f.I, f.I8, f.ld8, f.nstrips,
                                             static_cast<int>(Yc), S, f.alpha, f.rowpart, reinterpret_cast<uint4*>(f.colpart),
                                             f.t, f.c, f.a, f.b, f.ra, f.rb, f.codes, f.deq, f.zero_count,
                                             static_cast<FusedSync*>(f.sync), nonce);
    if (e != cudaSuccess) {
        cudaGetLastError();                                     // the caller falls back to the three launches
        return false;
    }
    return true;
}

template <int DT, int BITS>
static bool launch_fused_out(const FusedArgs& f, cudaStream_t st) {
    const bool hc = f.codes != nullptr, hz = f.zero_count != nullptr;
#define CQ_FUSED(D) \
    (hc ? (hz ? launch_fused_typed<DT, BITS, D, true, true>(f, st) : launch_fused_typed<DT, BITS, D, true, false>(f, st)) \
        : (hz ? launch_fused_typed<DT, BITS, D, false, true>(f, st) : launch_fused_typed<DT, BITS, D, false, false>(f, st)))
    if (f.deq_mode == 0) return CQ_FUSED(0);
    if (f.deq_mode == 1) return CQ_FUSED(1);
    return CQ_FUSED(2);
#undef CQ_FUSED
}

bool launch_fused(const FusedArgs& f, cudaStream_t st) {
    static_assert(sizeof(FusedSync) <= kFusedSyncBytes, "the workspace reserves too little for the barrier words");
    if (f.T < 1 || f.I8 < 1 || f.nstrips < 1) return false;
    if (f.dtype == CQ_F16) return f.bits == 8 ? launch_fused_out<CQ_F16, 8>(f, st) : launch_fused_out<CQ_F16, 4>(f, st);
    return f.bits == 8 ? launch_fused_out<CQ_BF16, 8>(f, st) : launch_fused_out<CQ_BF16, 4>(f, st);
}

int fused_fault(unsigned int* fault_host) {
    return cudaMemcpyFromSymbol(fault_host, g_fused_fault, sizeof(unsigned int)) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

}  // namespace cq
