// CrossQuant of a small activation matrix (a decode batch, a short prompt) in ONE launch (sm_100a).
//
// The three-launch path costs three launch latencies, which is all a matrix of a few hundred KB pays for.
// Here the whole grid is one thread-block cluster (8 CTAs, or 16 for three or four column strips: column
// strips x row chunks): every CTA keeps its tile of X in shared memory, the partial row and column maxima
// are exchanged through distributed shared memory behind a cluster barrier (a hardware barrier among
// co-scheduled CTAs: nothing spins on memory), the CTAs that share a column strip split its fp64 pow work
// (the long pole: one or two per thread) and exchange the scale factors the same way, and every CTA
// quantizes its tile from shared memory.  Arithmetic and results are those of the three-launch path
// (Section 4.2, CrossQuant equation).
#include <cooperative_groups.h>

#include "cq_common.cuh"
#include "cq_host.h"

namespace cg = cooperative_groups;

namespace cq {

constexpr int kSmallRows = 16;        // most rows of a tile one CTA may hold
constexpr int kSmallTileVecs = 1024;  // most 8-element vectors of a tile (4 rows of a full strip, 8-16 rows of a narrow one)
__device__ unsigned int g_small_stage_fault = 0;      // set if the bounded wait on the tile copy ever gave up
constexpr int kSmallStrips = 4;       // more column strips would leave each thread more than two pows

// Grid = cluster = (nstrips, RY).  CTA (x, y) owns vectors [x W, x W + W) of rows [y Tc, y Tc + Tc).
template <int DT, int BITS>
__global__ void __launch_bounds__(kThreads)
k_small(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8, int Tc, double alpha,
        float* __restrict__ t_out, float* __restrict__ c_out, float* __restrict__ a_out, float* __restrict__ b_out,
        void* __restrict__ codes, void* __restrict__ deq, int deq_mode, unsigned long long* __restrict__ zero_count) {
    constexpr int qmax = (1 << (BITS - 1)) - 1;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    uint4* s_x = reinterpret_cast<uint4*>(s_dyn);                 // [Tc][blockDim.x]
    __shared__ uint4 s_colmax[kThreads];                          // this CTA's column maxima (packed magnitudes)
    __shared__ uint16_t s_rowpart[kThreads / 32][kSmallRows];
    __shared__ uint16_t s_rowmax[kSmallRows];                     // this CTA's row maxima over its strip
    __shared__ float s_a[kSmallRows], s_ra[kSmallRows];
    __shared__ float s_b[8][kThreads], s_rb[8][kThreads];         // column factors this CTA computed: [element][thread]

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, Wv = blockDim.x;
    const int nstrips = gridDim.x, RY = gridDim.y;
    const int v = blockIdx.x * Wv + tid;
    const bool active = v < I8;
    const int vv = active ? v : I8 - 1;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * Tc;
    const int rows = static_cast<int>(max(int64_t(0), min(T - r0, static_cast<int64_t>(Tc))));

    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0 && zero_count != nullptr) *zero_count = 0ull;

    // ---- tile into shared memory by one asynchronous bulk copy per row (the whole tile in flight at once,
    // bounded wait), then the partial maxima from there
    __shared__ uint64_t s_bar;
    const int strip0 = blockIdx.x * Wv;
    const uint32_t seg_bytes = static_cast<uint32_t>(min(Wv, I8 - strip0)) * 16u;
    if (tid == 0) {
        mbar_init(&s_bar, 1);
        mbar_init_fence();
    }
    __syncthreads();
    if (tid == 0 && rows > 0) {
        mbar_expect_tx(&s_bar, static_cast<uint32_t>(rows) * seg_bytes);
        for (int r = 0; r < rows; ++r) bulk_load(s_x + r * Wv, X + (r0 + r) * ld8 + strip0, seg_bytes, &s_bar);
    }
    if (rows > 0 && !mbar_wait(&s_bar, 0u)) atomicExch(&g_small_stage_fault, 1u);
    uint4 cm = make_uint4(0, 0, 0, 0);
    for (int r = 0; r < rows; ++r) {
        uint4 m = active ? s_x[r * Wv + tid] : make_uint4(0, 0, 0, 0);      // lanes past the last column hold nothing
        m.x &= 0x7FFF7FFFu; m.y &= 0x7FFF7FFFu; m.z &= 0x7FFF7FFFu; m.w &= 0x7FFF7FFFu;
        cm.x = max_u16x2(cm.x, m.x); cm.y = max_u16x2(cm.y, m.y);
        cm.z = max_u16x2(cm.z, m.z); cm.w = max_u16x2(cm.w, m.w);
        const uint32_t mm = max_u16x2(max_u16x2(m.x, m.y), max_u16x2(m.z, m.w));
        const uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, max(mm & 0xFFFFu, mm >> 16));
        if (lane == 0) s_rowpart[warp][r] = static_cast<uint16_t>(wm);
    }
    s_colmax[tid] = cm;
    __syncthreads();
    if (tid < kSmallRows) {
        uint32_t m = 0;
        if (tid < rows)
            for (int wdx = 0; wdx < (Wv >> 5); ++wdx) m = max(m, static_cast<uint32_t>(s_rowpart[wdx][tid]));
        s_rowmax[tid] = static_cast<uint16_t>(m);
    }
    cluster.sync();                                               // every CTA's partial maxima are in place

    // ---- row scales of this CTA's rows: maxima over the strips (CTAs (x', y))
    if (tid < rows) {
        uint32_t m = 0;
        for (int xs = 0; xs < nstrips; ++xs) {
            const uint16_t* remote = cluster.map_shared_rank(s_rowmax, xs + blockIdx.y * nstrips);
            m = max(m, static_cast<uint32_t>(remote[tid]));
        }
        const float ti = cvt16<DT>(static_cast<uint16_t>(m));
        float ai, rai;
        row_scale_of(ti, alpha, qmax, ai, rai);
        s_a[tid] = ai;
        s_ra[tid] = rai;
        if (blockIdx.x == 0) {
            t_out[r0 + tid] = ti;
            a_out[r0 + tid] = ai;
        }
    }
    // ---- column scales of this CTA's strip: maxima over the row chunks (CTAs (x, y'))
    uint4 cg4 = make_uint4(0, 0, 0, 0);
    for (int ys = 0; ys < RY; ++ys) {
        const uint4* remote = cluster.map_shared_rank(s_colmax, blockIdx.x + ys * nstrips);
        const uint4 o = remote[tid];
        cg4.x = max_u16x2(cg4.x, o.x); cg4.y = max_u16x2(cg4.y, o.y);
        cg4.z = max_u16x2(cg4.z, o.z); cg4.w = max_u16x2(cg4.w, o.w);
    }
    {
        // element e of every vector is this CTA's if e % RY == blockIdx.y: 8 / RY pows per thread
        const uint32_t words[4] = {cg4.x, cg4.y, cg4.z, cg4.w};
        float cj[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            cj[2 * k] = cvt16<DT>(static_cast<uint16_t>(words[k] & 0xFFFFu));
            cj[2 * k + 1] = cvt16<DT>(static_cast<uint16_t>(words[k] >> 16));
        }
#pragma unroll 1
        for (int e = static_cast<int>(blockIdx.y); e < 8; e += RY) {
            float bj, rbj;
            col_scale_of(cj[e], alpha, qmax, bj, rbj);
            s_b[e][tid] = bj;
            s_rb[e][tid] = rbj;
            if (active) {
                c_out[static_cast<int64_t>(v) * 8 + e] = cj[e];
                b_out[static_cast<int64_t>(v) * 8 + e] = bj;
            }
        }
    }
    cluster.sync();                                               // every CTA's share of the scale factors is in place
    float2 b2[4], rb2[4];
    {
        float bj[8], rbj[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int owner = blockIdx.x + (e % RY) * nstrips;
            bj[e] = cluster.map_shared_rank(&s_b[0][0], owner)[e * kThreads + tid];
            rbj[e] = cluster.map_shared_rank(&s_rb[0][0], owner)[e * kThreads + tid];
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            b2[k] = make_float2(bj[2 * k], bj[2 * k + 1]);
            rb2[k] = make_float2(rbj[2 * k], rbj[2 * k + 1]);
        }
    }
    const bool cols_trusted = ((rb2[0].x + rb2[0].y) + (rb2[1].x + rb2[1].y)) +
                              ((rb2[2].x + rb2[2].y) + (rb2[3].x + rb2[3].y)) < INFINITY;
    // This CTA has read all it needs from the others; it may not exit before they have read what they need from it.
    // Arrive now, wait at the end: the quantize phase runs meanwhile (s_a / s_ra were in place at the barrier above).
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

    // ---- quantize the tile from shared memory
    unsigned int zeros = 0;
#pragma unroll 2
    for (int r = 0; r < rows; ++r) {
        const uint4 w = active ? s_x[r * Wv + tid] : make_uint4(0, 0, 0, 0);
        const float au = s_a[r], rau = s_ra[r];
        float2 y2[4], q2[4];
        quantize_row8<DT, BITS, true>(w, au, rau, b2, rb2, cols_trusted && rau == rau, y2, q2);
        const int64_t vec = (r0 + r) * I8 + v;
        if constexpr (BITS == 8) {
            const uint32_t c0 = pack_int8x4(y2[0].x, y2[0].y, y2[1].x, y2[1].y);
            const uint32_t c1 = pack_int8x4(y2[2].x, y2[2].y, y2[3].x, y2[3].y);
            if (active) zeros += zero_bytes(c0) + zero_bytes(c1);
            if (codes != nullptr && active) st_stream(reinterpret_cast<uint2*>(codes) + vec, make_uint2(c0, c1));
        } else {
            const uint32_t c0 = pack_int4x8(y2);
            if (active) zeros += zero_nibbles(c0);
            if (codes != nullptr && active) st_stream(reinterpret_cast<uint32_t*>(codes) + vec, c0);
        }
        if (deq_mode != 0 && active) {
            const float2 a2 = make_float2(au, au);
            float2 d2[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) d2[k] = __fmul2_rn(q2[k], __fmul2_rn(a2, b2[k]));
            if (deq_mode == 1) {
                uint4 o;
                o.x = pack16x2<DT>(d2[0].x, d2[0].y); o.y = pack16x2<DT>(d2[1].x, d2[1].y);
                o.z = pack16x2<DT>(d2[2].x, d2[2].y); o.w = pack16x2<DT>(d2[3].x, d2[3].y);
                st_stream(reinterpret_cast<uint4*>(deq) + vec, o);
            } else {
                float4* o = reinterpret_cast<float4*>(deq) + vec * 2;
                st_stream(o, make_float4(d2[0].x, d2[0].y, d2[1].x, d2[1].y));
                st_stream(o + 1, make_float4(d2[2].x, d2[2].y, d2[3].x, d2[3].y));
            }
        }
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int DT, int BITS>
static bool launch_small_typed(const SmallArgs& s, int RY, int Tc, cudaStream_t st) {
    auto kern = k_small<DT, BITS>;
    const size_t smem = static_cast<size_t>(Tc) * s.W * 16;
    static thread_local LaunchMemo memo;
    if (resident_ctas(kern, s.W, smem, static_cast<size_t>(kSmallRows) * kThreads * 16, memo) < 1) return false;
    if (s.nstrips * RY > 8) {                                    // 16 CTAs: a non-portable cluster size
        static thread_local int allowed_dev = -1;
        int dev = 0;
        cudaGetDevice(&dev);
        if (allowed_dev != dev) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
                cudaGetLastError();
                return false;
            }
            allowed_dev = dev;
        }
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(s.nstrips);
    attr[0].val.clusterDim.y = static_cast<unsigned>(RY);
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(s.nstrips), static_cast<unsigned>(RY));
    cfg.blockDim = dim3(static_cast<unsigned>(s.W));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, static_cast<const uint4*>(s.X), s.T, s.I8, s.ld8, Tc, s.alpha, s.t, s.c, s.a, s.b,
                           s.codes, s.deq, s.deq_mode, s.zero_count) != cudaSuccess) {
        cudaGetLastError();                                      // the caller falls back to the three-launch path
        return false;
    }
    return true;
}

int small_stage_fault(unsigned int* fault_host) {
    return cudaMemcpyFromSymbol(fault_host, g_small_stage_fault, sizeof(unsigned int)) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

bool launch_small(const SmallArgs& s, cudaStream_t st) {
    if (s.nstrips < 1 || s.nstrips > kSmallStrips || s.T < 1) return false;
    // row chunks: as many as the cluster has room for (a chunk may be empty: its CTA still takes its share of the pows);
    // one or two strips go from the portable 8-CTA cluster to 16 CTAs when that is what makes the tile small enough
    auto fits = [&](int64_t tc) { return tc <= kSmallRows && tc * s.W <= kSmallTileVecs; };
    int RY = (s.nstrips <= 2 ? 8 : 16) / s.nstrips;
    int64_t Tc64 = (s.T + RY - 1) / RY;
    if (!fits(Tc64) && s.nstrips <= 2) {
        RY = 16 / s.nstrips;
        Tc64 = (s.T + RY - 1) / RY;
    }
    if (!fits(Tc64)) return false;
    const int Tc = static_cast<int>(Tc64);
    if (s.dtype == CQ_F16)
        return s.bits == 8 ? launch_small_typed<CQ_F16, 8>(s, RY, Tc, st) : launch_small_typed<CQ_F16, 4>(s, RY, Tc, st);
    return s.bits == 8 ? launch_small_typed<CQ_BF16, 8>(s, RY, Tc, st) : launch_small_typed<CQ_BF16, 4>(s, RY, Tc, st);
}

}  // namespace cq
