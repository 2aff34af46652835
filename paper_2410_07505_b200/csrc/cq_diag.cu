// Diagnostics of the quantization kernel (Definition 1) that need no codes: the "Remove Kernel"
// operator (Figure 1, Appendix B) with the per-token and CrossQuant kernel sizes from one pass, and
// |K(CQ)| straight from X (Section 4.2).  Both only ask, per element, whether |fl32(x / s)| <= h.
#include <math.h>

#include "cq_common.cuh"
#include "cq_host.h"

#ifndef CQ_K9_MIN_CTAS
#define CQ_K9_MIN_CTAS 2
#endif

namespace cq {

// |fl32(x / s)| <= h, decided from a reciprocal product where that is safe.  With every scale factor
// in [2^-40, 2^40] the product v = x * (1/a_i) * (1/b_j) (or x * (1/s) for one scale) differs from the
// real quotient z by less than 5 * 2^-24 |z|, and fl32(z) from z by at most 2^-24 |z|; so for h in
// [2^-20, 2^20] (where nothing near h can be subnormal)
//     |v| < h (1 - 2^-16)  =>  |fl32(z)| <  h,        |v| > h (1 + 2^-16)  =>  |fl32(z)| > h,
// and only values inside that band (or a NaN, which fails both comparisons: the marker of an extreme
// scale factor) need the quotient itself.  For h outside that range the band is (-1, inf): every
// element takes the quotient.
struct ZeroBand { float lo, hi; };

static __device__ __noinline__ bool exact_at_most(float x, float s, float h) {
    if (s == 0.0f) return true;                       // the code of a zero scale is 0 by definition
    return fabsf(__fdiv_rn(x, s)) <= h;
}

// Same strip / resident-CTA layout and rolling four-row prefetch as the quantize pass; rows walked
// from the last full group backwards, the ragged last group first by CTA y = 0.
//   WRITE: out = x, or +0 where |fl32(x / s_ij)| <= half_bound         (counts[0] += removed)
//   DUAL : counts[1] += |K| of per-token quantization (scale fl32(t_i / qmax)), counts[2] += |K(CQ)|
//   SAME : half_bound == 1/2, so "removed" and "in K(CQ)" are one test
//   !WRITE && !DUAL: counts[0] += |K(CQ)| only
template <int DT, bool WRITE, bool DUAL, bool SAME>
__global__ void __launch_bounds__(kThreads, CQ_K9_MIN_CTAS)
k9_zero_tests(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8,
              const float* __restrict__ t, const float* __restrict__ a, const float* __restrict__ ra,
              const float* __restrict__ b, const float* __restrict__ rb, float qmaxf,
              float half_bound, ZeroBand band_h, ZeroBand band_half,
              uint4* __restrict__ out, unsigned long long* __restrict__ counts) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const bool warp_active = (v - lane) < I8;
    const int vv = active ? v : I8 - 1;
    const int64_t nfull = T >> 2;
    const int64_t Y = gridDim.y;
    unsigned int n_removed = 0, n_pt = 0, n_cq = 0;

    // the scale vectors come from the preceding kernel of the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp_active) {
        float2 rb2[4];
        {
            const float4* rp = reinterpret_cast<const float4*>(rb) + static_cast<int64_t>(vv) * 2;
            const float4 q0 = __ldg(rp), q1 = __ldg(rp + 1);
            rb2[0] = make_float2(q0.x, q0.y); rb2[1] = make_float2(q0.z, q0.w);
            rb2[2] = make_float2(q1.x, q1.y); rb2[3] = make_float2(q1.z, q1.w);
        }
        const uint4* xp = X + vv;

        auto do_row = [&](uint4& slot, const uint4* reload, bool has_next, float rau, float rpt, int64_t row, int vec) {
            const uint32_t words[4] = {slot.x, slot.y, slot.z, slot.w};
            if (has_next) slot = ld_stream(reload);
            const float2 ra2 = make_float2(rau, rau), rp2 = make_float2(rpt, rpt);
            unsigned int r_rm = 0, r_pt = 0, r_cq = 0;
            bool undecided = false;
            uint32_t ow[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 x = unpack16x2<DT>(words[k]);
                const float2 vq = __fmul2_rn(x, __fmul2_rn(ra2, rb2[k]));
                const float av[2] = {fabsf(vq.x), fabsf(vq.y)};
                uint32_t keep = 0xFFFFFFFFu;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const bool z = av[h] < band_half.lo, nz = av[h] > band_half.hi;
                    r_cq += z;
                    undecided |= !(z || nz);
                    bool gone = z;
                    if constexpr (!SAME) {
                        const bool g = av[h] < band_h.lo, ng = av[h] > band_h.hi;
                        undecided |= !(g || ng);
                        gone = g;
                    }
                    r_rm += gone;
                    if (gone) keep &= h ? 0x0000FFFFu : 0xFFFF0000u;
                }
                if constexpr (DUAL) {
                    const float2 vp = __fmul2_rn(x, rp2);
                    const float ap[2] = {fabsf(vp.x), fabsf(vp.y)};
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const bool z = ap[h] < band_half.lo, nz = ap[h] > band_half.hi;
                        r_pt += z;
                        undecided |= !(z || nz);
                    }
                }
                ow[k] = words[k] & keep;
            }
            if (undecided) {
                // Rare: some element sits within 2^-16 (relative) of a bound, or a scale factor is extreme.
                // The whole vector is decided again from the IEEE quotients.
                r_rm = r_pt = r_cq = 0;
                const float ai = __ldg(a + row);
                const float spt = DUAL ? __fdiv_rn(__ldg(t + row), qmaxf) : 0.0f;
                const float* bp = b + static_cast<int64_t>(vv) * 8;
#pragma unroll 1
                for (int k = 0; k < 4; ++k) {
                    const float2 x = unpack16x2<DT>(words[k]);
                    const float xs[2] = {x.x, x.y};
                    uint32_t keep = 0xFFFFFFFFu;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float s = __fmul_rn(ai, __ldg(bp + 2 * k + h));
                        const bool z = exact_at_most(xs[h], s, 0.5f);
                        const bool gone = SAME ? z : exact_at_most(xs[h], s, half_bound);
                        r_cq += z;
                        r_rm += gone;
                        if constexpr (DUAL) r_pt += exact_at_most(xs[h], spt, 0.5f);
                        if (gone) keep &= h ? 0x0000FFFFu : 0xFFFF0000u;
                    }
                    ow[k] = words[k] & keep;
                }
            }
            n_removed += r_rm; n_pt += r_pt; n_cq += r_cq;
            if constexpr (WRITE) {
                if (active) st_stream(out + vec, make_uint4(ow[0], ow[1], ow[2], ow[3]));
            }
        };
        // lanes 0-3: 1/a_i of a group's four rows; lanes 4-7: reciprocal of the per-token scale t_i / qmax
        auto load_scales = [&](int64_t g) {
            const int64_t row = min((g << 2) + (lane & 3), T - 1);
            float sv = 0.0f;
            if (lane < 4) sv = __ldg(ra + row);
            else if (DUAL && lane < 8) sv = guarded_rcp(__fdiv_rn(__ldg(t + row), qmaxf));
            return sv;
        };

        if ((T & 3) != 0 && blockIdx.y == 0) {                           // ragged last group
            const float sv = load_scales(nfull);
            for (int u = 0; u < static_cast<int>(T & 3); ++u) {
                const int64_t row = (nfull << 2) + u;
                uint4 slot = ld_stream(xp + row * ld8);
                do_row(slot, nullptr, false, __shfl_sync(0xFFFFFFFFu, sv, u), __shfl_sync(0xFFFFFFFFu, sv, 4 + u), row,
                       static_cast<int>(row * I8 + vv));
            }
        }

        int64_t pos = blockIdx.y;
        if (pos < nfull) {
            int64_t g = nfull - 1 - pos;
            const int64_t xstep = -4 * Y * ld8;
            const int ostep = static_cast<int>(-4 * Y * I8);
            const uint4* p = xp + (g << 2) * ld8;
            int vec = static_cast<int>((g << 2) * I8 + vv);
            uint4 w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) w[u] = ld_stream(p + u * ld8);
            float sv = load_scales(g);
            for (; pos < nfull; pos += Y) {
                const bool has_next = pos + Y < nfull;
                const uint4* pn = p + xstep;
                float svn = 0.0f;
                if (has_next) svn = load_scales(g - Y);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    do_row(w[u], pn + u * ld8, has_next, __shfl_sync(0xFFFFFFFFu, sv, u), __shfl_sync(0xFFFFFFFFu, sv, 4 + u),
                           (g << 2) + u, vec + u * I8);
                p = pn;
                vec += ostep;
                g -= Y;
                sv = svn;
            }
        }
        if (!active) { n_removed = 0; n_pt = 0; n_cq = 0; }
    }
    if constexpr (WRITE || DUAL) {
        cta_count_add(n_removed, counts);
        __syncthreads();
        cta_count_add(n_pt, counts + 1);
        __syncthreads();
        cta_count_add(n_cq, counts + 2);
    } else {
        cta_count_add(n_cq, counts);
    }
}

// General shapes / alignments: one thread per element, IEEE quotients.  counts as above; out unused
// when only |K(CQ)| is asked for.
template <int DT>
__global__ void __launch_bounds__(kThreads)
g9_zero_tests(const uint16_t* __restrict__ X, int64_t T, int64_t I, int64_t ld, const float* __restrict__ t,
              const float* __restrict__ a, const float* __restrict__ b, float qmaxf, float half_bound,
              uint16_t* __restrict__ out, unsigned long long* __restrict__ counts, int only_cq) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    unsigned int n_removed = 0, n_pt = 0, n_cq = 0;
    if (idx < T * I) {
        const int64_t i = idx / I, j = idx % I;
        const uint16_t bits16 = X[i * ld + j];
        const float x = cvt16<DT>(bits16);
        const float s = __fmul_rn(a[i], b[j]);
        n_cq = exact_at_most(x, s, 0.5f);
        if (!only_cq) {
            const bool gone = exact_at_most(x, s, half_bound);
            n_removed = gone;
            n_pt = exact_at_most(x, __fdiv_rn(t[i], qmaxf), 0.5f);
            out[idx] = gone ? static_cast<uint16_t>(0) : bits16;
        }
    }
    if (only_cq) {
        cta_count_add(n_cq, counts);
    } else {
        cta_count_add(n_removed, counts);
        __syncthreads();
        cta_count_add(n_pt, counts + 1);
        __syncthreads();
        cta_count_add(n_cq, counts + 2);
    }
}

// ============================================================================ host side
static ZeroBand band_of(float h) {
    if (h >= 9.5367431640625e-07f && h <= 1048576.0f)                 // [2^-20, 2^20]
        return ZeroBand{h * (1.0f - 1.52587890625e-05f), h * (1.0f + 1.52587890625e-05f)};
    return ZeroBand{-1.0f, INFINITY};
}

template <typename... KArgs, typename... Args>
static void launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = tuning_no_pdl() ? 0 : 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

struct ZeroArgs {
    const void* X; int64_t T; int64_t I; int64_t ld;
    const float *t, *a, *ra, *b, *rb;
    float qmaxf, half_bound;
    void* out; unsigned long long* counts;
};

template <int DT, bool WRITE, bool DUAL, bool SAME>
static void launch_k9(const Plan& p, const ZeroArgs& z, cudaStream_t st) {
    auto kern = k9_zero_tests<DT, WRITE, DUAL, SAME>;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, p.W, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    int64_t y = static_cast<int64_t>(sm_count()) * per_sm / p.nstrips;
    if (y > p.ngroups) y = p.ngroups;
    if (y > 65535) y = 65535;
    if (y < 1) y = 1;
    launch_after(kern, dim3(p.nstrips, static_cast<unsigned>(y)), dim3(p.W), st, static_cast<const uint4*>(z.X), z.T, p.I8,
                 z.ld / 8, z.t, z.a, z.ra, z.b, z.rb, z.qmaxf, z.half_bound, band_of(z.half_bound), band_of(0.5f),
                 static_cast<uint4*>(z.out), z.counts);
}

template <int DT>
static void launch_zero_tests(const Plan& p, const ZeroArgs& z, bool only_cq, bool fast, cudaStream_t st) {
    if (fast) {
        if (only_cq) launch_k9<DT, false, false, true>(p, z, st);
        else if (z.half_bound == 0.5f) launch_k9<DT, true, true, true>(p, z, st);
        else launch_k9<DT, true, true, false>(p, z, st);
    } else {
        const int64_t n = z.T * z.I;
        const unsigned blocks = static_cast<unsigned>((n + kThreads - 1) / kThreads);
        g9_zero_tests<DT><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(z.X), z.T, z.I, z.ld, z.t, z.a, z.b,
                                                       z.qmaxf, z.half_bound, static_cast<uint16_t*>(z.out), z.counts,
                                                       only_cq ? 1 : 0);
    }
}

static bool is_aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }

static ZeroArgs zero_args(const Plan& p, void* workspace, const void* X, int64_t T, int64_t I, int64_t ld, const float* t,
                          int bits, float half_bound, void* out, unsigned long long* counts) {
    char* ws = static_cast<char*>(workspace);
    return ZeroArgs{X, T, I, ld, t,
                    reinterpret_cast<const float*>(ws + p.off_a), reinterpret_cast<const float*>(ws + p.off_ra),
                    reinterpret_cast<const float*>(ws + p.off_b), reinterpret_cast<const float*>(ws + p.off_rb),
                    static_cast<float>((1 << (bits - 1)) - 1), half_bound, out, counts};
}

// vectors of 8 columns are indexed with 32-bit integers in the tiled kernel
static bool fast_shape(const Plan& p, const void* X, int64_t T, int64_t I, int64_t ld) {
    return is_aligned(X, 16) && (I % 8) == 0 && (ld % 8) == 0 && T * static_cast<int64_t>(p.I8) < (int64_t(1) << 31);
}

}  // namespace cq

extern "C" {

int cq_kernel_count_x(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                      const float* t, const float* c, unsigned long long* count,
                      void* workspace, size_t workspace_bytes, void* stream) {
    using namespace cq;
    int rc = check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (!(alpha >= 0.0 && alpha <= 1.0)) return CQ_ERR_ALPHA;
    if (count == nullptr) return CQ_ERR_NULL;
    if (!is_aligned(count, 8)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0 || I == 0)
        return cudaMemsetAsync(count, 0, sizeof(unsigned long long), st) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    if (t == nullptr || c == nullptr) return CQ_ERR_NULL;
    if (!is_aligned(t, 4) || !is_aligned(c, 4)) return CQ_ERR_ALIGN;
    rc = scales_from_vectors(T, I, t, c, alpha, bits, workspace, workspace_bytes, count, st);
    if (rc != CQ_OK) return rc;
    const Plan p = make_plan(T, I);
    const ZeroArgs z = zero_args(p, workspace, X, T, I, ld, t, bits, 0.5f, nullptr, count);
    const bool fast = fast_shape(p, X, T, I, ld);
    if (dtype == CQ_F16) launch_zero_tests<CQ_F16>(p, z, true, fast, st);
    else launch_zero_tests<CQ_BF16>(p, z, true, fast, st);
    return launch_status();
}

int cq_remove_kernel(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                     float bound_scale, void* out, unsigned long long* counts,
                     void* workspace, size_t workspace_bytes, void* stream) {
    using namespace cq;
    int rc = check_matrix(X, dtype, T, I, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (!(alpha >= 0.0 && alpha <= 1.0)) return CQ_ERR_ALPHA;
    if (!(bound_scale >= 0.0f)) return CQ_ERR_SHAPE;
    if (counts == nullptr) return CQ_ERR_NULL;
    if (!is_aligned(counts, 8)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T > 0 && I > 0) {
        if (out == nullptr) return CQ_ERR_NULL;
        if (!is_aligned(out, 2)) return CQ_ERR_ALIGN;
    }
    if (cudaMemsetAsync(counts, 0, 3 * sizeof(unsigned long long), st) != cudaSuccess) return CQ_ERR_CUDA;
    if (T == 0 || I == 0) return CQ_OK;
    // absmax pass and scale vectors into the workspace (no outputs requested: the quantize pass is skipped)
    rc = quantize_act_impl(X, dtype, T, I, ld, alpha, bits, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                           nullptr, nullptr, dtype, nullptr, workspace, workspace_bytes, st);
    if (rc != CQ_OK) return rc;
    const Plan p = make_plan(T, I);
    const float* t_dev = reinterpret_cast<const float*>(static_cast<char*>(workspace) + p.off_t);
    const ZeroArgs z = zero_args(p, workspace, X, T, I, ld, t_dev, bits, 0.5f * bound_scale, out, counts);
    const bool fast = fast_shape(p, X, T, I, ld) && is_aligned(out, 16);
    if (dtype == CQ_F16) launch_zero_tests<CQ_F16>(p, z, false, fast, st);
    else launch_zero_tests<CQ_BF16>(p, z, false, fast, st);
    return launch_status();
}

}  // extern "C"
