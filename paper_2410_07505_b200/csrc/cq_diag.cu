// Diagnostics of the quantization kernel (Definition 1) that need no codes: the "Remove Kernel"
// operator (Figure 1, Appendix B) with the per-token and CrossQuant kernel sizes from one pass, and
// |K(CQ)| straight from X (Section 4.2).  Both only ask, per element, whether |fl32(x / s)| <= h.
#include <math.h>

#include "cq_common.cuh"
#include "cq_host.h"

#ifndef CQ_K9_MIN_CTAS
#define CQ_K9_MIN_CTAS 4
#endif

namespace cq {

// Membership in the quantization kernel itself (h = 1/2) needs no division and no tolerance: for a 16-bit element x
// and a normal fp32 scale s,
//     |fl32(x / s)| <= 1/2   <=>   |x| <= s / 2.
// (<=: the quotient of x <= s/2 is at most 1/2 and rounding is monotone.  =>: x and s/2 are both fp32 numbers, so
// x > s/2 means x >= s/2 + ulp(s/2), i.e. x/s >= 1/2 + ulp(s/2)/s > 1/2 + 2^-25, which rounds to a float above 1/2;
// the tie 1/2 + 2^-25 itself would need x - s/2 = s 2^-25 < ulp(s/2), which no pair of floats has.)  And since |x| is
// a 16-bit float, |x| <= s/2 is an integer comparison of its 15-bit pattern with the largest 16-bit float not above
// s/2 (the fp32 value rounded toward zero to 16 bits).  So the CrossQuant kernel (s_ij = fl32(a_i b_j), its half formed
// exactly as fl32((a_i / 2) b_j)) and the per-token kernel (one threshold pattern per row from fl32(t_i / qmax) / 2) are
// decided on the packed 16-bit words: no unpacking, no band, nothing undecided.  Rows or columns whose scale factors
// lie outside [2^-40, 2^40] (where s / 2 might not be exact) are marked and take the IEEE quotients.
//
// A bound other than 1/2 (bound_scale != 1) has no such identity.  There, with a_i, b_j in [2^-40, 2^40],
// p = fl32(x * (1/b_j)) against the row's threshold m_i = fl32(h a_i) compares like |z| = |x / s_ij| against h
// up to a relative error of 4 * 2^-24 (the roundings of 1/b_j, p, m_i and s_ij = fl32(a_i b_j)), and fl32(z)
// lies within 2^-24 |z| of z; so for h in [2^-20, 2^20] (nothing near h can be subnormal) and
// e_i = fl32(2^-18 h a_i), six times that error,
//     |p| - m_i <= -e_i  =>  |fl32(z)| < h,        |p| - m_i >= e_i  =>  |fl32(z)| > h,
// and only elements with | |p| - m_i | < e_i need the quotient itself.  A zero scale gives (m, e) = (inf, 0):
// everything in the row is removed; a scale outside [2^-40, 2^40], or h outside [2^-20, 2^20], gives (0, inf): every
// element takes the quotient.  ZeroFactors: what a_i is multiplied with to get m_i and e_i.
struct ZeroFactors { float m, e; };

static __device__ __noinline__ bool exact_at_most(float x, float s, float h) {
    if (s == 0.0f) return true;                       // the code of a zero scale is 0 by definition
    return fabsf(__fdiv_rn(x, s)) <= h;
}

// Two stages of four rows and four or more resident CTAs per SM: measured against rings of 3, 4 and 6 stages with fewer
// CTAs (count-only pass 58.4 -> 52.2 us, Remove Kernel 125.4 -> 124.8 us on 4096x28672; more CTAs hide the barrier per group).
#ifndef CQ_K9_RING
#define CQ_K9_RING 2
#endif
constexpr int kRing = CQ_K9_RING;                  // stages of four rows per CTA
__device__ unsigned int g_diag_stage_fault = 0;    // set if a bounded wait on a stage ever gave up

// 0xFFFF in the low / high half of the result where d_lo / d_hi is negative (sign bit set), else 0:
// byte permute in its sign-replicating mode on the top bytes of the two values.
__device__ __forceinline__ uint32_t negative_halves(float d_lo, float d_hi) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, 0xFFBB;" : "=r"(r) : "r"(__float_as_uint(d_lo)), "r"(__float_as_uint(d_hi)));
    return r;
}

// The largest 16-bit values (fp16 or bf16 patterns) not above two non-negative floats, packed low | high << 16:
// conversion with rounding toward zero (it saturates at the largest finite fp16); for bf16 that is the upper half
// of the binary32 pattern.
template <int DT>
__device__ __forceinline__ uint32_t floor16x2(float lo, float hi) {
    if constexpr (DT == CQ_BF16) {
        return __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x7632);
    } else {
        uint32_t r;
        asm("cvt.rz.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
}

// 0xFFFF in each half of the result whose bit 15 is set in w, else 0 (byte permute replicating the sign of bytes 1 and 3).
__device__ __forceinline__ uint32_t sign_halves(uint32_t w) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %1, 0xBB99;" : "=r"(r) : "r"(w));
    return r;
}

// Same strip / resident-CTA layout as the quantize pass, rows staged the same way: groups of four rows
// arrive in a ring of shared-memory stages through asynchronous bulk copies issued by thread 0 (no
// tensor map, no multicast; waits bounded, a wait that gives up raises g_diag_stage_fault).  Rows are
// walked from the last full group backwards, the ragged last group first by CTA y = 0.
//   WRITE: out = x, or +0 where |fl32(x / s_ij)| <= half_bound         (counts[0] += removed)
//   DUAL : counts[1] += |K| of per-token quantization (scale fl32(t_i / qmax)), counts[2] += |K(CQ)|
//   SAME : half_bound == 1/2, so "removed" and "in K(CQ)" are one test
//   !WRITE && !DUAL: counts[0] += |K(CQ)| only
// The comparisons are subtractions whose sign bits are gathered into per-row bit masks (one bit pair
// per element pair): the masks give the output mask and the counts (popc); one chained comparison per
// element collects whether any difference is inside the band, i.e. whether the row needs the quotients.
template <int DT, bool WRITE, bool DUAL, bool SAME>
__global__ void __launch_bounds__(kThreads, CQ_K9_MIN_CTAS)
k9_zero_tests(const uint4* __restrict__ X, int64_t T, int I8, int64_t ld8,
              const float* __restrict__ t, const float* __restrict__ a,
              const float* __restrict__ b, const float* __restrict__ rb, float qmaxf,
              float half_bound, ZeroFactors zf,
              uint4* __restrict__ out, unsigned long long* __restrict__ counts) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int v = blockIdx.x * blockDim.x + tid;
    const bool active = v < I8;
    const bool warp_active = (v - lane) < I8;
    const int vv = active ? v : I8 - 1;
    const int64_t nfull = T >> 2;
    const int64_t Y = gridDim.y;
    unsigned int n_removed = 0, n_pt = 0, n_cq = 0;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ uint64_t s_full[kRing];
    __shared__ int s_abort;                      // a wait on a row copy gave up: the CTA stops issuing and leaves

    // Ring geometry, barriers and the first copies: X is an input of the call, not a product of the preceding
    // kernel (the scale vectors), so the ring fills while that kernel is still running.
    uint4* stage = reinterpret_cast<uint4*>(s_dyn);                   // [kRing][4 rows][blockDim.x]
    const int Wv = blockDim.x;
    const int strip0 = blockIdx.x * Wv;
    const uint32_t seg_bytes = static_cast<uint32_t>(min(Wv, I8 - strip0)) * 16u;
    const int64_t first = blockIdx.y;
    const int64_t mine = first < nfull ? (nfull - first + Y - 1) / Y : 0;          // groups of this CTA
    auto group_at = [&](int64_t k) { return nfull - 1 - (first + k * Y); };
    auto issue = [&](int64_t k) {                                     // thread 0 only
        if (k >= mine) return;
        const int st = static_cast<int>(k % kRing);
        const uint4* src = X + (group_at(k) << 2) * ld8 + strip0;
        mbar_expect_tx(&s_full[st], 4u * seg_bytes);
#pragma unroll
        for (int u = 0; u < 4; ++u) bulk_load(stage + (st * 4 + u) * Wv, src + u * ld8, seg_bytes, &s_full[st]);
    };
    if (tid == 0) {
        s_abort = 0;
#pragma unroll
        for (int st = 0; st < kRing; ++st) mbar_init(&s_full[st], 1);
        mbar_init_fence();
        for (int k = 0; k < kRing - 1; ++k) issue(k);
    }
    __syncthreads();

    // the scale vectors come from the preceding kernel of the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");

    {
        float2 rb2[4];
        {
            const float4* rp = reinterpret_cast<const float4*>(rb) + static_cast<int64_t>(vv) * 2;
            const float4 q0 = __ldg(rp), q1 = __ldg(rp + 1);
            rb2[0] = make_float2(q0.x, q0.y); rb2[1] = make_float2(q0.z, q0.w);
            rb2[2] = make_float2(q1.x, q1.y); rb2[3] = make_float2(q1.z, q1.w);
        }
        // a NaN among the column reciprocals (extreme b_j) sends all of this thread's vectors to the quotients
        const bool cols_trusted = ((rb2[0].x + rb2[0].y) + (rb2[1].x + rb2[1].y)) +
                                  ((rb2[2].x + rb2[2].y) + (rb2[3].x + rb2[3].y)) < INFINITY;
        const uint4* xp = X + vv;

        // column scale factors of this thread's eight columns
        float2 b2[4];
        {
            const float4* bp = reinterpret_cast<const float4*>(b) + static_cast<int64_t>(vv) * 2;
            const float4 b0 = __ldg(bp), b1 = __ldg(bp + 1);
            b2[0] = make_float2(b0.x, b0.y); b2[1] = make_float2(b0.z, b0.w);
            b2[2] = make_float2(b1.x, b1.y); b2[3] = make_float2(b1.z, b1.w);
        }

        // thr[]: a_i / 2 (NaN: a_i outside the range), per-token threshold pattern in both halves (all ones: outside
        // the range), (m, e) of CrossQuant for the caller's bound
        auto do_row = [&](const uint4& slot, const float (&thr)[4], int64_t row, int vec) {
            const uint32_t words[4] = {slot.x, slot.y, slot.z, slot.w};
            const float2 ah2 = make_float2(thr[0], thr[0]);
            const uint32_t tpt2 = __float_as_uint(thr[1]);
            uint32_t m_c = 0, m_p = 0, m_g = 0;
            float near_g = INFINITY;          // smallest distance of any element from the caller's bound (band test, once per row)
            uint32_t ow[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // |x| as a 15-bit pattern against the largest 16-bit value <= s / 2: bit 15 of each half of
                // (threshold + 0x8000 - magnitude) is set exactly where the element is in the kernel
                const uint32_t mag = words[k] & 0x7FFF7FFFu;
                const float2 th = __fmul2_rn(ah2, b2[k]);                     // s_ij / 2 (exact halving of fl32(a_i b_j))
                const uint32_t dc = floor16x2<DT>(th.x, th.y) + 0x80008000u - mag;
                m_c |= (dc & 0x80008000u) >> k;
                if constexpr (DUAL) m_p |= ((tpt2 + 0x80008000u - mag) & 0x80008000u) >> k;
                uint32_t gone;
                if constexpr (SAME) {
                    gone = sign_halves(dc);                                   // 0xFFFF in the halves whose bit 15 is set
                } else {
                    const uint32_t bit = 0x00010001u << k;
                    const float2 x = unpack16x2<DT>(words[k]);
                    const float2 p = __fmul2_rn(x, rb2[k]);
                    const float g0 = __fadd_rn(fabsf(p.x), -thr[2]), g1 = __fadd_rn(fabsf(p.y), -thr[2]);
                    near_g = fminf(near_g, fminf(fabsf(g0), fabsf(g1)));
                    gone = negative_halves(g0, g1);
                    m_g |= gone & bit;
                }
                ow[k] = words[k] & ~gone;
            }
            unsigned int r_cq = __popc(m_c), r_pt = __popc(m_p), r_rm = SAME ? r_cq : __popc(m_g);
            // rows and columns whose scale factors are outside [2^-40, 2^40] (markers), and for a scaled bound the
            // elements inside its band, go to the IEEE quotients
            bool undecided = !cols_trusted || !(thr[0] == thr[0]);
            if constexpr (DUAL) undecided |= tpt2 == 0xFFFFFFFFu;
            if constexpr (!SAME) undecided |= near_g < thr[3];
            if (undecided) {
                // Rare: some element sits within 2^-16 (relative) of a bound, or a scale factor is extreme.
                // The whole vector is decided again from the IEEE quotients.
                r_rm = r_pt = r_cq = 0;
                const float ai = __ldg(a + row);
                const float spt = DUAL ? __fdiv_rn(__ldg(t + row), qmaxf) : 0.0f;
                const float* bp = b + static_cast<int64_t>(vv) * 8;
#pragma unroll
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
        // Lane l holds threshold number l / 4 (order of thr[] above) of row l % 4 of the group.  The scale is
        // fetched one group ahead (load_scale) and turned into the threshold when its group comes up.
        constexpr int kKinds = SAME ? (DUAL ? 2 : 1) : 4;
        const int kind = lane >> 2;
        auto load_scale = [&](int64_t g) {
            if (kind >= kKinds) return 0.0f;
            const int64_t row = min((g << 2) + (lane & 3), T - 1);
            return kind == 1 ? __ldg(t + row) : __ldg(a + row);
        };
        auto threshold_of = [&](float raw) {
            const float nan = __int_as_float(0x7FC00000);
            if (kind == 0) {                                           // a_i / 2; a zero row has only zeros, which 0 admits
                if (raw == 0.0f) return 0.0f;
                return (raw >= kScaleLo && raw <= kScaleHi) ? __fmul_rn(0.5f, raw) : nan;
            }
            if (kind == 1) {                                           // per-token: largest 16-bit value <= fl32(t_i / qmax) / 2
                if (raw == 0.0f) return 0.0f;
                const float spt = __fdiv_rn(raw, qmaxf);
                if (!(spt >= kScaleLo && spt <= kScaleHi)) return __uint_as_float(0xFFFFFFFFu);
                const float h = __fmul_rn(0.5f, spt);
                return __uint_as_float(floor16x2<DT>(h, h));
            }
            const bool is_mid = kind == 2;                             // (m, e) of the caller's bound, as before
            if (raw == 0.0f) return is_mid ? INFINITY : 0.0f;
            if (raw >= kScaleLo && raw <= kScaleHi) return __fmul_rn(is_mid ? zf.m : zf.e, raw);
            return is_mid ? 0.0f : INFINITY;
        };
        auto row_thresholds = [&](float tv, int u, float (&thr)[4]) {
#pragma unroll
            for (int k = 0; k < 4; ++k) thr[k] = k < kKinds ? __shfl_sync(0xFFFFFFFFu, tv, 4 * k + u) : 0.0f;
        };

        if ((T & 3) != 0 && blockIdx.y == 0 && warp_active) {            // ragged last group
            const float tv = threshold_of(load_scale(nfull));
            for (int u = 0; u < static_cast<int>(T & 3); ++u) {
                const int64_t row = (nfull << 2) + u;
                const uint4 slot = ld_stream(xp + row * ld8);
                float thr[4];
                row_thresholds(tv, u, thr);
                do_row(slot, thr, row, static_cast<int>(row * I8 + vv));
            }
        }

        float raw = mine > 0 ? load_scale(group_at(0)) : 0.0f;
        int64_t k = 0;
        for (; k < mine; ++k) {
            const int64_t g = group_at(k);
            const float tv = threshold_of(raw);
            if (k + 1 < mine) raw = load_scale(group_at(k + 1));
            __syncthreads();                                              // everybody is done with group k-1: its stage is free
            if (s_abort) break;
            if (tid == 0) issue(k + kRing - 1);
            const int st = static_cast<int>(k % kRing);
            if (!mbar_wait(&s_full[st], static_cast<uint32_t>((k / kRing) & 1))) {
                atomicExch(&g_diag_stage_fault, 1u);
                s_abort = 1;                                              // seen by everybody after the next barrier
            }
            if (warp_active) {
                const int vec = static_cast<int>((g << 2) * I8 + vv);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint4 cur = stage[(st * 4 + u) * Wv + tid];
                    float thr[4];
                    row_thresholds(tv, u, thr);
                    do_row(cur, thr, (g << 2) + u, vec + u * I8);
                }
            }
        }
        if (k < mine && tid == 0) {
            // abandoned: nothing more is issued; one more bounded wait for each copy still in flight
            for (int64_t kk = k; kk < min(mine, k + kRing - 1); ++kk)
                mbar_wait(&s_full[kk % kRing], static_cast<uint32_t>((kk / kRing) & 1));
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
static ZeroFactors factors_of(float h) {
    ZeroFactors z{};
    if (h >= 9.5367431640625e-07f && h <= 1048576.0f) {              // [2^-20, 2^20]
        z.m = h;
        z.e = h * 3.814697265625e-06f;                                // 2^-18
    } else {
        z.m = 0.0f;
        z.e = INFINITY;
    }
    return z;
}

template <typename... KArgs, typename... Args>
static void launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = tuning_no_pdl() ? 0 : 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

struct ZeroArgs {
    const void* X; int64_t T; int64_t I; int64_t ld;
    const float *t, *a, *b, *rb;
    float qmaxf, half_bound;
    void* out; unsigned long long* counts;
};

template <int DT, bool WRITE, bool DUAL, bool SAME>
static bool launch_k9(const Plan& p, const ZeroArgs& z, cudaStream_t st) {
    auto kern = k9_zero_tests<DT, WRITE, DUAL, SAME>;
    const size_t smem = static_cast<size_t>(kRing) * 4 * p.W * 16;
    static thread_local LaunchMemo memo;
    const int per_sm = resident_ctas(kern, p.W, smem, static_cast<size_t>(kRing) * 4 * kThreads * 16, memo);
    if (per_sm < 1) return false;
    int64_t y = static_cast<int64_t>(sm_count()) * per_sm / p.nstrips;
    if (y > p.ngroups) y = p.ngroups;
    if (y > 65535) y = 65535;
    if (y < 1) y = 1;
    launch_after(kern, dim3(p.nstrips, static_cast<unsigned>(y)), dim3(p.W), smem, st, static_cast<const uint4*>(z.X), z.T,
                 p.I8, z.ld / 8, z.t, z.a, z.b, z.rb, z.qmaxf, z.half_bound, factors_of(z.half_bound),
                 static_cast<uint4*>(z.out), z.counts);
    return true;
}

template <int DT>
static void launch_zero_tests(const Plan& p, const ZeroArgs& z, bool only_cq, bool fast, cudaStream_t st) {
    if (fast) {
        if (only_cq) fast = launch_k9<DT, false, false, true>(p, z, st);
        else if (z.half_bound == 0.5f) fast = launch_k9<DT, true, true, true>(p, z, st);
        else fast = launch_k9<DT, true, true, false>(p, z, st);
    }
    if (!fast) {
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
                    reinterpret_cast<const float*>(ws + p.off_a), reinterpret_cast<const float*>(ws + p.off_b),
                    reinterpret_cast<const float*>(ws + p.off_rb),
                    static_cast<float>((1 << (bits - 1)) - 1), half_bound, out, counts};
}

// vectors of 8 columns are indexed with 32-bit integers in the tiled kernel
static bool fast_shape(const Plan& p, const void* X, int64_t T, int64_t I, int64_t ld) {
    return is_aligned(X, 16) && (I % 8) == 0 && (ld % 8) == 0 && T * static_cast<int64_t>(p.I8) < (int64_t(1) << 31);
}

int diag_stage_fault(unsigned int* fault_host) {
    return cudaMemcpyFromSymbol(fault_host, g_diag_stage_fault, sizeof(unsigned int)) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
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
