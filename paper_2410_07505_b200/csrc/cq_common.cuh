// Device-side helpers shared by the CrossQuant kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "cq.h"

namespace cq {

// Adding 1.5 * 2^23 to a float of magnitude < 2^22 leaves round-half-even(v) in the low mantissa
// bits: bits(v + kMagic) == kMagicBits + rint(v) as a two's-complement integer.
constexpr float kMagic = 12582912.0f;
constexpr uint32_t kMagicBits = 0x4B400000u;
// 1/2 - 2^-16: a candidate code q is accepted without the IEEE division when |x - q s| < s * kHalfMinus.
constexpr float kHalfMinus = 0.4999847412109375f;

constexpr float kScaleLoTie = 2.350988701644575e-38f;    // 2^-125: s / 2 is a normal number, hence exact, from here up
constexpr int kThreads = 256;      // largest CTA of the tiled kernels

__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint4 ld_nc(const uint4* p) { return __ldg(p); }

// streaming (evict-first) accesses for data touched once
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint2* p, uint2 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint32_t* p, uint32_t v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

// ---- asynchronous bulk copies into shared memory (TMA unit, no tensor map) --------------------
// One thread announces the byte count on an mbarrier and issues the copies; everybody waits on the
// barrier's phase parity.  Source, destination and size are multiples of 16 bytes.  No multicast.
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Bounded wait: gives up after ~2^22 polls (seconds) and reports it, so a kernel can never hang on it.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t polls = 0; polls < (1u << 22); ++polls) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// ---- 16-bit formats ------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ float2 unpack16x2(uint32_t w) {
    if constexpr (DT == CQ_BF16) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    } else {
        __half2 h = *reinterpret_cast<__half2*>(&w);
        return __half22float2(h);
    }
}

template <int DT>
__device__ __forceinline__ float cvt16(uint16_t bits) {
    if constexpr (DT == CQ_BF16) {
        return __uint_as_float(static_cast<uint32_t>(bits) << 16);
    } else {
        return __half2float(__ushort_as_half(bits));
    }
}

__device__ __forceinline__ float cvt16_rt(uint16_t bits, int dt) {
    return dt == CQ_BF16 ? cvt16<CQ_BF16>(bits) : cvt16<CQ_F16>(bits);
}

// two floats -> packed 16-bit pair, round to nearest even
template <int DT>
__device__ __forceinline__ uint32_t pack16x2(float lo, float hi) {
    if constexpr (DT == CQ_BF16) {
        __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&p);
    } else {
        __half2 p = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&p);
    }
}

template <int DT>
__device__ __forceinline__ uint16_t pack16(float v) {
    if constexpr (DT == CQ_BF16) {
        return __bfloat16_as_ushort(__float2bfloat16_rn(v));
    } else {
        return __half_as_ushort(__float2half_rn(v));
    }
}

// ---- one element ---------------------------------------------------------------------------
// Candidate code from a reciprocal product; returns kMagic + q.  `ok` tells whether q is proven
// equal to round-half-even(fl32(x / s)): with z = x/s and |z| <= 128, fl32(z) lies within 2^-17 of
// z, so |z - q| < 1/2 - 2^-16 (checked on the exactly computed residual x - q s) forces the IEEE
// quotient to round to q as well.  Any NaN or infinity in the candidate makes the test fail.
__device__ __forceinline__ float quant_candidate(float x, float s, float r, float qmaxf, bool& ok, float& e) {
    float v = __fmul_rn(x, r);
    v = fminf(fmaxf(v, -qmaxf), qmaxf);
    float y = __fadd_rn(v, kMagic);
    float qf = __fadd_rn(y, -kMagic);
    e = __fmaf_rn(-qf, s, x);
    ok = fabsf(e) < __fmul_rn(s, kHalfMinus);
    return y;
}

// The defining sequence: IEEE division, round half to even, clamp.  Returns kMagic + q.
static __device__ __noinline__ float quant_exact(float x, float s, float qmaxf) {
    if (s == 0.0f) return kMagic;
    float u = __fdiv_rn(x, s);
    float q = rintf(u);
    q = fminf(fmaxf(q, -qmaxf), qmaxf);
    return __fadd_rn(q, kMagic);        // (-0) + kMagic == kMagic
}

// For a candidate that failed its test.  First the exact tie: if the candidate's residual e = x - q s is
// exactly +-s/2, then x / s = q +- 1/2 (for q != 0 up to a relative 2^-24 of the 1/2, which fl32 absorbs),
// the IEEE quotient is that half-integer and round-half-even picks the even one of q and q +- 1.  16-bit
// inputs make such ties common (a weight row whose maximum has the mantissa 2 * 127 puts a quarter of
// its elements on one), so they are settled without the division.  Everything else takes quant_exact.
// y = kMagic + q with a finite q; s / 2 is exact for s >= 2^-125.
static __device__ __noinline__ float quant_settle(float x, float s, float qmaxf, float y, float e) {
    if (s >= kScaleLoTie && fabsf(e) == __fmul_rn(s, 0.5f)) {
        float qf = __fadd_rn(y, -kMagic);
        if ((__float_as_uint(y) & 1u) != 0u) qf = __fadd_rn(qf, e > 0.0f ? 1.0f : -1.0f);   // q odd: step to the even side
        qf = fminf(fmaxf(qf, -qmaxf), qmaxf);
        return __fadd_rn(qf, kMagic);
    }
    if (s == 0.0f) return kMagic;
    float u = __fdiv_rn(x, s);
    float q = rintf(u);
    q = fminf(fmaxf(q, -qmaxf), qmaxf);
    return __fadd_rn(q, kMagic);
}

// ---- eight elements of one row -------------------------------------------------------------
// Scale factors outside [2^-40, 2^40] get a NaN "reciprocal"; callers test for it (x != x) and send
// such rows / columns to the defining sequence.  A factor of exactly zero means the whole row or
// column is zero (t_i = 0 or c_j = 0), so its elements are zeros and any finite reciprocal gives the
// right candidate, code 0: it gets 0.
constexpr float kScaleLo = 9.094947017729282e-13f;     // 2^-40
constexpr float kScaleHi = 1.099511627776e12f;         // 2^40
__device__ __forceinline__ float guarded_rcp(float f) {
    if (f == 0.0f) return 0.0f;
    return (f >= kScaleLo && f <= kScaleHi) ? __fdiv_rn(1.0f, f) : __int_as_float(0x7FC00000);
}
// ---- scale factors -------------------------------------------------------------------------
//   a_i = fl32(pow(t_i, alpha) / qmax), b_j = fl32(pow(c_j, 1 - alpha)) in fp64, with alpha in {0, 1}
//   special-cased so that they reduce exactly to per-column / per-token quantization, plus the
//   reciprocals the quantize pass uses for its candidate codes.
__device__ __forceinline__ void row_scale_of(float ti, double alpha, int qmax, float& ai, float& rai) {
    if (alpha == 1.0) ai = __fdiv_rn(ti, static_cast<float>(qmax));
    else if (alpha == 0.0) ai = 1.0f;
    else ai = static_cast<float>(pow(static_cast<double>(ti), alpha) / static_cast<double>(qmax));
    rai = guarded_rcp(ai);
}

__device__ __forceinline__ void col_scale_of(float cj, double alpha, int qmax, float& bj, float& rbj) {
    if (alpha == 1.0) bj = 1.0f;
    else if (alpha == 0.0) bj = __fdiv_rn(cj, static_cast<float>(qmax));
    else bj = static_cast<float>(pow(static_cast<double>(cj), 1.0 - alpha));
    rbj = guarded_rcp(bj);
}

// The candidate q = round-half-even(v), v = x * (1/a_i) * (1/b_j), is accepted when |v - q| < 1/2 - 2^-14.
// With a_i, b_j in [2^-40, 2^40] they, their reciprocals, s_ij = fl32(a_i b_j) and the reciprocal product
// are all normal numbers, so v differs from z = x / s_ij by less than 5 * 2^-24 |z| < 3.8e-5 (five roundings,
// |z| <= 127.0001); hence |z - q| < 1/2 - 6.1e-5 + 3.8e-5 and the IEEE quotient fl32(z), which lies within
// 2^-17 = 0.8e-5 of z, stays 1.5e-5 short of the rounding boundary and rounds to the same q.
// |x| <= min(t_i, c_j) gives |z| <= qmax (1 + 2^-22), which keeps q within [-qmax, qmax].
constexpr float kAcceptBelow = 0.49993896484375f;       // 1/2 - 2^-14

// Packed fp32x2 arithmetic (bit-identical to the scalar IEEE operations, half the issue slots).
// y2[k] = kMagic + q and q2[k] = q for elements 2k, 2k+1; element e has the scale a * b2[e] (per-element scales:
// the activation path; rows under one scale take exact_codes_uniform_row8 below instead).
// `trusted`: none of the reciprocals involved is the NaN marker (a NaN would not
// survive the max below, so it has to be tested where the reciprocals are loaded).
template <int DT, int BITS, bool LEAN = false>
__device__ __forceinline__ void quantize_row8(const uint4& w, float a, float ra, const float2 (&b2)[4],
                                              const float2 (&rb2)[4], bool trusted,
                                              float2 (&y2)[4], float2 (&q2)[4]) {
    constexpr float qmaxf = static_cast<float>((1 << (BITS - 1)) - 1);
    const float2 ra2 = make_float2(ra, ra);
    const float2 m2 = make_float2(kMagic, kMagic), nm2 = make_float2(-kMagic, -kMagic);
    const float2 neg1 = make_float2(-1.0f, -1.0f);
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
    float worst = 0.0f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = unpack16x2<DT>(words[k]);
        const float2 r = __fmul2_rn(ra2, rb2[k]);
        const float2 v = __fmul2_rn(x, r);                    // x / s, approximately
        y2[k] = __fadd2_rn(v, m2);
        q2[k] = __fadd2_rn(y2[k], nm2);                       // round-half-even(v), exact
        const float2 f = __ffma2_rn(q2[k], neg1, v);          // v - q, exact
        worst = fmaxf(fmaxf(worst, fabsf(f.x)), fabsf(f.y));
    }
    if (!(trusted && worst < kAcceptBelow)) {
        // Some element is too close to a rounding boundary (or a scale factor is extreme) for the cheap
        // test to decide.  The pairs that hold such an element are found again; their elements are
        // re-examined with the exact residual, and the undecided ones are settled as exact ties or take
        // the defining sequence (IEEE division, round half to even, clamp).  LEAN re-examines all eight
        // elements instead: no fast result has to survive this region, which saves the registers a
        // kernel that lives on occupancy needs.
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 x = unpack16x2<DT>(words[k]);
            const float2 r = __fmul2_rn(ra2, rb2[k]);
            if constexpr (!LEAN) {
                const float2 f = __ffma2_rn(q2[k], neg1, __fmul2_rn(x, r));
                if (trusted && fmaxf(fabsf(f.x), fabsf(f.y)) < kAcceptBelow) continue;
            }
            const float xs[2] = {x.x, x.y};
            const float bs[2] = {b2[k].x, b2[k].y};
            const float rs[2] = {r.x, r.y};
            float ys[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float sh = __fmul_rn(a, bs[h]);
                bool good;
                float e;
                ys[h] = quant_candidate(xs[h], sh, rs[h], qmaxf, good, e);
                if (!good) ys[h] = quant_settle(xs[h], sh, qmaxf, ys[h], e);
            }
            y2[k] = make_float2(ys[0], ys[1]);
            q2[k] = __fadd2_rn(y2[k], nm2);
        }
    }
}

// ---- eight elements under ONE scale (a weight row or group): exact quotients, no test ----------
// With one scale s per row the correctly rounded reciprocal rs = fl32(1 / s) costs one division per row, and
// then   q0 = fl32(x rs),  r = x - q0 s  (one FMA, exact),  u = fl32(q0 + r rs)  (one FMA)
// is the correctly rounded quotient fl32(x / s) itself (the classical residual-corrected division; for this use
// it is not taken on faith: tests/test_exact_quotient_cpu.py checks it against the IEEE division for every pair
// of mantissas of up to 11 bits, i.e. every fp16 / bf16 element against every scale fl32(max / qmax) a 16-bit
// maximum can give, which is exhaustive because binary scaling changes nothing while all values stay normal).
// The magic-number add then rounds u half to even exactly as the defining sequence does, ties included, so no
// candidate has to be examined afterwards.  Valid for s in [2^-40, 2^40] (guarded_rcp marks anything else with a
// NaN, and the caller takes exact_codes_uniform_slow); s == 0 gives rs = 0 and codes 0.  No clamp is needed:
// |x| <= max and s >= (max / qmax)(1 - 2^-24) keep |u| <= qmax (1 + 2^-23), which rounds to qmax.
template <int DT>
__device__ __forceinline__ void exact_codes_uniform_row8(const uint4& w, float s, float rs, float2 (&y2)[4]) {
    const float2 rs2 = make_float2(rs, rs), ns2 = make_float2(-s, -s), m2 = make_float2(kMagic, kMagic);
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = unpack16x2<DT>(words[k]);
        const float2 q0 = __fmul2_rn(x, rs2);
        const float2 r = __ffma2_rn(q0, ns2, x);
        y2[k] = __fadd2_rn(__ffma2_rn(r, rs2, q0), m2);
    }
}

// The same codes by the defining sequence, element by element (scales outside [2^-40, 2^40]).  Only scalars cross
// the out-of-line calls, so the arrays of the caller stay in registers.
template <int DT, int BITS>
__device__ __forceinline__ void exact_codes_uniform_slow(const uint4& w, float s, float2 (&y2)[4]) {
    constexpr float qmaxf = static_cast<float>((1 << (BITS - 1)) - 1);
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = unpack16x2<DT>(words[k]);
        const float y0 = quant_exact(x.x, s, qmaxf), y1 = quant_exact(x.y, s, qmaxf);
        y2[k] = make_float2(y0, y1);
    }
}

__device__ __forceinline__ float code_as_float(float y) { return __fadd_rn(y, -kMagic); }
__device__ __forceinline__ int code_as_int(float y) {
    return static_cast<int>(__float_as_uint(y)) - static_cast<int>(kMagicBits);
}

// four codes (low bytes of four magic-biased floats) -> one word of int8
__device__ __forceinline__ uint32_t pack_int8x4(float y0, float y1, float y2, float y3) {
    uint32_t p01 = __byte_perm(__float_as_uint(y0), __float_as_uint(y1), 0x0040);
    uint32_t p23 = __byte_perm(__float_as_uint(y2), __float_as_uint(y3), 0x0040);
    return __byte_perm(p01, p23, 0x5410);
}

// eight codes -> one word of two's-complement nibbles, element e in bits [4e, 4e+4): each pair of
// magic-biased floats gives one byte (low nibble | high nibble << 4), the four bytes are then gathered
__device__ __forceinline__ uint32_t pack_int4x8(const float2 (&y2)[4]) {
    uint32_t t[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) t[k] = (__float_as_uint(y2[k].x) & 0xFu) + __float_as_uint(y2[k].y) * 16u;
    const uint32_t p01 = __byte_perm(t[0], t[1], 0x0040);
    const uint32_t p23 = __byte_perm(t[2], t[3], 0x0040);
    return __byte_perm(p01, p23, 0x5410);
}

__device__ __forceinline__ int zero_bytes(uint32_t w) {
    uint32_t t = (w & 0x7F7F7F7Fu) + 0x7F7F7F7Fu;
    t = ~(t | w | 0x7F7F7F7Fu);
    return __popc(t);
}

__device__ __forceinline__ int zero_nibbles(uint32_t w) {
    uint32_t nz = (w | (w >> 1) | (w >> 2) | (w >> 3)) & 0x11111111u;
    return 8 - __popc(nz);
}

// CTA-wide sum of per-thread counts, one atomic per CTA
__device__ __forceinline__ void cta_count_add(unsigned int cnt, unsigned long long* dst) {
    __shared__ unsigned int s_cnt[kThreads / 32];
    unsigned int w = __reduce_add_sync(0xFFFFFFFFu, cnt);
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s_cnt[warp] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long sum = 0;
        int nw = (blockDim.x + 31) >> 5;
        for (int k = 0; k < nw; ++k) sum += s_cnt[k];
        if (sum) atomicAdd(dst, sum);
    }
}

}  // namespace cq
