// Group-wise weight quantization (Section 3, "Background": the weight matrix is reshaped to
// (elements / g) x g and quantized per row, g = 128 in the paper's W4A8-g128 runs) for sm_100a.
//
// One thread owns one 8-element vector; the g/8 consecutive lanes that hold a group reduce its
// absolute maximum with shuffles, so the matrix is read from HBM exactly once and nothing is staged.
#include "cq_common.cuh"
#include "cq_host.h"

namespace cq {

#ifndef CQ_K7_VEC
#define CQ_K7_VEC 4
#endif
#ifndef CQ_K7_MIN_CTAS
#define CQ_K7_MIN_CTAS 1
#endif
constexpr int kVecPerThread = CQ_K7_VEC;

// LANES = g / 8 (a power of two <= 32).  Groups never straddle a stored row (C % g == 0).
template <int DT, int BITS, int DEQ, bool CODES, int LANES>
__global__ void __launch_bounds__(kThreads, CQ_K7_MIN_CTAS)
k7_weight_groups(const uint4* __restrict__ W, int64_t nvec, int C8, int64_t ld8,
                 void* __restrict__ codes, float* __restrict__ scale, void* __restrict__ deq,
                 unsigned long long* __restrict__ zero_count) {
    constexpr float qmaxf = static_cast<float>((1 << (BITS - 1)) - 1);
    const int lane = threadIdx.x & 31;
    const int64_t base = (static_cast<int64_t>(blockIdx.x) * kVecPerThread) * kThreads + threadIdx.x;
    const bool contiguous = ld8 == C8;
    uint4 w[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int64_t idx = base + static_cast<int64_t>(k) * kThreads;
        w[k] = make_uint4(0, 0, 0, 0);
        if (idx < nvec) w[k] = ld_stream(contiguous ? W + idx : W + (idx / C8) * ld8 + (idx % C8));
    }
    // group maxima: the LANES consecutive lanes of a group all end up with it
    uint32_t m16[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const uint32_t mm = max_u16x2(max_u16x2(w[k].x & 0x7FFF7FFFu, w[k].y & 0x7FFF7FFFu),
                                      max_u16x2(w[k].z & 0x7FFF7FFFu, w[k].w & 0x7FFF7FFFu));
        m16[k] = max(mm & 0xFFFFu, mm >> 16);
#pragma unroll
        for (int off = LANES / 2; off > 0; off >>= 1) m16[k] = max(m16[k], __shfl_xor_sync(0xFFFFFFFFu, m16[k], off));
    }
    // scales d = fl32(max / qmax) and their reciprocals.  A warp holds 32 / LANES groups per vector; with
    // LANES >= 4 the groups of all its vectors get one lane each, so the warp divides once, not once per vector.
    float dk[kVecPerThread], rdk[kVecPerThread];
    if constexpr (LANES >= kVecPerThread) {
        constexpr int G = 32 / LANES;
        uint32_t mine = DT == CQ_BF16 ? 0x3F80u : 0x3C00u;        // lanes without a group divide 1.0
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            const uint32_t mk = __shfl_sync(0xFFFFFFFFu, m16[k], (lane % G) * LANES);
            if (lane / G == k) mine = mk;
        }
        const float d = __fdiv_rn(cvt16<DT>(static_cast<uint16_t>(mine)), qmaxf);
        const float rd = guarded_rcp(d);                             // correctly rounded: the quotients below rely on it
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            dk[k] = __shfl_sync(0xFFFFFFFFu, d, k * G + lane / LANES);
            rdk[k] = __shfl_sync(0xFFFFFFFFu, rd, k * G + lane / LANES);
        }
    } else {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
            dk[k] = __fdiv_rn(cvt16<DT>(static_cast<uint16_t>(m16[k])), qmaxf);
            rdk[k] = guarded_rcp(dk[k]);
        }
    }
    // codes of all the thread's vectors: exact quotients in straight-line packed arithmetic; a group whose scale is
    // outside the range that covers (NaN marker in rdk) sends the thread's vectors to the defining sequence instead
    float2 y[kVecPerThread][4];
    bool scales_ok = true;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) scales_ok = scales_ok && rdk[k] == rdk[k];
    if (scales_ok) {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) exact_codes_uniform_row8<DT>(w[k], dk[k], rdk[k], y[k]);
    } else {
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) exact_codes_uniform_slow<DT, BITS>(w[k], dk[k], y[k]);
    }
    unsigned int zeros = 0;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const int64_t idx = base + static_cast<int64_t>(k) * kThreads;
        const float d = dk[k];
        if (idx < nvec) {
            if (scale != nullptr && (idx % LANES) == 0) scale[idx / LANES] = d;
            const float2 (&y2)[4] = y[k];
            if constexpr (BITS == 8) {
                const uint32_t c0 = pack_int8x4(y2[0].x, y2[0].y, y2[1].x, y2[1].y);
                const uint32_t c1 = pack_int8x4(y2[2].x, y2[2].y, y2[3].x, y2[3].y);
                zeros += zero_bytes(c0) + zero_bytes(c1);
                if constexpr (CODES) st_stream(reinterpret_cast<uint2*>(codes) + idx, make_uint2(c0, c1));
            } else {
                const uint32_t c0 = pack_int4x8(y2);
                zeros += zero_nibbles(c0);
                if constexpr (CODES) st_stream(reinterpret_cast<uint32_t*>(codes) + idx, c0);
            }
            if constexpr (DEQ != 0) {
                const float2 d2s = make_float2(d, d), nm2 = make_float2(-kMagic, -kMagic);
                float2 dq[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) dq[e] = __fmul2_rn(__fadd2_rn(y2[e], nm2), d2s);
                if constexpr (DEQ == 1) {
                    uint4 o;
                    o.x = pack16x2<DT>(dq[0].x, dq[0].y); o.y = pack16x2<DT>(dq[1].x, dq[1].y);
                    o.z = pack16x2<DT>(dq[2].x, dq[2].y); o.w = pack16x2<DT>(dq[3].x, dq[3].y);
                    st_stream(reinterpret_cast<uint4*>(deq) + idx, o);
                } else {
                    float4* o = reinterpret_cast<float4*>(deq) + idx * 2;
                    st_stream(o, make_float4(dq[0].x, dq[0].y, dq[1].x, dq[1].y));
                    st_stream(o + 1, make_float4(dq[2].x, dq[2].y, dq[3].x, dq[3].y));
                }
            }
        }
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
}

// Any group size / shape / alignment: one thread per group, scalar accesses, two reads of the group.
template <int DT>
__global__ void __launch_bounds__(kThreads)
g7_weight_groups(const uint16_t* __restrict__ W, int64_t ngroups, int64_t C, int64_t ld, int64_t g, int bits,
                 void* __restrict__ codes, float* __restrict__ scale, void* __restrict__ deq, int deq_dt,
                 unsigned long long* __restrict__ zero_count) {
    const float qmaxf = static_cast<float>((1 << (bits - 1)) - 1);
    const int64_t grp = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    unsigned int zeros = 0;
    if (grp < ngroups) {
        const int64_t per_row = C / g;
        const int64_t row = grp / per_row, col0 = (grp % per_row) * g;
        const uint16_t* p = W + row * ld + col0;
        uint32_t m = 0;
        for (int64_t k = 0; k < g; ++k) m = max(m, static_cast<uint32_t>(p[k] & 0x7FFFu));
        const float d = __fdiv_rn(cvt16<DT>(static_cast<uint16_t>(m)), qmaxf);
        if (scale != nullptr) scale[grp] = d;
        const int64_t out0 = row * C + col0;
        int prev = 0;
        for (int64_t k = 0; k < g; ++k) {
            const int q = code_as_int(quant_exact(cvt16<DT>(p[k]), d, qmaxf));
            zeros += (q == 0);
            const float dq = __fmul_rn(static_cast<float>(q), d);
            if (deq != nullptr) {
                if (deq_dt == CQ_F32) reinterpret_cast<float*>(deq)[out0 + k] = dq;
                else reinterpret_cast<uint16_t*>(deq)[out0 + k] = pack16<DT>(dq);
            }
            if (codes != nullptr) {
                if (bits == 8) reinterpret_cast<int8_t*>(codes)[out0 + k] = static_cast<int8_t>(q);
                else if (k & 1) reinterpret_cast<uint8_t*>(codes)[(out0 + k) / 2] = static_cast<uint8_t>((prev & 0xF) | ((q & 0xF) << 4));
            }
            prev = q;
        }
    }
    if (zero_count != nullptr) cta_count_add(zeros, zero_count);
}

static bool aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }

template <int DT, int BITS, int DEQ, bool CODES>
static void launch_k7_lanes(int lanes, unsigned blocks, cudaStream_t st, const uint4* W, int64_t nvec, int C8, int64_t ld8,
                            void* codes, float* scale, void* deq, unsigned long long* zc) {
    switch (lanes) {
        case 1: k7_weight_groups<DT, BITS, DEQ, CODES, 1><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
        case 2: k7_weight_groups<DT, BITS, DEQ, CODES, 2><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
        case 4: k7_weight_groups<DT, BITS, DEQ, CODES, 4><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
        case 8: k7_weight_groups<DT, BITS, DEQ, CODES, 8><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
        case 16: k7_weight_groups<DT, BITS, DEQ, CODES, 16><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
        default: k7_weight_groups<DT, BITS, DEQ, CODES, 32><<<blocks, kThreads, 0, st>>>(W, nvec, C8, ld8, codes, scale, deq, zc); break;
    }
}

template <int DT, int BITS>
static void launch_k7(int deq_mode, bool has_codes, int lanes, unsigned blocks, cudaStream_t st, const uint4* W, int64_t nvec,
                      int C8, int64_t ld8, void* codes, float* scale, void* deq, unsigned long long* zc) {
    if (has_codes) {
        if (deq_mode == 0) launch_k7_lanes<DT, BITS, 0, true>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
        else if (deq_mode == 1) launch_k7_lanes<DT, BITS, 1, true>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
        else launch_k7_lanes<DT, BITS, 2, true>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
    } else {
        if (deq_mode == 0) launch_k7_lanes<DT, BITS, 0, false>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
        else if (deq_mode == 1) launch_k7_lanes<DT, BITS, 1, false>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
        else launch_k7_lanes<DT, BITS, 2, false>(lanes, blocks, st, W, nvec, C8, ld8, codes, scale, deq, zc);
    }
}

}  // namespace cq

extern "C" int cq_quantize_weight_groupwise(const void* W, int dtype, int64_t R, int64_t C, int64_t ld, int64_t group,
                                            int bits, void* codes, float* scale, void* deq, int deq_dtype,
                                            unsigned long long* zero_count, void* stream) {
    using namespace cq;
    int rc = check_matrix(W, dtype, R, C, ld);
    if (rc != CQ_OK) return rc;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (group <= 0 || (C % group) != 0) return CQ_ERR_SHAPE;
    if (deq != nullptr && deq_dtype != dtype && deq_dtype != CQ_F32) return CQ_ERR_DTYPE;
    if (bits == 4 && (group % 2) != 0) return CQ_ERR_ALIGN;
    if (deq != nullptr && !aligned(deq, deq_dtype == CQ_F32 ? 4 : 2)) return CQ_ERR_ALIGN;
    if (scale != nullptr && !aligned(scale, 4)) return CQ_ERR_ALIGN;
    if (zero_count != nullptr && !aligned(zero_count, 8)) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (zero_count != nullptr && cudaMemsetAsync(zero_count, 0, sizeof(unsigned long long), st) != cudaSuccess)
        return CQ_ERR_CUDA;
    if (R == 0 || C == 0) return CQ_OK;
    const bool pow2 = (group & (group - 1)) == 0;
    const bool fast = pow2 && group >= 8 && group <= 256 && aligned(W, 16) && (ld % 8 == 0) &&
                      (codes == nullptr || aligned(codes, bits == 8 ? 8 : 4)) && (deq == nullptr || aligned(deq, 16));
    if (fast) {
        const int C8 = static_cast<int>(C / 8);
        const int64_t nvec = R * C8;
        const int lanes = static_cast<int>(group / 8);
        const int64_t per_block = static_cast<int64_t>(kThreads) * kVecPerThread;
        const unsigned blocks = static_cast<unsigned>((nvec + per_block - 1) / per_block);
        const int deq_mode = deq == nullptr ? 0 : (deq_dtype == CQ_F32 ? 2 : 1);
        const uint4* Wv = static_cast<const uint4*>(W);
        const bool hc = codes != nullptr;
        if (dtype == CQ_F16) {
            if (bits == 8) launch_k7<CQ_F16, 8>(deq_mode, hc, lanes, blocks, st, Wv, nvec, C8, ld / 8, codes, scale, deq, zero_count);
            else launch_k7<CQ_F16, 4>(deq_mode, hc, lanes, blocks, st, Wv, nvec, C8, ld / 8, codes, scale, deq, zero_count);
        } else {
            if (bits == 8) launch_k7<CQ_BF16, 8>(deq_mode, hc, lanes, blocks, st, Wv, nvec, C8, ld / 8, codes, scale, deq, zero_count);
            else launch_k7<CQ_BF16, 4>(deq_mode, hc, lanes, blocks, st, Wv, nvec, C8, ld / 8, codes, scale, deq, zero_count);
        }
    } else {
        const int64_t ngroups = R * (C / group);
        const unsigned blocks = static_cast<unsigned>((ngroups + kThreads - 1) / kThreads);
        if (dtype == CQ_F16)
            g7_weight_groups<CQ_F16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(W), ngroups, C, ld, group, bits,
                                                                 codes, scale, deq, deq_dtype, zero_count);
        else
            g7_weight_groups<CQ_BF16><<<blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(W), ngroups, C, ld, group, bits,
                                                                  codes, scale, deq, deq_dtype, zero_count);
    }
    return cudaGetLastError() == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}
