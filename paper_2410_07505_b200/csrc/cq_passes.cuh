// Device code shared by the activation kernels: the scale-vector step on the partial maxima of the absmax pass
// and the per-row quantize / pack / dequantize / count step (CrossQuant equation, Section 4.2).
#pragma once

#include "cq_common.cuh"

namespace cq {

// ---------------------------------------------------------------------------- scale vectors from partial maxima
// One block of the scale-vector step.  Blocks [0, col_ctas): 64 columns each; thread (vx, grp) reduces every 32nd
// partial row of vector column vx (8 vector columns x 32 groups per block, so even ~300 partial rows cost a thread
// only ~10 independent loads), shared memory combines the 32 groups, then one thread per column forms
// c_j, b_j = fl32(pow(c_j, 1 - alpha)) and 1 / b_j.  Blocks [col_ctas, ...): one thread per row: t_i, a_i, 1 / a_i.
// `vb` is the block's number; every thread of the CTA calls this with the same vb (it synchronises the CTA).
constexpr int kK2Cols = 8;       // vector columns per block
constexpr int kK2Groups = 32;    // partial-row groups per block
constexpr int kK2Batch = 12;     // partial rows a thread loads at once

template <int DT>
__device__ __forceinline__ void scales_block(int vb, int64_t T, int64_t I, int I8, int nstrips, int Y, int col_ctas,
                                             const uint16_t* __restrict__ rowpart, const uint4* __restrict__ colpart,
                                             double alpha, int qmax,
                                             float* __restrict__ t_out, float* __restrict__ c_out,
                                             float* __restrict__ a, float* __restrict__ b,
                                             float* __restrict__ ra, float* __restrict__ rb,
                                             uint4 (&s_part)[kK2Groups][kK2Cols]) {
    const int tid = threadIdx.x;
    if (vb < col_ctas) {
        const int nthreads = blockDim.x;
        // (vx, grp) pairs are dealt to the threads in rounds, so blocks narrower than 256 threads cover all 256 pairs
        for (int pr = tid; pr < kK2Cols * kK2Groups; pr += nthreads) {
            const int vx = pr & (kK2Cols - 1), grp = pr / kK2Cols;
            const int vcol = vb * kK2Cols + vx;
            uint4 m = make_uint4(0, 0, 0, 0);
            if (vcol < I8) {
                // all of a thread's loads (up to kK2Batch per round) are issued before the first is used: the partial
                // rows come from L2, and a chain of dependent rounds is what this latency-bound step must not have
                for (int y0 = grp; y0 < Y; y0 += kK2Groups * kK2Batch) {
                    uint4 w[kK2Batch];
#pragma unroll
                    for (int i = 0; i < kK2Batch; ++i) {
                        const int y = y0 + i * kK2Groups;
                        w[i] = y < Y ? __ldcg(colpart + static_cast<int64_t>(y) * I8 + vcol) : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int i = 0; i < kK2Batch; ++i) {
                        m.x = max_u16x2(m.x, w[i].x); m.y = max_u16x2(m.y, w[i].y);
                        m.z = max_u16x2(m.z, w[i].z); m.w = max_u16x2(m.w, w[i].w);
                    }
                }
            }
            s_part[grp][vx] = m;
        }
        __syncthreads();
        for (int col = tid; col < kK2Cols * 8; col += nthreads) {
            const int64_t j = static_cast<int64_t>(vb) * (kK2Cols * 8) + col;
            if (j < I) {
                const uint16_t* sp = reinterpret_cast<const uint16_t*>(&s_part[0][0]);
                uint32_t mx = 0;
#pragma unroll
                for (int k = 0; k < kK2Groups; ++k) mx = max(mx, static_cast<uint32_t>(sp[k * (kK2Cols * 8) + col]));
                const float cj = cvt16<DT>(static_cast<uint16_t>(mx));
                if (c_out != nullptr) c_out[j] = cj;
                float bj, rbj;
                col_scale_of(cj, alpha, qmax, bj, rbj);
                b[j] = bj;
                rb[j] = rbj;
            }
        }
        __syncthreads();                 // s_part may be refilled by the caller's next block
    } else {
        for (int r = tid; r < kThreads; r += blockDim.x) {            // kThreads rows per block, whatever the CTA's width
            const int64_t i = static_cast<int64_t>(vb - col_ctas) * kThreads + r;
            if (i < T) {
                uint32_t m = 0;
                for (int sx = 0; sx < nstrips; ++sx) m = max(m, static_cast<uint32_t>(__ldcg(rowpart + i * nstrips + sx)));
                const float ti = cvt16<DT>(static_cast<uint16_t>(m));
                if (t_out != nullptr) t_out[i] = ti;
                float ai, rai;
                row_scale_of(ti, alpha, qmax, ai, rai);
                a[i] = ai;
                ra[i] = rai;
            }
        }
    }
}

// ---------------------------------------------------------------------------- one row of eight elements
// The scale factors of a thread's eight columns, read once per kernel.
struct ColumnScales {
    float2 b2[4], rb2[4];
    bool trusted;          // none of the eight reciprocals is the NaN marker of an extreme scale factor
};

__device__ __forceinline__ ColumnScales load_column_scales(const float* __restrict__ b, const float* __restrict__ rb, int vv) {
    ColumnScales cs;
    const float4* bp = reinterpret_cast<const float4*>(b) + static_cast<int64_t>(vv) * 2;
    const float4* rp = reinterpret_cast<const float4*>(rb) + static_cast<int64_t>(vv) * 2;
    const float4 b0 = __ldcg(bp), b1 = __ldcg(bp + 1), q0 = __ldcg(rp), q1 = __ldcg(rp + 1);
    cs.b2[0] = make_float2(b0.x, b0.y); cs.b2[1] = make_float2(b0.z, b0.w);
    cs.b2[2] = make_float2(b1.x, b1.y); cs.b2[3] = make_float2(b1.z, b1.w);
    cs.rb2[0] = make_float2(q0.x, q0.y); cs.rb2[1] = make_float2(q0.z, q0.w);
    cs.rb2[2] = make_float2(q1.x, q1.y); cs.rb2[3] = make_float2(q1.z, q1.w);
    cs.trusted = ((cs.rb2[0].x + cs.rb2[0].y) + (cs.rb2[1].x + cs.rb2[1].y)) +
                 ((cs.rb2[2].x + cs.rb2[2].y) + (cs.rb2[3].x + cs.rb2[3].y)) < INFINITY;
    return cs;
}

// Quantize the eight elements `x` of row scale (au, 1 / au), pack and store the codes, store the dequantized values,
// count the zero codes.  `vec` indexes 8-element vectors of the outputs; only `active` lanes store.
// DEQ: 0 none, 1 same 16-bit type as X, 2 fp32.
template <int DT, int BITS, int DEQ, bool CODES, bool COUNT, bool LEAN = false>
__device__ __forceinline__ void quantize_store_row8(const uint4& x, float au, float rau, const ColumnScales& cs, bool active,
                                                    int64_t vec, void* __restrict__ codes, void* __restrict__ deq,
                                                    unsigned int& zeros) {
    float2 y2[4], q2[4];
    quantize_row8<DT, BITS, LEAN>(x, au, rau, cs.b2, cs.rb2, cs.trusted && rau == rau, y2, q2);
    if constexpr (BITS == 8) {
        const uint32_t c0 = pack_int8x4(y2[0].x, y2[0].y, y2[1].x, y2[1].y);
        const uint32_t c1 = pack_int8x4(y2[2].x, y2[2].y, y2[3].x, y2[3].y);
        if constexpr (COUNT) zeros += zero_bytes(c0) + zero_bytes(c1);
        if constexpr (CODES) { if (active) st_stream(reinterpret_cast<uint2*>(codes) + vec, make_uint2(c0, c1)); }
    } else {
        const uint32_t c0 = pack_int4x8(y2);
        if constexpr (COUNT) zeros += zero_nibbles(c0);
        if constexpr (CODES) { if (active) st_stream(reinterpret_cast<uint32_t*>(codes) + vec, c0); }
    }
    if constexpr (DEQ != 0) {
        const float2 a2 = make_float2(au, au);
        float2 d2[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) d2[k] = __fmul2_rn(q2[k], __fmul2_rn(a2, cs.b2[k]));
        if constexpr (DEQ == 1) {
            uint4 o;
            o.x = pack16x2<DT>(d2[0].x, d2[0].y); o.y = pack16x2<DT>(d2[1].x, d2[1].y);
            o.z = pack16x2<DT>(d2[2].x, d2[2].y); o.w = pack16x2<DT>(d2[3].x, d2[3].y);
            if (active) st_stream(reinterpret_cast<uint4*>(deq) + vec, o);
        } else {
            float4* o = reinterpret_cast<float4*>(deq) + vec * 2;
            if (active) {
                st_stream(o, make_float4(d2[0].x, d2[0].y, d2[1].x, d2[1].y));
                st_stream(o + 1, make_float4(d2[2].x, d2[2].y, d2[3].x, d2[3].y));
            }
        }
    }
}

}  // namespace cq
