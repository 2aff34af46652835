// Diagnostics the paper derives from the absmax vectors (Table 1 of Section 4.2) for sm_100a.
#include "cq_common.cuh"
#include "cq_host.h"

namespace cq {

constexpr int kPairRows = 64;     // rows per CTA tile of the pair count

// counts[0] += #{(i,j) : c_j >= t_i},  counts[1] += #{(i,j) : s_ij / 2 < fl32(t_i / qmax) / 2}.
// One thread per column, a tile of rows per CTA staged in shared memory.
__global__ void __launch_bounds__(kThreads)
k8_case_indicators(const float* __restrict__ t, const float* __restrict__ c, const float* __restrict__ a,
                   const float* __restrict__ b, int64_t T, int64_t I, float qmaxf,
                   unsigned long long* __restrict__ counts) {
    __shared__ float s_t[kPairRows], s_a[kPairRows], s_half_pt[kPairRows];
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kPairRows;
    const int rows = static_cast<int>(min(static_cast<int64_t>(kPairRows), T - r0));
    if (threadIdx.x < rows) {
        const float ti = t[r0 + threadIdx.x];
        s_t[threadIdx.x] = ti;
        s_a[threadIdx.x] = a[r0 + threadIdx.x];
        s_half_pt[threadIdx.x] = __fmul_rn(0.5f, __fdiv_rn(ti, qmaxf));
    }
    __syncthreads();
    unsigned int n_case2 = 0, n_smaller = 0;
    if (j < I) {
        const float cj = c[j], bj = b[j];
        for (int r = 0; r < rows; ++r) {
            n_case2 += (cj >= s_t[r]);
            n_smaller += (__fmul_rn(0.5f, __fmul_rn(s_a[r], bj)) < s_half_pt[r]);
        }
    }
    cta_count_add(n_case2, counts);
    __syncthreads();
    cta_count_add(n_smaller, counts + 1);
}

}  // namespace cq

extern "C" int cq_case_indicators(const float* t, const float* c, const float* row_scale, const float* col_scale,
                                  int64_t T, int64_t I, int bits, unsigned long long* counts, void* stream) {
    using namespace cq;
    if (T < 0 || I < 0 || T > (int64_t(1) << 31) || I > (int64_t(1) << 31)) return CQ_ERR_SHAPE;
    if (bits != 4 && bits != 8) return CQ_ERR_BITS;
    if (counts == nullptr) return CQ_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(counts) % 8) != 0) return CQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(counts, 0, 2 * sizeof(unsigned long long), st) != cudaSuccess) return CQ_ERR_CUDA;
    if (T == 0 || I == 0) return CQ_OK;
    if (t == nullptr || c == nullptr || row_scale == nullptr || col_scale == nullptr) return CQ_ERR_NULL;
    for (const float* f : {t, c, row_scale, col_scale})
        if ((reinterpret_cast<uintptr_t>(f) % 4) != 0) return CQ_ERR_ALIGN;
    const dim3 grid(static_cast<unsigned>((I + kThreads - 1) / kThreads), static_cast<unsigned>((T + kPairRows - 1) / kPairRows));
    if (grid.y > 65535) return CQ_ERR_SHAPE;
    k8_case_indicators<<<grid, kThreads, 0, st>>>(t, c, row_scale, col_scale, T, I,
                                                  static_cast<float>((1 << (bits - 1)) - 1), counts);
    return cudaGetLastError() == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}
