// Host-side declarations shared by the translation units of libcq.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace cq {

// Tiling of a T x I matrix and the carving of the caller's workspace.
struct Plan {
    int I8;        // vectors of 8 columns per row
    int W;         // threads per CTA = vectors per column strip
    int nstrips;   // column strips
    int64_t ngroups;  // groups of 4 rows
    int ycap;      // most CTAs per strip the absmax pass may use (rows of the column-partial buffer)
    size_t off_t, off_c, off_a, off_b, off_ra, off_rb, off_rowpart, off_colpart, total;
};

Plan make_plan(int64_t T, int64_t I);
int check_matrix(const void* X, int dtype, int64_t T, int64_t I, int64_t ld);
int quantize_act_impl(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                      const float* t_given, const float* c_given,
                      float* t, float* c, float* row_scale, float* col_scale,
                      void* codes, void* deq, int deq_dtype, unsigned long long* zero_count,
                      void* workspace, size_t ws_bytes, cudaStream_t st);

// The single-launch path for small matrices (cq_small.cu).  Returns false, having launched nothing, when
// the shape is not eligible.  All pointers except codes / deq / zero_count are non-null device pointers.
struct SmallArgs {
    const void* X; int dtype; int64_t T; int I8; int64_t ld8; int W; int nstrips; double alpha; int bits;
    float *t, *c, *a, *b;
    void* codes; void* deq; int deq_mode; unsigned long long* zero_count;
};
bool launch_small(const SmallArgs& s, cudaStream_t st);
int small_stage_fault(unsigned int* fault_host);   // flag of its tile copy

int scales_from_vectors(int64_t T, int64_t I, const float* t, const float* c, double alpha, int bits,
                        void* workspace, size_t ws_bytes, unsigned long long* to_zero, cudaStream_t st);
int sm_count();
int launch_status();
int diag_stage_fault(unsigned int* fault_host);   // flag of the staged diagnostics kernels
int weight_stage_fault(unsigned int* fault_host); // flag of the bulk-copy weight kernel
bool tuning_no_stage();   // staged (bulk-copy) variants switched off through cq_set_tuning
bool tuning_no_pdl();     // programmatic dependent launch switched off through cq_set_tuning

// What the runtime answered for one kernel at (device, block size, dynamic shared memory): resident CTAs
// per SM, after raising the kernel's dynamic shared-memory limit to `smem_limit` (the most any launch of
// that kernel asks for, so the limit never shrinks whatever the order of shapes and threads).
// One memo per launch site (a thread_local static there), so repeated calls of one shape ask only once.
struct LaunchMemo { int dev = -1; int block = 0; size_t smem = 0; int per_sm = 0; };

template <typename Kernel>
inline int resident_ctas(Kernel kern, int block, size_t smem, size_t smem_limit, LaunchMemo& memo) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (memo.dev == dev && memo.block == block && memo.smem == smem) return memo.per_sm;
    int per_sm = 0;
    if (smem_limit > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_limit)) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, block, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        return 0;
    }
    memo = LaunchMemo{dev, block, smem, per_sm};
    return per_sm;
}

}  // namespace cq
