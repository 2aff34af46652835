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

int scales_from_vectors(int64_t T, int64_t I, const float* t, const float* c, double alpha, int bits,
                        void* workspace, size_t ws_bytes, unsigned long long* to_zero, cudaStream_t st);
int sm_count();
int launch_status();
int diag_stage_fault(unsigned int* fault_host);   // flag of the staged diagnostics kernels
int weight_stage_fault(unsigned int* fault_host); // flag of the bulk-copy weight kernel
bool tuning_no_stage();   // staged (bulk-copy) variants switched off through cq_set_tuning
bool tuning_no_pdl();     // programmatic dependent launch switched off through cq_set_tuning

}  // namespace cq
