/*
 * cq.h -- C ABI of the CrossQuant activation cross-quantizer for NVIDIA B200 (sm_100a).
 *
 * The operations follow the paper "CrossQuant" (arXiv 2410.07505): Eq. 1 (per-token
 * quantization), Eq. 2 (per-channel weight quantization), Definition 1 (the quantization
 * kernel: the set of elements whose code is 0) and the CrossQuant equation of Section 4.2,
 *
 *     CQ(X_ij) = round( X_ij / D_ij ),   D_ij = t_i^alpha * c_j^(1-alpha) / (2^(N-1) - 1),
 *     t_i = max_j |X_ij| ,  c_j = max_i |X_ij| ,  0 <= alpha <= 1.
 *
 * Conventions that hold for every function unless it says otherwise
 *   - Matrices are row-major, 16-bit (IEEE binary16 or bfloat16), `ld` = distance between rows
 *     in elements (ld >= columns).  Sizes are 64-bit.  Inputs are expected to be finite.
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library allocates
 *     nothing, frees nothing and keeps no per-call state.  The only state it has is process-wide
 *     and for measurement: the knobs of cq_set_tuning and the event pair of cq_set_timing_events
 *     (both thread-safe, neither changes a result), the sticky health flag read by cq_stage_fault,
 *     and the fixed scratch array of cq_quantize_act_noalloc.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All work is
 *     enqueued on it; no call synchronises; scalar results are written to device memory.
 *   - The return value is a cq_status.  On any status other than CQ_OK no kernel was launched
 *     by that call (CQ_ERR_CUDA excepted: it reports a launch the driver refused).
 *   - Arithmetic (identical for every alpha, bit width and shape):
 *         qmax = 2^(bits-1) - 1
 *         alpha == 1 : a_i = fl32(t_i / qmax), b_j = 1        (Eq. 1 exactly)
 *         alpha == 0 : a_i = 1, b_j = fl32(c_j / qmax)        (per-column quantization)
 *         else       : a_i = fl32(pow_fp64(t_i, alpha) / qmax), b_j = fl32(pow_fp64(c_j, 1-alpha))
 *         s_ij = fl32(a_i * b_j);  s_ij == 0 -> code 0, dequantized 0
 *         code = round-half-even(fl32(x_ij / s_ij)) clamped to [-qmax, qmax]
 *         xhat = fl32(code * s_ij), rounded once more (nearest-even) when a 16-bit output is asked
 *   - INT4 storage: two codes per byte; element (i, 2k) in the low nibble and (i, 2k+1) in the
 *     high nibble of byte i*(I/2)+k; two's-complement nibbles in [-7, 7].  I must be even.
 *   - Fast kernels need 16-byte aligned matrix pointers and I, ld multiples of 8; any other
 *     shape or alignment (2-byte aligned at least) is served by slower general kernels with
 *     identical results.
 */
#ifndef CQ_H_
#define CQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CQ_OK = 0,
    CQ_ERR_NULL = 1,       /* a required pointer is NULL                                   */
    CQ_ERR_SHAPE = 2,      /* negative size, ld < columns, or a size beyond what is supported */
    CQ_ERR_DTYPE = 3,      /* dtype not valid for that argument                            */
    CQ_ERR_BITS = 4,       /* bits not in {4, 8}                                           */
    CQ_ERR_ALPHA = 5,      /* alpha outside [0, 1] or NaN                                  */
    CQ_ERR_ALIGN = 6,      /* pointer not aligned to its element size, or odd I with INT4  */
    CQ_ERR_WORKSPACE = 7,  /* workspace NULL, misaligned (256 B) or smaller than required  */
    CQ_ERR_CUDA = 8,       /* the CUDA runtime reported an error at launch                 */
    CQ_ERR_TOO_LARGE = 9   /* the matrix needs more scratch than the built-in buffer of
                              cq_quantize_act_noalloc holds                                */
} cq_status;

typedef enum { CQ_F16 = 0, CQ_BF16 = 1, CQ_F32 = 2 /* outputs only */ } cq_dtype;

int cq_version(void);
const char* cq_status_string(int status);

/* t_i = max_j |X_ij| (Eq. 1).  X: device [T x ld] 16-bit.  t: device float[T], overwritten. */
int cq_absmax_rows(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t, void* stream);

/* c_j = max_i |X_ij| (CrossQuant equation, Section 4.2).  c: device float[I], overwritten. */
int cq_absmax_cols(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, float* c, void* stream);

/* Both vectors from a single read of X. */
int cq_absmax_rows_cols(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                        float* t, float* c, void* stream);

/* Bytes of device workspace cq_quantize_act / cq_kernel_count_x need for a T x I matrix
 * (scale vectors, their reciprocals and the partial maxima of the first pass). */
size_t cq_workspace_bytes(int64_t T, int64_t I);

/*
 * The CrossQuant activation quantizer (Section 4.2): absmax vectors, scale vectors, codes,
 * dequantized matrix and the size of the quantization kernel (Definition 1), in three launches
 * (decode-sized matrices: one launch of one thread-block cluster, same results).
 *   X          in   device [T x ld], dtype CQ_F16 or CQ_BF16
 *   alpha      in   exponent of the row maxima, [0, 1]; 1 = per-token (Eq. 1), 0 = per-column
 *   bits       in   8 or 4
 *   t, c       out  device float[T], float[I]; nullable
 *   row_scale  out  device float[T], a_i;  col_scale out device float[I], b_j; nullable
 *   codes      out  device int8[T*I] (bits = 8) or uint8[T*I/2] (bits = 4); nullable
 *   deq        out  device [T*I] of deq_dtype (X's dtype or CQ_F32); nullable
 *   zero_count out  device uint64, number of zero codes = |K(CQ)|; nullable
 *   workspace  in   device, 256-byte aligned, >= cq_workspace_bytes(T, I); contents undefined after
 * T == 0 or I == 0 is valid: zero_count = 0, and the vectors of the non-empty dimension are still written
 * (maxima over nothing are 0: t = 0 or c = 0, with the scale factors that follow from them), so that an empty
 * row block contributes zeros when the blocks' column maxima are combined.
 * The call only enqueues kernels (and at most two small device-to-device copies) on `stream`; after one
 * ordinary call per shape on a device (which settles the kernels' launch attributes) it can be captured
 * in a CUDA graph and replayed.
 */
int cq_quantize_act(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                    double alpha, int bits,
                    float* t, float* c, float* row_scale, float* col_scale,
                    void* codes, void* deq, int deq_dtype,
                    unsigned long long* zero_count,
                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * One matrix held in several row blocks (tokens split over GPUs, or X streamed through the device in
 * chunks): c_j of the CrossQuant equation (Section 4.2) is the maximum over ALL tokens, so the blocks'
 * column maxima have to be combined before any code is formed; t_i stays local to the block that holds
 * row i.  These two calls are the per-block steps; what moves the vector between GPUs (an all-reduce
 * with MAX) is the caller's.
 *
 * cq_vector_max: acc_j = max(acc_j, v_j) for j < n, device pointers, in place (acc and v may not overlap
 * unless equal).  Use it to keep a running c over chunks, or after gathering other blocks' vectors.
 *
 * cq_quantize_act_given: cq_quantize_act without its first pass, with t (float[T], this block's rows)
 * and c (float[I], the combined column maxima) supplied.  Requires t_i >= max_j |X_ij| and
 * c_j >= max_i |X_ij| for the block (true for maxima combined as above); elements that exceed either
 * bound get unspecified codes (nothing is checked, nothing faults).  Other arguments, outputs, workspace
 * and errors as for cq_quantize_act; zero_count counts this block only.
 */
int cq_vector_max(float* acc, const float* v, int64_t n, void* stream);
int cq_quantize_act_given(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                          double alpha, int bits, const float* t, const float* c,
                          float* row_scale, float* col_scale,
                          void* codes, void* deq, int deq_dtype,
                          unsigned long long* zero_count,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * cq_quantize_act for callers that cannot allocate device memory.  (The paper has no counterpart to
 * this function: it exists for deployment, not for the method.)
 *
 * Who needs it: a process that gave the whole GPU to one memory pool at start-up and has no allocator of
 * its own to ask; a plug-in on a latency-critical path where the host application forbids cudaMalloc
 * (which synchronises the device and may fail when memory is fragmented); any component whose device
 * memory budget was fixed before it was loaded.  Such a caller still owns X and every output buffer it
 * passes, but has nowhere to take the scratch space from that cq_quantize_act asks for.
 *
 * Here the scratch is a fixed array of CQ_NOALLOC_SCRATCH_BYTES (8 MiB) inside the library image: every
 * GPU on which the library is loaded holds that much until the process exits.  Arguments and results
 * are exactly those of cq_quantize_act without `workspace` / `workspace_bytes`.  The function calls no
 * cudaMalloc, cudaFree or other allocating routine, on any call.
 *
 *   - Limit: shapes with cq_workspace_bytes(T, I) > CQ_NOALLOC_SCRATCH_BYTES return CQ_ERR_TOO_LARGE and
 *     enqueue nothing.  (4096 x 28672 needs 4.5 MiB; every benchmark configuration fits.)
 *   - First call on a device: it looks up the array's address on the current device (one
 *     cudaGetSymbolAddress, remembered afterwards).  Make that first call with the right device current
 *     and before starting any stream capture.  Make it EARLY, too: the CUDA runtime may load the library's
 *     device code, and with it these 8 MiB, onto a GPU only when it is first needed there, so a process that
 *     has already handed the rest of the device's memory to its pool could see CQ_ERR_CUDA from the first
 *     call.  After that first call nothing more is ever taken (free device memory stays where it was).
 *   - All calls on a device share the one array and find the previous call's contents in it; nothing in
 *     it needs clearing between calls.  Two calls whose kernels may overlap on the GPU (different
 *     streams without an ordering between them) race on the array and give undefined results: keep
 *     calls on one device ordered, e.g. on one stream.
 */
#define CQ_NOALLOC_SCRATCH_BYTES (8u << 20)
int cq_quantize_act_noalloc(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                            double alpha, int bits,
                            float* t, float* c, float* row_scale, float* col_scale,
                            void* codes, void* deq, int deq_dtype,
                            unsigned long long* zero_count, void* stream);

/*
 * Same operation on HOST buffers: copies X to the device, runs cq_quantize_act and copies
 * every requested output back, all on `stream`.  Host pointers should be page-locked for the
 * copies to be asynchronous.  `device_scratch` (device, 256-byte aligned) must hold
 * cq_host_scratch_bytes(...) bytes.  Outputs are complete once `stream` has been synchronised
 * by the caller.  zero_count is a HOST uint64 here.
 */
size_t cq_host_scratch_bytes(int64_t T, int64_t I, int bits, int want_codes, int want_deq, int deq_dtype);
int cq_quantize_act_host(const void* X_host, int dtype, int64_t T, int64_t I, int64_t ld,
                         double alpha, int bits,
                         float* t_host, float* c_host, float* row_scale_host, float* col_scale_host,
                         void* codes_host, void* deq_host, int deq_dtype,
                         unsigned long long* zero_count_host,
                         void* device_scratch, size_t scratch_bytes, void* stream);

/* xhat_ij = fl32(code_ij * fl32(row_scale_i * col_scale_j)) from stored codes (the last step of
 * the Appendix B.1 listing).  out: device [T*I] of out_dtype (CQ_F16, CQ_BF16 or CQ_F32). */
int cq_dequantize(const void* codes, int bits, int64_t T, int64_t I,
                  const float* row_scale, const float* col_scale,
                  void* out, int out_dtype, void* stream);

/* |K| = number of zero codes (Definition 1) in stored codes.  count: device uint64. */
int cq_kernel_count(const void* codes, int bits, int64_t T, int64_t I,
                    unsigned long long* count, void* stream);

/* |K(CQ)| straight from X, without storing codes (the kernel-proportion analysis of
 * Section 4.2).  t, c: device, as produced by cq_absmax_rows_cols on the same X. */
int cq_kernel_count_x(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                      double alpha, int bits, const float* t, const float* c,
                      unsigned long long* count,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Per-channel weight quantization (Eq. 2): one scale per STORED row r,
 *   d_r = fl32(max_k |W_rk| / qmax), code = round-half-even(fl32(W_rk / d_r)), what = fl32(code * d_r).
 * Store weights as [output channels x input channels] to get one scale per output channel.
 *   W in device [R x ld]; codes out int8[R*C] or packed uint8[R*C/2]; scale out float[R];
 *   deq out [R*C] of deq_dtype (W's dtype or CQ_F32); zero_count out device uint64.
 *   codes, scale, deq, zero_count are nullable.  Each row is read from HBM once while it fits
 *   in shared memory (C <= 110,592), twice otherwise; rows of 32 KB or more arrive through one
 *   asynchronous bulk copy each.
 */
int cq_quantize_weight_per_channel(const void* W, int dtype, int64_t R, int64_t C, int64_t ld, int bits,
                                   void* codes, float* scale, void* deq, int deq_dtype,
                                   unsigned long long* zero_count, void* stream);

/*
 * Group-wise weight quantization (Section 3: W is reshaped to (elements / g) x g and then quantized per
 * row as in Eq. 2; g = 128 in the paper's W4A8-g128 experiments).  `group` must divide C, so every group
 * lies inside one stored row; groups are numbered row by row.
 *   scale out float[R * C / group]; codes / deq as in cq_quantize_weight_per_channel (dense [R x C]).
 * One read of W for group sizes 8..256 that are powers of two; other sizes take a slower general kernel.
 */
int cq_quantize_weight_groupwise(const void* W, int dtype, int64_t R, int64_t C, int64_t ld, int64_t group, int bits,
                                 void* codes, float* scale, void* deq, int deq_dtype,
                                 unsigned long long* zero_count, void* stream);

/*
 * The "Remove Kernel" operator (Figure 1 and Appendix B): the elements of the quantization kernel are set
 * to zero, every other element is passed through unquantized.  An element is removed when
 * |fl32(x_ij / s_ij)| <= bound_scale / 2 (s_ij the CrossQuant scale for `alpha`, s_ij == 0 counts as removed).
 * bound_scale = 1 removes exactly K(CQ) (alpha = 1: the kernel of per-token quantization, Eq. 1); other
 * values scale the zero bound and so sweep the removed proportion as in Section 4.3.
 *   out    device [T*I] of X's dtype: x_ij or +0
 *   counts device uint64[3]: removed elements, |K(Q)| of per-token quantization, |K(CQ)| for `alpha`
 *          -- the two kernel proportions of Figure 4 from the same pass over X
 *   workspace as for cq_quantize_act.
 */
int cq_remove_kernel(const void* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                     float bound_scale, void* out, unsigned long long* counts,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * The two indicators of Table 1 (Section 4.2, Cases I and II) from the vectors of one matrix:
 *   counts[0] = #{(i,j) : c_j >= t_i}                              (Case II)
 *   counts[1] = #{(i,j) : B~_ij < B_ij}, the CrossQuant zero bound s_ij / 2 (s_ij = fl32(row_scale_i *
 *               col_scale_j)) against the per-token one, fl32(t_i / qmax) / 2.
 * t, c, row_scale, col_scale: device vectors as written by cq_quantize_act.  counts: device uint64[2].
 * Divide by T * I for the proportions the table prints.
 */
int cq_case_indicators(const float* t, const float* c, const float* row_scale, const float* col_scale,
                       int64_t T, int64_t I, int bits, unsigned long long* counts, void* stream);

/* Launch-shape knobs for measurement.  Results never depend on them.  They are PROCESS-WIDE: every later call
 * of every thread uses them (each call reads a knob once, atomically); leave them alone in production.  key:
 *   "k1_ctas_per_sm", "k3_ctas_per_sm"  resident CTAs per SM the two passes size their grids for (1..64); for the
 *                                       staged quantize pass 2 or 3 picks the build for that occupancy
 *   "k3_forward"  1: the quantize pass walks the rows in ascending order
 *   "no_pdl"      1: no programmatic dependent launch (quantize pass and diagnostics passes)
 *   "no_stage"    1: the quantize pass loads rows straight into registers instead of staging them in shared memory
 *                    with bulk copies; the weight quantizer uses plain loads for long rows too
 *   "no_small"    1: decode-sized matrices (up to 8192 columns and 16-256 rows) take the three launches too
 *                    instead of the single thread-block-cluster launch
 * value <= 0 restores the built-in choice.  Returns CQ_OK or CQ_ERR_SHAPE (unknown key). */
int cq_set_tuning(const char* key, int value);

/* Health check.  The quantize pass, the single-launch path for small matrices, the diagnostics passes
 * (cq_remove_kernel, cq_kernel_count_x) and the weight quantizer on long rows wait for their asynchronous
 * row copies with a bounded number of polls;
 * if a wait ever gives up, a device flag is raised (results of that call are then undefined).  This
 * copies the flag of the current device to *fault_host (0 = never happened).  Synchronises the device.
 * A CTA whose wait gave up stops issuing copies, waits once more (bounded) for those in flight and leaves; the
 * flag is sticky for the life of the process. */
int cq_stage_fault(unsigned int* fault_host);

/* Measurement hook, PROCESS-WIDE like the knobs above: while both are non-NULL, every cq_quantize_act (of any
 * thread) records the two cudaEvent_t (passed as void*, owned by the caller) on its stream immediately before and
 * after the quantize pass, so that pass can be timed inside a real call.  While the hook is set, decode-sized
 * matrices take the three launches too (the single-launch path has no separate quantize pass to bracket); results
 * are the same.  Pass NULL, NULL to switch it off (the default).  Setting and reading the pair is thread-safe. */
int cq_set_timing_events(void* before_quantize_pass, void* after_quantize_pass);

#ifdef __cplusplus
}
#endif
#endif /* CQ_H_ */
