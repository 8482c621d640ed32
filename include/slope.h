/*
 * slope.h -- C ABI of the B200 (sm_100a) SLoPe 2:4-sparse linear layer.
 *
 * The calls follow the thesis chapter "SLoPe: Double-Pruned Sparse Plus Lazy
 * Low-Rank Adapter Pretraining of LLMs": Eq. (sparse_forward),
 * Eq. (sparse_backward_weight), Eq. (sparse_backward_input), Eq. (concat),
 * Algorithm 1 and the supplementary section "Implementation details".
 *
 * Common rules
 *  - Every pointer is DEVICE memory owned by the caller unless a comment says
 *    "host".  The library allocates no device memory (on the host each calling
 *    thread keeps a small table of tensor-map encodings it has already made).
 *    Base pointers must be 16-byte aligned.  Matrices are dense, row-major,
 *    contiguous.
 *  - bf16 = the upper 16 bits of an IEEE fp32.  GEMMs accumulate in fp32 and
 *    round once (nearest-even) to bf16.
 *  - `stream` is a cudaStream_t (NULL = the legacy default stream).  Calls are
 *    asynchronous with respect to the host.
 *  - Argument, shape, alignment and architecture errors are returned before
 *    anything is launched.  d_out, d_in must be multiples of 128; any number of
 *    tokens b >= 1; adapter rank r in {0, 16, 32, ..., 256}.
 *    There is no CPU fallback: on a device that is not sm_100 the calls return
 *    SLOPE_ERR_UNSUPPORTED_ARCH.
 *  - Device-side waits are bounded; a wait that runs out makes the kernel stop
 *    and record SLOPE_ERR_TIMEOUT in a sticky status word, read (and cleared)
 *    by slope_poll_status().
 *  - Same inputs on the same device give bit-identical outputs.
 *
 * Compressed 2:4 format of a matrix A[rows x cols] pruned along its columns
 *  - values  [rows x cols/2] bf16: for each group of 4 consecutive columns the
 *    two kept entries, in ascending column order (bit copies of the source);
 *  - metadata, rows*cols/8 bytes: one 4-bit code p0 | p1<<2 (p0 < p1 the kept
 *    positions) per group, stored in the order the sparse tensor-core
 *    instruction reads it.  The matrix is cut into 128x128 blocks, block
 *    (rb, cb) at byte ((rb*(cols/128)) + cb) * 2048; inside a block the four
 *    codes of row rr, columns [16*cs, 16*cs+16) form a 16-bit unit placed in
 *    32-bit word (16*(rr/16) + 8*(cs%2) + rr%8)*4 + cs/2, low half if
 *    (rr/8)%2 == 0, else high half;
 *  - mask, [rows x cols/8] bytes: bit (j%8) of byte [i][j/8] is set when
 *    element (i, j) was kept.  Masks are always in W's orientation.
 */
#ifndef SLOPE_H_
#define SLOPE_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SLOPE_OK = 0,
    SLOPE_ERR_INVALID_ARG = 1,      /* null pointer, bad enum value            */
    SLOPE_ERR_SHAPE = 2,            /* dimension not supported                 */
    SLOPE_ERR_ALIGNMENT = 3,        /* pointer not 16-byte aligned             */
    SLOPE_ERR_UNSUPPORTED_ARCH = 4, /* current device is not sm_100            */
    SLOPE_ERR_CUDA = 5,             /* a CUDA runtime / driver call failed     */
    SLOPE_ERR_TIMEOUT = 6           /* a bounded device-side wait ran out      */
} slope_status_t;

/* Buffer sizes in bytes of the compressed format of a [rows x cols] matrix. */
size_t slope_values_bytes(int rows, int cols);
size_t slope_meta_bytes(int rows, int cols);
size_t slope_mask_bytes(int rows, int cols);

/*
 * First pruning pass + compression (Algorithm 1, "backend.setup(W)"; the
 * compression is described in the supplementary section on cuSPARSELt
 * initialisation overhead).  For every row of W[d_out x d_in] and every group
 * of 4 consecutive columns keep the two entries of largest magnitude (equal
 * magnitudes: the lower column wins).  Writes the compressed W^R: values,
 * metadata and (if mask1_bits != NULL) the element mask.
 */
slope_status_t slope_prune_24(const void* W, int d_out, int d_in,
                              void* Wc_vals, void* Wc_meta, void* mask1_bits, void* stream);

/*
 * Second pruning pass (Section "Double-pruned Backward Pass"): transpose the
 * already pruned W^R = W (.) mask1 and impose 2:4 again, now along d_out.
 * Entries removed by the first pass take part with magnitude 0 and value +0.
 * Writes the compressed TRANSPOSED matrix (W^{R,C})^T [d_in x d_out]: values
 * [d_in x d_out/2], metadata, and (if mask2_bits != NULL) the mask of
 * W^{R,C} in W's orientation [d_out x d_in/8] (a subset of mask1).
 */
slope_status_t slope_double_prune(const void* W, const void* mask1_bits, int d_out, int d_in,
                                  void* WTc_vals, void* WTc_meta, void* mask2_bits, void* stream);

/*
 * Both pruning passes in one launch (Algorithm 1 calls "backend.setup" twice, once for W and once
 * for its transpose; Section "Double-pruned Backward Pass" makes the second a function of the
 * first): every output of slope_prune_24 followed by slope_double_prune, bit for bit, while W is
 * read once and the first mask is never read back (4.375 instead of 6.5 bytes of HBM traffic per
 * weight element).  mask1_bits and mask2_bits may be NULL.
 */
slope_status_t slope_prune_24_double(const void* W, int d_out, int d_in,
                                     void* Wc_vals, void* Wc_meta, void* mask1_bits,
                                     void* WTc_vals, void* WTc_meta, void* mask2_bits, void* stream);

/*
 * Forward, Eq. (sparse_forward), optionally with the lazy adapter fused as in
 * Eq. (concat):  Y[b x d_out] = X[b x d_in] (W^R)^T  (+ T[b x r] R[r x d_out]).
 * Wc_vals / Wc_meta come from slope_prune_24.  T = X L is produced by
 * slope_adapter_fwd_bwd(phase 0).  r = 0 (T, R ignored) leaves the adapter out.
 * With few tokens (inference, decode: the paper's forward-only inference measurements; always up
 * to 16 tokens, up to 128 where it is estimated faster than the tile kernels) the same call
 * runs on a kernel that streams the compressed weight once from HBM and splits the
 * reduction over a thread-block cluster.  All GEMM launches of this library are issued with
 * programmatic stream serialisation (their set-up may overlap the previous kernel's tail) and
 * synchronise on the device before they touch memory (the second launch of
 * slope_linear_fwd_adapter relies on its first one having done so and waits only for that one's
 * output), so stream order holds as for any other launch.  Every compute call of this library
 * can be captured in a CUDA graph
 * (slope_poll_status synchronises the stream and cannot).
 */
slope_status_t slope_linear_fwd(const void* X, int b, const void* Wc_vals, const void* Wc_meta,
                                int d_out, int d_in, const void* T, const void* R, int r,
                                void* Y, void* stream);

/*
 * The forward with its lazy adapter in one call, Eq. (concat):
 *   T[b x r] = X L,   Y[b x d_out] = X (W^R)^T + T R      (L[d_in x r], R[r x d_out], r > 0).
 * The same sums as slope_adapter_fwd_bwd(phase 0) followed by slope_linear_fwd: T bit for bit; Y up
 * to the order of fp32 partial sums (a fused pair may split the reduction differently), and
 * deterministic like every other call.
 * T is caller-owned scratch that holds X L afterwards.  At inference sizes (decode, and prefill
 * up to a few thousand tokens: as long as the T launch is small enough to run beside the forward
 * and an estimate says it pays) the two launches are issued as a fused pair: the forward streams
 * its operands and runs its sparse reduction while T is still being computed and waits only for
 * T itself, which takes the adapter's extra launch off the critical path (Sec. "Efficient
 * inference": the adapter multiplications are what limits the inference speedup).  With more
 * tokens it issues the same two launches as the separate calls.  The stream must not receive
 * work from another host thread while the call runs.
 */
slope_status_t slope_linear_fwd_adapter(const void* X, int b, const void* Wc_vals, const void* Wc_meta,
                                        int d_out, int d_in, const void* L, const void* R, int r,
                                        void* T, void* Y, void* stream);

/*
 * Input gradient, Eq. (sparse_backward_input), with the double-pruned weight:
 *   dX[b x d_in] = dY[b x d_out] W^{R,C}  (+ dT[b x r] L^T, L[d_in x r]).
 * WTc_vals / WTc_meta come from slope_double_prune.  dT = dY R^T is produced by
 * slope_adapter_fwd_bwd(phase 1).
 */
slope_status_t slope_linear_bwd_dx(const void* dY, int b, const void* WTc_vals, const void* WTc_meta,
                                   int d_out, int d_in, const void* dT, const void* L, int r,
                                   void* dX, void* stream);

/*
 * Weight gradient, Eq. (sparse_backward_weight), restricted to the first-pass
 * mask and stored compressed (Algorithm 1 "pruneAndCompress"; output shape
 * d_out x d_in/2 per "Implementation details"):
 *   dWc[i][2g+t] = sum_n dY[n][i] X[n][4g + p_t(i,g)],  p_0 < p_1 kept by mask1.
 */
slope_status_t slope_linear_bwd_dw_masked(const void* dY, const void* X, int b, int d_out, int d_in,
                                          const void* mask1_bits, void* dWc_vals, void* stream);

/*
 * Dense low-rank adapter GEMMs of Section "Lazy Low-rank Adapters" in the
 * orientation of Eq. (concat): L[d_in x r], R[r x d_out].
 *   phase 0:  T[b x r]  = X L
 *   phase 1:  dT[b x r] = dY R^T,  dL[d_in x r] = X^T dT,  dR[r x d_out] = T^T dY
 *             (dT and T are the bf16 tensors written by this call / phase 0).
 *   phase 2:  dT[b x r] = dY R^T only (dL and dR then come from slope_linear_bwd_dw_adapter).
 * `workspace` is device scratch of at least slope_adapter_workspace_bytes()
 * bytes, used by phase 1 for fixed-order split-K partial sums; unused pointers
 * of the other phase may be NULL.
 */
size_t slope_adapter_workspace_bytes(int b, int d_out, int d_in, int r);
slope_status_t slope_adapter_fwd_bwd(int phase, const void* X, const void* dY,
                                     const void* L, const void* R,
                                     int b, int d_out, int d_in, int r,
                                     void* T, void* dT, void* dL, void* dR,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Weight gradient and the adapter's factor gradients in one pass over X and dY:
 *   dWc          as slope_linear_bwd_dw_masked              Eq. (sparse_backward_weight)
 *   dL[d_in x r]  = X^T dT,  dR[r x d_out] = T^T dY          chain rule on Eq. (concat), as phase 1
 * T and dT are the bf16 tensors of slope_adapter_fwd_bwd phases 0 and 2.  All three products contract
 * over the tokens and the two small ones use the operand tiles the weight-gradient GEMM has staged
 * anyway, so X and dY are not streamed from HBM a second time (Sec. "Efficient implementation" names
 * the adapter's extra low-intensity kernel calls as what limits the speed-up).  For r <= 128 and
 * weight matrices large enough for the 256 x 256 tile kernel the work is one GEMM launch plus the
 * fixed-order reduction of fp32 partial sums; other shapes run the separate launches.  Same sums as
 * the separate calls; dL and dR may differ from phase 1 in the last bit because the token
 * reduction is cut into different slices, and are deterministic like every other output.
 * `workspace`: device scratch of at least slope_bwd_dw_adapter_workspace_bytes() bytes.
 */
size_t slope_bwd_dw_adapter_workspace_bytes(int b, int d_out, int d_in, int r);
slope_status_t slope_linear_bwd_dw_adapter(const void* dY, const void* X, const void* T, const void* dT,
                                           int b, int d_out, int d_in, int r,
                                           const void* mask1_bits, void* dWc_vals, void* dL, void* dR,
                                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Optimizer tail of Algorithm 1 ("sparseAdd", supplementary "Sparse matrix addition"):
 *   out = beta * A + gamma * B
 * element-wise on two compressed value arrays [rows x cols/2] bf16 that share one sparsity
 * pattern, e.g. (1/gamma_scale) * dWc + alpha * Wc for weight decay under gradient scaling.
 * fp32 arithmetic, one rounding to bf16.  out may alias A or B.
 */
slope_status_t slope_sparse_add(const void* A_vals, const void* B_vals, float beta, float gamma,
                                int rows, int cols, void* out_vals, void* stream);

/*
 * Optimizer tail of Algorithm 1 ("updateSparseMatrix", supplementary "Update Sparse Matrix").
 * The optimizer writes the new weights straight into the forward copy's values Wc_vals (the
 * pattern is static, so that copy needs nothing else); this call refreshes the values of the
 * transposed double-pruned copy from them: slot t of group h of row j of WTc_vals becomes
 * W_new[4h + q_t][j] if that element survived both pruning passes, else +0 (q_t from
 * WTc_meta; existence and position inside Wc_vals from mask1_bits).  Metadata and masks are
 * not modified.  d_out * d_in must stay below 2^35 (SLOPE_ERR_SHAPE otherwise).
 */
slope_status_t slope_update_sparse_matrix(const void* Wc_vals, const void* mask1_bits, const void* WTc_meta,
                                          int d_out, int d_in, void* WTc_vals, void* stream);

/*
 * General N:M magnitude pruning to masked-dense matrices: the matrices A^R and A^{R,C} of
 * Lemma 1 / Eq. (sparsity_ratio) for any pattern, and the emulation of N:M sparsity on dense
 * GEMMs that the accuracy experiments use (Sec. "Experiment Setup").  m in {2, 4, 8, 16},
 * 0 < n < m; d_out, d_in multiples of 128.  Selection as for 2:4: largest 15-bit bf16
 * magnitude, the lower position wins ties.  All matrices dense row-major bf16 [d_out x d_in],
 * masks [d_out x d_in/8] bytes (bit j%8 of byte j/8), W's orientation.
 *
 *   slope_prune_nm         W_R  = W with, in every group of m consecutive entries of a ROW, all but
 *                          the n largest set to +0; mask1_bits (optional, may be NULL) = kept.
 *   slope_double_prune_nm  W_RC = second pass on the already pruned matrix (entries outside
 *                          mask1_bits count as zeros): in every group of m consecutive entries
 *                          of a COLUMN keep the n largest; mask2_bits (optional) = kept by
 *                          both passes.
 *   slope_apply_mask       out = G where the mask bit is set, +0 elsewhere (a dense weight
 *                          gradient restricted to a static pattern, Eq. (sparse_backward_weight)).
 * The output may be the input matrix itself (in-place); calling slope_prune_nm on the dense
 * master weight every step gives the dynamic-mask (re-selection) variants.
 */
slope_status_t slope_prune_nm(const void* W, int d_out, int d_in, int n, int m,
                              void* W_R, void* mask1_bits, void* stream);
slope_status_t slope_double_prune_nm(const void* W, const void* mask1_bits, int d_out, int d_in,
                                     int n, int m, void* W_RC, void* mask2_bits, void* stream);
slope_status_t slope_apply_mask(const void* G, const void* mask_bits, int d_out, int d_in,
                                void* out, void* stream);

/*
 * Mask difference (supplementary "Comparison with Dynamic Sparsity: SR-STE": how many mask
 * elements an iteration's mask differs in from the converged one): writes to the device
 * uint64 *count_out (8-byte aligned) the number of element positions whose bits differ in
 * the two masks [rows x cols/8].  With slope_prune_nm on the dense weight every step this
 * measures how much a dynamically re-selected mask still moves.
 */
slope_status_t slope_mask_difference(const void* mask_a, const void* mask_b, int rows, int cols,
                                     void* count_out, void* stream);

/*
 * The dense bf16 layer on the same tcgen05 pipeline (CTA-pair 256 x 256 tiles, no sparsity):
 *   slope_dense_linear_fwd      Y [b x d_out]    = X  W^T
 *   slope_dense_linear_bwd_dx   dX[b x d_in]     = dY W
 *   slope_dense_linear_bwd_dw   dW[d_out x d_in] = dY^T X
 * for a dense row-major W[d_out x d_in]; fp32 accumulation, one rounding to bf16.  They are the
 * dense layer of Eq. (forward) / Eq. (backward_input) / Eq. (backward_weight) that the sparse
 * path is compared with, and they run N:M-emulated layers on the masked-dense matrices of
 * slope_prune_nm / slope_double_prune_nm (mask the weight gradient with slope_apply_mask).
 */
slope_status_t slope_dense_linear_fwd(const void* X, int b, const void* W, int d_out, int d_in,
                                      void* Y, void* stream);
slope_status_t slope_dense_linear_bwd_dx(const void* dY, int b, const void* W, int d_out, int d_in,
                                         void* dX, void* stream);
slope_status_t slope_dense_linear_bwd_dw(const void* dY, const void* X, int b, int d_out, int d_in,
                                         void* dW, void* stream);

/*
 * dL[d_in x r] = X[b x d_in]^T dT[b x r] without any allocation, for callers that cannot
 * call cudaMalloc or hand over a workspace (code running inside a host application whose
 * memory pool is closed to it, or in a section where allocation is forbidden).
 * The thesis has no counterpart of this call; it computes the same dL as phase 1 of
 * slope_adapter_fwd_bwd from the same bf16 dT.
 *  - The split-K partial sums live in a fixed 16 MiB array inside the library image
 *    (slope_adapter_dl_noalloc_max_scratch_bytes()); every GPU that loads the library
 *    holds that array until the process exits.
 *  - Sizes whose partial sums do not fit (splits * d_in * r * 4 bytes, with at most 16
 *    splits) are rejected with SLOPE_ERR_SHAPE before anything is launched; use
 *    slope_adapter_fwd_bwd with a workspace for those.
 *  - The first call on a device looks up the array's device address (once per device,
 *    with that device current); make that first call before any stream capture.
 *  - All calls on a device share the one array.  Nothing in it needs clearing between
 *    calls, but two calls whose kernels overlap on the GPU (different streams) race on
 *    it: serialise them.
 * Calls no cudaMalloc / cudaFree and no allocating library routine.
 */
size_t slope_adapter_dl_noalloc_max_scratch_bytes(void);
slope_status_t slope_adapter_dl_noalloc(const void* X, const void* dT, int b, int d_in, int r,
                                        void* dL, void* stream);

/*
 * Diagnostic: rewrite tensor-core-order metadata as canonical metadata
 * (uint16 [rows x cols/16], group g of a row at bits 4*(g%4) of unit g/4).
 * Paper counterpart: none (the index storage of Eq. (index_bits) in a
 * readable order).
 */
slope_status_t slope_meta_to_canonical(const void* meta_hw, int rows, int cols,
                                       void* meta_canon, void* stream);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper): launches one warp
 * that waits, for at most limit_us microseconds (1..100000), on a barrier nothing ever
 * completes.  The kernel then returns normally, writes 1 to the device int *gave_up_flag and
 * leaves SLOPE_ERR_TIMEOUT in the sticky status; the context stays usable.
 */
slope_status_t slope_selftest_wait_timeout(unsigned int limit_us, void* gave_up_flag, void* stream);

/*
 * Diagnostic (no counterpart in the paper): the mean SM clock in MHz that the tensor-core tile
 * kernels actually ran at, over all launches that completed on the current device since the
 * previous call for that kind (or since the library was loaded) -- kind 0: the sparse forward /
 * input-gradient tile kernels, kind 1: the dense CTA-pair kernel (masked weight gradient, dense
 * layer).  The MMA-issuing thread of each launch's first CTA pair reads its SM cycle counter and
 * the global timer at its first and after its last MMA; the ratio of the summed differences is the
 * clock, weighted by kernel time.  Under the power cap the hardware lowers the SM clock within
 * microseconds of the tensor cores becoming busy, which no host-side sampler resolves; a fraction of
 * the tensor peak is only meaningful beside this clock.  Synchronises `stream`; *mhz_host (host
 * memory) is 0 when no such kernel has run since the previous call.
 */
slope_status_t slope_kernel_clock_mhz(int kind, void* stream, double* mhz_host);

/* Synchronises `stream`, returns and clears the sticky device status. */
slope_status_t slope_poll_status(void* stream);

/* Number of kernel launches issued by this library since load (host counter). */
unsigned long long slope_launch_count(void);

const char* slope_status_string(slope_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* SLOPE_H_ */
