/*
 * libmdbf — Multi-Envelope Double Binary Factorization (MDBF) linear forward
 * for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The layer is the paper's format (Eq. me-dbf-basis), in the column convention
 *
 *     y = W_hat x,   W_hat = (S_A (.) U_A V_A^T) (S_B (.) U_B V_B^T)
 *
 *     S_A  d_out x k   +-1      (paper: S_a,  N x R)
 *     S_B  k x d_in    +-1      (paper: S_b^T, R x M)
 *     U_A  d_out x l,  V_A  k x l      (paper: A, Q)
 *     U_B  k x l,      V_B  d_in x l   (paper: G, B)
 *
 * evaluated in the interleaved order of Eq. DBF-inference-form generalised by
 * Eq. me-dbf-expand: scale, sign contraction with S_B, scale, sign contraction
 * with S_A, scale — each stage being  sum_r diag(u_r) S diag(v_r)  with the
 * sign matrix shared by the l envelope modes.
 *
 * Conventions
 *   - All matrices are dense row-major.
 *   - Activations are token-contiguous: x[tau * d_in + i], y[tau * d_out + n]
 *     (a row-major [T, d] array).
 *   - Canonical sign packing: 32 signs per uint32 along the reduction
 *     dimension (k for S_A, d_in for S_B); column c of a row lives in word
 *     c / 32 at bit c % 32 (bit 0 = least significant); bit set <=> sign -1;
 *     padding bits of the last word are 0.  The paper only says the sign
 *     matrices are stored bit-packed (paragraph "Inference"); this layout is
 *     the library's.
 *   - Every function returns mdbf_status_t (0 = OK, negative = error), never
 *     throws, aborts or exits.  mdbf_last_error() returns a thread-local,
 *     NUL-terminated description of the last failure on the calling thread.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *   - There is no CPU fallback: every entry point that computes needs a CUDA
 *     device of compute capability 10.x and fails with MDBF_ERR_ARCH otherwise
 *     (the host-side sign packer, on_device = 0, is the one exception).
 */
#ifndef MDBF_H
#define MDBF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t mdbf_status_t;
enum {
    MDBF_OK = 0,
    MDBF_ERR_INVALID_ARG = -1, /* NULL pointer, bad handle, bad selector          */
    MDBF_ERR_SHAPE = -2,       /* non-positive size, T < 1, T > max_T, l > 64     */
    MDBF_ERR_DTYPE = -3,       /* unsupported element type                        */
    MDBF_ERR_ALLOC = -4,       /* device or host allocation failed                */
    MDBF_ERR_CUDA = -5,        /* a CUDA runtime call failed (see last_error)     */
    MDBF_ERR_ARCH = -6,        /* no CUDA device, or not compute capability 10.x  */
    MDBF_ERR_TIMEOUT = -7,     /* a bounded device-side wait expired              */
    MDBF_ERR_VALUE = -8,       /* a sign that is neither +1 nor -1                */
    MDBF_ERR_BOUNDS = -9       /* bounds-checked build only: a kernel computed a   */
                               /* store index outside its buffer (store skipped)  */
};

typedef enum { MDBF_F32 = 0, MDBF_F16 = 1, MDBF_BF16 = 2 } mdbf_dtype_t;

/* Kernel selector for mdbf_set_kernel. */
typedef enum {
    MDBF_KERNEL_AUTO = 0,   /* T = 1: TMEM or I8 per stage, by size; T >= 2: MAT (PREFILL / ALU where MAT cannot run); fp32 / l > 32: ALU */
    MDBF_KERNEL_ALU = 1,    /* fp32 CUDA-core path, sign applied by XOR of the IEEE sign bit      */
                            /* 2: retired (a warp-level MMA kernel for T <= 4)                     */
    MDBF_KERNEL_PREFILL = 3, /* T >= 2 (max_T >= 2): expanded order, tcgen05 GEMM of width l*T, TMEM accumulator, TMA operand */
    MDBF_KERNEL_TMEM = 4,   /* T = 1: tcgen05 MMA, sign (.) activation as bf16 operand in TMEM, one launch per stage */
    MDBF_KERNEL_MAT = 5,    /* T >= 2: W_hat tiles rebuilt on the fly (rank-l mini-MMA + sign XOR), one GEMM of width T */
    MDBF_KERNEL_I8 = 6      /* T = 1, l <= 16: packed bits as the 8-bit integer tcgen05 operand, 21-bit fixed-point scaled input;
                             * two launches per stage (operand images, contraction on one CTA per SM) */
} mdbf_kernel_t;

typedef struct {
    int32_t d_out;     /* rows of W_hat (paper: N)                         */
    int32_t d_in;      /* columns of W_hat (paper: M)                      */
    int32_t k;         /* inner rank (paper: R)                            */
    int32_t l;         /* envelope rank, 1 <= l <= 64                      */
    int32_t env_dtype; /* mdbf_dtype_t the envelope factors are stored in  */
    int32_t max_T;     /* largest token count a forward call may pass      */
} mdbf_desc_t;

typedef struct mdbf_handle_s *mdbf_handle_t;

/* ---------------------------------------------------------------- packing
 * Canonical sign packing (layout above; storage statement: paragraph
 * "Inference", effective bits-per-weight).
 *   s     rows x cols int8, every entry +1 or -1
 *   out   rows x ceil(cols/32) uint32
 * on_device = 0: both pointers are host memory, the work is done on the host
 * (no GPU needed); a value other than +-1 returns MDBF_ERR_VALUE.
 * on_device = 1: both are device memory, the kernel runs asynchronously on
 * `stream`; values other than -1 are treated as +1.
 * Caller owns both buffers. */
mdbf_status_t mdbf_pack_signs(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out,
                              int on_device, void *stream);

/* Inverse of mdbf_pack_signs: p rows x ceil(cols/32) uint32 -> out rows x cols int8. */
mdbf_status_t mdbf_unpack_signs(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out,
                                int on_device, void *stream);

/* ------------------------------------------------------------------ layer
 * Build a layer (Eq. me-dbf-basis).  Copies everything: the caller keeps
 * ownership of all inputs and may free them on return.
 *   S_A d_out x k, S_B k x d_in   int8 +-1
 *   U_A d_out x l, V_A k x l, U_B k x l, V_B d_in x l   float32; rounded
 *   (round-to-nearest-even) to desc->env_dtype — the rounded values are the
 *   layer and can be read back with mdbf_get_envelope.
 * inputs_on_device: 0 = all seven pointers are host memory, 1 = all device.
 * The handle owns one device copy of the sign words (in the layout its kernels
 * read; canonical words are produced on request by mdbf_get_packed), the
 * envelopes with their operand layouts, and scratch for the k x T
 * intermediate sized for max_T: about one bit per sign plus the envelopes.
 * One forward per handle may be in flight at a time.  Synchronises `stream`
 * before returning.
 * Errors: INVALID_ARG (NULL), SHAPE, DTYPE, VALUE (host inputs only), ALLOC,
 * CUDA, ARCH. */
mdbf_status_t mdbf_pack(const mdbf_desc_t *desc, const int8_t *S_A, const int8_t *S_B,
                        const float *U_A, const float *V_A, const float *U_B, const float *V_B,
                        int inputs_on_device, void *stream, mdbf_handle_t *out);

/* Copy the canonical packed words of S_A (which = 0, d_out x ceil(k/32)) or
 * S_B (which = 1, k x ceil(d_in/32)) to `out` (host if out_on_device = 0). */
mdbf_status_t mdbf_get_packed(mdbf_handle_t h, int which, uint32_t *out, int out_on_device,
                              void *stream);

/* Stored (rounded) envelope factor as float32: which = 0 U_A, 1 V_A, 2 U_B, 3 V_B. */
mdbf_status_t mdbf_get_envelope(mdbf_handle_t h, int which, float *out, int out_on_device,
                                void *stream);

/* Read the layer's descriptor back. */
mdbf_status_t mdbf_get_desc(mdbf_handle_t h, mdbf_desc_t *out);

/* Force a kernel for later forwards on this handle (tests, benchmarks).  MDBF_KERNEL_PREFILL
 * allocates that kernel's scratch (max_T * l * (d_in + k) * 2 bytes of pre-scaled operands) on the
 * first request, which synchronises the device; no forward ever does (a forward that is forced to
 * that kernel on a handle without the scratch returns MDBF_ERR_INVALID_ARG; a handle packed with
 * max_T = 1 never has the scratch). */
mdbf_status_t mdbf_set_kernel(mdbf_handle_t h, int32_t kernel /* mdbf_kernel_t */);

/* ---------------------------------------------------------------- forward
 * y = W_hat x, evaluated stage by stage, z = (S_B (.) U_B V_B^T) x, y = (S_A (.) U_A V_A^T) z
 * (Eq. DBF-inference-form).  One token and the selectable expanded-order kernels follow
 * Eq. me-dbf-expand (scale by V, sign contraction with S, contract the l modes with U); from two
 * tokens on the default kernels rebuild each factor S (.) U V^T of Eq. me-dbf-basis tile by tile
 * and multiply it by the activations once.  Both orders compute the same y up to rounding.
 *   x  device, T x d_in  of act_dtype (token-contiguous), read only
 *   y  device, T x d_out of act_dtype, written (round-to-nearest-even)
 *   act_dtype  MDBF_BF16 or MDBF_F32 (MDBF_F16 is accepted by the ALU path)
 * Precision.  Accumulation is fp32 (one token, integer kernel: exact int32 sums of 21-bit fixed-point
 * operands).  What is rounded to bf16 on the way, besides y itself: T >= 2, default order: every
 * entry of the two rebuilt factors and the intermediate z (four roundings with y); T >= 2, expanded
 * order: the pre-scaled x and z (three); one token, TMEM-operand kernel: V_B, z and V_A (four);
 * one token, integer kernel: nothing (one).  fp16 envelopes are re-rounded to bf16 where they become
 * bf16 MMA operands.  Measured against the fp64 definition: 1.6e-3 to 3.7e-3 relative Frobenius
 * error on the 7B- and 70B-class shapes, bound 5e-3.  x is expected to be finite: the integer
 * kernel scales its operand by max|x| (and max|z|), so an Inf or NaN in x gives an unspecified y
 * there, where the floating-point kernels would propagate it.
 * Asynchronous on `stream`; never allocates and never synchronises.  With the library choosing the
 * kernel, an x that the default kernels cannot take (T >= 2 and x not 16-byte aligned) is served
 * by the expanded order if mdbf_set_kernel(PREFILL) has prepared its scratch on this handle, else
 * by the CUDA-core kernel.  x and y must not alias; the current device must be the one the layer
 * was packed on.
 * Errors: INVALID_ARG, SHAPE (T < 1 or T > max_T), DTYPE, CUDA. */
mdbf_status_t mdbf_linear_forward(mdbf_handle_t h, const void *x, void *y, int32_t T,
                                  int32_t act_dtype, void *stream);

/* Sum of P layers on the same input, y = (W_hat^(1) + ... + W_hat^(P)) x: the residual-compensation
 * form (Eq. dbf-residual-comp: a DBF term plus a DBF term fitted to the residual, (l, P) = (1, 2);
 * the paper's (l, P) sweep uses the same sum with MDBF terms).  Every term is evaluated by the same
 * kernels as mdbf_linear_forward with an fp32 output: term 1 stores into `acc`, the others add to
 * it, and one pass rounds `acc` to y - so y carries a single rounding whatever P is.  With one
 * token, bf16 activations and at most four terms of one envelope-rank bucket, the first stage of
 * all terms shares a launch and the last term's epilogue does the final add and rounding
 * (P + 1 launches instead of 2P + 1, same result).
 *   terms  P handles of equal d_out and d_in (k, l and env_dtype may differ), all distinct
 *   x, y   device, T x d_in read, T x d_out written, of act_dtype
 *   acc    device, T x d_out float32 scratch owned by the caller, overwritten
 * Asynchronous on `stream`, allocates nothing.  Errors: INVALID_ARG, SHAPE, DTYPE, CUDA. */
mdbf_status_t mdbf_linear_forward_sum(const mdbf_handle_t *terms, int32_t P, const void *x, void *y, float *acc,
                                      int32_t T, int32_t act_dtype, void *stream);

/* Sibling projections: n layers applied to the same input, ys[i] = W_hat_i x (q/k/v, or gate/up, of a
 * decoder block; the paper quantises each linear layer separately, so this is n forwards of
 * Eq. DBF-inference-form / Eq. me-dbf-expand on a shared x).  With one token, bf16 activations and
 * layers of equal envelope-rank bucket the stages of up to four layers share a launch (their row
 * blocks side by side in one grid): two launches instead of 2n, and small layers no longer leave
 * most SMs idle.  Otherwise the layers run one after the other, exactly as n calls of
 * mdbf_linear_forward.
 *   layers  n distinct handles of equal d_in          ys  n device pointers, ys[i] is T x d_out_i
 * Asynchronous on `stream`, allocates nothing.  Errors: INVALID_ARG, SHAPE, DTYPE, CUDA. */
mdbf_status_t mdbf_linear_forward_siblings(const mdbf_handle_t *layers, int32_t n, const void *x, void *const *ys,
                                           int32_t T, int32_t act_dtype, void *stream);

/* Independent layers, each with its own input: ys[i] = W_hat_i xs[i] for n layers whose forwards do not depend on
 * one another (projections of different requests, or of different places of a model whose inputs are all at hand).
 * The arithmetic is n forwards of Eq. DBF-inference-form / Eq. me-dbf-expand; only the launch structure changes:
 * with one token, bf16 activations and layers of equal envelope-rank bucket (l <= 16, 16-bit envelopes) up to
 * eight layers share the four launches of the integer one-token kernel (operand images and contraction, per stage),
 * every CTA walking its share of every layer, so that the fixed cost of a forward is paid once and small layers no
 * longer leave SMs idle.  Otherwise the layers run one after the other, exactly as n calls of mdbf_linear_forward.
 *   layers  n distinct handles          xs, ys  n device pointers each: xs[i] is T x d_in_i, ys[i] is T x d_out_i
 * Asynchronous on `stream`, allocates nothing.  Errors: INVALID_ARG, SHAPE, DTYPE, CUDA. */
mdbf_status_t mdbf_linear_forward_group(const mdbf_handle_t *layers, int32_t n, const void *const *xs, void *const *ys,
                                        int32_t T, int32_t act_dtype, void *stream);

/* Device staging buffers for mdbf_linear_forward_host (max_T * (d_in + d_out) * 4 bytes): allocated
 * here, once, so that the host-buffer forward itself allocates nothing.  Errors: ALLOC, CUDA. */
mdbf_status_t mdbf_prepare_host_staging(mdbf_handle_t h);

/* Same computation with HOST buffers: copies x to the handle's device staging buffer, runs the
 * forward, copies y back, all on `stream`, and synchronises the stream before returning.  x_host /
 * y_host should be pinned for full copy bandwidth.  Needs mdbf_prepare_host_staging once per handle
 * (MDBF_ERR_INVALID_ARG otherwise). */
mdbf_status_t mdbf_linear_forward_host(mdbf_handle_t h, const void *x_host, void *y_host, int32_t T,
                                       int32_t act_dtype, void *stream);

/* The same without the final synchronisation: the two copies and the kernels are enqueued on
 * `stream` and the call returns; y_host holds the result once the caller has synchronised the
 * stream (or an event recorded after the call).  x_host must stay unchanged and both buffers
 * allocated until then; pageable buffers make the copies synchronous, so use pinned memory.  Calls
 * on different handles pipeline on one stream: the next layer's input copy overlaps this layer's
 * kernels.  Two calls on the SAME handle share its staging buffers and are ordered by the stream. */
mdbf_status_t mdbf_linear_forward_host_async(mdbf_handle_t h, const void *x_host, void *y_host, int32_t T,
                                             int32_t act_dtype, void *stream);

/* ------------------------------------------------- forward without allocation
 * (The paper has no counterpart: this entry point exists for deployment, not
 * for the method.)
 *
 * Some callers may not allocate device memory: a serving runtime that has
 * given every byte to its own arena and forbids cudaMalloc from then on, a
 * plug-in that only ever receives buffers from its host application, a
 * real-time loop that cannot afford the device-wide synchronisation an
 * allocation implies.  They cannot use mdbf_pack, which allocates the handle's
 * buffers.  This call computes the same y = W_hat x from buffers the caller
 * already owns and needs no handle:
 *
 *   desc       shape and env_dtype of the layer (max_T is ignored)
 *   wA, wB     device; canonical packed words of S_A (d_out x ceil(k/32)) and
 *              S_B (k x ceil(d_in/32)), as mdbf_pack_signs writes them
 *   U_A..V_B   device; envelope factors stored in desc->env_dtype, row-major
 *              d_out x l, k x l, k x l, d_in x l
 *   x, y       device; T x d_in read, T x d_out written, of act_dtype
 *              (MDBF_F32, MDBF_F16 or MDBF_BF16); fp32 accumulation
 *
 * The k x T intermediate between the two stages is kept in a fixed array
 * inside the library image (MDBF_STATIC_MAX_KT floats = 1 MiB, resident on
 * every GPU that loads the library until the process exits); a call with
 * k * T above that limit returns MDBF_ERR_SHAPE.  The call runs the fp32
 * CUDA-core kernels (sign applied by XOR of the IEEE sign bit), asynchronously
 * on `stream`, and calls neither cudaMalloc nor cudaFree nor any allocating
 * library routine.
 *
 * The first call on each device looks the array's device address up (with
 * that device current) and keeps it for the life of the process; make that
 * first call outside any stream capture.  cudaDeviceReset() destroys the
 * array with the context: do not call this function again on that device
 * afterwards (the kept address would be stale).
 * Every call on a device shares the one array, which keeps whatever the
 * previous call left in it: each call overwrites all the entries it later
 * reads, so nothing has to be cleared, but two calls that overlap on the GPU
 * (different streams, no dependency between them) race on it and both may
 * return wrong results.  Serialise them.
 * Errors: INVALID_ARG (NULL), SHAPE, DTYPE, ARCH, CUDA. */
#define MDBF_STATIC_MAX_KT 262144
mdbf_status_t mdbf_linear_forward_static(const mdbf_desc_t *desc, const uint32_t *wA, const uint32_t *wB,
                                         const void *U_A, const void *V_A, const void *U_B,
                                         const void *V_B, const void *x, void *y, int32_t T,
                                         int32_t act_dtype, void *stream);

/* The k x T intermediate z of the last forward on this handle (after the
 * stage with S_B), as float32 token-contiguous T x k, for tests that localise
 * a disagreement to one stage.  Synchronises `stream`. */
mdbf_status_t mdbf_get_intermediate(mdbf_handle_t h, float *z, int32_t T, int out_on_device,
                                    void *stream);

/* Dense W_hat (Eq. me-dbf-basis), fp32, d_out x d_in row-major, device memory,
 * asynchronous on `stream`.  Check path, not a hot path. */
mdbf_status_t mdbf_reconstruct(mdbf_handle_t h, float *W, void *stream);

/* Device-side status word of the handle (0, or MDBF_ERR_TIMEOUT when a bounded
 * wait inside a kernel expired; the kernel then returns without completing y).
 * Synchronises the device.  Reading clears the word. */
mdbf_status_t mdbf_poll_status(mdbf_handle_t h, int32_t *device_status);

/* ---------------------------------------------------------------- quantizer, first step
 * Multi-Envelope SVID of a device matrix (Eq. msvid-def):  MSVID_l[Z] = sign(Z) (.) TSVD_l(|Z|),  sign(0) = +1.
 * It is the operator the paper applies to each balanced factor of W's truncated SVD to initialise MDBF
 * (Eq. mesvid-init-compact); by Theorem 1 (Eq. rankl-error, Eq. Ustar) its result is the best approximation of Z
 * among the matrices that keep Z's sign mask and have an envelope of rank <= l, with error
 * (sum_{i > l} sigma_i(|Z|)^2)^(1/2).
 *   Z         device, rows x cols fp32, row-major, read only
 *   l         envelope rank, 1 <= l <= min(32, rows, cols)
 *   n_iter    subspace iterations (two passes over Z each), >= 1; 2 already fixes the leading singular value,
 *             8 leaves the squared error within a fraction of a per cent to about one per cent of the optimum
 *   Q0        device, cols x l fp32: the start block of the iteration (e.g. i.i.d. Gaussian; the caller draws it,
 *             so that a run is reproducible from its inputs alone); needs full column rank
 *   S_packed  device, rows x ceil(cols / 32) uint32, written: the sign mask in the canonical packing of
 *             mdbf_pack_signs (bit set <=> entry negative); exact
 *   U, V      device, rows x l and cols x l fp32, written: balanced factors of the truncated envelope,
 *             TSVD_l(|Z|) ~ U V^T, columns ordered by decreasing singular value (each pair is unique up to a
 *             common sign only, and up to rotations inside a group of equal singular values)
 *   sigma     device, l fp32, written: the estimated singular values; each is a lower bound of the exact one
 *   workspace device, at least mdbf_msvid_workspace_bytes(rows, cols, l) bytes on a 256-byte boundary, scratch of the
 *             call (the two blocks, the partial sums of a product - up to 16 per output row - and operand images:
 *             ask mdbf_msvid_workspace_bytes); free again when the stream has passed it
 * The truncated SVD is computed by block subspace iteration, not to machine precision: see n_iter.  The two products
 * with |Z| run on the tensor cores (TF32 operands in a three-term split, fp32 accumulation; within a few 1e-6 of the
 * scalar fp32 kernels' results)
 * when cols is a multiple of 4 and Z sits on a 16-byte boundary, else in scalar fp32 kernels; the small Gram matrices
 * are fp64.  Results do not depend on scheduling (no floating-point atomics).  Asynchronous on `stream`; allocates
 * nothing and does not synchronise.  Should one of the kernel's bounded waits expire (not expected), the outputs are
 * NaN.  Errors: INVALID_ARG (NULL pointer, workspace too small or misaligned), SHAPE, ARCH, CUDA. */
mdbf_status_t mdbf_msvid(const float *Z, int64_t rows, int64_t cols, int32_t l, int32_t n_iter, const float *Q0,
                         uint32_t *S_packed, float *U, float *V, float *sigma, void *workspace, size_t workspace_bytes,
                         void *stream);

/* Projection onto the matrices that share a GIVEN sign mask and have an envelope of rank <= l (Theorem 1, Eq. Ustar):
 *   Pi(Z) = S (.) TSVD_l(S (.) Z),   error (sum_{i > l} sigma_i(S (.) Z)^2)^(1/2)   (Eq. rankl-error)
 * - the step the paper's refinement repeats with the mask held fixed; mdbf_msvid is the special case S = sign(Z).
 * Arguments as for mdbf_msvid, except that S_packed (rows x ceil(cols / 32) words, canonical packing, bit set <=> -1) is
 * read, not written.  U V^T approximates the demodulated envelope S (.) Z, so the projection itself is S (.) (U V^T).
 * The same workspace size serves.  Asynchronous on `stream`, allocates nothing.  Errors as for mdbf_msvid. */
mdbf_status_t mdbf_project_fixed_mask(const float *Z, const uint32_t *S_packed, int64_t rows, int64_t cols, int32_t l,
                                      int32_t n_iter, const float *Q0, float *U, float *V, float *sigma, void *workspace,
                                      size_t workspace_bytes, void *stream);

/* Size of the workspace mdbf_msvid needs for this shape (host computation, no device needed).  Errors: INVALID_ARG, SHAPE. */
mdbf_status_t mdbf_msvid_workspace_bytes(int64_t rows, int64_t cols, int32_t l, size_t *bytes);

/* ---------------------------------------------------------------- quantizer, refinement
 * n_inner ADMM inner iterations on one factor with the other held fixed (Section "ADMM Refinement"), for the
 * objective ||W - U V^T||_F^2 with the multi-envelope structure imposed by MSVID_l:
 *     U_tilde = (W V + rho (U - Lam)) (V^T V + rho I)^-1        (Eq. admm-U-tilde)
 *     U       = MSVID_l[U_tilde + Lam]                          (Eq. admm-U-prox)
 *     Lam     = Lam + U_tilde - U                               (Eq. admm-U-dual)
 * With N x M = the shape of op(W): op(W) = W (w_rows x w_cols) for transpose_w = 0 and W^T for transpose_w != 0 -
 * the update of the other factor is this call on the transposed problem, with the roles of the factors exchanged.
 *   W          device, w_rows x w_cols fp32 row-major, read only
 *   V          device, M x R fp32 row-major: the dense values of the fixed factor, read only
 *   U, Lambda  device, N x R fp32 row-major, read and written: the dense values of the factor being refined and the
 *              scaled dual variable (zeros to start with)
 *   rho        penalty, > 0
 *   l, n_iter, Q0 (R x l)   as for mdbf_msvid, which performs the prox step (the same Q0 starts every inner iteration)
 *   S_packed (N x ceil(R / 32)), Ul (N x l), Vl (R x l), sigma (l)   device, written: the compact form of the new U,
 *              U = S (.) (Ul Vl^T), as mdbf_msvid returns it in the last inner iteration
 *   U_tilde    device, N x R fp32, written with the last inner iteration's least-squares iterate; may be NULL
 *   workspace  device, mdbf_admm_workspace_bytes(N, M, R, l) bytes on a 256-byte boundary (three N x R matrices, the R x R
 *              system, the operand images of op(W) and V - twice their size - and mdbf_msvid's workspace)
 * The dense products (W V, V^T V, the inverse of the system and its application) run on the tensor cores (TF32
 * operands in a three-term split, fp32 accumulation in chunks of 128 contraction indices; U_tilde comes out within a few
 * 1e-6 of its largest entry of the exact result); the Cholesky factorisation and the solves of the R x R system are cuSOLVER calls in
 * fp32; the MSVID step, the elementwise passes and the reconstruction of the dense factor fused with the dual update
 * are this library's kernels.  Asynchronous on `stream`; part of the work runs on a stream of the library's own that
 * is forked from `stream` and joined to it by events inside the call.  The first call on a host thread creates the
 * solver's handles, that stream and its events, and allocates the scratch the factorisation asks for (kept for later calls; a larger request synchronises
 * the stream and reallocates).  A failed factorisation (not expected for rho > 0) or an expired wait of a kernel turns
 * sigma into NaN.
 * Errors: INVALID_ARG (NULL pointer, rho <= 0, counts out of range, workspace too small or misaligned), SHAPE, ARCH, CUDA. */
mdbf_status_t mdbf_admm_factor_update(const float *W, int64_t w_rows, int64_t w_cols, int32_t transpose_w, const float *V, int64_t r,
                                      float *U, float *Lambda, float rho, int32_t l, int32_t n_inner, int32_t n_iter,
                                      const float *Q0, uint32_t *S_packed, float *Ul, float *Vl, float *sigma, float *U_tilde,
                                      void *workspace, size_t workspace_bytes, void *stream);

/* Size of the workspace mdbf_admm_factor_update needs for an N x R factor of an N x M matrix (host computation, no device
 * needed).
 * Errors: INVALID_ARG, SHAPE. */
mdbf_status_t mdbf_admm_workspace_bytes(int64_t n, int64_t m, int64_t r, int32_t l, size_t *bytes);

/* Test hook (no counterpart in the paper): the `nth` device allocation that the calling thread makes
 * inside this library from now on fails with MDBF_ERR_ALLOC without touching the device; nth <= 0
 * cancels a pending request.  A call that fails this way frees what it had allocated, publishes
 * nothing half-built to the handle and leaves the handle (if any) as usable as before. */
void mdbf_debug_fail_alloc(int nth);

/* Self-test of the bounded device-side wait the tcgen05 kernels use (no counterpart in the paper):
 * launches one warp that waits on a barrier nothing arrives at.  After the time limit (about one
 * second) the kernel records MDBF_ERR_TIMEOUT in the handle's status word and returns normally; the
 * context stays usable and mdbf_poll_status reports (and clears) the code.  Asynchronous on
 * `stream`. */
mdbf_status_t mdbf_selftest_wait_timeout(mdbf_handle_t h, void *stream);

/* Number of kernels the last forward on this handle launched. */
mdbf_status_t mdbf_last_launch_count(mdbf_handle_t h, int32_t *count);

/* Which kernel (an mdbf_kernel_t other than AUTO) the last forward on this handle ran; 0 before the
 * first forward. */
mdbf_status_t mdbf_last_kernel(mdbf_handle_t h, int32_t *kernel);

/* Free everything the handle owns.  Synchronises the device. */
mdbf_status_t mdbf_destroy(mdbf_handle_t h);

const char *mdbf_last_error(void);

/* Library version string. */
const char *mdbf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MDBF_H */
