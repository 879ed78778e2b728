/*
 * dk.h - C ABI of libdk: DarKnight's masked linear-algebra path on one GPU.
 *
 * A virtual batch of K private inputs plus one noise tensor is mixed by a
 * small coefficient matrix (Eq. 1), the dense linear layer runs on the
 * encoded inputs, the outputs are decoded with the inverse coefficients
 * (Eq. 2) and checked against one redundant equation (Section 4.4); the
 * weight gradient is computed on the stored encodings and decoded with the
 * (B, Gamma) coefficients of Eq. 4-6.
 *
 * General conventions
 *  - Every entry point returns a dk_status and never throws or exits.
 *  - All tensors are fp32, contiguous, 16-byte aligned DEVICE pointers owned
 *    by the caller.  Coefficient arrays (C, gamma) are small HOST pointers,
 *    read before the call returns.
 *  - Calls are asynchronous on the CUDA stream passed as `stream`
 *    (a cudaStream_t cast to void*, NULL = default stream).  Outputs and the
 *    dk_verdict are valid after that stream is synchronised.
 *  - A batch holds G virtual batches ("groups") of K consecutive samples.
 *    Sample tensors are stored row by row: x[G*K][n_in], r[G][n_in],
 *    xbar[G*(K+2)][n_in], ybar[G*(K+2)][n_out], y[G*K][n_out].
 *    For DK_CONV2D one row is an image; with layout DK_NHWC it is stored
 *    [h][w][channels] and weights are [cout][kh][kw][cin]; with DK_NCHW it
 *    is [channels][h][w] and weights are [cout][cin][kh][kw].  For DK_FC a
 *    row is a vector of cin values and W is [cout][cin].
 *  - Coefficients: C[g][i][k], g < G, i < K+2, k < K+1, is the weight of
 *    source k (k < K: private input k of the group, k = K: the noise) in
 *    encoding i.  Rows 0..K are the square, invertible part used for
 *    decoding (the transpose of the paper's A in X_bar = X.A); row K+1 is
 *    the redundant encoding used only by the integrity check.
 *  - Colluding accelerators (Section 4.5: M noise vectors, S = K_p + M
 *    encodings of K_p private inputs, plus the redundant one).  No separate
 *    entry point is needed: call with K = K_p + M - 1, store per group the
 *    K_p private inputs followed by the first M - 1 noise vectors in x, the
 *    M-th noise vector in r, and pass C[g] = [A^T; redundant row] with
 *    A = [A1; A2].  Rows K_p..K-1 of each group's y then hold <W, r_m>
 *    (to be dropped; with option DK_OPT_NOISE_ROWS = M - 1 they are not even
 *    computed or stored), and dk_linear_bwd_wgrad takes zero deltas for those rows.
 *    K_p + M - 1 <= DK_MAX_K.
 *  - An integrity violation is a RESULT (dk_verdict.ok = 0), not an error:
 *    the call still returns DK_OK.
 *  - The library allocates only small per-context buffers in dk_create.
 *    Large scratch memory is provided by the caller through
 *    dk_set_workspace (size from dk_workspace_bytes).
 *  - A context is not thread-safe, and calls that share a context but run
 *    on different streams race on its scratch buffers.
 *  - The library reads no environment variable and keeps no state outside its
 *    contexts (dk_decode_verify_static's fixed scratch array excepted); what
 *    can be tuned is a per-context option (dk_set_option).
 */
#ifndef DK_H_
#define DK_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DK_API __attribute__((visibility("default")))
#else
#define DK_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DK_OK = 0,
  DK_ERR_INVALID_ARG = 1,  /* NULL pointer, misaligned pointer, bad enum          */
  DK_ERR_SHAPE = 2,        /* geometry out of the supported range                 */
  DK_ERR_SINGULAR = 3,     /* a group's square coefficient block is not invertible */
  DK_ERR_WORKSPACE = 4,    /* workspace missing or too small                      */
  DK_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed                   */
  DK_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired                  */
  DK_ERR_UNSUPPORTED = 7   /* valid request that this build cannot serve          */
} dk_status;

enum { DK_FC = 0, DK_CONV2D = 1 };
enum { DK_NHWC = 0, DK_NCHW = 1 };
/* Arithmetic of the dense contraction.  DK_TF32X3 (default) runs on the
 * tensor cores with each fp32 operand split into two TF32 terms and three
 * products kept (error ~2^-22 per product); DK_FP32_SIMT uses plain fp32 FMAs
 * and accepts every geometry.  A request the tensor-core path cannot serve
 * (see dk_linear_fwd) is executed by the SIMT path. */
enum { DK_PREC_DEFAULT = 0, DK_TF32X3 = 1, DK_FP32_SIMT = 2, DK_FP64_SIMT = 3, DK_TF32X2_WUNSPLIT = 4 };
/* DK_TF32X2_WUNSPLIT (forward calls only; the weight gradient and everything the
 * tensor-core kernels do not take run as under DK_TF32X3): W enters as ONE TF32
 * term, the encodings stay split, two products per step instead of three.
 * Rounding W is exact under decoding, decode(<W', x_bar>) = <W', x>: the result
 * is the layer's output for weights rounded to 11 significant bits, an error of
 * ~1e-4 of the output's scale that does not grow with the noise.  Opt-in.
 * DK_FP64_SIMT exists for the regime in which fp32 itself cannot hold the
 * signal next to the noise: with noise 1000x the inputs and K = 8, one fp32
 * rounding of an encoded value (2^-24 * 2000) decodes to ~1e-3 of the result.
 * In dk_masked_linear it encodes, contracts and decodes in fp64 (encodings and
 * y_bar live in the workspace as doubles); the calls that exchange fp32 tensors
 * (dk_encode, dk_linear_fwd, dk_decode_verify, dk_linear_bwd_wgrad) treat it
 * as DK_FP32_SIMT. */

#define DK_MAX_K 8

typedef struct {
  int32_t kind;       /* DK_FC | DK_CONV2D                                        */
  int32_t layout;     /* DK_NHWC | DK_NCHW (ignored for DK_FC)                    */
  int32_t cin, cout;  /* FC: input / output features                              */
  int32_t h, w;       /* conv input height / width (FC: 1, 1)                     */
  int32_t kh, kw;     /* filter size (FC: 1, 1)                                   */
  int32_t stride, pad;/* same in both directions (FC: 1, 0)                       */
  int32_t K, G;       /* virtual batch size (1..DK_MAX_K), number of groups       */
  int32_t precision;  /* DK_PREC_DEFAULT | DK_TF32X3 | DK_FP32_SIMT | DK_FP64_SIMT | DK_TF32X2_WUNSPLIT */
  float tol;          /* integrity threshold tau; <= 0 selects 1e-4               */
} dk_problem;

/* Result of the integrity check, written to caller-provided device memory. */
typedef struct {
  int32_t ok;           /* 1 = every element consistent, 0 = at least one flagged */
  uint32_t n_flagged;   /* number of flagged (group, output element) pairs        */
  int64_t first_index;  /* smallest flagged g*n_out + e (e in memory order), or -1 */
  float max_ratio;      /* max over elements of |rho| / s_g (see dk_decode_verify) */
  int32_t status;       /* dk_status raised on the device (0 = none)              */
} dk_verdict;

/* Test hook modelling an accelerator that returns one wrong value (threat
 * model, Section 3): delta is added to ybar[group*(K+2)+enc][out_index]
 * before decoding. */
typedef struct {
  int32_t group, enc;
  int64_t out_index;
  float delta;
} dk_fault;

typedef struct dk_ctx dk_ctx;

/* Create / destroy a context bound to CUDA device `device`.  The context owns
 * a few MB of device and pinned host memory for coefficient upload. */
DK_API dk_status dk_create(dk_ctx** ctx, int device);
DK_API dk_status dk_destroy(dk_ctx* ctx);

/* Per-context options.  None is needed in normal use: the defaults are the
 * measured best.  They exist for measurements (what a tiling choice costs), for
 * cross-checks in the tests (another kernel for the same result) and for the
 * failure-handling test.  A value outside an option's range is clamped.
 *   DK_OPT_TC_CHUNK   the most 32-wide k-blocks accumulated in tensor memory between
 *                     two promotions to fp32 registers in the forward kernels
 *                     (default 8, 1..64; see DK_OPT_TC_CHUNK_ADAPT).  CHANGES THE
 *                     ARITHMETIC: the tensor pipe truncates when it adds, so the
 *                     error of y_bar grows with the chunk length.
 *   DK_OPT_WG_CHUNK   the same for the weight-gradient kernel (default 2, 1..64);
 *                     changes the arithmetic likewise.
 *   DK_OPT_TC_BK      k-block of the forward kernel: 32 (default) or 16 floats.
 *   DK_OPT_TC_PAIR    1 (default): layers with more than 128 output channels and
 *                     even K run on pairs of CTAs; 0: one CTA per tile.
 *   DK_OPT_WG_PACK    1 (default): the weight-gradient kernel puts several filter
 *                     taps side by side for layers with few input channels.
 *   DK_OPT_WG_PAIR    1 (default): CTA pairs in the weight-gradient kernel.
 *   DK_OPT_TC_STEM    forward pass of layers with 1-3 input channels (the stems):
 *                     1 (default) one fused fp32 kernel (encode, contraction, decode
 *                     and check in registers and shared memory) when the contraction
 *                     has at most 64 elements, else the tensor-core kernels through
 *                     patch rows; 2 always the latter; 0 the generic fp32 kernels.
 *   DK_OPT_FIELD_PATH contraction kernels of the finite-field calls: 0 (default)
 *                     tensor cores (tcgen05 with operands fetched by TMA from digit
 *                     planes where the shape allows: channels-last, stride 1,
 *                     cin % 64 == 0; else tcgen05 with operands split in registers;
 *                     else mma.sync), 1 the 64-bit integer-ALU kernels, 2 mma.sync
 *                     only, 3 as 0 without the TMA-fed kernels (1-3 are
 *                     cross-checks of the default).
 *   DK_OPT_SPIN_LIMIT polls after which a device-side wait gives up and the call
 *                     reports DK_ERR_TIMEOUT (default 2^22, 2^10..2^26).
 *   DK_OPT_XBAR_HI    how the tensor-core kernels get the leading TF32 term of an
 *                     encoded activation: 1 (default) they read the fp32 encodings
 *                     themselves (the tensor core ignores the 13 low mantissa bits
 *                     of a TF32 operand) and the pre-pass writes only the second
 *                     term tf32(v - trunc(v)); 0: the pre-pass also writes a
 *                     rounded copy tf32(v) and the second term is tf32(v - tf32(v)).
 *   DK_OPT_TC_MPACK   1 (default): a stride-1 convolution with at most 64 output
 *                     channels fills the 128 rows of the forward kernel's tiles with
 *                     two output rows of the image (rows 64-127 hold the filters of
 *                     the tap one row up, so one activation box serves both); 0: one
 *                     output row per tile, half of every product unused.
 *                     The weight-gradient kernel does the same with an even and
 *                     an odd row of the gradients.
 *   DK_OPT_TC_CHUNK_ADAPT  1 (default): DK_OPT_TC_CHUNK is the most the forward kernels add
 *                     up in tensor memory; a virtual batch whose coefficients
 *                     amplify errors in the noise term of the encoded outputs
 *                     (a = max_k sum_i |Cinv[k][i]| |C[i][K]|, in exact arithmetic
 *                     the noise cancels: sum_i Cinv[k][i] C[i][K] = 0) takes shorter
 *                     chunks: 8 k-blocks up to a = 12, 4 up to 20, 2 up to 30, 1
 *                     beyond.  Measured at noise 100x the inputs, the decoded error is
 *                     about (2.2e-5 + 0.5e-5 x k-blocks) x a of the output scale, so
 *                     this keeps it below 1e-3 up to a = 30.  0: every tile uses
 *                     DK_OPT_TC_CHUNK.
 *   DK_OPT_TC_LO_INKERNEL  default 0: the pre-pass writes the second TF32 term of the
 *                     encoded activations.  1: that term is derived inside the forward
 *                     GEMM kernels instead (two warps per CTA compute
 *                     tf32(v - trunc(v)) from the fp32 values a stage's copy brought, in
 *                     shared memory): a third less traffic into the SMs and no second
 *                     array in HBM, same results bit for bit, but measured 15-20 %
 *                     slower kernels (the derivation lengthens the way of every stage
 *                     through a pipeline of two to four stages), which outweighs the
 *                     shorter pre-pass.  2: only in the CTA-pair kernel.  Needs
 *                     DK_OPT_XBAR_HI = 1.
 *   DK_OPT_TC_SPLIT_RING  1 (default): the single-CTA forward kernel keeps the W tiles and
 *                     the activations of its k-blocks in two rings of shared-memory
 *                     slots filled by two producer warps, the activations' ring one
 *                     slot deeper (two and three slots for K = 4, where three whole
 *                     stages do not fit); 0: one ring of whole stages.
 *   DK_OPT_NOISE_ROWS default 0.  n > 0: the last n of the K inputs of every virtual batch
 *                     are noise vectors (the relabelling of Section 4.5's colluding-
 *                     accelerator scheme onto these calls, see above): dk_masked_linear,
 *                     dk_decode_verify, dk_field_masked_linear and
 *                     dk_field_decode_verify neither compute nor store the decoded rows
 *                     of those inputs (rows K-n .. K-1 of each group of y are left as
 *                     they were); encoding, the products and the integrity check are
 *                     unchanged.  At most K-1.
 *   DK_OPT_WG_PACE    1 (default): the persistent CTAs of the tensor-core weight-gradient
 *                     kernel start each round of work items together (a bounded wait
 *                     on a device counter, a hint only), so that the items that read
 *                     the same operands stay close in time and share them in L2;
 *                     0: every CTA runs ahead as it can.
 *   DK_OPT_TC_PACE    default 8.  n > 0: the persistent CTAs (CTA pairs) of the
 *                     tensor-core forward kernels (fused call and dk_linear_fwd) meet every n tiles (the same bounded
 *                     wait on a device counter, a hint only): the tiles in flight stay
 *                     neighbours in the image and share their halo rows in L2 (measured
 *                     on a 224x224 layer of 64 channels: 15.0 -> 9.9 GB read from DRAM,
 *                     the activations' bytes once).  0: off.  Calls whose CTAs walk
 *                     fewer than 2n tiles, and split-K calls, are never paced.
 *   DK_OPT_SLABS      default 1: one pre-pass launch, then one GEMM launch.  n > 1:
 *                     the tensor-core forward and weight-gradient calls may be cut
 *                     into up to n ranges of virtual batches (at most 8): the
 *                     HBM-bound pre-pass (Eq. 1 / Eq. 4 mixing, second TF32 terms)
 *                     of a later range runs on a stream owned by the context while
 *                     the GEMM of an earlier range runs on the caller's stream; the
 *                     call leaves both joined (it is still one unit of work on the
 *                     caller's stream, and can be captured).  The library picks
 *                     the count per layer from the sizes.  Outputs, stored
 *                     encodings and verdicts do not depend on it; dW does within
 *                     the error of its arithmetic (the contraction is sliced
 *                     differently).  Off by default because it measured slower on
 *                     every large layer: the GEMM kernels lose more to the
 *                     pre-pass's traffic through L2 than the overlap hides.
 *   DK_OPT_SLABS_FORCE  default 0: the library picks the count; n >= 1: exactly
 *                     min(n, DK_OPT_SLABS, tiles along the virtual batches) launches,
 *                     whatever the sizes (for tests and measurements).
 *   DK_OPT_TEST_WITHHOLD  test hook, default -1 (off): the producer warp of the
 *                     next tensor-core forward or weight-gradient kernel arms the
 *                     barrier of its n-th pipeline stage but issues no copy for
 *                     it and stops, so every consumer's wait runs out; nothing is
 *                     read or written out of bounds.  The option switches itself
 *                     off after one launch. */
enum {
  DK_OPT_TC_CHUNK = 0, DK_OPT_WG_CHUNK = 1, DK_OPT_TC_BK = 2, DK_OPT_TC_PAIR = 3, DK_OPT_WG_PACK = 4,
  DK_OPT_WG_PAIR = 5, DK_OPT_TC_STEM = 6, DK_OPT_FIELD_PATH = 7, DK_OPT_SPIN_LIMIT = 8,
  DK_OPT_TEST_WITHHOLD = 9, DK_OPT_XBAR_HI = 10, DK_OPT_TC_MPACK = 11, DK_OPT_SLABS = 12, DK_OPT_SLABS_FORCE = 13,
  DK_OPT_TC_CHUNK_ADAPT = 14, DK_OPT_WG_PACE = 15, DK_OPT_TC_LO_INKERNEL = 16,
  DK_OPT_TC_SPLIT_RING = 17, DK_OPT_NOISE_ROWS = 18, DK_OPT_TC_PACE = 19, DK_OPT_COUNT = 20
};
DK_API dk_status dk_set_option(dk_ctx* ctx, int32_t option, int32_t value);
DK_API dk_status dk_get_option(dk_ctx* ctx, int32_t option, int32_t* value);

/* Human-readable name of a status code (static storage). */
DK_API const char* dk_status_string(dk_status s);

/* Scratch bytes the calls below may need for problem `p` (the maximum over
 * all entry points), and registration of a caller-owned device buffer of at
 * least that size (256-byte aligned).  The buffer must stay valid until it is
 * replaced or the context is destroyed. */
DK_API dk_status dk_workspace_bytes(const dk_problem* p, size_t* bytes);
DK_API dk_status dk_set_workspace(dk_ctx* ctx, void* dev_ptr, size_t bytes);

/* Eq. 1 and the redundant encoding of Section 4.4:
 *   xbar[g*(K+2)+i][e] = sum_{k<K} C[g][i][k]*x[g*K+k][e] + C[g][i][K]*r[g][e]
 * x: [G*K][n_in], r: [G][n_in]  ->  xbar: [G*(K+2)][n_in].  HBM-bound. */
DK_API dk_status dk_encode(dk_ctx* ctx, const dk_problem* p, const float* x, const float* r,
                           const float* C_host, float* xbar, void* stream);

/* The bilinear operation <W, xbar> of Section 4.1 on all G*(K+2) encoded
 * samples (the untrusted accelerator's role; knows nothing about C):
 *   FC:   ybar[n][o] = sum_c W[o][c]*xbar[n][c]
 *   conv: ybar[n][o][p][q] = sum_{c,u,v} W[o][c][u][v]*xbar[n][c][p*s+u-pad][q*s+v-pad]
 * (cross-correlation, zero padding).  The tensor-core path serves DK_FC and
 * DK_CONV2D/DK_NHWC with stride <= 4 and cin % 4 == 0 and needs the workspace
 * (in dk_masked_linear also the 3-channel stems: cin % 4 != 0 with a
 * contraction of at most 256 elements and cout % 4 == 0); everything else runs
 * on the SIMT path. */
DK_API dk_status dk_linear_fwd(dk_ctx* ctx, const dk_problem* p, const float* W,
                               const float* xbar, float* ybar, void* stream);

/* Eq. 2 and Section 4.4.  Per group and output element e:
 *   [y_0..y_{K-1}, z] = C_sq^{-1} . [ybar_0..ybar_K]      (z = <W,r> is dropped)
 *   rho = sum_i n[i]*ybar_i with n^T C = 0, n[K+1] = 1     (redundant equation)
 *   s_e = sum_i |n[i]|*|ybar_i[e]|,  s_g = sum_i |n[i]|*rms_e(ybar_i)
 *   flagged iff not (|rho| <= tau * max(s_e, s_g)), or s_e is not finite
 * (the paper compares exactly in a finite field; in floating point the
 * residual is compared with the scale of the numbers it was formed from).
 * ybar: [G*(K+2)][n_out] -> y: [G*K][n_out]; bias[cout] (nullable) is added
 * after decoding; *verdict (device) receives the summary.  HBM-bound. */
DK_API dk_status dk_decode_verify(dk_ctx* ctx, const dk_problem* p, const float* ybar,
                                  const float* C_host, const float* bias, float* y,
                                  dk_verdict* verdict, void* stream);

/* Encode -> linear -> decode -> verify for one layer in one call (flow steps
 * 3-6 of Section 3.1 without leaving the device).  xbar_save (nullable)
 * receives all K+2 encodings per group, [G*(K+2)][n_in], for later use by
 * dk_linear_bwd_wgrad (Section 6, "Encoded Data Storage"); for a 1x1
 * convolution with stride s > 1 on the tensor-core path only the rows and
 * columns the layer reads (every s-th) are encoded and written, the rest of
 * xbar_save is left as it is.  fault (host
 * pointer, nullable) injects one wrong accelerator output.  Needs the
 * workspace. */
DK_API dk_status dk_masked_linear(dk_ctx* ctx, const dk_problem* p, const float* W,
                                  const float* x, const float* r, const float* C_host,
                                  const float* bias, float* y, float* xbar_save,
                                  dk_verdict* verdict, const dk_fault* fault, void* stream);

/* Eq. 4-6 summed over the virtual batches of the batch (Section 6, "Large
 * Batch Aggregation"):
 *   B[j][i] = (C_sq^{-1})[i][j] / gamma[g][j]          (the unique B of Eq. 5)
 *   dW = scale * sum_g sum_{j<=K} gamma[g][j] * < sum_i B[j][i]*delta[g*K+i], xbar[g*rows+j] >
 * delta: [G*K][n_out]; xbar holds `xbar_rows` (K+1 or K+2) encodings per
 * group of which the first K+1 are used; gamma_host: [G][K+1], non-zero;
 * dW has the shape of W.  Needs the workspace. */
DK_API dk_status dk_linear_bwd_wgrad(dk_ctx* ctx, const dk_problem* p, const float* delta,
                                     const float* xbar, int32_t xbar_rows, const float* C_host,
                                     const float* gamma_host, float scale, float* dW,
                                     void* stream);

/* The weight gradient with an integrity check.  Section 4.4 verifies a result
 * "by computing it redundantly at least twice using at least two sets of
 * equations" and states this for the forward outputs; this call applies the
 * same idea to Eq. 4-6: dW is decoded from encodings 0..K of every group (as
 * dk_linear_bwd_wgrad does) and a second time, into workspace scratch, from
 * encodings 1..K+1 with the B of that set (square part = rows 1..K+1 of C,
 * gammas rotated by one); any K+1 rows of C are independent because no
 * component of its null vector vanishes.  The two agree up to rounding unless a
 * term <delta_bar, x_bar^(j)> came back wrong.  Element e is flagged iff
 *   not (|dW[e] - dW_second[e]| <= tol_w * rms(dW)),
 * and *verdict (device) receives ok, the number of flagged elements, the
 * smallest flagged index into dW as stored, max |difference| / rms(dW), and
 * the device status.  tol_w > 0; honest fp32-class differences are ~1e-3 of
 * rms(dW), 1e-2 is a reasonable setting (the threshold and the normaliser are
 * this library's choice, the paper gives none).  xbar: all K+2 encodings per
 * group, [G*(K+2)][n_in], n_in a multiple of 4 (else DK_ERR_UNSUPPORTED).
 * fault (host pointer, nullable) adds fault->delta to element fault->out_index
 * of result fault->enc (0: dW, 1: the second one) before the comparison;
 * fault->group is ignored.  Costs two weight-gradient products.  Needs the
 * workspace. */
DK_API dk_status dk_linear_bwd_wgrad_verify(dk_ctx* ctx, const dk_problem* p, const float* delta,
                                            const float* xbar, const float* C_host,
                                            const float* gamma_host, float scale, float tol_w,
                                            float* dW, dk_verdict* verdict, const dk_fault* fault,
                                            void* stream);

/* dk_linear_bwd_wgrad that ADDS to what dW holds instead of overwriting it:
 *   dW += scale * sum_g sum_{j<=K} gamma[g][j] * < ... >       (same terms)
 * Section 6, "Large Batch Aggregation" (Algorithm 2): the gradient of a batch
 * is the sum of the gradients of its virtual batches, so a batch larger than
 * what one call holds is processed as several calls on slices of its groups,
 * the first through dk_linear_bwd_wgrad and the others through this call (the
 * paper's paging of partial sums in and out of the enclave is not needed
 * here: the running sum stays in device memory). */
DK_API dk_status dk_linear_bwd_wgrad_accumulate(dk_ctx* ctx, const dk_problem* p, const float* delta,
                                                const float* xbar, int32_t xbar_rows, const float* C_host,
                                                const float* gamma_host, float scale, float* dW,
                                                void* stream);

/* Back-propagation of the output gradient through the layer (Section 4.2: the
 * gradient with respect to the layer's input is computed from delta and W
 * "without encoding", since neither is private):
 *   FC:   dx[n][c] = sum_o delta[n][o]*W[o][c]
 *   conv: dx[n][c][i][j] = sum over (o,u,v,p,q) with i = p*s+u-pad, j = q*s+v-pad
 *                          of delta[n][o][p][q]*W[o][c][u][v]
 * (the adjoint of dk_linear_fwd's operation).  delta: [G*K][n_out], dx:
 * [G*K][n_in], layouts as in dk_problem.  Stride-1 channels-last layers with
 * cin % 4 == 0 and cout % 4 == 0 run on the tensor-core kernel (plain 3xTF32;
 * needs the workspace of dk_workspace_bytes(p)); others run in fp32 FMAs. */
DK_API dk_status dk_linear_bwd_dgrad(dk_ctx* ctx, const dk_problem* p, const float* W, const float* delta,
                                     float* dx, void* stream);

/* The non-linear layers between the masked products (the paper keeps ReLU and
 * MaxPool on the trusted side, Section 3.1 flow; here they run on the same
 * device).  x: [n][h][w][c] channels-last (a vector per sample: h = w = 1).
 *   fwd: y = relu(x), or with pool != 0 the 2x2/stride-2 max pooling of relu(x),
 *        y: [n][h/2][w/2][c] (a last odd row or column is dropped).
 *   bwd: dx = dy where x > 0, else 0; with pool != 0, dy[n][p][q][c] goes to the
 *        first maximum of relu(x) in its 2x2 window (row-major order) if that
 *        x > 0, every other position gets 0.  dy has the shape of y, dx of x.
 * HBM-bound. */
DK_API dk_status dk_relu_pool_fwd(dk_ctx* ctx, const float* x, int64_t n, int32_t h, int32_t w, int32_t c,
                                  int32_t pool, float* y, void* stream);
DK_API dk_status dk_relu_pool_bwd(dk_ctx* ctx, const float* dy, const float* x, int64_t n, int32_t h, int32_t w,
                                  int32_t c, int32_t pool, float* dx, void* stream);

/* Errors raised ON THE DEVICE by calls that have no dk_verdict to carry them
 * (dk_linear_fwd, dk_linear_bwd_wgrad): every wait inside the kernels is
 * bounded, and a kernel whose wait expires stops, leaves its output incomplete
 * and records DK_ERR_TIMEOUT.  dk_device_status synchronises the device,
 * returns the recorded code (0 = none) in *status and clears it. */
DK_API dk_status dk_device_status(dk_ctx* ctx, int32_t* status);

/* dk_decode_verify without allocation and without a context.  The paper has
 * no counterpart for this call; it exists for callers that may not allocate
 * device memory where they need the check: code confined to a fixed memory
 * budget, sections where the device-wide synchronisation implied by an
 * allocation is not acceptable, and processes that must not create a dk_ctx
 * (dk_create allocates).  It computes exactly what dk_decode_verify computes,
 * with the same arguments except that the CUDA device ordinal replaces the
 * context.  All scratch memory (coefficient tables, per-group statistics, the
 * suspect list) is one fixed array of about 1.2 MiB inside the library image,
 * which every GPU that loads the library holds until the process exits.
 *  - Limits: G*K*(K+1)*2 + G*(K+2) <= 16384 and G*(K+3) <= 16384; larger
 *    problems are refused with DK_ERR_WORKSPACE and nothing is launched.
 *  - The first call on a device looks up the array's device address (once per
 *    device); make that first call outside any stream capture.  No call may
 *    be made on a stream that is being captured: the coefficient tables are
 *    copied from the call's own stack frame, so such a call is refused with
 *    DK_ERR_UNSUPPORTED.  The call needs about 70 KiB of host stack.
 *  - The one-time address look-up is not synchronised: make the first call on
 *    a device from one thread.
 *  - Every call uses the same array: two calls whose kernels can overlap on
 *    the GPU (different streams, different threads) race on it.  Calls on
 *    one stream are safe; each call clears the state it needs.
 *  - It calls no cudaMalloc/cudaFree and no allocating library routine; the
 *    caller still provides ybar, y, bias and the dk_verdict on the device. */
DK_API dk_status dk_decode_verify_static(int device, const dk_problem* p, const float* ybar,
                                         const float* C_host, const float* bias, float* y,
                                         dk_verdict* verdict, void* stream);

/* ---------------------------------------------------------------------------
 * The same path in the finite field F_p (Section 5, "Privacy Guarantee", and
 * Algorithm 1).  The paper quantises inputs and weights to l fractional bits
 * (l = 8), maps them to residues modulo the prime p = 2^25 - 39, draws the
 * noise, the coefficients A and Gamma uniformly in F_p and runs Eq. 1, the
 * linear operation, Eq. 2 and Eq. 4-6 modulo p; a result then decodes exactly
 * and the integrity test of Section 4.4 is an exact comparison.
 *  - Residues are uint32 in [0, p) on the device, laid out like their fp32
 *    counterparts.  `prime` must be an odd prime below 2^30 (checked by trial
 *    division; DK_ERR_INVALID_ARG otherwise).  Coefficient arrays C_host
 *    [G][K+2][K+1] and gamma_host [G][K+1] are HOST arrays of residues
 *    (gamma non-zero); the index convention is the one of the fp32 calls.
 *  - DK_ERR_SINGULAR: a group's square block is not invertible modulo p, or a
 *    component of its null vector is zero (a fault in that encoding would be
 *    invisible to the redundant equation).
 *  - A decoded value is meaningful as a number only while the true integer
 *    result lies in (-p/2, p/2); the calls compute modulo p regardless, so
 *    keeping the scaled values in range is the caller's job (the paper
 *    normalises VGG activations for this reason).
 *  - dk_verdict: ok, n_flagged and first_index as for the fp32 calls;
 *    max_ratio is 0 when clean and 1 otherwise (the comparison is exact).
 *  - dk_field_masked_linear and dk_field_linear_bwd_wgrad need a workspace of
 *    dk_field_workspace_bytes registered with dk_set_workspace.
 * ------------------------------------------------------------------------- */

/* An accelerator that returns one wrong residue: delta (mod p) is added to
 * ybar[group*(K+2)+enc][out_index] before decoding. */
typedef struct {
  int32_t group, enc;
  int64_t out_index;
  uint32_t delta;
} dk_field_fault;

DK_API dk_status dk_field_workspace_bytes(const dk_problem* p, size_t* bytes);

/* Algorithm 1, procedures Round and Field: vq[i] = Field(Round(v[i]*2^scale_bits)),
 * Round(t) = floor(t) if t - floor(t) < 0.5 else floor(t) + 1, Field = residue
 * in [0, p).  scale_bits = l for inputs, weights and output gradients, 2l for a
 * bias.  v: n fp32 values (device), finite; a value whose scaled magnitude
 * is not below 4e18 maps to 0.  HBM-bound. */
DK_API dk_status dk_field_quantize(dk_ctx* ctx, const float* v, int64_t n, int32_t scale_bits,
                                   uint32_t prime, uint32_t* vq, void* stream);

/* The way back for a tensor of residues (Section 5: "subtracts p from all the
 * elements larger than p/2 to restore negative numbers"): v[i] = c*2^-scale_bits
 * with c the representative of vq[i] in (-p/2, p/2).  Used for the weight
 * gradient, whose residues carry 2l fractional bits. */
DK_API dk_status dk_field_dequantize(dk_ctx* ctx, const uint32_t* vq, int64_t n, int32_t scale_bits,
                                     uint32_t prime, float* v, void* stream);

/* Eq. 1 and the redundant encoding of Section 4.4 modulo p:
 *   xbar[g*(K+2)+i][e] = sum_{k<K} C[g][i][k]*xq[g*K+k][e] + C[g][i][K]*rq[g][e]  (mod p)
 * xq: [G*K][n_in], rq: [G][n_in] (uniform residues drawn by the caller)
 * -> xbar: [G*(K+2)][n_in]. */
DK_API dk_status dk_field_encode(dk_ctx* ctx, const dk_problem* p, uint32_t prime, const uint32_t* xq,
                                 const uint32_t* rq, const uint32_t* C_host, uint32_t* xbar, void* stream);

/* The bilinear operation of Section 4.1 on residues (step "GPUs compute" of
 * Algorithm 1): ybar = <Wq, xbar> modulo p for all G*(K+2) encoded samples,
 * FC or convolution as in dk_linear_fwd, every layout and stride.  Exact:
 * residues are multiplied digit by digit (base 256) on the integer tensor
 * cores and the partial sums reduced modulo p before they can overflow.
 * Shapes with contiguous channels (DK_FC, DK_NHWC with cin % 4 == 0) run on
 * the tcgen05 path when a workspace of dk_field_workspace_bytes is registered
 * (it holds W_q's digit planes); others, or calls without a workspace, run
 * on the mma.sync path.  A bounded device-side wait that expires is reported
 * by dk_device_status as DK_ERR_TIMEOUT. */
DK_API dk_status dk_field_linear_fwd(dk_ctx* ctx, const dk_problem* p, uint32_t prime, const uint32_t* Wq,
                                     const uint32_t* xbar, uint32_t* ybar, void* stream);

/* Eq. 2 and Section 4.4 modulo p, then the last steps of Algorithm 1.  Per
 * group and output element e:
 *   [y_0..y_{K-1}, z] = C_sq^{-1} . [ybar_0..ybar_K]  (mod p),  z dropped
 *   flagged iff sum_i n[i]*ybar_i != 0 (mod p), n^T C = 0, n[K+1] = 1
 *   y_k += bias_q[channel(e)] (mod p) when bias_q is given (device, [cout],
 *          residues quantised with 2l bits)
 *   yq (nullable, int32 [G*K][n_out]) = representative of y_k in (-p/2, p/2)
 *   y  (nullable, fp32  [G*K][n_out]) = Round(yq*2^-l)*2^-l
 * At least one of yq, y must be given.  *verdict (device) receives the summary. */
DK_API dk_status dk_field_decode_verify(dk_ctx* ctx, const dk_problem* p, uint32_t prime, int32_t l,
                                        const uint32_t* ybar, const uint32_t* C_host,
                                        const uint32_t* bias_q, int32_t* yq, float* y,
                                        dk_verdict* verdict, void* stream);

/* Procedure "Linear Operations" of Algorithm 1 in one call: quantise W, x
 * (l bits) and bias (2l bits, nullable, fp32 [cout]), encode with the noise rq,
 * run the linear operation on the encodings, decode, check, return to floating
 * point.  W, x: fp32 as in dk_masked_linear; xbar_save (nullable) receives the
 * K+2 encodings per group as residues for dk_field_linear_bwd_wgrad; fault
 * (host pointer, nullable) injects one wrong accelerator output. */
DK_API dk_status dk_field_masked_linear(dk_ctx* ctx, const dk_problem* p, uint32_t prime, int32_t l,
                                        const float* W, const float* x, const uint32_t* rq,
                                        const uint32_t* C_host, const float* bias, float* y, int32_t* yq,
                                        uint32_t* xbar_save, dk_verdict* verdict,
                                        const dk_field_fault* fault, void* stream);

/* Eq. 4-6 modulo p, summed over the virtual batches:
 *   B[j][i] = (C_sq^{-1})[i][j] / gamma[g][j]                       (mod p)
 *   dWq = sum_g sum_{j<=K} gamma[g][j] * < sum_i B[j][i]*deltaq[g*K+i], xbar[g*rows+j] >  (mod p)
 * deltaq: [G*K][n_out] residues (quantise the output gradients with
 * dk_field_quantize); xbar: xbar_rows (K+1 or K+2) encodings per group; dWq has
 * the shape of W and equals sum_i <deltaq_i, xq_i> modulo p exactly; apply
 * dk_field_dequantize with 2l bits and the batch scale afterwards. */
DK_API dk_status dk_field_linear_bwd_wgrad(dk_ctx* ctx, const dk_problem* p, uint32_t prime,
                                           const uint32_t* deltaq, const uint32_t* xbar, int32_t xbar_rows,
                                           const uint32_t* C_host, const uint32_t* gamma_host,
                                           uint32_t* dWq, void* stream);

/* Measurement aids (the paper reports time per class of operation, Table 3;
 * these give the same breakdown per kernel class).  The library always counts
 * the kernels it launches; with profiling enabled it also brackets every
 * launch with CUDA events on the launching stream (up to a few thousand
 * launches between two reads).  dk_profile_read synchronises on the recorded
 * events, returns the time and number of timed launches of `kind` since the
 * last reset together with the number of all launches of that kind, and
 * leaves the records in place; dk_profile_reset clears records and counters. */
enum {
  DK_KERNEL_ENCODE = 0,
  DK_KERNEL_LINEAR_FWD = 1,
  DK_KERNEL_DECODE_VERIFY = 2,
  DK_KERNEL_MIX_DELTA = 3,
  DK_KERNEL_WGRAD = 4,
  DK_KERNEL_OTHER = 5,
  DK_KERNEL_KINDS = 6
};
DK_API dk_status dk_profile_enable(dk_ctx* ctx, int on);
DK_API dk_status dk_profile_read(dk_ctx* ctx, int kind, double* ms_total, int64_t* timed_launches,
                                 int64_t* all_launches);
DK_API dk_status dk_profile_reset(dk_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* DK_H_ */
