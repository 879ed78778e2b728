// Internal declarations shared by the translation units of libdk.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "dk.h"

struct CUtensorMap_st;      // the driver's tensor-map type (cuda.h)

namespace dk {

// Geometry of one layer, derived once from dk_problem.
struct Geom {
  int kind, layout;
  int cin, cout, h, w, kh, kw, stride, pad, ho, wo;
  int K, G, E;              // E = K + 2
  long long n_in, n_out;    // elements per input / output sample
  int kc;                   // contraction length cin*kh*kw
  int precision;
  int mpack;                // forward tensor-core kernel: two output rows of the image per 128-row tile (cout <= 64)
  int nprod;                // TF32 products per step of the forward tensor-core kernels: 3, or 2 (W as one term)
  int kstore;               // decoded rows k < kstore of each group are computed and stored (K, or K minus the noise
                            // vectors that stand in the place of private inputs, Section 4.5)
  float tol;
  // element strides of one sample: activation (channel, row, col), weights
  // (cout, cin, u, v), output (channel, row, col)
  long long xs_c, xs_h, xs_w;
  long long ws_o, ws_c, ws_u, ws_v;
  long long ys_c, ys_h, ys_w;
};

dk_status make_geom(const dk_problem* p, Geom* g);

// Per-call coefficient tables in device memory (all fp32), one block per group.
// enc : [G][K+2][K+1]   encoding coefficients as given
// dec : [G][K][K+1]     rows 0..K-1 of C_sq^{-1}, fp32 head of the fp64 value
// decl: [G][K][K+1]     fp32 remainder of the same fp64 value
// nul : [G][K+2]        null vector n (n[K+1] = 1)
// dmix: [G][K+1][K]     gamma[j]*B[j][i], the delta mixing weights of Eq. 4
struct CoefView {
  const float* enc;
  const float* dec;
  const float* decl;
  const float* nul;
  const float* dmix;
  int chunk_cap;         // k-blocks (of 32 contraction elements) the forward kernels may add up in tensor memory
                         // between promotions with these coefficients: the worst group's value, and
  const unsigned char* chunk_tab;   // one value per group (device; null when the tables were not derived)
};

constexpr int kCoefSlots = 8;
constexpr int kMaxSlabs = 8;       // most launches one call's groups are cut into
constexpr size_t kCoefSlotBytes = 512 * 1024;

// Scratch of the integrity check.  The decision for an element needs the rms
// of every encoded output row of its group, which is only known once the whole
// tensor has been seen; so the pass that decodes accumulates the sums of
// squares and appends every element that fails the per-element test to a
// candidate list, and a one-block kernel takes the final decisions.
struct Candidate {
  long long index;   // g*n_out + e
  float absrho;      // |rho|
  float s_e;         // sum_i |n_i||ybar_i[e]|
};
constexpr unsigned int kCandCap = 1u << 16;
constexpr size_t kVerifyStatFloats = 1u << 18;   // >= G*(K+3)

struct VerifyScratch {
  float* sumsq;          // [G][K+2] sum of squares of the finite values of each row
  int* maxrho;           // [G] bit pattern of max |rho|
  unsigned int* count;   // candidates appended (may exceed kCandCap)
  Candidate* cand;       // [kCandCap]
};

struct ProfState;

// Per-context options (dk_set_option), indexed by DK_OPT_*.
struct Options {
  int v[DK_OPT_COUNT];
};

}  // namespace dk

struct dk_ctx {
  int device;
  int sm_count;
  void* ws;
  size_t ws_bytes;
  char* h_stage;   // pinned, kCoefSlots * kCoefSlotBytes
  char* d_stage;   // device, same size
  cudaEvent_t slot_ev[dk::kCoefSlots];
  bool slot_used[dk::kCoefSlots];
  int cur_slot;
  float* d_vstats;            // kVerifyStatFloats floats + one counter
  dk::Candidate* d_cand;      // kCandCap entries
  void* tc_state;             // tensor-core path state
  dk::ProfState* prof;        // launch counters and event records
  dk::Options opt;
  // second stream on which the pre-passes of a call's later group ranges run beside the GEMM of the earlier ones
  cudaStream_t side;
  cudaEvent_t ev_fork;
  cudaEvent_t ev_slab[dk::kMaxSlabs];
};

namespace dk {

// Host-side coefficient algebra in fp64; fills a staging slot and enqueues
// its upload.  want_dec / want_mix select which tables are derived.
dk_status upload_coefficients(dk_ctx* ctx, const Geom& g, const float* C_host,
                              const float* gamma_host, bool want_dec, bool want_mix,
                              cudaStream_t st, CoefView* view);

// elementwise kernels (dk_elementwise.cu)
dk_status launch_encode(const Geom& g, const float* x, const float* r, const float* enc,
                        float* xbar, int sm_count, cudaStream_t st);
VerifyScratch verify_scratch(const dk_ctx* ctx, const Geom& g);
// begin: clears the statistics; finalize: decides the candidates, writes *v
dk_status launch_verify_begin(const Geom& g, const VerifyScratch& vs, cudaStream_t st);
dk_status launch_decode_verify(const Geom& g, const float* ybar, const CoefView& cv,
                               const float* bias, float* y, const VerifyScratch& vs,
                               int sm_count, cudaStream_t st);
dk_status launch_verify_finalize(const Geom& g, const float* nul, const VerifyScratch& vs,
                                 dk_verdict* v, cudaStream_t st);
dk_status launch_add_fault(float* ybar, long long index, float delta, cudaStream_t st);
dk_status launch_mix_delta(const Geom& g, const float* delta, const float* dmix, float* dtil,
                           int sm_count, cudaStream_t st);

// dk_wgverify.cu: elementwise comparison of two weight gradients (n elements)
// against tol * rms(a); `scratch32` = 32 bytes of device scratch; the verdict
// also carries *status_word when that is given
dk_status launch_wgrad_compare(const float* a, const float* b, long long n, float tol, void* scratch32,
                               const int* status_word, dk_verdict* v, int sm_count, cudaStream_t st);

// fp64 variants for DK_FP64_SIMT (dk_fp64.cu, dk_simt.cu)
dk_status launch_encode64(const Geom& g, const float* x, const float* r, const float* enc, double* out64,
                          float* full32, int sm_count, cudaStream_t st);
dk_status launch_decode_verify64(const Geom& g, const double* ybar, const CoefView& cv, const float* bias,
                                 float* y, const VerifyScratch& vs, int sm_count, cudaStream_t st);
dk_status launch_add_fault64(double* ybar, long long index, float delta, cudaStream_t st);
dk_status launch_simt_fwd64(const Geom& g, const float* W, const double* xbar, double* ybar,
                            int nsamples, cudaStream_t st);

// DK_FP64_SIMT for pointwise convolutions in one kernel (dk_fp64_fused.cu): Eq. 1 in the prologue, the
// contraction on the fp64 tensor path, Eq. 2 and the integrity statistics in the epilogue
bool fused64_supported(const Geom& g);
dk_status launch_fused64(const Geom& g, const float* W, const float* x, const float* r, const CoefView& cv,
                         const float* bias, float* y, float* xsave, const VerifyScratch& vs, const dk_fault* fault,
                         int sm_count, cudaStream_t st);

// Layers with 1-3 input channels (the stems) in one fp32 kernel each way (dk_stem.cu)
bool stem_fused_supported(const Geom& g, int smem_optin);
dk_status launch_stem_fwd(const Geom& g, const float* W, const float* x, const float* r, const CoefView& cv,
                          const float* bias, float* y, const VerifyScratch& vs, const dk_fault* fault, int sm_count,
                          cudaStream_t st);
bool stem_wgrad_fused_supported(const Geom& g, int smem_optin);      // 3x3 filters on 3 channels
dk_status launch_stem_wgrad(const Geom& g, const float* delta, const float* xbar, int xbar_rows, const float* dmix,
                            float scale, float* dW, bool clear, int sm_count, cudaStream_t st);
int tc_smem_optin(const dk_ctx* ctx);      // opt-in shared memory per block of the context's device (dk_tc.cu)

// SIMT dense kernels (dk_simt.cu)
dk_status launch_simt_fwd(const Geom& g, const float* W, const float* xbar, float* ybar,
                          int nsamples, cudaStream_t st);
// dW = scale * sum_n <dtil[n], xbar[row(n)]> with row(n) = (n/(K+1))*xbar_rows + n%(K+1)
// (clear = false adds to what dW holds)
dk_status launch_simt_wgrad(const Geom& g, const float* dtil, const float* xbar, int xbar_rows,
                            float scale, float* dW, int sm_count, cudaStream_t st, bool clear = true);

// the context's status word (see dk_device_status) and the offsets of workspace regions that
// other translation units borrow (dk_api.cu)
int* device_status_word(dk_ctx* ctx);
void workspace_offsets(const Geom& g, size_t* ybar, size_t* w_hi, size_t* w_lo);

// Launch accounting: counts `nkernels` launches of `kind` and, when profiling
// is on, brackets them with a pair of events on `st`.
struct ProfScope {
  dk_ctx* ctx;
  int slot;
  cudaStream_t st;
  ProfScope(dk_ctx* c, int kind, int nkernels, cudaStream_t s);
  ~ProfScope();
};

// tensor-core path (dk_tc.cu)
dk_status tc_init(dk_ctx* ctx);
// tiled tensor map over bytes, 64- or 128-byte swizzle, zero fill outside (false: the driver refused it)
bool tc_encode_map_bytes(const dk_ctx* ctx, ::CUtensorMap_st* m, const void* base, int rank,
                         const unsigned long long* dims, const unsigned long long* strides_bytes,
                         const unsigned int* box, int swz_bytes);
void tc_destroy(dk_ctx* ctx);
// true when the tensor-core kernel takes this geometry (channels-last,
// stride 1, cin % 4 == 0, not DK_FP32_SIMT)
bool tc_fwd_supported(const dk_ctx* ctx, const Geom& g);
// shapes whose forward tiles can hold two output rows (stride-1 convolution, cout <= 64, power-of-two pixel tile)
bool tc_mpack_eligible(const Geom& g);
// hi = tf32(src), lo = tf32(src - hi); n % 4 == 0
// (hi = nullptr, raw = 1: only lo = tf32(src - trunc(src)) is written, the reader takes src itself as hi)
dk_status tc_split(const float* src, float* hi, float* lo, long long n, int sm_count, cudaStream_t st, int raw = 0);
// Eq. 1 with the split fused in; `full` (nullable) also receives the fp32 encodings
dk_status tc_encode_split(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                          float* hi, float* lo, int sm_count, cudaStream_t st);
// y_bar = <W, x_bar> from split operands; ksplit > 1 slices the contraction
// (the slices add into y_bar with atomics; it is cleared here unless the caller has done so)
int tc_fwd_ksplit(const dk_ctx* ctx, const Geom& g);
dk_status tc_linear_fwd(dk_ctx* ctx, const Geom& g, const float* w_hi, const float* w_lo,
                        const float* xb_hi, const float* xb_lo, float* ybar, int ksplit, bool ybar_cleared,
                        int* status_word, cudaStream_t st, int chunk_cap = 0, bool lo_inkernel = false);
// (lo_inkernel: xb_lo is neither read nor needed, the kernel derives the second term from the fp32 values in xb_hi;
// ask tc_fwd_lo_inkernel whether the kernel that serves the geometry can)
bool tc_fwd_lo_inkernel(const dk_ctx* ctx, const Geom& g);
// (chunk_cap > 0: cap on the k-blocks of 32 added up in tensor memory, see CoefView::chunk_cap)
// weight gradient on tensor cores (channels-last, stride 1, cin % 4 == 0, cout % 4 == 0)
bool tc_wgrad_supported(const dk_ctx* ctx, const Geom& g);
// Eq. 4 delta mixing written as a TF32 hi/lo pair, [G*(K+1)][n_out] each
dk_status tc_mix_split(const Geom& g, const float* delta, const float* dmix, float* hi, float* lo,
                       int sm_count, cudaStream_t st);
// dW = scale * sum <dtil, xbar> from split operands; adds into dW, which the
// caller has cleared (tc_wgrad_prepass does)
dk_status tc_wgrad(dk_ctx* ctx, const Geom& g, const float* dt_hi, const float* dt_lo,
                   const float* xb_hi, const float* xb_lo, int xbar_rows, float scale, float* dW,
                   int* status_word, cudaStream_t st, int gt_lo = 0, int gt_cnt = -1);
// (gt_cnt >= 0: only the pixel blocks of group tiles [gt_lo, gt_lo + gt_cnt); tc_wgrad_group_tiles gives the
// number of group tiles, the groups per tile and the rounds of work items a whole launch deals to a CTA)
bool tc_wgrad_group_tiles(const dk_ctx* ctx, const Geom& g, int* GT, int* bg, long long* rounds);
// One launch for everything a masked forward call prepares (dk_tc_prepass.cu):
// Eq. 1 encodings as hi/lo pairs (and in full when `full` is given), W as a
// hi/lo pair, cleared integrity statistics, and (ybar_clear != nullptr) the
// y_bar buffer of a split-K call cleared.
dk_status tc_fwd_prepass(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                         float* xb_hi, float* xb_lo, const float* W, float* w_hi, float* w_lo,
                         const VerifyScratch& vs, float* ybar_clear, int sm_count, cudaStream_t st, int raw = 0,
                         int g_lo = 0, int g_cnt = -1, bool beside = false);
// (g_lo, g_cnt: only the encodings of groups [g_lo, g_lo + g_cnt); the launch with g_lo = 0 does the rest.
// beside: the launch is to run next to a GEMM kernel on another stream and takes a small grid of small blocks.)
// (raw != 0: xb_hi is not written; the reader takes the fp32 encodings in `full` as leading term and
// xb_lo holds tf32(v - trunc(v)))
// One launch for what a weight-gradient call prepares: Eq. 4 delta mixing and
// the stored encodings as hi/lo pairs, dW cleared (dW = nullptr: left as it is).
dk_status tc_wgrad_prepass(const Geom& g, const float* delta, const float* dmix, float* dt_hi, float* dt_lo,
                           const float* xbar, long long xbar_elems, float* xb_hi, float* xb_lo, float* dW,
                           int sm_count, cudaStream_t st, int raw = 0, int xbar_rows = 0, int g_lo = 0,
                           int g_cnt = -1, bool beside = false);
// (g_lo, g_cnt: only groups [g_lo, g_lo + g_cnt); the launch with g_lo = 0 clears dW)
// (raw != 0: only xb_lo is written, and only for the K+1 encodings of each group that Eq. 4 uses)
// same contraction with decode + integrity statistics in the epilogue; when
// `verdict` is given the kernel's last CTA also writes it (no finalize launch)
dk_status tc_masked_fwd(dk_ctx* ctx, const Geom& g, const float* w_hi, const float* w_lo,
                        const float* xb_hi, const float* xb_lo, const CoefView& cv, const float* bias,
                        float* y, const VerifyScratch& vs, int* status_word, const dk_fault* fault,
                        dk_verdict* verdict, cudaStream_t st, int gt_lo = 0, int gt_cnt = -1,
                        bool lo_inkernel = false);
// (gt_cnt >= 0: only group tiles [gt_lo, gt_lo + gt_cnt) of the tiling; a call served by several such launches
// gives `verdict` to the last one.  tc_fwd_group_tiles: group tiles, groups per tile, rounds of tiles per CTA.)
bool tc_fwd_group_tiles(const dk_ctx* ctx, const Geom& g, int* GT, int* bg, long long* rounds);

// Forward pass of layers with cin % 4 != 0 (3-channel stems) on the tensor-core kernels: the
// pre-pass lays the kc inputs under the filter out as rows of Kp = kc rounded
// up to 32 (hi/lo pairs), and the GEMM kernels run the 1x1 convolution that
// tc_stem_gemm_geom describes (dk_tc_prepass.cu).
bool tc_stem_supported(const dk_ctx* ctx, const Geom& g);
int tc_stem_padded_kc(const Geom& g);
Geom tc_stem_gemm_geom(const Geom& g);
dk_status tc_stem_fwd_prepass(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                              float* col_hi, float* col_lo, const float* W, float* w_hi, float* w_lo,
                              const VerifyScratch& vs, int sm_count, cudaStream_t st);

}  // namespace dk

#define DK_CUDA_CHECK(expr)                     \
  do {                                           \
    cudaError_t _e = (expr);                     \
    if (_e != cudaSuccess) return DK_ERR_CUDA;   \
  } while (0)
