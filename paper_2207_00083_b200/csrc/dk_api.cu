// C-ABI entry points of libdk: argument checks, fp64 coefficient algebra on
// the host, workspace carving and kernel dispatch.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "dk_internal.h"

namespace dk {

dk_status make_geom(const dk_problem* p, Geom* g) {
  if (!p || !g) return DK_ERR_INVALID_ARG;
  if (p->kind != DK_FC && p->kind != DK_CONV2D) return DK_ERR_INVALID_ARG;
  if (p->layout != DK_NHWC && p->layout != DK_NCHW) return DK_ERR_INVALID_ARG;
  if (p->precision < DK_PREC_DEFAULT || p->precision > DK_TF32X2_WUNSPLIT) return DK_ERR_INVALID_ARG;
  if (p->K < 1 || p->K > DK_MAX_K || p->G < 1) return DK_ERR_SHAPE;
  if (p->cin < 1 || p->cout < 1) return DK_ERR_SHAPE;
  memset(g, 0, sizeof(*g));
  g->kind = p->kind;
  g->layout = (p->kind == DK_FC) ? DK_NHWC : p->layout;
  g->cin = p->cin;
  g->cout = p->cout;
  g->K = p->K;
  g->G = p->G;
  g->E = p->K + 2;
  g->precision = (p->precision == DK_PREC_DEFAULT || p->precision == DK_TF32X2_WUNSPLIT) ? DK_TF32X3 : p->precision;
  g->nprod = p->precision == DK_TF32X2_WUNSPLIT ? 2 : 3;
  g->kstore = p->K;
  g->tol = p->tol > 0.f ? p->tol : 1e-4f;
  if (p->kind == DK_FC) {
    g->h = g->w = g->kh = g->kw = g->stride = 1;
    g->pad = 0;
  } else {
    if (p->h < 1 || p->w < 1 || p->kh < 1 || p->kw < 1 || p->stride < 1 || p->pad < 0)
      return DK_ERR_SHAPE;
    if (p->kh > 16 || p->kw > 16) return DK_ERR_SHAPE;
    g->h = p->h; g->w = p->w; g->kh = p->kh; g->kw = p->kw;
    g->stride = p->stride; g->pad = p->pad;
  }
  int eh = g->h + 2 * g->pad - g->kh, ew = g->w + 2 * g->pad - g->kw;
  if (eh < 0 || ew < 0) return DK_ERR_SHAPE;
  g->ho = eh / g->stride + 1;
  g->wo = ew / g->stride + 1;
  g->n_in = (long long)g->cin * g->h * g->w;
  g->n_out = (long long)g->cout * g->ho * g->wo;
  long long kc = (long long)g->cin * g->kh * g->kw;
  if (kc > (1LL << 30)) return DK_ERR_SHAPE;
  g->kc = (int)kc;
  if ((size_t)g->G * (g->E + 1) > kVerifyStatFloats) return DK_ERR_SHAPE;
  if ((long long)g->G * g->E * g->n_in >= (1LL << 40) ||
      (long long)g->G * g->E * g->n_out >= (1LL << 40))
    return DK_ERR_SHAPE;
  if ((long long)g->G * g->E * g->ho * g->wo >= (1LL << 31)) return DK_ERR_SHAPE;
  if (g->layout == DK_NHWC) {
    g->xs_c = 1; g->xs_w = g->cin; g->xs_h = (long long)g->cin * g->w;
    g->ws_c = 1; g->ws_v = g->cin; g->ws_u = (long long)g->cin * g->kw; g->ws_o = kc;
    g->ys_c = 1; g->ys_w = g->cout; g->ys_h = (long long)g->cout * g->wo;
  } else {
    g->xs_w = 1; g->xs_h = g->w; g->xs_c = (long long)g->h * g->w;
    g->ws_v = 1; g->ws_u = g->kw; g->ws_c = (long long)g->kh * g->kw; g->ws_o = kc;
    g->ys_w = 1; g->ys_h = g->wo; g->ys_c = (long long)g->ho * g->wo;
  }
  return DK_OK;
}

// Gauss-Jordan inverse with partial pivoting, n <= DK_MAX_K+1, fp64.
static bool invert_small(const double* M, int n, double* inv) {
  double a[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
  double amax = 0.0;
  for (int i = 0; i < n * n; ++i) { a[i] = M[i]; amax = fmax(amax, fabs(M[i])); }
  if (!(amax > 0.0) || !isfinite(amax)) return false;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) inv[i * n + j] = (i == j) ? 1.0 : 0.0;
  for (int c = 0; c < n; ++c) {
    int piv = c;
    for (int r = c + 1; r < n; ++r)
      if (fabs(a[r * n + c]) > fabs(a[piv * n + c])) piv = r;
    double pv = a[piv * n + c];
    if (!(fabs(pv) > 1e-10 * amax)) return false;
    if (piv != c)
      for (int j = 0; j < n; ++j) {
        double t = a[c * n + j]; a[c * n + j] = a[piv * n + j]; a[piv * n + j] = t;
        t = inv[c * n + j]; inv[c * n + j] = inv[piv * n + j]; inv[piv * n + j] = t;
      }
    double ip = 1.0 / pv;
    for (int j = 0; j < n; ++j) { a[c * n + j] *= ip; inv[c * n + j] *= ip; }
    for (int r = 0; r < n; ++r) {
      if (r == c) continue;
      double f = a[r * n + c];
      if (f == 0.0) continue;
      for (int j = 0; j < n; ++j) {
        a[r * n + j] -= f * a[c * n + j];
        inv[r * n + j] -= f * inv[c * n + j];
      }
    }
  }
  return true;
}

dk_status upload_coefficients(dk_ctx* ctx, const Geom& g, const float* C_host,
                              const float* gamma_host, bool want_dec, bool want_mix,
                              cudaStream_t st, CoefView* view) {
  const int K = g.K, K1 = K + 1, E = K + 2, G = g.G;
  const size_t n_enc = (size_t)G * E * K1, n_dec = (size_t)G * K * K1, n_nul = (size_t)G * E,
               n_mix = (size_t)G * K1 * K;
  const size_t n_chk = ((size_t)G + 3) / 4;      // one byte per group
  const size_t total = n_enc + 2 * n_dec + n_nul + n_mix + n_chk;
  if (total * sizeof(float) > kCoefSlotBytes) return DK_ERR_SHAPE;
  if (!C_host) return DK_ERR_INVALID_ARG;
  if (want_mix && !gamma_host) return DK_ERR_INVALID_ARG;

  int s = ctx->cur_slot;
  ctx->cur_slot = (s + 1) % kCoefSlots;
  if (ctx->slot_used[s]) DK_CUDA_CHECK(cudaEventSynchronize(ctx->slot_ev[s]));
  float* h = reinterpret_cast<float*>(ctx->h_stage + (size_t)s * kCoefSlotBytes);
  float* d = reinterpret_cast<float*>(ctx->d_stage + (size_t)s * kCoefSlotBytes);
  float* h_enc = h;
  float* h_dec = h_enc + n_enc;
  float* h_decl = h_dec + n_dec;
  float* h_nul = h_decl + n_dec;
  float* h_mix = h_nul + n_nul;
  memcpy(h_enc, C_host, n_enc * sizeof(float));
  memset(h_dec, 0, (2 * n_dec + n_nul + n_mix) * sizeof(float));
  unsigned char* h_chunk = reinterpret_cast<unsigned char*>(h_mix + n_mix);
  memset(h_chunk, 8, n_chk * 4);
  view->chunk_cap = 8;
  view->chunk_tab = nullptr;

  if (want_dec || want_mix) {
    double sq[(DK_MAX_K + 1) * (DK_MAX_K + 1)], inv[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
    for (int gi = 0; gi < G; ++gi) {
      const float* Cg = C_host + (size_t)gi * E * K1;
      for (int i = 0; i < K1 * K1; ++i) sq[i] = (double)Cg[i];
      if (!invert_small(sq, K1, inv)) return DK_ERR_SINGULAR;
      // decode rows: y_k = sum_i inv[k][i] ybar_i
      for (int k = 0; k < K; ++k)
        for (int i = 0; i < K1; ++i) {
          double v = inv[k * K1 + i];
          float hi = (float)v;
          h_dec[((size_t)gi * K + k) * K1 + i] = hi;
          h_decl[((size_t)gi * K + k) * K1 + i] = (float)(v - (double)hi);
        }
      // How strongly decoding amplifies an error that is relative to the noise term of the encoded outputs:
      // a = max_k sum_i |inv[k][i]| |C[i][K]| (in exact arithmetic sum_i inv[k][i] C[i][K] = 0: the noise
      // cancels).  The forward kernels' accumulator in tensor memory truncates when it adds, a bias that grows
      // with the k-blocks added there; measured at noise 100x the inputs, the decoded error is about
      // (2.2e-5 + 0.5e-5 x k-blocks) x a of the output scale for a short contraction (288 elements; less for
      // long ones).  The chunk lengths below keep that under 1e-3 up to a = 30 (beyond, one k-block per chunk
      // is the best this arithmetic does): 7.4e-4 at a = 12 with 8 k-blocks, 8.4e-4 at 20 with 4, 9.6e-4 at 30
      // with 2.
      {
        double amp = 0.0;
        for (int k = 0; k < K; ++k) {
          double a = 0.0;
          for (int i = 0; i < K1; ++i) a += fabs(inv[k * K1 + i]) * fabs((double)Cg[i * K1 + K]);
          amp = a > amp ? a : amp;
        }
        const int cap = amp <= 12.0 ? 8 : (amp <= 20.0 ? 4 : (amp <= 30.0 ? 2 : 1));
        if (cap < view->chunk_cap) view->chunk_cap = cap;
        h_chunk[gi] = (unsigned char)cap;
      }
      // null vector: n[0..K] = -C[K+1] . C_sq^{-1}, n[K+1] = 1
      for (int i = 0; i < K1; ++i) {
        double acc = 0.0;
        for (int k = 0; k < K1; ++k) acc += (double)Cg[(size_t)K1 * K1 + k] * inv[k * K1 + i];
        h_nul[(size_t)gi * E + i] = (float)(-acc);
      }
      h_nul[(size_t)gi * E + K1] = 1.f;
      if (want_mix) {
        // Eq. 5: B[j][i] = inv[i][j] / gamma[j]; mixing weight gamma[j]*B[j][i]
        for (int j = 0; j < K1; ++j) {
          double gm = (double)gamma_host[(size_t)gi * K1 + j];
          if (gm == 0.0 || !isfinite(gm)) return DK_ERR_INVALID_ARG;
          for (int i = 0; i < K; ++i) {
            double B = inv[i * K1 + j] / gm;
            h_mix[((size_t)gi * K1 + j) * K + i] = (float)(gm * B);
          }
        }
      }
    }
  }
  DK_CUDA_CHECK(cudaMemcpyAsync(d, h, total * sizeof(float), cudaMemcpyHostToDevice, st));
  DK_CUDA_CHECK(cudaEventRecord(ctx->slot_ev[s], st));
  ctx->slot_used[s] = true;
  view->enc = d;
  view->dec = d + n_enc;
  view->decl = view->dec + n_dec;
  view->nul = view->decl + n_dec;
  view->dmix = view->nul + n_nul;
  if ((want_dec || want_mix) && ctx->opt.v[DK_OPT_TC_CHUNK_ADAPT])
    view->chunk_tab = reinterpret_cast<const unsigned char*>(view->dmix + n_mix);
  else
    view->chunk_cap = 64;
  return DK_OK;
}

struct ProfState {
  bool on = false;
  long long launches[DK_KERNEL_KINDS] = {0, 0, 0, 0, 0, 0};
  std::vector<cudaEvent_t> ev;      // 2 per slot
  std::vector<int> kind_of;         // per used slot
  static constexpr size_t kMaxSlots = 8192;
};

ProfScope::ProfScope(dk_ctx* c, int kind, int nkernels, cudaStream_t s) : ctx(c), slot(-1), st(s) {
  ProfState* ps = c->prof;
  if (!ps) return;
  ps->launches[kind] += nkernels;
  if (!ps->on || ps->kind_of.size() >= ProfState::kMaxSlots) return;
  size_t i = ps->kind_of.size();
  while (ps->ev.size() < 2 * (i + 1)) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    ps->ev.push_back(e);
  }
  if (cudaEventRecord(ps->ev[2 * i], st) != cudaSuccess) return;
  ps->kind_of.push_back(kind);
  slot = (int)i;
}

ProfScope::~ProfScope() {
  if (slot >= 0) cudaEventRecord(ctx->prof->ev[2 * slot + 1], st);
}

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct WsPlan {
  size_t xbar, ybar, dtil, w_hi, w_lo, xb_hi, xb_lo, total;
};

// Geometry of the layers that go through the patch-row pre-pass (3-channel
// stems): channels-last convolution, cin not a multiple of four, a contraction
// of at most 256 elements, default arithmetic.  Independent of the context so
// that dk_workspace_bytes can size for it.
static bool stem_shape(const Geom& g) {
  return g.kind == DK_CONV2D && g.layout == DK_NHWC && g.precision == DK_TF32X3 && (g.cin % 4) != 0 &&
         g.kc <= 256 && (g.cout % 4) == 0;
}

// One layout serves every entry point: fp32 encodings (when the caller does
// not store them), y_bar of the unfused path, mixed deltas of wgrad, and the
// TF32 hi/lo split copies of W and x_bar that feed the tensor-core kernel.
static WsPlan plan_workspace(const Geom& g) {
  WsPlan w;
  size_t off = 0;
  // (a stem layer's hi/lo regions hold its patch rows and padded weights instead)
  size_t xe = (size_t)g.G * g.E * g.n_in, we = (size_t)g.cout * g.kc;
  if (stem_shape(g)) {
    const size_t Kp = (size_t)tc_stem_padded_kc(g);
    const size_t rows = (size_t)g.G * g.E * g.ho * g.wo * Kp;
    if (rows > xe) xe = rows;
    we = (size_t)g.cout * Kp;
  }
  if (g.kind == DK_CONV2D && g.cout <= 64 && g.kh >= 2) {
    // two-output-row tiles of the forward kernel: 128 rows x (kh+1)*kw taps x cin packed weights
    const size_t packed = (size_t)128 * (g.kh + 1) * g.kw * g.cin;
    if (packed > we) we = packed;
  }
  const size_t xb = align_up(xe * sizeof(float), 1024);
  const size_t wb = align_up(we * sizeof(float), 1024);
  w.xbar = off; off += xb;
  // y_bar: sized for doubles (DK_FP64_SIMT keeps it in fp64)
  w.ybar = off; off += align_up((size_t)g.G * g.E * g.n_out * sizeof(double), 1024);
  w.dtil = off; off += align_up((size_t)g.G * (g.K + 1) * g.n_out * sizeof(float), 1024);
  w.w_hi = off; off += wb;
  w.w_lo = off; off += wb;
  w.xb_hi = off; off += xb;
  w.xb_lo = off; off += xb;
  w.total = off;
  return w;
}

// Device word that kernels without a dk_verdict raise on a bounded-wait expiry
// (third word after the verify statistics; read and cleared by dk_device_status).
static int* ctx_status_word(dk_ctx* ctx) {
  return reinterpret_cast<int*>(ctx->d_vstats + kVerifyStatFloats) + 2;
}
int* device_status_word(dk_ctx* ctx) { return ctx_status_word(ctx); }

void workspace_offsets(const Geom& g, size_t* ybar, size_t* w_hi, size_t* w_lo) {
  const WsPlan wp = plan_workspace(g);
  *ybar = wp.ybar; *w_hi = wp.w_hi; *w_lo = wp.w_lo;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct DeviceGuard {
  int prev;
  bool ok;
  explicit DeviceGuard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) return;
    ok = true;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (ok && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

}  // namespace dk

using namespace dk;

extern "C" {

const char* dk_status_string(dk_status s) {
  switch (s) {
    case DK_OK: return "DK_OK";
    case DK_ERR_INVALID_ARG: return "DK_ERR_INVALID_ARG";
    case DK_ERR_SHAPE: return "DK_ERR_SHAPE";
    case DK_ERR_SINGULAR: return "DK_ERR_SINGULAR";
    case DK_ERR_WORKSPACE: return "DK_ERR_WORKSPACE";
    case DK_ERR_CUDA: return "DK_ERR_CUDA";
    case DK_ERR_TIMEOUT: return "DK_ERR_TIMEOUT";
    case DK_ERR_UNSUPPORTED: return "DK_ERR_UNSUPPORTED";
  }
  return "DK_ERR_UNKNOWN";
}

dk_status dk_create(dk_ctx** out, int device) {
  if (!out) return DK_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return DK_ERR_CUDA;
  DeviceGuard dg(device);
  if (!dg.ok) return DK_ERR_CUDA;
  dk_ctx* c = new (std::nothrow) dk_ctx();
  if (!c) return DK_ERR_CUDA;
  memset(c, 0, sizeof(*c));
  c->device = device;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
    delete c;
    return DK_ERR_CUDA;
  }
  c->sm_count = sms;
  static const int kOptDefault[DK_OPT_COUNT] = {8, 2, 32, 1, 1, 1, 1, 0, 1 << 22, -1, 1, 1, 1, 0, 1, 1, 0, 1, 0, 8};
  for (int i = 0; i < DK_OPT_COUNT; ++i) c->opt.v[i] = kOptDefault[i];
  bool ok = cudaMallocHost(&c->h_stage, kCoefSlots * kCoefSlotBytes) == cudaSuccess &&
            cudaMalloc(&c->d_stage, kCoefSlots * kCoefSlotBytes) == cudaSuccess &&
            cudaMalloc(&c->d_vstats, (kVerifyStatFloats + 64) * sizeof(float)) == cudaSuccess &&
            cudaMemset(c->d_vstats, 0, (kVerifyStatFloats + 64) * sizeof(float)) == cudaSuccess &&
            cudaMalloc(&c->d_cand, kCandCap * sizeof(Candidate)) == cudaSuccess;
  for (int i = 0; ok && i < kCoefSlots; ++i)
    ok = cudaEventCreateWithFlags(&c->slot_ev[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess &&
       cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < kMaxSlabs; ++i)
    ok = cudaEventCreateWithFlags(&c->ev_slab[i], cudaEventDisableTiming) == cudaSuccess;
  c->prof = new (std::nothrow) ProfState();
  ok = ok && c->prof != nullptr;
  if (ok) ok = tc_init(c) == DK_OK;
  if (!ok) { dk_destroy(c); return DK_ERR_CUDA; }
  *out = c;
  return DK_OK;
}

dk_status dk_destroy(dk_ctx* c) {
  if (!c) return DK_OK;
  DeviceGuard dg(c->device);
  cudaDeviceSynchronize();
  tc_destroy(c);
  for (int i = 0; i < kCoefSlots; ++i)
    if (c->slot_ev[i]) cudaEventDestroy(c->slot_ev[i]);
  for (int i = 0; i < kMaxSlabs; ++i)
    if (c->ev_slab[i]) cudaEventDestroy(c->ev_slab[i]);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->side) cudaStreamDestroy(c->side);
  if (c->prof) {
    for (cudaEvent_t e : c->prof->ev) cudaEventDestroy(e);
    delete c->prof;
  }
  if (c->h_stage) cudaFreeHost(c->h_stage);
  if (c->d_stage) cudaFree(c->d_stage);
  if (c->d_vstats) cudaFree(c->d_vstats);
  if (c->d_cand) cudaFree(c->d_cand);
  delete c;
  return DK_OK;
}

// Section 4.5 relabelling: the last DK_OPT_NOISE_ROWS inputs of every group are noise vectors, whose decoded
// outputs are neither computed nor stored (at least one row stays).
static void apply_noise_rows(const dk_ctx* ctx, Geom* g) {
  int n = ctx->opt.v[DK_OPT_NOISE_ROWS];
  if (n > g->K - 1) n = g->K - 1;
  g->kstore = g->K - (n > 0 ? n : 0);
}

dk_status dk_set_option(dk_ctx* ctx, int32_t option, int32_t value) {
  if (!ctx || option < 0 || option >= DK_OPT_COUNT) return DK_ERR_INVALID_ARG;
  static const int lo[DK_OPT_COUNT] = {1, 1, 16, 0, 0, 0, 0, 0, 1 << 10, -1, 0, 0, 1, 0, 0, 0, 0, 0, 0, 0};
  static const int hi[DK_OPT_COUNT] = {64, 64, 32, 1, 1, 1, 2, 3, 1 << 26, 1 << 20, 1, 1, kMaxSlabs, kMaxSlabs, 1, 1, 2, 1, DK_MAX_K - 1, 1024};
  int v = value < lo[option] ? lo[option] : (value > hi[option] ? hi[option] : value);
  if (option == DK_OPT_TC_BK) v = v == 16 ? 16 : 32;
  ctx->opt.v[option] = v;
  return DK_OK;
}

dk_status dk_get_option(dk_ctx* ctx, int32_t option, int32_t* value) {
  if (!ctx || !value || option < 0 || option >= DK_OPT_COUNT) return DK_ERR_INVALID_ARG;
  *value = ctx->opt.v[option];
  return DK_OK;
}

dk_status dk_workspace_bytes(const dk_problem* p, size_t* bytes) {
  if (!bytes) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  *bytes = plan_workspace(g).total;
  return DK_OK;
}

dk_status dk_set_workspace(dk_ctx* ctx, void* dev_ptr, size_t bytes) {
  if (!ctx) return DK_ERR_INVALID_ARG;
  if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255)) return DK_ERR_INVALID_ARG;
  ctx->ws = dev_ptr;
  ctx->ws_bytes = dev_ptr ? bytes : 0;
  return DK_OK;
}

dk_status dk_encode(dk_ctx* ctx, const dk_problem* p, const float* x, const float* r,
                    const float* C_host, float* xbar, void* stream) {
  if (!ctx || !x || !r || !C_host || !xbar) return DK_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(r) || !aligned16(xbar)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CoefView cv;
  s = upload_coefficients(ctx, g, C_host, nullptr, false, false, st, &cv);
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
  return launch_encode(g, x, r, cv.enc, xbar, ctx->sm_count, st);
}

dk_status dk_linear_fwd(dk_ctx* ctx, const dk_problem* p, const float* W, const float* xbar,
                        float* ybar, void* stream) {
  if (!ctx || !W || !xbar || !ybar) return DK_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(xbar) || !aligned16(ybar)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (tc_fwd_supported(ctx, g)) {
    WsPlan wp = plan_workspace(g);
    if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
    char* ws = static_cast<char*>(ctx->ws);
    float* w_hi = reinterpret_cast<float*>(ws + wp.w_hi);
    float* w_lo = reinterpret_cast<float*>(ws + wp.w_lo);
    float* xb_hi = reinterpret_cast<float*>(ws + wp.xb_hi);
    float* xb_lo = reinterpret_cast<float*>(ws + wp.xb_lo);
    const bool lo_in = tc_fwd_lo_inkernel(ctx, g);
    {
      ProfScope ps(ctx, DK_KERNEL_OTHER, 2, st);
      const int raw = ctx->opt.v[DK_OPT_XBAR_HI];
      s = tc_split(W, w_hi, w_lo, (long long)g.cout * g.kc, ctx->sm_count, st);
      // (a kernel that derives the second term itself needs no pass over the encodings at all)
      if (s == DK_OK && !lo_in)
        s = tc_split(xbar, raw ? nullptr : xb_hi, xb_lo, (long long)g.G * g.E * g.n_in, ctx->sm_count, st, raw);
      if (raw) xb_hi = const_cast<float*>(xbar);      // the kernel reads the caller's encodings as leading term
    }
    if (s != DK_OK) return s;
    ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
    return tc_linear_fwd(ctx, g, w_hi, w_lo, xb_hi, xb_lo, ybar, tc_fwd_ksplit(ctx, g), false, ctx_status_word(ctx),
                         st, 0, lo_in);
  }
  ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
  return launch_simt_fwd(g, W, xbar, ybar, g.G * g.E, st);
}

dk_status dk_decode_verify(dk_ctx* ctx, const dk_problem* p, const float* ybar,
                           const float* C_host, const float* bias, float* y,
                           dk_verdict* verdict, void* stream) {
  if (!ctx || !ybar || !C_host || !y || !verdict) return DK_ERR_INVALID_ARG;
  if (!aligned16(ybar) || !aligned16(y) || !aligned16(verdict)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  apply_noise_rows(ctx, &g);
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CoefView cv;
  s = upload_coefficients(ctx, g, C_host, nullptr, true, false, st, &cv);
  if (s != DK_OK) return s;
  VerifyScratch vs = verify_scratch(ctx, g);
  {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    s = launch_verify_begin(g, vs, st);
  }
  if (s != DK_OK) return s;
  {
    ProfScope ps(ctx, DK_KERNEL_DECODE_VERIFY, 1, st);
    s = launch_decode_verify(g, ybar, cv, bias, y, vs, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
  return launch_verify_finalize(g, cv.nul, vs, verdict, st);
}

// Launches a call's groups are cut into: the pre-pass of a later range runs beside the GEMM of an earlier one,
// so n launches leave 1/n of the pre-pass exposed, and each launch but the last ends with CTAs idle for about
// half the time of one of its work items.  prep_bytes at a nominal 5.5 TB/s against gemm_flops (as issued) at a
// nominal 600 TFLOP/s: only the ratio matters.
static int plan_slabs(const dk_ctx* ctx, int GT, long long rounds, double prep_bytes, double gemm_flops,
                      double tail_floor = 5e-6) {
  int cap = ctx->opt.v[DK_OPT_SLABS];
  if (cap > kMaxSlabs) cap = kMaxSlabs;
  if (cap > GT) cap = GT;
  const int force = ctx->opt.v[DK_OPT_SLABS_FORCE];
  if (force > 0) return force < cap ? force : (cap < 1 ? 1 : cap);
  if (cap < 2 || rounds < 1) return 1;
  const double tp = prep_bytes / 5.5e12;
  double tail = 0.5 * (gemm_flops / 6.0e14) / (double)rounds;
  if (tail < tail_floor) tail = tail_floor;
  int best = 1;
  double best_cost = tp;
  for (int n = 2; n <= cap; ++n) {
    const double cost = tp / n + (n - 1) * tail;
    if (cost < best_cost * 0.98) { best_cost = cost; best = n; }
  }
  return best;
}

// The context's second stream joins the caller's stream for the duration of one call: it starts behind
// everything already enqueued there, and the caller's stream waits for its last piece of work before the
// call returns, whatever happens in between.
struct SideStream {
  dk_ctx* ctx;
  cudaStream_t main;
  bool forked;
  SideStream(dk_ctx* c, cudaStream_t st) : ctx(c), main(st), forked(false) {
    forked = cudaEventRecord(c->ev_fork, st) == cudaSuccess && cudaStreamWaitEvent(c->side, c->ev_fork, 0) == cudaSuccess;
  }
  ~SideStream() {
    if (forked && cudaEventRecord(ctx->ev_fork, ctx->side) == cudaSuccess) cudaStreamWaitEvent(main, ctx->ev_fork, 0);
  }
};

dk_status dk_masked_linear(dk_ctx* ctx, const dk_problem* p, const float* W, const float* x,
                           const float* r, const float* C_host, const float* bias, float* y,
                           float* xbar_save, dk_verdict* verdict, const dk_fault* fault,
                           void* stream) {
  if (!ctx || !W || !x || !r || !C_host || !y || !verdict) return DK_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(x) || !aligned16(r) || !aligned16(y) || !aligned16(verdict) ||
      !aligned16(xbar_save))
    return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  apply_noise_rows(ctx, &g);
  if (fault) {
    if (fault->group < 0 || fault->group >= g.G || fault->enc < 0 || fault->enc >= g.E ||
        fault->out_index < 0 || fault->out_index >= g.n_out)
      return DK_ERR_INVALID_ARG;
  }
  WsPlan wp = plan_workspace(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CoefView cv;
  s = upload_coefficients(ctx, g, C_host, nullptr, true, false, st, &cv);
  if (s != DK_OK) return s;
  char* ws = static_cast<char*>(ctx->ws);
  if (g.precision == DK_TF32X3 && ctx->opt.v[DK_OPT_TC_STEM] == 1 && stem_fused_supported(g, tc_smem_optin(ctx))) {
    // 1-3 input channels: one fp32 kernel encodes the input patch, contracts, decodes and checks; the
    // encodings, when the caller stores them, come from the streaming encoder (they are tiny here)
    VerifyScratch vs = verify_scratch(ctx, g);
    {
      ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
      s = launch_verify_begin(g, vs, st);
    }
    if (s == DK_OK && xbar_save) {
      ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
      s = launch_encode(g, x, r, cv.enc, xbar_save, ctx->sm_count, st);
    }
    if (s != DK_OK) return s;
    {
      ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
      s = launch_stem_fwd(g, W, x, r, cv, bias, y, vs, fault, ctx->sm_count, st);
    }
    if (s != DK_OK) return s;
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    return launch_verify_finalize(g, cv.nul, vs, verdict, st);
  }
  const bool stem = stem_shape(g) && tc_stem_supported(ctx, g);
  // layers with at most 64 output channels: two output rows per 128-row tile (see dk_tc.cu)
  if (!stem && ctx->opt.v[DK_OPT_TC_MPACK] && tc_mpack_eligible(g)) g.mpack = 1;
  const Geom g_stem = stem ? tc_stem_gemm_geom(g) : g;
  if (stem || tc_fwd_supported(ctx, g)) {
    // tensor-core path: encode+split pre-pass, then one GEMM whose epilogue
    // decodes and gathers the integrity statistics; y_bar never reaches HBM.
    // (A stem layer's pre-pass writes patch rows, and the GEMM runs on the
    // 1x1 geometry over them; outputs and statistics are laid out the same.)
    const Geom& gg = g_stem;
    float* w_hi = reinterpret_cast<float*>(ws + wp.w_hi);
    float* w_lo = reinterpret_cast<float*>(ws + wp.w_lo);
    float* xb_hi = reinterpret_cast<float*>(ws + wp.xb_hi);
    float* xb_lo = reinterpret_cast<float*>(ws + wp.xb_lo);
    VerifyScratch vs = verify_scratch(ctx, g);
    const int ksplit = tc_fwd_ksplit(ctx, gg);
    float* ybar = reinterpret_cast<float*>(ws + wp.ybar);
    const bool prepass_clears = ksplit > 1 && !stem;     // the pre-pass also clears y_bar for the slices
    // leading TF32 term of the encodings: the fp32 encodings themselves (stored by the caller, or in the
    // workspace), or a rounded copy
    const int raw = stem ? 0 : ctx->opt.v[DK_OPT_XBAR_HI];
    float* full = xbar_save;
    if (raw && !full) full = reinterpret_cast<float*>(ws + wp.xbar);
    // the second term: written by the pre-pass, or derived inside the GEMM kernel (then the array is unused)
    const bool lo_in = raw && tc_fwd_lo_inkernel(ctx, gg);
    if (lo_in) xb_lo = nullptr;
    // Large layers: the groups are cut into ranges; the pre-passes run in order on the context's second stream,
    // the GEMM of a range starts on the caller's stream as soon as its pre-pass has finished, and the kernel
    // of the last range takes the final decisions of the check.
    int nslab = 1, GT = 0, bg = 1;
    if (!stem && ksplit == 1) {
      long long rounds = 0;
      if (tc_fwd_group_tiles(ctx, gg, &GT, &bg, &rounds)) {
        const double prep = ((double)(g.K + 1) + (raw ? 2.0 : 3.0) * g.E) * g.G * (double)g.n_in * 4.0;
        nslab = plan_slabs(ctx, GT, rounds, prep, 6.0 * g.G * g.E * (double)g.n_out * g.kc);
      }
    }
    if (nslab > 1) {
      SideStream fork(ctx, st);
      if (!fork.forked) return DK_ERR_CUDA;
      int gt_lo[kMaxSlabs + 1];
      for (int i = 0; i <= nslab; ++i) gt_lo[i] = (int)((long long)GT * i / nslab);
      for (int i = 0; i < nslab && s == DK_OK; ++i) {
        const int g_lo = gt_lo[i] * bg, g_hi = gt_lo[i + 1] * bg < g.G ? gt_lo[i + 1] * bg : g.G;
        {
          ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, ctx->side);
          s = tc_fwd_prepass(gg, x, r, cv.enc, full, raw ? nullptr : xb_hi, xb_lo, W, w_hi, w_lo, vs, nullptr,
                             ctx->sm_count, ctx->side, raw, g_lo, g_hi - g_lo, i > 0);
        }
        if (s == DK_OK && cudaEventRecord(ctx->ev_slab[i], ctx->side) != cudaSuccess) s = DK_ERR_CUDA;
      }
      if (raw) xb_hi = full;
      for (int i = 0; i < nslab && s == DK_OK; ++i) {
        if (cudaStreamWaitEvent(st, ctx->ev_slab[i], 0) != cudaSuccess) { s = DK_ERR_CUDA; break; }
        ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
        s = tc_masked_fwd(ctx, gg, w_hi, w_lo, xb_hi, xb_lo, cv, bias, y, vs, reinterpret_cast<int*>(vs.count + 1),
                          fault, i == nslab - 1 ? verdict : nullptr, st, gt_lo[i], gt_lo[i + 1] - gt_lo[i], lo_in);
      }
      return s;
    }
    {
      // one launch: encodings and weights as hi/lo pairs, integrity statistics cleared
      ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
      s = stem ? tc_stem_fwd_prepass(g, x, r, cv.enc, xbar_save, xb_hi, xb_lo, W, w_hi, w_lo, vs, ctx->sm_count, st)
               : tc_fwd_prepass(gg, x, r, cv.enc, full, raw ? nullptr : xb_hi, xb_lo, W, w_hi, w_lo, vs,
                                prepass_clears ? ybar : nullptr, ctx->sm_count, st, raw);
      if (raw) xb_hi = full;
    }
    if (s != DK_OK) return s;
    if (ksplit > 1) {
      // too few tiles to fill the GPU: slice the contraction, let the slices
      // meet in y_bar (small here by construction) and decode in a second kernel
      {
        ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
        s = tc_linear_fwd(ctx, gg, w_hi, w_lo, xb_hi, xb_lo, ybar, ksplit, prepass_clears,
                          reinterpret_cast<int*>(vs.count + 1), st, cv.chunk_cap, lo_in);
      }
      if (s != DK_OK) return s;
      if (fault) {
        long long idx = ((long long)fault->group * g.E + fault->enc) * g.n_out + fault->out_index;
        ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
        s = launch_add_fault(ybar, idx, fault->delta, st);
        if (s != DK_OK) return s;
      }
      {
        ProfScope ps(ctx, DK_KERNEL_DECODE_VERIFY, 1, st);
        s = launch_decode_verify(gg, ybar, cv, bias, y, vs, ctx->sm_count, st);
      }
      if (s != DK_OK) return s;
      ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
      return launch_verify_finalize(gg, cv.nul, vs, verdict, st);
    }
    {
      ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
      s = tc_masked_fwd(ctx, gg, w_hi, w_lo, xb_hi, xb_lo, cv, bias, y, vs,
                        reinterpret_cast<int*>(vs.count + 1), fault, verdict, st, 0, -1, lo_in);
    }
    return s;      // the kernel's last CTA has written the verdict
  }
  if (g.precision == DK_FP64_SIMT && fused64_supported(g)) {
    // pointwise layers: one kernel encodes, contracts and decodes in fp64; nothing but x, r, W and y
    // (and the fp32 encodings, when stored) touches memory
    VerifyScratch vs = verify_scratch(ctx, g);
    {
      ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
      s = launch_verify_begin(g, vs, st);
    }
    if (s != DK_OK) return s;
    {
      ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
      s = launch_fused64(g, W, x, r, cv, bias, y, xbar_save, vs, fault, ctx->sm_count, st);
    }
    if (s != DK_OK) return s;
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    return launch_verify_finalize(g, cv.nul, vs, verdict, st);
  }
  if (g.precision == DK_FP64_SIMT) {
    // beyond-fp32 path: encodings and y_bar stay in the workspace as doubles
    // (the two adjacent hi/lo regions hold the fp64 encodings)
    double* x64 = reinterpret_cast<double*>(ws + wp.xb_hi);
    double* y64 = reinterpret_cast<double*>(ws + wp.ybar);
    VerifyScratch vs = verify_scratch(ctx, g);
    {
      ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
      s = launch_encode64(g, x, r, cv.enc, x64, xbar_save, ctx->sm_count, st);
    }
    if (s != DK_OK) return s;
    {
      ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
      s = launch_simt_fwd64(g, W, x64, y64, g.G * g.E, st);
    }
    if (s != DK_OK) return s;
    {
      ProfScope ps(ctx, DK_KERNEL_OTHER, fault ? 2 : 1, st);
      if (fault) {
        long long idx = ((long long)fault->group * g.E + fault->enc) * g.n_out + fault->out_index;
        s = launch_add_fault64(y64, idx, fault->delta, st);
      }
      if (s == DK_OK) s = launch_verify_begin(g, vs, st);
    }
    if (s != DK_OK) return s;
    {
      ProfScope ps(ctx, DK_KERNEL_DECODE_VERIFY, 1, st);
      s = launch_decode_verify64(g, y64, cv, bias, y, vs, ctx->sm_count, st);
    }
    if (s != DK_OK) return s;
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    return launch_verify_finalize(g, cv.nul, vs, verdict, st);
  }
  float* xbar = xbar_save ? xbar_save : reinterpret_cast<float*>(ws + wp.xbar);
  float* ybar = reinterpret_cast<float*>(ws + wp.ybar);
  {
    ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
    s = launch_encode(g, x, r, cv.enc, xbar, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  {
    ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
    s = launch_simt_fwd(g, W, xbar, ybar, g.G * g.E, st);
  }
  if (s != DK_OK) return s;
  if (fault) {
    long long idx = ((long long)fault->group * g.E + fault->enc) * g.n_out + fault->out_index;
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    s = launch_add_fault(ybar, idx, fault->delta, st);
    if (s != DK_OK) return s;
  }
  VerifyScratch vs = verify_scratch(ctx, g);
  {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    s = launch_verify_begin(g, vs, st);
  }
  if (s != DK_OK) return s;
  {
    ProfScope ps(ctx, DK_KERNEL_DECODE_VERIFY, 1, st);
    s = launch_decode_verify(g, ybar, cv, bias, y, vs, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
  return launch_verify_finalize(g, cv.nul, vs, verdict, st);
}

// Eq. 4-6 on encodings 0..K of every group of `xbar` (xbar_rows rows per group,
// `xbar_elems` readable elements from `xbar` on).
static dk_status wgrad_impl(dk_ctx* ctx, const Geom& g, const WsPlan& wp, const float* delta, const float* xbar,
                            int xbar_rows, long long xbar_elems, const float* C_host, const float* gamma_host,
                            float scale, float* dW, cudaStream_t st, bool accumulate = false) {
  CoefView cv;
  dk_status s = upload_coefficients(ctx, g, C_host, gamma_host, true, true, st, &cv);
  if (s != DK_OK) return s;
  float* dtil = reinterpret_cast<float*>(static_cast<char*>(ctx->ws) + wp.dtil);
  if (tc_wgrad_supported(ctx, g)) {
    // tensor-core path: mixed deltas and encodings as TF32 hi/lo pairs (the
    // y_bar region of the workspace, unused here, holds the lo part of dtil)
    char* ws = static_cast<char*>(ctx->ws);
    float* dt_lo = reinterpret_cast<float*>(ws + wp.ybar);
    float* xb_hi = reinterpret_cast<float*>(ws + wp.xb_hi);
    float* xb_lo = reinterpret_cast<float*>(ws + wp.xb_lo);
    const int raw = ctx->opt.v[DK_OPT_XBAR_HI];
    int nslab = 1, GT = 0, bg = 1;
    {
      long long rounds = 0;
      if (tc_wgrad_group_tiles(ctx, g, &GT, &bg, &rounds)) {
        const double prep = (g.K + 2.0 * (g.K + 1)) * g.G * (double)g.n_out * 4.0 +
                            (raw ? 2.0 : 3.0) * (g.K + 1) * g.G * (double)g.n_in * 4.0;
        // (every launch slices its own part of the contraction to fill the device, so what a further launch
        // costs is its fixed part: pipeline fill and the reductions into dW, about 15 us)
        nslab = plan_slabs(ctx, GT, 1LL << 30, prep, 6.0 * g.G * (g.K + 1) * (double)g.n_out * g.kc, 15e-6);
      }
    }
    if (nslab > 1) {
      // ranges of groups: the pre-passes in order on the second stream, each range's products on the caller's
      // stream once its pre-pass has finished (they add into dW, which the first pre-pass clears)
      SideStream fork(ctx, st);
      if (!fork.forked) return DK_ERR_CUDA;
      int gt_lo[kMaxSlabs + 1];
      for (int i = 0; i <= nslab; ++i) gt_lo[i] = (int)((long long)GT * i / nslab);
      for (int i = 0; i < nslab && s == DK_OK; ++i) {
        const int g_lo = gt_lo[i] * bg, g_hi = gt_lo[i + 1] * bg < g.G ? gt_lo[i + 1] * bg : g.G;
        {
          ProfScope ps(ctx, DK_KERNEL_MIX_DELTA, 1, ctx->side);
          s = tc_wgrad_prepass(g, delta, cv.dmix, dtil, dt_lo, xbar, xbar_elems, raw ? nullptr : xb_hi, xb_lo,
                               accumulate ? nullptr : dW, ctx->sm_count, ctx->side, raw, xbar_rows, g_lo, g_hi - g_lo,
                               i > 0);
        }
        if (s == DK_OK && cudaEventRecord(ctx->ev_slab[i], ctx->side) != cudaSuccess) s = DK_ERR_CUDA;
      }
      if (raw) xb_hi = const_cast<float*>(xbar);
      for (int i = 0; i < nslab && s == DK_OK; ++i) {
        if (cudaStreamWaitEvent(st, ctx->ev_slab[i], 0) != cudaSuccess) { s = DK_ERR_CUDA; break; }
        ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
        s = tc_wgrad(ctx, g, dtil, dt_lo, xb_hi, xb_lo, xbar_rows, scale, dW, ctx_status_word(ctx), st, gt_lo[i],
                     gt_lo[i + 1] - gt_lo[i]);
      }
      return s;
    }
    {
      // one launch: mixed deltas and stored encodings as hi/lo pairs, dW cleared
      ProfScope ps(ctx, DK_KERNEL_MIX_DELTA, 1, st);
      s = tc_wgrad_prepass(g, delta, cv.dmix, dtil, dt_lo, xbar, xbar_elems, raw ? nullptr : xb_hi, xb_lo,
                           accumulate ? nullptr : dW, ctx->sm_count, st, raw, xbar_rows);
      if (raw) xb_hi = const_cast<float*>(xbar);      // the stored encodings are the leading term
    }
    if (s != DK_OK) return s;
    ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
    return tc_wgrad(ctx, g, dtil, dt_lo, xb_hi, xb_lo, xbar_rows, scale, dW, ctx_status_word(ctx), st);
  }
  if (ctx->opt.v[DK_OPT_TC_STEM] == 1 && stem_wgrad_fused_supported(g, tc_smem_optin(ctx))) {
    // 3x3 stem on 3 channels: one fp32 kernel mixes the gradients (Eq. 4) and forms the products
    ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
    return launch_stem_wgrad(g, delta, xbar, xbar_rows, cv.dmix, scale, dW, !accumulate, ctx->sm_count, st);
  }
  {
    ProfScope ps(ctx, DK_KERNEL_MIX_DELTA, 1, st);
    s = launch_mix_delta(g, delta, cv.dmix, dtil, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
  return launch_simt_wgrad(g, dtil, xbar, xbar_rows, scale, dW, ctx->sm_count, st, !accumulate);
}

dk_status dk_linear_bwd_wgrad(dk_ctx* ctx, const dk_problem* p, const float* delta,
                              const float* xbar, int32_t xbar_rows, const float* C_host,
                              const float* gamma_host, float scale, float* dW, void* stream) {
  if (!ctx || !delta || !xbar || !C_host || !gamma_host || !dW) return DK_ERR_INVALID_ARG;
  if (!aligned16(delta) || !aligned16(xbar) || !aligned16(dW)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  if (xbar_rows != g.K + 1 && xbar_rows != g.K + 2) return DK_ERR_INVALID_ARG;
  WsPlan wp = plan_workspace(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  return wgrad_impl(ctx, g, wp, delta, xbar, xbar_rows, (long long)g.G * xbar_rows * g.n_in, C_host, gamma_host,
                    scale, dW, static_cast<cudaStream_t>(stream));
}

dk_status dk_linear_bwd_wgrad_accumulate(dk_ctx* ctx, const dk_problem* p, const float* delta, const float* xbar,
                                         int32_t xbar_rows, const float* C_host, const float* gamma_host,
                                         float scale, float* dW, void* stream) {
  if (!ctx || !delta || !xbar || !C_host || !gamma_host || !dW) return DK_ERR_INVALID_ARG;
  if (!aligned16(delta) || !aligned16(xbar) || !aligned16(dW)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  if (xbar_rows != g.K + 1 && xbar_rows != g.K + 2) return DK_ERR_INVALID_ARG;
  WsPlan wp = plan_workspace(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  return wgrad_impl(ctx, g, wp, delta, xbar, xbar_rows, (long long)g.G * xbar_rows * g.n_in, C_host, gamma_host,
                    scale, dW, static_cast<cudaStream_t>(stream), true);
}

dk_status dk_linear_bwd_wgrad_verify(dk_ctx* ctx, const dk_problem* p, const float* delta, const float* xbar,
                                     const float* C_host, const float* gamma_host, float scale, float tol_w,
                                     float* dW, dk_verdict* verdict, const dk_fault* fault, void* stream) {
  if (!ctx || !delta || !xbar || !C_host || !gamma_host || !dW || !verdict) return DK_ERR_INVALID_ARG;
  if (!aligned16(delta) || !aligned16(xbar) || !aligned16(dW) || !aligned16(verdict)) return DK_ERR_INVALID_ARG;
  if (!(tol_w > 0.f)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  if (g.n_in % 4) return DK_ERR_UNSUPPORTED;      // the second set starts one row into xbar: keep it 16-byte aligned
  const long long n_dw = (long long)g.cout * g.kc;
  if (fault && (fault->enc < 0 || fault->enc > 1 || fault->out_index < 0 || fault->out_index >= n_dw))
    return DK_ERR_INVALID_ARG;
  WsPlan wp = plan_workspace(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int K1 = g.K + 1, E = g.E;
  // first set: encodings 0..K with C and gamma as given
  s = wgrad_impl(ctx, g, wp, delta, xbar, E, (long long)g.G * E * g.n_in, C_host, gamma_host, scale, dW, st);
  if (s != DK_OK) return s;
  // second set: encodings 1..K+1 = rows 0..K of the tensor that starts one row
  // later; its square coefficient part is rows 1..K+1 of C, its gammas rotated
  std::vector<float> C2((size_t)g.G * E * K1), g2((size_t)g.G * K1);
  for (int gi = 0; gi < g.G; ++gi) {
    for (int i = 0; i < E; ++i)
      for (int k = 0; k < K1; ++k)
        C2[((size_t)gi * E + i) * K1 + k] = C_host[((size_t)gi * E + (i + 1) % E) * K1 + k];
    for (int j = 0; j < K1; ++j) g2[(size_t)gi * K1 + j] = gamma_host[(size_t)gi * K1 + (j + 1) % K1];
  }
  float* dW2 = reinterpret_cast<float*>(static_cast<char*>(ctx->ws) + wp.w_hi);      // unused by the wgrad path
  s = wgrad_impl(ctx, g, wp, delta, xbar + g.n_in, E, ((long long)g.G * E - 1) * g.n_in, C2.data(), g2.data(), scale,
                 dW2, st);
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_OTHER, fault ? 4 : 3, st);
  if (fault) {
    s = launch_add_fault(fault->enc == 0 ? dW : dW2, fault->out_index, fault->delta, st);
    if (s != DK_OK) return s;
  }
  // 32 bytes of scratch behind the integrity statistics' counters
  void* scratch = ctx->d_vstats + kVerifyStatFloats + 16;
  return launch_wgrad_compare(dW, dW2, n_dw, tol_w, scratch, ctx_status_word(ctx), verdict, ctx->sm_count, st);
}

dk_status dk_device_status(dk_ctx* ctx, int32_t* status) {
  if (!ctx || !status) return DK_ERR_INVALID_ARG;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  int v = 0;
  DK_CUDA_CHECK(cudaDeviceSynchronize());
  DK_CUDA_CHECK(cudaMemcpy(&v, ctx_status_word(ctx), sizeof(int), cudaMemcpyDeviceToHost));
  if (v != 0) DK_CUDA_CHECK(cudaMemset(ctx_status_word(ctx), 0, sizeof(int)));
  *status = v;
  return DK_OK;
}

dk_status dk_profile_enable(dk_ctx* ctx, int on) {
  if (!ctx || !ctx->prof) return DK_ERR_INVALID_ARG;
  ctx->prof->on = on != 0;
  return DK_OK;
}

dk_status dk_profile_read(dk_ctx* ctx, int kind, double* ms_total, int64_t* timed_launches,
                          int64_t* all_launches) {
  if (!ctx || !ctx->prof || kind < 0 || kind >= DK_KERNEL_KINDS) return DK_ERR_INVALID_ARG;
  DeviceGuard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  ProfState* ps = ctx->prof;
  double ms = 0.0;
  int64_t n = 0;
  for (size_t i = 0; i < ps->kind_of.size(); ++i) {
    if (ps->kind_of[i] != kind) continue;
    float t = 0.f;
    DK_CUDA_CHECK(cudaEventSynchronize(ps->ev[2 * i + 1]));
    DK_CUDA_CHECK(cudaEventElapsedTime(&t, ps->ev[2 * i], ps->ev[2 * i + 1]));
    ms += t;
    ++n;
  }
  if (ms_total) *ms_total = ms;
  if (timed_launches) *timed_launches = n;
  if (all_launches) *all_launches = ps->launches[kind];
  return DK_OK;
}

dk_status dk_profile_reset(dk_ctx* ctx) {
  if (!ctx || !ctx->prof) return DK_ERR_INVALID_ARG;
  ctx->prof->kind_of.clear();
  for (int k = 0; k < DK_KERNEL_KINDS; ++k) ctx->prof->launches[k] = 0;
  return DK_OK;
}

}  // extern "C"
