// The unmasked steps that chain the masked products into a training step:
// back-propagation of the output gradient through a linear layer (Section 4.2:
// computed from delta and W "without encoding"), ReLU / 2x2 max pooling (the
// non-linear layers of the Section 3.1 flow), forward and backward.
//
// dgrad.  dx = <delta, W> is the adjoint of the layer.  For a stride-1
// convolution it is itself a convolution of delta with the filters flipped and
// their channel roles exchanged, with padding k-1-pad; that form runs on the
// tensor-core implicit-GEMM kernel (plain 3xTF32, no decode), the batch being
// presented to it as virtual batches of E' samples.  Everything else (strides,
// layouts, channel counts the tensor-core kernel does not take) runs on a
// gather kernel in fp32.
#include "dk_internal.h"
#include "dk_tc_kernel.cuh"

namespace dk {
namespace {

using tc::to_tf32;

// Wt[c][kh-1-u][kw-1-v][o] = W[o][u][v][c], written as a TF32 hi/lo pair.
// One 32x32 tile of the (o, c) plane of one filter tap per block.
__global__ void __launch_bounds__(256)
dgrad_weights_kernel(const float* __restrict__ W, float* __restrict__ hi, float* __restrict__ lo, int cout, int cin,
                     int kh, int kw) {
  __shared__ float tile[32][33];
  const int tap = blockIdx.z, u = tap / kw, v = tap - u * kw;
  const int tap_t = (kh - 1 - u) * kw + (kw - 1 - v);
  const int o0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int taps = kh * kw;
  for (int r = ty; r < 32; r += 8) {
    const int o = o0 + r, c = c0 + tx;
    tile[r][tx] = (o < cout && c < cin) ? __ldg(W + ((size_t)o * taps + tap) * cin + c) : 0.f;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int c = c0 + r, o = o0 + tx;
    if (c < cin && o < cout) {
      const float val = tile[tx][r];
      const float h = to_tf32(val);
      const size_t idx = ((size_t)c * taps + tap_t) * cout + o;
      hi[idx] = h;
      lo[idx] = to_tf32(val - h);
    }
  }
}

struct DgradParams {
  const float* W;
  const float* d;
  float* dx;
  int cin, cout, h, w, kh, kw, stride, pad, ho, wo;
  long long total;          // samples * n_in
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
};

// dx[n][c][i][j] = sum over (o, u, v) with i = p*stride + u - pad, j = q*stride + v - pad
// of delta[n][o][p][q] * W[o][c][u][v]; one thread per input element.
__global__ void __launch_bounds__(256) simt_dgrad_kernel(const DgradParams p) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < p.total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long n = e / p.n_in;
    long long r = e - n * p.n_in;
    int c, i, j;
    if (p.xs_c == 1) {            // channels-last (and FC)
      c = (int)(r % p.cin); r /= p.cin;
      j = (int)(r % p.w); i = (int)(r / p.w);
    } else {
      j = (int)(r % p.w); r /= p.w;
      i = (int)(r % p.h); c = (int)(r / p.h);
    }
    const float* dn = p.d + n * p.n_out;
    float tot = 0.f;
    for (int u = 0; u < p.kh; ++u) {
      const int a = i + p.pad - u;
      if (a < 0 || a % p.stride) continue;
      const int pp = a / p.stride;
      if (pp >= p.ho) continue;
      for (int v = 0; v < p.kw; ++v) {
        const int b = j + p.pad - v;
        if (b < 0 || b % p.stride) continue;
        const int q = b / p.stride;
        if (q >= p.wo) continue;
        const float* dpq = dn + (long long)pp * p.ys_h + (long long)q * p.ys_w;
        const float* wuv = p.W + (long long)c * p.ws_c + (long long)u * p.ws_u + (long long)v * p.ws_v;
        float acc = 0.f;
        for (int o = 0; o < p.cout; ++o)
          acc = fmaf(__ldg(dpq + (long long)o * p.ys_c), __ldg(wuv + (long long)o * p.ws_o), acc);
        tot += acc;
      }
    }
    p.dx[n * p.n_in + (long long)c * p.xs_c + (long long)i * p.xs_h + (long long)j * p.xs_w] = tot;
  }
}

template <int VEC>
__device__ __forceinline__ void ldv(const float* p, float* out) {
  if constexpr (VEC == 4) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
  } else {
    out[0] = __ldg(p);
  }
}
template <int VEC>
__device__ __forceinline__ void stv(float* p, const float* v) {
  if constexpr (VEC == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  else p[0] = v[0];
}

// y = relu(x) (POOL = false) or maxpool2x2(relu(x)); channels-last, VEC floats per thread along c.
template <bool POOL, int VEC>
__global__ void __launch_bounds__(256)
relu_pool_fwd_kernel(const float* __restrict__ x, float* __restrict__ y, long long n, int h, int w, int c) {
  const int cv = c / VEC;
  const int ho = POOL ? h / 2 : h, wo = POOL ? w / 2 : w;
  const long long total = n * ho * wo * cv;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const int ch = (int)(e % cv) * VEC;
    long long r = e / cv;
    const int q = (int)(r % wo); r /= wo;
    const int pp = (int)(r % ho);
    const long long s = r / ho;
    float out[VEC], in[VEC];
    if (!POOL) {
      ldv<VEC>(x + ((s * h + pp) * w + q) * c + ch, in);
#pragma unroll
      for (int k = 0; k < VEC; ++k) out[k] = fmaxf(in[k], 0.f);
    } else {
#pragma unroll
      for (int k = 0; k < VEC; ++k) out[k] = 0.f;           // relu >= 0, so 0 is the identity of the max
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        ldv<VEC>(x + ((s * h + 2 * pp + (t >> 1)) * w + 2 * q + (t & 1)) * c + ch, in);
#pragma unroll
        for (int k = 0; k < VEC; ++k) out[k] = fmaxf(out[k], in[k]);
      }
    }
    stv<VEC>(y + ((s * ho + pp) * wo + q) * c + ch, out);
  }
}

// dx = relu'(x) . dy (POOL = false), or the gradient of maxpool2x2(relu(x)): dy goes to the first
// maximum of relu(x) in the window (row-major order) and passes only where x > 0.  Rows and columns of
// an odd-sized image that no window covers get zero.
template <bool POOL, int VEC>
__global__ void __launch_bounds__(256)
relu_pool_bwd_kernel(const float* __restrict__ dy, const float* __restrict__ x, float* __restrict__ dx, long long n,
                     int h, int w, int c) {
  const int cv = c / VEC;
  const int ho = POOL ? (h + 1) / 2 : h, wo = POOL ? (w + 1) / 2 : w;      // windows incl. the ragged border
  const int hp = h / 2, wp = w / 2;
  const long long total = n * ho * wo * cv;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const int ch = (int)(e % cv) * VEC;
    long long r = e / cv;
    const int q = (int)(r % wo); r /= wo;
    const int pp = (int)(r % ho);
    const long long s = r / ho;
    if (!POOL) {
      const long long off = ((s * h + pp) * w + q) * c + ch;
      float xv[VEC], gv[VEC];
      ldv<VEC>(x + off, xv);
      ldv<VEC>(dy + off, gv);
#pragma unroll
      for (int k = 0; k < VEC; ++k) gv[k] = xv[k] > 0.f ? gv[k] : 0.f;
      stv<VEC>(dx + off, gv);
      continue;
    }
    const bool covered = pp < hp && q < wp;
    float g[VEC], xv[4][VEC], out[4][VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) g[k] = 0.f;
    if (covered) ldv<VEC>(dy + ((s * hp + pp) * wp + q) * c + ch, g);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int i = 2 * pp + (t >> 1), j = 2 * q + (t & 1);
#pragma unroll
      for (int k = 0; k < VEC; ++k) xv[t][k] = 0.f;
      if (i < h && j < w) ldv<VEC>(x + ((s * h + i) * w + j) * c + ch, xv[t]);
    }
#pragma unroll
    for (int k = 0; k < VEC; ++k) {
      float best = fmaxf(xv[0][k], 0.f);
      int arg = 0;
#pragma unroll
      for (int t = 1; t < 4; ++t) {
        const float rv = fmaxf(xv[t][k], 0.f);
        if (rv > best) { best = rv; arg = t; }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) out[t][k] = (covered && t == arg && xv[t][k] > 0.f) ? g[k] : 0.f;
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int i = 2 * pp + (t >> 1), j = 2 * q + (t & 1);
      if (i < h && j < w) stv<VEC>(dx + ((s * h + i) * w + j) * c + ch, out[t]);
    }
  }
}

int grid_for(long long items, int sm_count) {
  long long b = (items + 255) / 256;
  const long long cap = (long long)sm_count * 16;
  if (b > cap) b = cap;
  return b < 1 ? 1 : (int)b;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

// Geometry of the convolution that computes dx from delta on the tensor-core
// kernel: `batch` samples as G' virtual batches of E' = K' + 2.  Returns false
// when the layer has no such form (stride > 1, non-square filter, pad > k-1,
// batch without a divisor in 3..10).
static bool dgrad_conv_geom(const Geom& g, Geom* t) {
  if (g.layout != DK_NHWC || g.stride != 1 || g.kh != g.kw || g.pad > g.kh - 1) return false;
  if ((g.cout % 4) != 0 || (g.cin % 4) != 0) return false;
  const long long batch = (long long)g.G * g.K;
  int E2 = 0;
  for (int e : {4, 6, 8, 10, 3, 5, 7, 9})
    if (batch % e == 0) { E2 = e; break; }
  if (!E2) return false;
  dk_problem q;
  q.kind = g.kind; q.layout = DK_NHWC;
  q.cin = g.cout; q.cout = g.cin;
  q.h = g.ho; q.w = g.wo; q.kh = g.kh; q.kw = g.kw; q.stride = 1; q.pad = g.kh - 1 - g.pad;
  q.K = E2 - 2; q.G = (int)(batch / E2);
  q.precision = DK_TF32X3; q.tol = 0.f;
  if (make_geom(&q, t) != DK_OK) return false;
  return t->ho == g.h && t->wo == g.w;
}

}  // namespace dk

using namespace dk;

extern "C" {

dk_status dk_linear_bwd_dgrad(dk_ctx* ctx, const dk_problem* p, const float* W, const float* delta, float* dx,
                              void* stream) {
  if (!ctx || !W || !delta || !dx) return DK_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(delta) || !aligned16(dx)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return DK_ERR_CUDA;
  if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Geom t;
  const long long batch = (long long)g.G * g.K;
  if (g.precision == DK_TF32X3 && dgrad_conv_geom(g, &t) && tc_fwd_supported(ctx, t)) {
    // workspace (sized by dk_workspace_bytes for this layer): the y_bar region holds delta as a hi/lo
    // pair, the W regions hold the flipped filters
    size_t need = 0;
    s = dk_workspace_bytes(p, &need);
    if (s == DK_OK && (!ctx->ws || ctx->ws_bytes < need)) s = DK_ERR_WORKSPACE;
    if (s == DK_OK) {
      char* ws = static_cast<char*>(ctx->ws);
      size_t off_ybar = 0, off_whi = 0, off_wlo = 0;
      workspace_offsets(g, &off_ybar, &off_whi, &off_wlo);
      float* d_hi = reinterpret_cast<float*>(ws + off_ybar);
      float* d_lo = d_hi + (((size_t)batch * g.n_out + 3) / 4) * 4;
      float* w_hi = reinterpret_cast<float*>(ws + off_whi);
      float* w_lo = reinterpret_cast<float*>(ws + off_wlo);
      {
        ProfScope ps(ctx, DK_KERNEL_OTHER, 2, st);
        dim3 grid((unsigned)((g.cin + 31) / 32), (unsigned)((g.cout + 31) / 32), (unsigned)(g.kh * g.kw));
        dgrad_weights_kernel<<<grid, 256, 0, st>>>(W, w_hi, w_lo, g.cout, g.cin, g.kh, g.kw);
        if (cudaGetLastError() != cudaSuccess) s = DK_ERR_CUDA;
        if (s == DK_OK) s = tc_split(delta, d_hi, d_lo, batch * g.n_out, ctx->sm_count, st);
      }
      if (s == DK_OK) {
        ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
        s = tc_linear_fwd(ctx, t, w_hi, w_lo, d_hi, d_lo, dx, tc_fwd_ksplit(ctx, t), false, device_status_word(ctx), st);
      }
    }
  } else {
    DgradParams q;
    q.W = W; q.d = delta; q.dx = dx;
    q.cin = g.cin; q.cout = g.cout; q.h = g.h; q.w = g.w; q.kh = g.kh; q.kw = g.kw;
    q.stride = g.stride; q.pad = g.pad; q.ho = g.ho; q.wo = g.wo;
    q.total = batch * g.n_in; q.n_in = g.n_in; q.n_out = g.n_out;
    q.xs_c = g.xs_c; q.xs_h = g.xs_h; q.xs_w = g.xs_w;
    q.ws_o = g.ws_o; q.ws_c = g.ws_c; q.ws_u = g.ws_u; q.ws_v = g.ws_v;
    q.ys_c = g.ys_c; q.ys_h = g.ys_h; q.ys_w = g.ys_w;
    ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
    simt_dgrad_kernel<<<grid_for(q.total, ctx->sm_count), 256, 0, st>>>(q);
    if (cudaGetLastError() != cudaSuccess) s = DK_ERR_CUDA;
  }
  if (prev != ctx->device) cudaSetDevice(prev);
  return s;
}

static dk_status relu_pool_args(dk_ctx* ctx, const void* a, const void* b, const void* c, int64_t n, int32_t h,
                                int32_t w, int32_t ch, int32_t pool) {
  if (!ctx || !a || !b || !c) return DK_ERR_INVALID_ARG;
  if (!aligned16(a) || !aligned16(b) || !aligned16(c)) return DK_ERR_INVALID_ARG;
  if (n < 1 || h < 1 || w < 1 || ch < 1) return DK_ERR_SHAPE;
  if (pool && (h < 2 || w < 2)) return DK_ERR_SHAPE;
  return DK_OK;
}

dk_status dk_relu_pool_fwd(dk_ctx* ctx, const float* x, int64_t n, int32_t h, int32_t w, int32_t c, int32_t pool,
                           float* y, void* stream) {
  dk_status s = relu_pool_args(ctx, x, y, y, n, h, w, c, pool);
  if (s != DK_OK) return s;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return DK_ERR_CUDA;
  if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int ho = pool ? h / 2 : h, wo = pool ? w / 2 : w;
  {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    if (c % 4 == 0) {
      const int grid = grid_for((long long)n * ho * wo * (c / 4), ctx->sm_count);
      if (pool) relu_pool_fwd_kernel<true, 4><<<grid, 256, 0, st>>>(x, y, n, h, w, c);
      else relu_pool_fwd_kernel<false, 4><<<grid, 256, 0, st>>>(x, y, n, h, w, c);
    } else {
      const int grid = grid_for((long long)n * ho * wo * c, ctx->sm_count);
      if (pool) relu_pool_fwd_kernel<true, 1><<<grid, 256, 0, st>>>(x, y, n, h, w, c);
      else relu_pool_fwd_kernel<false, 1><<<grid, 256, 0, st>>>(x, y, n, h, w, c);
    }
    if (cudaGetLastError() != cudaSuccess) s = DK_ERR_CUDA;
  }
  if (prev != ctx->device) cudaSetDevice(prev);
  return s;
}

dk_status dk_relu_pool_bwd(dk_ctx* ctx, const float* dy, const float* x, int64_t n, int32_t h, int32_t w, int32_t c,
                           int32_t pool, float* dx, void* stream) {
  dk_status s = relu_pool_args(ctx, dy, x, dx, n, h, w, c, pool);
  if (s != DK_OK) return s;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return DK_ERR_CUDA;
  if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int ho = pool ? (h + 1) / 2 : h, wo = pool ? (w + 1) / 2 : w;
  {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    if (c % 4 == 0) {
      const int grid = grid_for((long long)n * ho * wo * (c / 4), ctx->sm_count);
      if (pool) relu_pool_bwd_kernel<true, 4><<<grid, 256, 0, st>>>(dy, x, dx, n, h, w, c);
      else relu_pool_bwd_kernel<false, 4><<<grid, 256, 0, st>>>(dy, x, dx, n, h, w, c);
    } else {
      const int grid = grid_for((long long)n * ho * wo * c, ctx->sm_count);
      if (pool) relu_pool_bwd_kernel<true, 1><<<grid, 256, 0, st>>>(dy, x, dx, n, h, w, c);
      else relu_pool_bwd_kernel<false, 1><<<grid, 256, 0, st>>>(dy, x, dx, n, h, w, c);
    }
    if (cudaGetLastError() != cudaSuccess) s = DK_ERR_CUDA;
  }
  if (prev != ctx->device) cudaSetDevice(prev);
  return s;
}

}  // extern "C"
