// fp32 SIMT implicit-GEMM kernels for the bilinear operation <W, x> and for
// the weight-gradient product <delta, x>.  They accept every geometry and
// layout (addresses go through element strides) and are the DK_FP32_SIMT
// arithmetic as well as the fallback for shapes the tensor-core path does not
// take.  Accumulation is two-level (a short running sum is folded into the
// total every few k-tiles) so that rounding at the scale of the masking noise
// grows with the square root of the chunk length rather than of the whole
// contraction.
#include "dk_internal.h"

namespace dk {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;
constexpr int kFold = 4;   // fold the running sum every kFold k-tiles

__device__ __forceinline__ float fma_t(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double fma_t(double a, double b, double c) { return fma(a, b, c); }

// T = type of the activations, of the accumulators and of the output: float,
// or double for the regime in which fp32 cannot hold the signal next to the noise.
template <typename T>
struct FwdParams {
  const float* W;
  const T* x;
  T* y;
  int cin, cout, h, w, kw, stride, pad, ho, wo, kc;
  long long N;           // samples * ho * wo
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
};

template <typename T>
__global__ void __launch_bounds__(NT) simt_fwd_kernel(FwdParams<T> p) {
  __shared__ T As[BK][BM + 4];
  __shared__ T Bs[BK][BN + 4];
  const int t = threadIdx.x;
  const int tx = t % 16, ty = t / 16;
  const int m0 = blockIdx.y * BM;
  const long long n0 = (long long)blockIdx.x * BN;

  // load slots: element (kk, mm) with kk = t % 16, mm = t / 16 + 16*i
  const int kk = t % BK;
  long long a_off[4];
  bool a_ok[4];
  long long b_base[4];
  int b_ih0[4], b_iw0[4];
  bool b_ok[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int mm = t / BK + 16 * i;
    a_ok[i] = (m0 + mm) < p.cout;
    a_off[i] = (long long)(m0 + mm) * p.ws_o;
    long long n = n0 + mm;
    b_ok[i] = n < p.N;
    long long nn = b_ok[i] ? n : 0;
    int ow = (int)(nn % p.wo);
    long long r = nn / p.wo;
    int oh = (int)(r % p.ho);
    long long s = r / p.ho;
    b_base[i] = s * p.n_in;
    b_ih0[i] = oh * p.stride - p.pad;
    b_iw0[i] = ow * p.stride - p.pad;
  }

  T tot[4][4], acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) tot[i][j] = acc[i][j] = T(0);

  int fold = 0;
  for (int k0 = 0; k0 < p.kc; k0 += BK) {
    const int k = k0 + kk;
    const bool kok = k < p.kc;
    int tap = kok ? k / p.cin : 0;
    int ci = kok ? k - tap * p.cin : 0;
    int u = tap / p.kw, v = tap - u * p.kw;
    long long woff = (long long)ci * p.ws_c + (long long)u * p.ws_u + (long long)v * p.ws_v;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int mm = t / BK + 16 * i;
      As[kk][mm] = (kok && a_ok[i]) ? T(__ldg(p.W + a_off[i] + woff)) : T(0);
      int ih = b_ih0[i] + u, iw = b_iw0[i] + v;
      bool ok = kok && b_ok[i] && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
      Bs[kk][mm] = ok ? __ldg(p.x + b_base[i] + (long long)ci * p.xs_c + (long long)ih * p.xs_h +
                              (long long)iw * p.xs_w)
                      : T(0);
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < BK; ++q) {
      T a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[q][ty * 4 + i]; b[i] = Bs[q][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma_t(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
    if (++fold == kFold) {
      fold = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { tot[i][j] += acc[i][j]; acc[i][j] = T(0); }
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    long long n = n0 + tx * 4 + j;
    if (n >= p.N) continue;
    int ow = (int)(n % p.wo);
    long long r = n / p.wo;
    int oh = (int)(r % p.ho);
    long long s = r / p.ho;
    T* yo = p.y + s * p.n_out + (long long)oh * p.ys_h + (long long)ow * p.ys_w;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int m = m0 + ty * 4 + i;
      if (m < p.cout) yo[(long long)m * p.ys_c] = tot[i][j] + acc[i][j];
    }
  }
}

struct WgParams {
  const float* d;     // mixed deltas [G*(K+1)][n_out]
  const float* x;     // encodings, xbar_rows per group
  float* dW;
  int cin, cout, h, w, kw, stride, pad, ho, wo, kc;
  int K1, xbar_rows, P, PC;   // P = ho*wo pixels, PC = ceil(P/BK)
  long long GP;               // G * PC contraction blocks
  long long per_split;
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
  float scale;
};

// dW[m][k] += scale * sum over (group, pixel block, encoding j) with j
// innermost, so that the noise carried by the K+1 encodings cancels within
// K+1 consecutive k-tiles and the accumulators stay at signal scale.
__global__ void __launch_bounds__(NT) simt_wgrad_kernel(WgParams p) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int t = threadIdx.x;
  const int tx = t % 16, ty = t / 16;
  const int m0 = blockIdx.y * BM;
  const int kb0 = blockIdx.x * BN;
  const long long gp_lo = (long long)blockIdx.z * p.per_split;
  long long gp_hi = gp_lo + p.per_split;
  if (gp_hi > p.GP) gp_hi = p.GP;

  // load slots: (pixel pp = t / 64 + 4*i, column cc = t % 64)
  const int cc = t % 64;
  const bool a_ok = (m0 + cc) < p.cout;
  const long long a_off = (long long)(m0 + cc) * p.ys_c;
  const int kcol = kb0 + cc;
  const bool b_ok = kcol < p.kc;
  int tap = b_ok ? kcol / p.cin : 0;
  int ci = b_ok ? kcol - tap * p.cin : 0;
  const int u = tap / p.kw, v = tap - u * p.kw;
  const long long b_off = (long long)ci * p.xs_c;

  float tot[4][4], acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) tot[i][j] = acc[i][j] = 0.f;

  for (long long gp = gp_lo; gp < gp_hi; ++gp) {
    const long long g = gp / p.PC;
    const int pc = (int)(gp - g * p.PC);
    int oh[4], ow[4];
    bool pok[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int pix = pc * BK + t / 64 + 4 * i;
      pok[i] = pix < p.P;
      int pp = pok[i] ? pix : 0;
      oh[i] = pp / p.wo;
      ow[i] = pp - oh[i] * p.wo;
    }
    for (int j = 0; j < p.K1; ++j) {
      const float* dj = p.d + (g * p.K1 + j) * p.n_out;
      const float* xj = p.x + (g * p.xbar_rows + j) * p.n_in;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int pp = t / 64 + 4 * i;
        As[pp][cc] = (pok[i] && a_ok)
                         ? __ldg(dj + a_off + (long long)oh[i] * p.ys_h + (long long)ow[i] * p.ys_w)
                         : 0.f;
        int ih = oh[i] * p.stride + u - p.pad, iw = ow[i] * p.stride + v - p.pad;
        bool ok = pok[i] && b_ok && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
        Bs[pp][cc] = ok ? __ldg(xj + b_off + (long long)ih * p.xs_h + (long long)iw * p.xs_w) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < BK; ++q) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { a[i] = As[q][ty * 4 + i]; b[i] = Bs[q][tx * 4 + i]; }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(a[i], b[jj], acc[i][jj]);
      }
      __syncthreads();
    }
    // one whole cycle of encodings done: the noise has cancelled, fold
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) { tot[i][jj] += acc[i][jj]; acc[i][jj] = 0.f; }
  }
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    int kcol2 = kb0 + tx * 4 + jj;
    if (kcol2 >= p.kc) continue;
    int tap2 = kcol2 / p.cin, ci2 = kcol2 - tap2 * p.cin;
    int u2 = tap2 / p.kw, v2 = tap2 - u2 * p.kw;
    long long woff = (long long)ci2 * p.ws_c + (long long)u2 * p.ws_u + (long long)v2 * p.ws_v;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int m = m0 + ty * 4 + i;
      if (m < p.cout) atomicAdd(p.dW + (long long)m * p.ws_o + woff, p.scale * tot[i][jj]);
    }
  }
}

}  // namespace

namespace {
template <typename T>
dk_status launch_fwd_t(const Geom& g, const float* W, const T* xbar, T* ybar, int nsamples,
                       cudaStream_t st) {
  FwdParams<T> p;
  p.W = W; p.x = xbar; p.y = ybar;
  p.cin = g.cin; p.cout = g.cout; p.h = g.h; p.w = g.w; p.kw = g.kw; p.stride = g.stride;
  p.pad = g.pad; p.ho = g.ho; p.wo = g.wo; p.kc = g.kc;
  p.N = (long long)nsamples * g.ho * g.wo;
  p.n_in = g.n_in; p.n_out = g.n_out;
  p.xs_c = g.xs_c; p.xs_h = g.xs_h; p.xs_w = g.xs_w;
  p.ws_o = g.ws_o; p.ws_c = g.ws_c; p.ws_u = g.ws_u; p.ws_v = g.ws_v;
  p.ys_c = g.ys_c; p.ys_h = g.ys_h; p.ys_w = g.ys_w;
  long long nb = (p.N + BN - 1) / BN;
  if (nb > 2147483647LL) return DK_ERR_SHAPE;
  dim3 grid((unsigned)nb, (unsigned)((g.cout + BM - 1) / BM));
  if (grid.y > 65535) return DK_ERR_SHAPE;
  simt_fwd_kernel<T><<<grid, NT, 0, st>>>(p);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}
}  // namespace

dk_status launch_simt_fwd(const Geom& g, const float* W, const float* xbar, float* ybar,
                          int nsamples, cudaStream_t st) {
  return launch_fwd_t<float>(g, W, xbar, ybar, nsamples, st);
}

dk_status launch_simt_fwd64(const Geom& g, const float* W, const double* xbar, double* ybar,
                            int nsamples, cudaStream_t st) {
  return launch_fwd_t<double>(g, W, xbar, ybar, nsamples, st);
}

dk_status launch_simt_wgrad(const Geom& g, const float* dtil, const float* xbar, int xbar_rows,
                            float scale, float* dW, int sm_count, cudaStream_t st, bool clear) {
  WgParams p;
  p.d = dtil; p.x = xbar; p.dW = dW;
  p.cin = g.cin; p.cout = g.cout; p.h = g.h; p.w = g.w; p.kw = g.kw; p.stride = g.stride;
  p.pad = g.pad; p.ho = g.ho; p.wo = g.wo; p.kc = g.kc;
  p.K1 = g.K + 1; p.xbar_rows = xbar_rows;
  p.P = g.ho * g.wo;
  p.PC = (p.P + BK - 1) / BK;
  p.GP = (long long)g.G * p.PC;
  p.n_in = g.n_in; p.n_out = g.n_out;
  p.xs_c = g.xs_c; p.xs_h = g.xs_h; p.xs_w = g.xs_w;
  p.ws_o = g.ws_o; p.ws_c = g.ws_c; p.ws_u = g.ws_u; p.ws_v = g.ws_v;
  p.ys_c = g.ys_c; p.ys_h = g.ys_h; p.ys_w = g.ys_w;
  p.scale = scale;
  long long tiles = (long long)((g.cout + BM - 1) / BM) * ((g.kc + BN - 1) / BN);
  long long splits = (4LL * sm_count + tiles - 1) / tiles;
  if (splits > p.GP) splits = p.GP;
  if (splits > 65535) splits = 65535;
  if (splits < 1) splits = 1;
  p.per_split = (p.GP + splits - 1) / splits;
  splits = (p.GP + p.per_split - 1) / p.per_split;
  if (clear) DK_CUDA_CHECK(cudaMemsetAsync(dW, 0, (size_t)g.cout * g.kc * sizeof(float), st));
  dim3 grid((unsigned)((g.kc + BN - 1) / BN), (unsigned)((g.cout + BM - 1) / BM), (unsigned)splits);
  if (grid.y > 65535) return DK_ERR_SHAPE;
  simt_wgrad_kernel<<<grid, NT, 0, st>>>(p);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
