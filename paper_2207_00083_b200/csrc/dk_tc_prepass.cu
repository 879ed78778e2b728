// Fused HBM-bound pre-passes of the tensor-core path.
//
// A masked forward call needs three independent pieces of preparation: the
// encodings of Eq. 1 as TF32 hi/lo pairs, the weights as a hi/lo pair, and
// cleared integrity statistics; a weight-gradient call needs the mixed deltas
// of Eq. 4 and the stored encodings as hi/lo pairs and a cleared dW.  Each
// piece is a grid-stride loop with nothing to share with the others, so one
// launch serves all three with disjoint ranges of blocks.  On small layers
// every launch saved is a few microseconds of a call that lasts ~100.
#include "dk_internal.h"
#include "dk_tc_kernel.cuh"

namespace dk {
namespace {

using tc::to_tf32;

__device__ __forceinline__ void split4(const float4& v, float4& h, float4& l) {
  h.x = to_tf32(v.x); l.x = to_tf32(v.x - h.x);
  h.y = to_tf32(v.y); l.y = to_tf32(v.y - h.y);
  h.z = to_tf32(v.z); l.z = to_tf32(v.z - h.z);
  h.w = to_tf32(v.w); l.w = to_tf32(v.w - h.w);
}

// blocks [first, first + nblocks) split src into hi = tf32(src), lo = tf32(src - hi)
__device__ __forceinline__ void split_job(const float4* __restrict__ src, float4* __restrict__ hi,
                                          float4* __restrict__ lo, long long n4, int block, int nblocks) {
  for (long long i = (long long)block * blockDim.x + threadIdx.x; i < n4; i += (long long)nblocks * blockDim.x) {
    float4 h, l;
    split4(__ldg(src + i), h, l);
    hi[i] = h;
    lo[i] = l;
  }
}

// out[g][i] = sum_k coef[g][i][k] * in[g][k] for ROWS outputs from COLS inputs
// (Eq. 1: ROWS = K+2, COLS = K+1 with the noise as last input; Eq. 4:
// ROWS = K+1, COLS = K), written as a hi/lo pair and optionally in full.
template <int ROWS, int COLS, bool LAST_SEPARATE>
__device__ __forceinline__ void mix_job(const float* __restrict__ in, const float* __restrict__ last,
                                        const float* __restrict__ coef, float* __restrict__ full,
                                        float* __restrict__ hi, float* __restrict__ lo, long long n, int g,
                                        int chunk, int nchunks) {
  float c[ROWS][COLS];
#pragma unroll
  for (int i = 0; i < ROWS; ++i)
#pragma unroll
    for (int k = 0; k < COLS; ++k) c[i][k] = __ldg(coef + ((size_t)g * ROWS + i) * COLS + k);
  constexpr int NIN = LAST_SEPARATE ? COLS - 1 : COLS;      // inputs taken from `in`
  const float* ig = in + (size_t)g * NIN * n;
  const size_t ob = (size_t)g * ROWS * n;
  const long long n4 = n / 4;
  for (long long q = (long long)chunk * blockDim.x + threadIdx.x; q < n4; q += (long long)nchunks * blockDim.x) {
    float4 s[COLS];
#pragma unroll
    for (int k = 0; k < NIN; ++k) s[k] = __ldg(reinterpret_cast<const float4*>(ig + (size_t)k * n) + q);
    if (LAST_SEPARATE) s[COLS - 1] = __ldg(reinterpret_cast<const float4*>(last + (size_t)g * n) + q);
#pragma unroll
    for (int i = 0; i < ROWS; ++i) {
      float4 o, h, l;
      o.x = c[i][COLS - 1] * s[COLS - 1].x; o.y = c[i][COLS - 1] * s[COLS - 1].y;
      o.z = c[i][COLS - 1] * s[COLS - 1].z; o.w = c[i][COLS - 1] * s[COLS - 1].w;
#pragma unroll
      for (int k = 0; k < COLS - 1; ++k) {
        o.x = fmaf(c[i][k], s[k].x, o.x); o.y = fmaf(c[i][k], s[k].y, o.y);
        o.z = fmaf(c[i][k], s[k].z, o.z); o.w = fmaf(c[i][k], s[k].w, o.w);
      }
      split4(o, h, l);
      const size_t off = ob + (size_t)i * n;
      if (full != nullptr) reinterpret_cast<float4*>(full + off)[q] = o;
      reinterpret_cast<float4*>(hi + off)[q] = h;
      reinterpret_cast<float4*>(lo + off)[q] = l;
    }
  }
}

struct FwdPrepass {
  const float* x; const float* r; const float* enc; float* full; float* xb_hi; float* xb_lo;
  long long n_in; int G, per_g;                    // blocks [0, G*per_g): encode
  const float* W; float* w_hi; float* w_lo; long long w4; int w_blocks;   // then w_blocks blocks: split W
  float* stats; int nstats; unsigned int* count;   // cleared by block 0
};

template <int K>
__global__ void __launch_bounds__(256) fwd_prepass_kernel(const FwdPrepass a) {
  const int enc_blocks = a.G * a.per_g;
  if ((int)blockIdx.x < enc_blocks) {
    if (blockIdx.x == 0) {
      for (int i = threadIdx.x; i < a.nstats; i += blockDim.x) a.stats[i] = 0.f;
      if (threadIdx.x == 0) { a.count[0] = 0u; a.count[1] = 0u; }
    }
    const int g = blockIdx.x / a.per_g, chunk = blockIdx.x - g * a.per_g;
    mix_job<K + 2, K + 1, true>(a.x, a.r, a.enc, a.full, a.xb_hi, a.xb_lo, a.n_in, g, chunk, a.per_g);
  } else {
    split_job(reinterpret_cast<const float4*>(a.W), reinterpret_cast<float4*>(a.w_hi),
              reinterpret_cast<float4*>(a.w_lo), a.w4, (int)blockIdx.x - enc_blocks, a.w_blocks);
  }
}

struct WgPrepass {
  const float* delta; const float* dmix; float* dt_hi; float* dt_lo;
  long long n_out; int G, per_g;                   // blocks [0, G*per_g): delta mixing
  const float* xbar; float* xb_hi; float* xb_lo; long long x4; int x_blocks;   // then: split xbar
  float4* dW; long long dw4; int z_blocks;         // then: clear dW
};

template <int K>
__global__ void __launch_bounds__(256) wgrad_prepass_kernel(const WgPrepass a) {
  const int mix_blocks = a.G * a.per_g;
  int b = blockIdx.x;
  if (b < mix_blocks) {
    const int g = b / a.per_g, chunk = b - g * a.per_g;
    mix_job<K + 1, K, false>(a.delta, nullptr, a.dmix, nullptr, a.dt_hi, a.dt_lo, a.n_out, g, chunk, a.per_g);
    return;
  }
  b -= mix_blocks;
  if (b < a.x_blocks) {
    split_job(reinterpret_cast<const float4*>(a.xbar), reinterpret_cast<float4*>(a.xb_hi),
              reinterpret_cast<float4*>(a.xb_lo), a.x4, b, a.x_blocks);
    return;
  }
  b -= a.x_blocks;
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  for (long long i = (long long)b * blockDim.x + threadIdx.x; i < a.dw4; i += (long long)a.z_blocks * blockDim.x)
    a.dW[i] = z;
}

// blocks for a grid-stride job over n4 vectors: enough to cover it, at most `cap`
int job_blocks(long long n4, long long cap) {
  long long b = (n4 + 255) / 256;
  if (b > cap) b = cap;
  return b < 1 ? 1 : (int)b;
}

}  // namespace

dk_status tc_fwd_prepass(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                         float* xb_hi, float* xb_lo, const float* W, float* w_hi, float* w_lo,
                         const VerifyScratch& vs, int sm_count, cudaStream_t st) {
  const long long wn = (long long)g.cout * g.kc;
  if (g.n_in % 4 || wn % 4) return DK_ERR_SHAPE;
  FwdPrepass a;
  a.x = x; a.r = r; a.enc = enc; a.full = full; a.xb_hi = xb_hi; a.xb_lo = xb_lo;
  a.n_in = g.n_in; a.G = g.G;
  const long long cap = (long long)sm_count * 16;
  a.per_g = job_blocks(g.n_in / 4, (cap + g.G - 1) / g.G);
  a.W = W; a.w_hi = w_hi; a.w_lo = w_lo; a.w4 = wn / 4;
  a.w_blocks = job_blocks(a.w4, cap);
  a.stats = vs.sumsq; a.nstats = g.G * (g.E + 1); a.count = vs.count;
  const long long blocks = (long long)a.G * a.per_g + a.w_blocks;
  if (blocks > 0x7fffffffLL) return DK_ERR_SHAPE;
#define DK_PRE_CASE(KK) \
  case KK: fwd_prepass_kernel<KK><<<(unsigned)blocks, 256, 0, st>>>(a); break;
  switch (g.K) {
    DK_PRE_CASE(1) DK_PRE_CASE(2) DK_PRE_CASE(3) DK_PRE_CASE(4)
    DK_PRE_CASE(5) DK_PRE_CASE(6) DK_PRE_CASE(7) DK_PRE_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_PRE_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status tc_wgrad_prepass(const Geom& g, const float* delta, const float* dmix, float* dt_hi, float* dt_lo,
                           const float* xbar, long long xbar_elems, float* xb_hi, float* xb_lo, float* dW,
                           int sm_count, cudaStream_t st) {
  const long long dwn = (long long)g.cout * g.kc;
  if (g.n_out % 4 || xbar_elems % 4 || dwn % 4) return DK_ERR_SHAPE;
  WgPrepass a;
  a.delta = delta; a.dmix = dmix; a.dt_hi = dt_hi; a.dt_lo = dt_lo;
  a.n_out = g.n_out; a.G = g.G;
  const long long cap = (long long)sm_count * 16;
  a.per_g = job_blocks(g.n_out / 4, (cap + g.G - 1) / g.G);
  a.xbar = xbar; a.xb_hi = xb_hi; a.xb_lo = xb_lo; a.x4 = xbar_elems / 4;
  a.x_blocks = job_blocks(a.x4, cap);
  a.dW = reinterpret_cast<float4*>(dW); a.dw4 = dwn / 4;
  a.z_blocks = job_blocks(a.dw4, (long long)sm_count * 4);
  const long long blocks = (long long)a.G * a.per_g + a.x_blocks + a.z_blocks;
  if (blocks > 0x7fffffffLL) return DK_ERR_SHAPE;
#define DK_PRE_CASE(KK) \
  case KK: wgrad_prepass_kernel<KK><<<(unsigned)blocks, 256, 0, st>>>(a); break;
  switch (g.K) {
    DK_PRE_CASE(1) DK_PRE_CASE(2) DK_PRE_CASE(3) DK_PRE_CASE(4)
    DK_PRE_CASE(5) DK_PRE_CASE(6) DK_PRE_CASE(7) DK_PRE_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_PRE_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
