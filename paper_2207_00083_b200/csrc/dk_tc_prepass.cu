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

// The second TF32 term when the reader takes the fp32 value itself as the first: the tensor core ignores
// the 13 low mantissa bits of a TF32 operand, i.e. it sees trunc(v).  (Measured: with the term
// tf32(v - tf32(v)), which would be right if it rounded, y_bar is off by 5e-4; with this one the error
// equals that of a separately stored rounded first term.)
__device__ __forceinline__ float lo_of_raw(float v) {
  return to_tf32(v - __uint_as_float(__float_as_uint(v) & 0xffffe000u));
}
__device__ __forceinline__ float4 lo4_of_raw(const float4& v) {
  return make_float4(lo_of_raw(v.x), lo_of_raw(v.y), lo_of_raw(v.z), lo_of_raw(v.w));
}

// blocks [first, first + nblocks) split src into hi = tf32(src), lo = tf32(src - hi); with raw != 0 only the
// second term (see lo_of_raw) is written, and rows (of row4 vectors) whose index modulo `period` is >= `used`
// are skipped
__device__ __forceinline__ void split_job(const float4* __restrict__ src, float4* __restrict__ hi,
                                          float4* __restrict__ lo, long long n4, int block, int nblocks, int raw = 0,
                                          long long row4 = 0, int period = 1, int used = 1) {
  for (long long i = (long long)block * blockDim.x + threadIdx.x; i < n4; i += (long long)nblocks * blockDim.x) {
    if (raw) {
      if (period > used && (int)((i / row4) % period) >= used) continue;
      lo[i] = lo4_of_raw(__ldg(src + i));
      continue;
    }
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
                                        int chunk, int nchunks, int raw = 0, int pix4 = 0, int width = 0,
                                        int step = 1) {
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
    if (step > 1) {
      // a strided 1x1 convolution reads every step-th row and column only: the others are neither encoded
      // nor written (pix4 = 16-byte vectors per pixel, width = pixels per row)
      const long long pix = q / pix4;
      if ((pix % width) % step != 0 || (pix / width) % step != 0) continue;
    }
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
      const size_t off = ob + (size_t)i * n;
      if (full != nullptr) reinterpret_cast<float4*>(full + off)[q] = o;
      if (raw) {
        if (lo != nullptr) reinterpret_cast<float4*>(lo + off)[q] = lo4_of_raw(o);
      } else {
        split4(o, h, l);
        reinterpret_cast<float4*>(hi + off)[q] = h;
        reinterpret_cast<float4*>(lo + off)[q] = l;
      }
    }
  }
}

struct FwdPrepass {
  const float* x; const float* r; const float* enc; float* full; float* xb_hi; float* xb_lo;
  long long n_in; int G, per_g;                    // blocks [0, G*per_g): encode
  const float* W; float* w_hi; float* w_lo; long long w4; int w_blocks;   // then w_blocks blocks: split W
  float* stats; int nstats; unsigned int* count;   // cleared by block 0
  float4* zero; long long z4; int z_blocks;        // then z_blocks blocks: clear y_bar (split-K calls)
  int raw;                                         // the encodings in `full` serve as leading term (see lo_of_raw)
  int pix4, width, step;                           // step > 1: only every step-th row and column is encoded
  int wpack, cout, cin4, kh, kw;                   // wpack: W is laid out for two-output-row tiles (see wpack_job)
};

// Weights of a layer with at most 64 output channels for tiles that hold two output rows of the image:
// 128 rows x (kh+1)*kw taps x cin.  Row co < 64 holds W[co][dy][v] at tap (dy, v) (zero at dy = kh); row
// 64 + co holds W[co][dy-1][v] (zero at dy = 0): the activation box at vertical offset dy is tap dy of the upper
// output row and tap dy-1 of the lower one.
__device__ __forceinline__ void wpack_job(const FwdPrepass& a, int block, int nblocks) {
  const int taps2 = (a.kh + 1) * a.kw;
  const long long n4 = (long long)128 * taps2 * a.cin4;
  for (long long i = (long long)block * blockDim.x + threadIdx.x; i < n4; i += (long long)nblocks * blockDim.x) {
    const int c4 = (int)(i % a.cin4);
    const int tap = (int)((i / a.cin4) % taps2), row = (int)(i / ((long long)a.cin4 * taps2));
    const int dy = tap / a.kw, v = tap - dy * a.kw;
    const int co = row & 63, u = row < 64 ? dy : dy - 1;
    float4 w = make_float4(0.f, 0.f, 0.f, 0.f), h, l;
    if (co < a.cout && u >= 0 && u < a.kh)
      w = __ldg(reinterpret_cast<const float4*>(a.W) + ((long long)(co * a.kh + u) * a.kw + v) * a.cin4 + c4);
    split4(w, h, l);
    reinterpret_cast<float4*>(a.w_hi)[i] = h;
    reinterpret_cast<float4*>(a.w_lo)[i] = l;
  }
}

template <int K>
__global__ void __launch_bounds__(256) fwd_prepass_kernel(const FwdPrepass a) {
  const int enc_blocks = a.G * a.per_g;
  if ((int)blockIdx.x >= enc_blocks + a.w_blocks) {
    const int b = (int)blockIdx.x - enc_blocks - a.w_blocks;
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (long long i = (long long)b * blockDim.x + threadIdx.x; i < a.z4; i += (long long)a.z_blocks * blockDim.x)
      a.zero[i] = z;
    return;
  }
  if ((int)blockIdx.x < enc_blocks) {
    if (blockIdx.x == 0 && a.count != nullptr) {
      for (int i = threadIdx.x; i < a.nstats; i += blockDim.x) a.stats[i] = 0.f;
      if (threadIdx.x == 0) { a.count[0] = 0u; a.count[1] = 0u; }
    }
    const int g = blockIdx.x / a.per_g, chunk = blockIdx.x - g * a.per_g;
    mix_job<K + 2, K + 1, true>(a.x, a.r, a.enc, a.full, a.xb_hi, a.xb_lo, a.n_in, g, chunk, a.per_g, a.raw, a.pix4, a.width,
                                a.step);
  } else if (a.wpack) {
    wpack_job(a, (int)blockIdx.x - enc_blocks, a.w_blocks);
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
  int raw; long long row4; int period, used;       // raw: only the second term of the used encodings is written
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
              reinterpret_cast<float4*>(a.xb_lo), a.x4, b, a.x_blocks, a.raw, a.row4, a.period, a.used);
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
                         const VerifyScratch& vs, float* ybar_clear, int sm_count, cudaStream_t st, int raw,
                         int g_lo, int g_cnt, bool beside) {
  // groups [g_lo, g_lo + g_cnt) only (g_cnt < 0: all); the launch for g_lo = 0 also splits W and clears
  const bool first = g_lo == 0;
  if (g_cnt < 0) g_cnt = g.G - g_lo;
  const long long wn = (long long)g.cout * g.kc;
  if (g.n_in % 4 || wn % 4) return DK_ERR_SHAPE;
  if (raw && full == nullptr) return DK_ERR_INVALID_ARG;
  FwdPrepass a;
  a.raw = raw;
  const bool strided_1x1 = g.kind == DK_CONV2D && g.kh == 1 && g.kw == 1 && g.pad == 0 && g.stride > 1;
  a.pix4 = g.cin / 4; a.width = g.w; a.step = strided_1x1 ? g.stride : 1;
  const long long yn = (long long)g.G * g.E * g.n_out;
  if (!first) ybar_clear = nullptr;
  a.zero = reinterpret_cast<float4*>(ybar_clear);
  a.z4 = ybar_clear ? (yn + 3) / 4 : 0;           // the y_bar region is padded to 1 KiB
  a.z_blocks = ybar_clear ? job_blocks(a.z4, (long long)sm_count * 4) : 0;
  const size_t eoff = (size_t)g_lo * g.E * g.n_in;
  a.x = x + (size_t)g_lo * g.K * g.n_in; a.r = r + (size_t)g_lo * g.n_in;
  a.enc = enc + (size_t)g_lo * g.E * (g.K + 1);
  a.full = full ? full + eoff : nullptr; a.xb_hi = xb_hi ? xb_hi + eoff : nullptr;
  a.xb_lo = xb_lo ? xb_lo + eoff : nullptr;      // (null with raw: the GEMM kernel derives the second term itself)
  if (xb_lo == nullptr && !raw) return DK_ERR_INVALID_ARG;
  a.n_in = g.n_in; a.G = g_cnt;
  // beside a GEMM kernel (one persistent CTA of 32K registers per SM) only a few small blocks fit on an SM, and a
  // larger grid would keep the GEMM's CTAs off the SMs until this kernel has ended: blocks of 128 threads, two
  // per SM up to K = 4 (at most 80 registers a thread), one beyond (at most 165)
  const int threads = beside ? 128 : 256;
  const long long cap = beside ? (long long)sm_count * (g.K <= 4 ? 2 : 1) : (long long)sm_count * 16;
  a.per_g = job_blocks(g.n_in / 4, (cap + g_cnt - 1) / g_cnt);
  a.W = W; a.w_hi = w_hi; a.w_lo = w_lo; a.w4 = wn / 4;
  a.wpack = g.mpack; a.cout = g.cout; a.cin4 = g.cin / 4; a.kh = g.kh; a.kw = g.kw;
  a.w_blocks = first ? job_blocks(g.mpack ? (long long)128 * (g.kh + 1) * g.kw * a.cin4 : a.w4, cap) : 0;
  a.stats = vs.sumsq; a.nstats = first ? g.G * (g.E + 1) : 0; a.count = first ? vs.count : nullptr;
  const long long blocks = (long long)a.G * a.per_g + a.w_blocks + a.z_blocks;
  if (blocks > 0x7fffffffLL) return DK_ERR_SHAPE;
#define DK_PRE_CASE(KK) \
  case KK: fwd_prepass_kernel<KK><<<(unsigned)blocks, threads, 0, st>>>(a); break;
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
                           int sm_count, cudaStream_t st, int raw, int xbar_rows, int g_lo, int g_cnt, bool beside) {
  const long long dwn = (long long)g.cout * g.kc;
  if (g.n_out % 4 || xbar_elems % 4 || dwn % 4 || g.n_in % 4) return DK_ERR_SHAPE;
  // groups [g_lo, g_lo + g_cnt) only (g_cnt < 0: all); the launch for g_lo = 0 also clears dW
  if (g_cnt < 0) g_cnt = g.G - g_lo;
  if (g_lo > 0 || g_cnt < g.G) {
    const int rows = xbar_rows > 0 ? xbar_rows : g.K + 1;
    const long long xoff = (long long)g_lo * rows * g.n_in;
    long long xe = (long long)g_cnt * rows * g.n_in;
    if (xoff + xe > xbar_elems) xe = xbar_elems - xoff;
    const long long doff = (long long)g_lo * (g.K + 1) * g.n_out;
    delta += (long long)g_lo * g.K * g.n_out; dmix += (long long)g_lo * (g.K + 1) * g.K;
    dt_hi += doff; dt_lo += doff;
    xbar += xoff; if (xb_hi) xb_hi += xoff;
    xb_lo += xoff;
    xbar_elems = xe;
    if (g_lo > 0) dW = nullptr;
  }
  WgPrepass a;
  a.raw = raw; a.row4 = g.n_in / 4; a.period = xbar_rows > 0 ? xbar_rows : 1; a.used = xbar_rows > 0 ? g.K + 1 : 1;
  a.delta = delta; a.dmix = dmix; a.dt_hi = dt_hi; a.dt_lo = dt_lo;
  a.n_out = g.n_out; a.G = g_cnt;
  // (beside a GEMM kernel: few small blocks, see tc_fwd_prepass; the cap is shared by the two jobs)
  const int threads = beside ? 128 : 256;
  const long long cap = beside ? (long long)sm_count * (g.K <= 4 ? 2 : 1) / 2 + 1 : (long long)sm_count * 16;
  a.per_g = job_blocks(g.n_out / 4, (cap + g_cnt - 1) / g_cnt);
  a.xbar = xbar; a.xb_hi = xb_hi; a.xb_lo = xb_lo; a.x4 = xbar_elems / 4;
  a.x_blocks = job_blocks(a.x4, cap);
  a.dW = reinterpret_cast<float4*>(dW); a.dw4 = dW ? dwn / 4 : 0;
  a.z_blocks = dW ? job_blocks(a.dw4, (long long)sm_count * 4) : 0;
  const long long blocks = (long long)a.G * a.per_g + a.x_blocks + a.z_blocks;
  if (blocks > 0x7fffffffLL) return DK_ERR_SHAPE;
#define DK_PRE_CASE(KK) \
  case KK: wgrad_prepass_kernel<KK><<<(unsigned)blocks, threads, 0, st>>>(a); break;
  switch (g.K) {
    DK_PRE_CASE(1) DK_PRE_CASE(2) DK_PRE_CASE(3) DK_PRE_CASE(4)
    DK_PRE_CASE(5) DK_PRE_CASE(6) DK_PRE_CASE(7) DK_PRE_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_PRE_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

// ---------------------------------------------------------------------------
// Layers whose input has a channel count that is not a multiple of four (the
// 3-channel stems).  Their contraction is short (kc = 27 or 147), which the
// tensor-core kernels cannot fetch as 16-byte aligned channel runs.  The
// pre-pass therefore writes, per encoded sample and output pixel, the kc
// inputs under the filter as one row padded to a multiple of 32, already as a
// hi/lo pair; the GEMM kernels then see a 1x1 convolution over ho x wo pixels
// with Kp input channels.  (The weight gradient of these layers stays on the
// fp32 kernels: its operands would have to be rewritten as patch rows too,
// which costs more HBM traffic than the tensor cores save.)
// ---------------------------------------------------------------------------
namespace {

struct PatchGeom {
  int cin, h, w, kw, stride, pad, ho, wo, kc, Kp;
  long long n_in;
};

// offset inside one sample of the input under filter position k of output pixel pix, or -1 (padding / k >= kc)
__device__ __forceinline__ long long patch_offset(const PatchGeom& q, int pix, int k) {
  if (k >= q.kc) return -1;
  const int c = k % q.cin, t = k / q.cin;
  const int v = t % q.kw, u = t / q.kw;
  const int oy = pix / q.wo, ox = pix - oy * q.wo;
  const int iy = oy * q.stride + u - q.pad, ix = ox * q.stride + v - q.pad;
  if (iy < 0 || iy >= q.h || ix < 0 || ix >= q.w) return -1;
  return ((long long)iy * q.w + ix) * q.cin + c;
}

struct StemFwd {
  PatchGeom q;
  const float* x; const float* r; const float* enc; float* full; float* col_hi; float* col_lo;
  int G, per_g;                                    // blocks [0, G*per_g): patches of the encodings
  int full_blocks;                                 // then: encodings in their own layout (when stored)
  const float* W; float* w_hi; float* w_lo; int cout; int w_blocks;   // then: padded weights
  float* stats; int nstats; unsigned int* count;   // cleared by block 0
};

template <int K>
__global__ void __launch_bounds__(256) stem_fwd_prepass_kernel(const StemFwd a) {
  constexpr int K1 = K + 1, E = K + 2;
  const PatchGeom& q = a.q;
  const int npix = q.ho * q.wo, kq = q.Kp / 4;
  int b = blockIdx.x;
  if (b < a.G * a.per_g) {
    if (b == 0) {
      for (int i = threadIdx.x; i < a.nstats; i += blockDim.x) a.stats[i] = 0.f;
      if (threadIdx.x == 0) { a.count[0] = 0u; a.count[1] = 0u; }
    }
    const int g = b / a.per_g, chunk = b - g * a.per_g;
    float c[E][K1];
#pragma unroll
    for (int i = 0; i < E; ++i)
#pragma unroll
      for (int k = 0; k < K1; ++k) c[i][k] = __ldg(a.enc + ((size_t)g * E + i) * K1 + k);
    const float* xg = a.x + (size_t)g * K * q.n_in;
    const float* rg = a.r + (size_t)g * q.n_in;
    const long long items = (long long)npix * kq;
    for (long long it = (long long)chunk * blockDim.x + threadIdx.x; it < items; it += (long long)a.per_g * blockDim.x) {
      const int pix = (int)(it / kq), k0 = (int)(it - (long long)pix * kq) * 4;
      float s[K1][4];
#pragma unroll
      for (int d = 0; d < 4; ++d) {
        const long long off = patch_offset(q, pix, k0 + d);
#pragma unroll
        for (int k = 0; k < K; ++k) s[k][d] = off >= 0 ? __ldg(xg + (size_t)k * q.n_in + off) : 0.f;
        s[K][d] = off >= 0 ? __ldg(rg + off) : 0.f;
      }
#pragma unroll
      for (int i = 0; i < E; ++i) {
        float4 o, hh, ll;
        float t[4];
#pragma unroll
        for (int d = 0; d < 4; ++d) {
          float acc = c[i][K] * s[K][d];
#pragma unroll
          for (int k = 0; k < K; ++k) acc = fmaf(c[i][k], s[k][d], acc);
          t[d] = acc;
        }
        o = make_float4(t[0], t[1], t[2], t[3]);
        split4(o, hh, ll);
        const size_t row = ((size_t)g * E + i) * npix + pix;
        reinterpret_cast<float4*>(a.col_hi + row * q.Kp)[k0 / 4] = hh;
        reinterpret_cast<float4*>(a.col_lo + row * q.Kp)[k0 / 4] = ll;
      }
    }
    return;
  }
  b -= a.G * a.per_g;
  if (b < a.full_blocks) {
    // Eq. 1 in the tensor's own layout, for the caller who stores the encodings
    const long long total = (long long)a.G * q.n_in;
    for (long long i = (long long)b * blockDim.x + threadIdx.x; i < total; i += (long long)a.full_blocks * blockDim.x) {
      const int g = (int)(i / q.n_in);
      const long long off = i - (long long)g * q.n_in;
      float s[K1];
#pragma unroll
      for (int k = 0; k < K; ++k) s[k] = __ldg(a.x + ((size_t)g * K + k) * q.n_in + off);
      s[K] = __ldg(a.r + (size_t)g * q.n_in + off);
#pragma unroll
      for (int e = 0; e < E; ++e) {
        const float* ce = a.enc + ((size_t)g * E + e) * K1;
        float acc = __ldg(ce + K) * s[K];
#pragma unroll
        for (int k = 0; k < K; ++k) acc = fmaf(__ldg(ce + k), s[k], acc);
        a.full[((size_t)g * E + e) * q.n_in + off] = acc;
      }
    }
    return;
  }
  b -= a.full_blocks;
  const long long witems = (long long)a.cout * kq;
  for (long long it = (long long)b * blockDim.x + threadIdx.x; it < witems; it += (long long)a.w_blocks * blockDim.x) {
    const int co = (int)(it / kq), k0 = (int)(it - (long long)co * kq) * 4;
    float t[4];
#pragma unroll
    for (int d = 0; d < 4; ++d) t[d] = k0 + d < q.kc ? __ldg(a.W + (size_t)co * q.kc + k0 + d) : 0.f;
    float4 hh, ll;
    split4(make_float4(t[0], t[1], t[2], t[3]), hh, ll);
    reinterpret_cast<float4*>(a.w_hi + (size_t)co * q.Kp)[k0 / 4] = hh;
    reinterpret_cast<float4*>(a.w_lo + (size_t)co * q.Kp)[k0 / 4] = ll;
  }
}

PatchGeom patch_geom(const Geom& g) {
  PatchGeom q;
  q.cin = g.cin; q.h = g.h; q.w = g.w; q.kw = g.kw; q.stride = g.stride; q.pad = g.pad;
  q.ho = g.ho; q.wo = g.wo; q.kc = g.kc; q.Kp = tc_stem_padded_kc(g); q.n_in = g.n_in;
  return q;
}

}  // namespace

int tc_stem_padded_kc(const Geom& g) { return (g.kc + 31) / 32 * 32; }

Geom tc_stem_gemm_geom(const Geom& g) {
  Geom s = g;
  const int Kp = tc_stem_padded_kc(g);
  s.kind = DK_CONV2D; s.layout = DK_NHWC;
  s.cin = Kp; s.h = g.ho; s.w = g.wo; s.kh = s.kw = 1; s.stride = 1; s.pad = 0;
  s.n_in = (long long)Kp * g.ho * g.wo;
  s.kc = Kp;
  s.xs_c = 1; s.xs_w = Kp; s.xs_h = (long long)Kp * g.wo;
  s.ws_c = 1; s.ws_v = Kp; s.ws_u = Kp; s.ws_o = Kp;
  return s;
}

dk_status tc_stem_fwd_prepass(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                              float* col_hi, float* col_lo, const float* W, float* w_hi, float* w_lo,
                              const VerifyScratch& vs, int sm_count, cudaStream_t st) {
  StemFwd a;
  a.q = patch_geom(g);
  a.x = x; a.r = r; a.enc = enc; a.full = full; a.col_hi = col_hi; a.col_lo = col_lo;
  a.G = g.G;
  const long long cap = (long long)sm_count * 16;
  const long long items = (long long)g.ho * g.wo * (a.q.Kp / 4);
  a.per_g = job_blocks(items, (cap + g.G - 1) / g.G);
  a.full_blocks = full ? job_blocks((long long)g.G * g.n_in, cap) : 0;
  a.W = W; a.w_hi = w_hi; a.w_lo = w_lo; a.cout = g.cout;
  a.w_blocks = job_blocks((long long)g.cout * (a.q.Kp / 4), cap);
  a.stats = vs.sumsq; a.nstats = g.G * (g.E + 1); a.count = vs.count;
  const long long blocks = (long long)a.G * a.per_g + a.full_blocks + a.w_blocks;
  if (blocks > 0x7fffffffLL) return DK_ERR_SHAPE;
#define DK_PRE_CASE(KK) \
  case KK: stem_fwd_prepass_kernel<KK><<<(unsigned)blocks, 256, 0, st>>>(a); break;
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
