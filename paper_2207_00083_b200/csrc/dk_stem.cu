// Layers with very few input channels (the 3-channel stems: cin % 4 != 0) in
// ONE kernel each way.  Such a layer is bound by writing its output (forward)
// or by reading the output gradients (weight gradient), not by its arithmetic:
// 27 or 147 multiply-adds per output value.  fp32 FMAs are accurate enough here
// without any operand splitting, so the kernels below do everything in
// registers and shared memory and touch HBM once per tensor:
//
//  forward  Eq. 1 on the input patch of a row of 32 output pixels (the K+2
//           encodings of every input value side by side in shared memory), the
//           cross-correlation in fp32 FMAs with an 8-channel x (K+2)-encoding
//           register tile per thread, Eq. 2 and the redundant equation of
//           Section 4.4 on that tile, decoded outputs stored as 32-byte runs.
//  wgrad    Eq. 4 on a row of 32 pixels of the output gradients (the K+1 mixed
//           gradients in shared memory), the stored encodings' patch beside
//           them, 4 output channels x all kc filter taps per thread, pixels
//           dealt to 16 streams that meet in shared memory at the end.
#include "dk_internal.h"

namespace dk {
namespace {

constexpr int kThreads = 256;
constexpr int kTileW = 32;        // output pixels per CTA step (one row segment)

struct StemFwdParams {
  const float* W; const float* x; const float* r; const float* bias; float* y;
  const float* enc; const float* dec; const float* nul;
  VerifyScratch vs;
  float tau;
  int cin, cout, h, w, kh, kw, stride, pad, ho, wo, kc, G;
  int PW;                      // patch width in input pixels: (kTileW - 1) * stride + kw
  int tiles_w;
  long long ntiles;            // G * ho * tiles_w
  int f_group, f_enc;
  long long f_index;
  float f_delta;
  int kstore;                  // decoded rows k >= kstore of a group are neither computed nor stored
};

template <int K>
__global__ void __launch_bounds__(kThreads, 2) stem_fwd_kernel(const StemFwdParams p) {
  constexpr int K1 = K + 1, E = K + 2, EP = (E + 3) / 4 * 4;
  extern __shared__ float4 smem4[];
  float* Xs = reinterpret_cast<float*>(smem4);               // [kh][PW][cin][EP] encoded patch
  const int patch = p.kh * p.PW * p.cin;
  float* Ws = Xs + (size_t)patch * EP;                       // [kc][2][8][4]: weights of the current 64 channels; a thread's
                                                             // 8 channels are two 16-byte pieces 128 bytes apart (conflict-free)
  float* cenc = Ws + (size_t)p.kc * 64;                      // [E][K1]
  float* cdec = cenc + E * K1;                               // [K][K1]
  float* cnul = cdec + K * K1;                               // [E]
  const int tid = threadIdx.x, lane = tid & 31;
  const int cog = tid & 7, pl = tid >> 3;                    // 8 output channels, pixel of the row segment
  const long long n_in = (long long)p.h * p.w * p.cin, n_out = (long long)p.ho * p.wo * p.cout;
  const float kInf = __int_as_float(0x7f800000);
  int loaded_g = -1;
  bool w_loaded = false;

  const int roww = p.PW * p.cin;     // a patch row is that many consecutive values of the image
  for (long long t = blockIdx.x; t < p.ntiles; t += gridDim.x) {
    const int ti = (int)t;           // (the host checked that the tile count fits 31 bits)
    const int tw = ti % p.tiles_w, rest = ti / p.tiles_w;
    const int oy = rest % p.ho, g = rest / p.ho;
    const int ox0 = tw * kTileW;
    __syncthreads();                 // the previous tile's reads of Xs, Ws and the tables are done
    if (g != loaded_g) {
      for (int i = tid; i < E * K1; i += kThreads) cenc[i] = __ldg(p.enc + (size_t)g * E * K1 + i);
      for (int i = tid; i < K * K1; i += kThreads) cdec[i] = __ldg(p.dec + (size_t)g * K * K1 + i);
      for (int i = tid; i < E; i += kThreads) cnul[i] = __ldg(p.nul + (size_t)g * E + i);
      loaded_g = g;
      __syncthreads();
    }
    // Eq. 1 on the patch: input rows oy*stride - pad + u, columns ox0*stride - pad + 0 .. PW-1
    {
      const float* xg = p.x + (size_t)g * K * n_in;
      const float* rg = p.r + (size_t)g * n_in;
      const int iy0 = oy * p.stride - p.pad, ix0 = ox0 * p.stride - p.pad;
      // (element e of a patch row lies in the image when e_lo <= e < e_hi: no division per element)
      const int e_lo = max(0, -ix0) * p.cin, e_hi = min(p.PW, p.w - ix0) * p.cin;
      for (int i = tid; i < patch; i += kThreads) {
        int u = 0, e = i;
        while (e >= roww) { e -= roww; ++u; }
        const int iy = iy0 + u;
        float s[K1];
        const bool in = iy >= 0 && iy < p.h && e >= e_lo && e < e_hi;
        const long long off = ((long long)iy * p.w + ix0) * p.cin + e;
#pragma unroll
        for (int k = 0; k < K; ++k) s[k] = in ? __ldg(xg + (size_t)k * n_in + off) : 0.f;
        s[K] = in ? __ldg(rg + off) : 0.f;
        float* dst = Xs + (size_t)i * EP;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          float a = cenc[e * K1 + K] * s[K];
#pragma unroll
          for (int k = 0; k < K; ++k) a = fmaf(cenc[e * K1 + k], s[k], a);
          dst[e] = a;
        }
#pragma unroll
        for (int e = E; e < EP; ++e) dst[e] = 0.f;
      }
    }
    const int ox = ox0 + pl;
    for (int cb = 0; cb < p.cout; cb += 64) {
      if (cb > 0) __syncthreads();   // the previous block's reads of Ws are done
      if (p.cout > 64 || !w_loaded) {      // a layer with at most 64 output channels keeps its weights for all tiles
        for (int i = tid; i < p.kc * 64; i += kThreads) {
          const int k = i >> 6, c64 = i & 63, co = cb + c64;
          Ws[k * 64 + ((c64 >> 2) & 1) * 32 + (c64 >> 3) * 4 + (c64 & 3)] = co < p.cout ? __ldg(p.W + (size_t)co * p.kc + k) : 0.f;
        }
        w_loaded = true;
      }
      __syncthreads();
      float acc[E][8];
#pragma unroll
      for (int e = 0; e < E; ++e)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[e][j] = 0.f;
      {
        // one filter element: the K+2 encodings of this thread's pixel against its 8 channels
        auto element = [&](const float* xrow, int vc, int k) {
          float xe[EP];
#pragma unroll
          for (int q = 0; q < EP / 4; ++q)
            *reinterpret_cast<float4*>(xe + 4 * q) = *reinterpret_cast<const float4*>(xrow + (size_t)vc * EP + 4 * q);
          const float4 w0 = *reinterpret_cast<const float4*>(Ws + k * 64 + cog * 4);
          const float4 w1 = *reinterpret_cast<const float4*>(Ws + k * 64 + 32 + cog * 4);
          const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
          for (int e = 0; e < E; ++e)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[e][j] = fmaf(xe[e], wv[j], acc[e][j]);
        };
        const int rowk = p.kw * p.cin;
        for (int u = 0; u < p.kh; ++u) {
          const float* xrow = Xs + ((size_t)u * p.PW + (size_t)pl * p.stride) * p.cin * EP;
          if (rowk == 9) {             // 3 taps x 3 channels, the usual stem: straight-line code
#pragma unroll
            for (int vc = 0; vc < 9; ++vc) element(xrow, vc, u * 9 + vc);
          } else {
#pragma unroll 3
            for (int vc = 0; vc < rowk; ++vc) element(xrow, vc, u * rowk + vc);
          }
        }
      }
      // ---- epilogue on the register tile: fault hook, Eq. 2, redundant equation, statistics
      const int co0 = cb + cog * 8;
      const bool pix_ok = ox < p.wo;
      const long long obase = ((long long)oy * p.wo + ox) * p.cout;
      if (p.f_group == g && pix_ok) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (obase + co0 + j == p.f_index && co0 + j < p.cout) {
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e][j] += (e == p.f_enc) ? p.f_delta : 0.f;
          }
      }
      float sq[E], maxrho = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) sq[e] = 0.f;
      const bool whole = co0 + 8 <= p.cout && (p.cout & 3) == 0;      // this thread's 8 channels as two 16-byte stores
      float bj[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) bj[j] = (p.bias && co0 + j < p.cout) ? __ldg(p.bias + co0 + j) : 0.f;
      if (pix_ok) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
          if (k >= p.kstore) continue;
          float yv[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) yv[j] = cdec[k * K1] * acc[0][j];
#pragma unroll
          for (int i = 1; i < K1; ++i) {
            const float c = cdec[k * K1 + i];
#pragma unroll
            for (int j = 0; j < 8; ++j) yv[j] = fmaf(c, acc[i][j], yv[j]);
          }
          float* dst = p.y + ((size_t)g * K + k) * n_out + obase + co0;
          if (whole) {
            *reinterpret_cast<float4*>(dst) = make_float4(yv[0] + bj[0], yv[1] + bj[1], yv[2] + bj[2], yv[3] + bj[3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(yv[4] + bj[4], yv[5] + bj[5], yv[6] + bj[6], yv[7] + bj[7]);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (co0 + j < p.cout) dst[j] = yv[j] + bj[j];
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (co0 + j >= p.cout) continue;
          float rho = 0.f, sc = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) {
            const float v = acc[e][j];
            rho = fmaf(cnul[e], v, rho);
            sc = fmaf(fabsf(cnul[e]), fabsf(v), sc);
            if (fabsf(v) < kInf) sq[e] = fmaf(v, v, sq[e]);
          }
          const float ar = fabsf(rho);
          maxrho = fmaxf(maxrho, ar);
          if (!(ar <= p.tau * sc) || !(sc < kInf)) {
            const unsigned int slot = atomicAdd(p.vs.count, 1u);
            if (slot < kCandCap) {
              Candidate cd;
              cd.index = (long long)g * n_out + obase + co0 + j;
              cd.absrho = ar;
              cd.s_e = sc;
              p.vs.cand[slot] = cd;
            }
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int e = 0; e < E; ++e) sq[e] += __shfl_xor_sync(0xffffffffu, sq[e], o);
        maxrho = fmaxf(maxrho, __shfl_xor_sync(0xffffffffu, maxrho, o));
      }
      {
        float tsum = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) tsum = lane == e ? sq[e] : tsum;
        if (lane < E && tsum != 0.f) atomicAdd(p.vs.sumsq + (size_t)g * E + lane, tsum);
      }
      if (lane == 0 && maxrho > 0.f) atomicMax(p.vs.maxrho + g, __float_as_int(maxrho));
    }
  }
}

size_t stem_fwd_smem(const Geom& g) {
  const int E = g.E, EP = (E + 3) / 4 * 4, K1 = g.K + 1;
  const int PW = (kTileW - 1) * g.stride + g.kw;
  return ((size_t)g.kh * PW * g.cin * EP + (size_t)g.kc * 64 + (size_t)E * K1 + (size_t)g.K * K1 + E + 4) * sizeof(float);
}

// ---------------------------------------------------------------------------
// weight gradient of a 3x3 stem with 3 input channels (Eq. 4-6)
// ---------------------------------------------------------------------------
struct StemWgParams {
  const float* delta; const float* xbar; const float* dmix; float* dW;
  int cout, h, w, stride, pad, ho, wo, G, xbar_rows;
  int PW, tiles_w;
  long long ntiles;
  float scale;
};

constexpr int kWgKH = 3, kWgKWC = 9, kWgKC = kWgKH * kWgKWC;      // 3 x 3 taps x 3 channels

// grid.y = blocks of 64 output channels; thread = 4 channels x all 27 filter elements, one of 16 pixel streams
template <int K>
__global__ void __launch_bounds__(kThreads, 1) stem_wgrad_kernel(const StemWgParams p) {
  constexpr int K1 = K + 1, CIN = 3;
  extern __shared__ float4 smem4[];
  float* Ds = reinterpret_cast<float*>(smem4);                 // [K1][32][64] mixed gradients of the row segment
  // stored encodings under it, two buffers: [K1][3][PW][4] (a pixel's 3 channels in a 16-byte slot, so that the
  // three taps of a filter row are three aligned 16-byte reads); the next tile's patch arrives by asynchronous
  // copies while this tile is contracted
  float* Xs0 = Ds + (size_t)K1 * kTileW * 64;
  const int xbuf = K1 * kWgKH * p.PW * 4;                      // floats of one buffer
  float* cmix = Xs0 + 2 * (size_t)xbuf;                        // [K1][K]
  const int tid = threadIdx.x, cog = tid & 15, stream = tid >> 4;
  const int cb = blockIdx.y * 64;
  const long long n_in = (long long)p.h * p.w * CIN, n_out = (long long)p.ho * p.wo * p.cout;
  float acc[kWgKC][4];
#pragma unroll
  for (int k = 0; k < kWgKC; ++k) acc[k][0] = acc[k][1] = acc[k][2] = acc[k][3] = 0.f;
  int loaded_g = -1;
  static_assert(kTileW * 16 == 2 * kThreads, "two 16-byte units of the gradients per thread");
  // the gradients of a tile are fetched into registers while the previous tile is being contracted
  float4 dn[2][K];
  auto fetch = [&](long long t) {
    const int ti = (int)(t < p.ntiles ? t : 0);
    const int tw = ti % p.tiles_w, rest = ti / p.tiles_w;
    const int oy = rest % p.ho, g = rest / p.ho;
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      const int u4 = tid + h2 * kThreads;
      const int px = u4 >> 4, c4 = (u4 & 15) * 4;
      const int ox = tw * kTileW + px, co = cb + c4;
      const bool ok = t < p.ntiles && ox < p.wo && co < p.cout;       // cout % 4 == 0: a group of four is inside or outside
#pragma unroll
      for (int i = 0; i < K; ++i)
        dn[h2][i] = ok ? __ldg(reinterpret_cast<const float4*>(p.delta + ((size_t)g * K + i) * n_out +
                                                               ((size_t)oy * p.wo + ox) * p.cout + co))
                       : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  // asynchronous 4-byte copies of tile t's patch of the stored encodings 0..K into buffer `b` (zeros outside the image)
  auto stage_patch = [&](long long t, int b) {
    if (t < p.ntiles) {
      const int ti = (int)t;                                   // (the host checked that the tile count fits 31 bits)
      const int tw = ti % p.tiles_w, rest = ti / p.tiles_w;
      const int oy = rest % p.ho, g = rest / p.ho;
      const int iy0 = oy * p.stride - p.pad, ix0 = tw * kTileW * p.stride - p.pad;
      float* xb = Xs0 + (size_t)b * xbuf;
      // a patch row of one encoding is PW * 3 consecutive values of the image: one warp per row, no division by
      // run-time values per element
      const int roww = p.PW * CIN;
      for (int row = tid >> 5; row < K1 * kWgKH; row += kThreads / 32) {
        const int j = row / kWgKH, u = row - j * kWgKH;
        const int iy = iy0 + u;
        const bool row_in = iy >= 0 && iy < p.h;
        const float* srow = p.xbar + ((size_t)g * p.xbar_rows + j) * n_in + ((long long)iy * p.w + ix0) * CIN;
        float* drow = xb + (size_t)row * p.PW * 4;
        for (int e = tid & 31; e < roww; e += 32) {
          const int px = e / CIN, c = e - px * CIN;
          const int ix = ix0 + px;
          const bool in = row_in && ix >= 0 && ix < p.w;
          const uint32_t dst = (uint32_t)__cvta_generic_to_shared(drow + px * 4 + c);
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(in ? srow + e : p.xbar), "r"(in ? 4 : 0));
        }
      }
    }
    asm volatile("cp.async.commit_group;\n" ::);
  };
  fetch(blockIdx.x);
  stage_patch(blockIdx.x, 0);
  int cur = 0;

  for (long long t = blockIdx.x; t < p.ntiles; t += gridDim.x, cur ^= 1) {
    const int g = (int)t / p.tiles_w / p.ho;
    __syncthreads();
    if (g != loaded_g) {
      for (int i = tid; i < K1 * K; i += kThreads) cmix[i] = __ldg(p.dmix + (size_t)g * K1 * K + i);
      loaded_g = g;
      __syncthreads();
    }
    // Eq. 4: the K+1 mixed gradients of the segment's pixels, 64 channels of this block
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      const int u4 = tid + h2 * kThreads;
      const int px = u4 >> 4, c4 = (u4 & 15) * 4;
      const float4* d = dn[h2];
#pragma unroll
      for (int j = 0; j < K1; ++j) {
        float4 o;
        const float c0 = cmix[j * K];
        o.x = c0 * d[0].x; o.y = c0 * d[0].y; o.z = c0 * d[0].z; o.w = c0 * d[0].w;
#pragma unroll
        for (int i = 1; i < K; ++i) {
          const float c = cmix[j * K + i];
          o.x = fmaf(c, d[i].x, o.x); o.y = fmaf(c, d[i].y, o.y); o.z = fmaf(c, d[i].z, o.z); o.w = fmaf(c, d[i].w, o.w);
        }
        *reinterpret_cast<float4*>(Ds + ((size_t)j * kTileW + px) * 64 + c4) = o;
      }
    }
    stage_patch(t + gridDim.x, cur ^ 1);   // (that buffer's last readers passed the barrier above)
    fetch(t + gridDim.x);                  // in flight during the products below
    asm volatile("cp.async.wait_group 1;\n" ::: "memory");      // this tile's patch has landed (the next one may be in flight)
    __syncthreads();
    const float* Xs = Xs0 + (size_t)cur * xbuf;
#pragma unroll 1
    for (int pp = 0; pp < kTileW / 16; ++pp) {
      const int px = stream + 16 * pp;
      // (unrolled: the loads of the next encoding are issued under the products of this one)
#pragma unroll
      for (int j = 0; j < K1; ++j) {
        const float4 d = *reinterpret_cast<const float4*>(Ds + ((size_t)j * kTileW + px) * 64 + cog * 4);
        const float4* xp = reinterpret_cast<const float4*>(Xs) + (size_t)j * kWgKH * p.PW + (size_t)px * p.stride;
#pragma unroll
        for (int u = 0; u < kWgKH; ++u) {
          const float4 x0 = xp[u * p.PW], x1 = xp[u * p.PW + 1], x2 = xp[u * p.PW + 2];
          const float xv[kWgKWC] = {x0.x, x0.y, x0.z, x1.x, x1.y, x1.z, x2.x, x2.y, x2.z};
#pragma unroll
          for (int vc = 0; vc < kWgKWC; ++vc) {
            float* a = acc[u * kWgKWC + vc];
            a[0] = fmaf(xv[vc], d.x, a[0]); a[1] = fmaf(xv[vc], d.y, a[1]);
            a[2] = fmaf(xv[vc], d.z, a[2]); a[3] = fmaf(xv[vc], d.w, a[3]);
          }
        }
      }
    }
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  // the two streams of a warp meet by shuffle, the eight warps in shared memory, the CTAs in dW
  __syncthreads();
#pragma unroll
  for (int k = 0; k < kWgKC; ++k)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[k][q] += __shfl_xor_sync(0xffffffffu, acc[k][q], 16);
  float* red = Ds;                                  // [8 warps][64 channels][27]
  if ((tid & 16) == 0) {
    const int warp = tid >> 5;
#pragma unroll
    for (int k = 0; k < kWgKC; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) red[((size_t)warp * 64 + cog * 4 + q) * kWgKC + k] = acc[k][q];
  }
  __syncthreads();
  for (int i = tid; i < 64 * kWgKC; i += kThreads) {
    float s = 0.f;
#pragma unroll
    for (int wp = 0; wp < kThreads / 32; ++wp) s += red[(size_t)wp * 64 * kWgKC + i];
    const int co = cb + i / kWgKC;
    if (co < p.cout && s != 0.f) atomicAdd(p.dW + (size_t)co * kWgKC + (i % kWgKC), p.scale * s);
  }
}

size_t stem_wgrad_smem(const Geom& g) {
  const int K1 = g.K + 1;
  const int PW = (kTileW - 1) * g.stride + g.kw;
  size_t ds = (size_t)K1 * kTileW * 64;
  const size_t red = (size_t)(kThreads / 32) * 64 * kWgKC;
  if (ds < red) ds = red;
  return (ds + 2 * (size_t)K1 * kWgKH * PW * 4 + (size_t)K1 * g.K + 4) * sizeof(float);
}

}  // namespace

bool stem_fused_supported(const Geom& g, int smem_optin) {
  if (g.kind != DK_CONV2D || g.layout != DK_NHWC || g.precision != DK_TF32X3) return false;
  // (longer contractions, e.g. a 7x7 stem, measured faster on the tensor-core kernels through patch rows)
  if ((g.cin % 4) == 0 || g.cin > 4 || g.kc > 64) return false;
  if ((long long)g.G * g.ho * ((g.wo + kTileW - 1) / kTileW) >= (1LL << 31)) return false;   // tile indices in 32 bits
  return stem_fwd_smem(g) <= (size_t)smem_optin / 2 - 1024;      // two CTAs per SM
}

dk_status launch_stem_fwd(const Geom& g, const float* W, const float* x, const float* r, const CoefView& cv,
                          const float* bias, float* y, const VerifyScratch& vs, const dk_fault* fault, int sm_count,
                          cudaStream_t st) {
  StemFwdParams p;
  p.W = W; p.x = x; p.r = r; p.bias = bias; p.y = y;
  p.enc = cv.enc; p.dec = cv.dec; p.nul = cv.nul; p.vs = vs; p.tau = g.tol;
  p.cin = g.cin; p.cout = g.cout; p.h = g.h; p.w = g.w; p.kh = g.kh; p.kw = g.kw; p.stride = g.stride; p.pad = g.pad;
  p.ho = g.ho; p.wo = g.wo; p.kc = g.kc; p.G = g.G;
  p.PW = (kTileW - 1) * g.stride + g.kw;
  p.tiles_w = (g.wo + kTileW - 1) / kTileW;
  p.ntiles = (long long)g.G * g.ho * p.tiles_w;
  p.f_group = -1; p.f_enc = 0; p.f_index = -1; p.f_delta = 0.f;
  p.kstore = g.kstore;
  if (fault) { p.f_group = fault->group; p.f_enc = fault->enc; p.f_index = fault->out_index; p.f_delta = fault->delta; }
  const size_t smem = stem_fwd_smem(g);
  const long long cap = 2LL * sm_count;
  const unsigned grid = (unsigned)(p.ntiles < cap ? p.ntiles : cap);
#define DK_STEM_CASE(KK)                                                                                     \
  case KK:                                                                                                   \
    if (smem > 48 * 1024)                                                                                    \
      DK_CUDA_CHECK(cudaFuncSetAttribute(stem_fwd_kernel<KK>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                         (int)smem));                                                        \
    stem_fwd_kernel<KK><<<grid, kThreads, smem, st>>>(p);                                                    \
    break;
  switch (g.K) {
    DK_STEM_CASE(1) DK_STEM_CASE(2) DK_STEM_CASE(3) DK_STEM_CASE(4)
    DK_STEM_CASE(5) DK_STEM_CASE(6) DK_STEM_CASE(7) DK_STEM_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_STEM_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk

namespace dk {

bool stem_wgrad_fused_supported(const Geom& g, int smem_optin) {
  if (g.kind != DK_CONV2D || g.layout != DK_NHWC || g.precision != DK_TF32X3) return false;
  if (g.cin != 3 || g.kh != kWgKH || g.kw != 3 || (g.cout % 4) != 0) return false;
  if ((long long)g.G * g.ho * ((g.wo + kTileW - 1) / kTileW) >= (1LL << 31)) return false;   // tile indices in 32 bits
  return stem_wgrad_smem(g) <= (size_t)smem_optin - 1024;
}

// dW = (accumulate ? dW : 0) + scale * sum over groups and encodings 0..K of <mixed delta, stored encoding>
dk_status launch_stem_wgrad(const Geom& g, const float* delta, const float* xbar, int xbar_rows, const float* dmix,
                            float scale, float* dW, bool clear, int sm_count, cudaStream_t st) {
  StemWgParams p;
  p.delta = delta; p.xbar = xbar; p.dmix = dmix; p.dW = dW;
  p.cout = g.cout; p.h = g.h; p.w = g.w; p.stride = g.stride; p.pad = g.pad; p.ho = g.ho; p.wo = g.wo; p.G = g.G;
  p.xbar_rows = xbar_rows;
  p.PW = (kTileW - 1) * g.stride + g.kw;
  p.tiles_w = (g.wo + kTileW - 1) / kTileW;
  p.ntiles = (long long)g.G * g.ho * p.tiles_w;
  p.scale = scale;
  if (clear) DK_CUDA_CHECK(cudaMemsetAsync(dW, 0, (size_t)g.cout * g.kc * sizeof(float), st));
  const size_t smem = stem_wgrad_smem(g);
  const int cblocks = (g.cout + 63) / 64;
  long long gx = sm_count / cblocks;
  if (gx < 1) gx = 1;
  if (gx > p.ntiles) gx = p.ntiles;
  dim3 grid((unsigned)gx, (unsigned)cblocks);
#define DK_STEMW_CASE(KK)                                                                                      \
  case KK:                                                                                                     \
    if (smem > 48 * 1024)                                                                                      \
      DK_CUDA_CHECK(cudaFuncSetAttribute(stem_wgrad_kernel<KK>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                         (int)smem));                                                          \
    stem_wgrad_kernel<KK><<<grid, kThreads, smem, st>>>(p);                                                    \
    break;
  switch (g.K) {
    DK_STEMW_CASE(1) DK_STEMW_CASE(2) DK_STEMW_CASE(3) DK_STEMW_CASE(4)
    DK_STEMW_CASE(5) DK_STEMW_CASE(6) DK_STEMW_CASE(7) DK_STEMW_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_STEMW_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
