// The masked path in the finite field F_p (Section 5 of the paper, Algorithm 1):
// quantisation to residues, Eq. 1 / Eq. 2 / the redundant equation of
// Section 4.4 and Eq. 4-6 modulo a prime p, with an exact equality test.
//
// Residues are uint32 in [0, p), p < 2^30.  A product of two residues is below
// 2^60; every contraction accumulates such products in uint64 and reduces
// before the sum can pass 2^64 (the host derives how many terms fit).
// Reduction is Barrett's: q = mulhi(x, floor(2^64 / p)) is the true quotient
// or one less, so x - q*p lies in [0, 2p).
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "dk_internal.h"
#include "dk_tc_kernel.cuh"

namespace dk {
namespace {

typedef unsigned int u32;
typedef unsigned long long u64;

struct Modulus {
  u64 m;     // floor(2^64 / p)
  u32 p;
  u32 m32;   // floor(2^(32+s) / p) with 2^s <= p < 2^(s+1); valid when s >= 0
  int s;     // -1 when p >= 2^27 (the short reduction is not offered)
};

__host__ __device__ __forceinline__ u32 reduce64(u64 x, Modulus md) {
#ifdef __CUDA_ARCH__
  u64 q = __umul64hi(x, md.m);
#else
  u64 q = (u64)(((unsigned __int128)x * md.m) >> 64);
#endif
  u64 r = x - q * md.p;
  if (r >= md.p) r -= md.p;
  if (r >= md.p) r -= md.p;
  return (u32)r;
}

// Short Barrett reduction for x < 2^(32+s): q = mulhi32(x >> s, m32) is the true
// quotient or up to two less, and x - q*p < 3p < 2^32 needs only the low words.
// The elementwise kernels' sums qualify when p < 2^27: at most 16 products
// below p^2 < 2^(2s+2) stay below 2^(32+s).
__device__ __forceinline__ u32 reduce_short(u64 x, Modulus md) {
  const u32 q = __umulhi((u32)(x >> md.s), md.m32);
  u32 r = (u32)x - q * md.p;
  if (r >= md.p) r -= md.p;
  if (r >= md.p) r -= md.p;
  return r;
}
__device__ __forceinline__ u32 reduce_sum(u64 x, Modulus md) {
  return md.s >= 0 ? reduce_short(x, md) : reduce64(x, md);
}

// ---------------------------------------------------------------------------
// host-side algebra in F_p (tiny matrices)
// ---------------------------------------------------------------------------
bool prime_by_trial_division(u32 p) {
  if (p < 3 || (p & 1) == 0) return false;
  for (u32 d = 3; (u64)d * d <= p; d += 2)
    if (p % d == 0) return false;
  return true;
}

u32 mulmod(u32 a, u32 b, u32 p) { return (u32)(((u64)a * b) % p); }

// a^(p-2) mod p: the inverse by Fermat's little theorem
u32 invmod(u32 a, u32 p) {
  u32 result = 1, base = a % p;
  u32 e = p - 2;
  while (e) {
    if (e & 1) result = mulmod(result, base, p);
    base = mulmod(base, base, p);
    e >>= 1;
  }
  return result;
}

// Gauss-Jordan elimination over F_p; false when singular.
bool invert_mod(const u32* M, int n, u32 p, u32* inv) {
  u32 a[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
  for (int i = 0; i < n * n; ++i) a[i] = M[i] % p;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) inv[i * n + j] = (i == j);
  for (int c = 0; c < n; ++c) {
    int piv = -1;
    for (int r = c; r < n && piv < 0; ++r)
      if (a[r * n + c]) piv = r;
    if (piv < 0) return false;
    if (piv != c)
      for (int j = 0; j < n; ++j) {
        u32 t = a[c * n + j]; a[c * n + j] = a[piv * n + j]; a[piv * n + j] = t;
        t = inv[c * n + j]; inv[c * n + j] = inv[piv * n + j]; inv[piv * n + j] = t;
      }
    const u32 ip = invmod(a[c * n + c], p);
    for (int j = 0; j < n; ++j) {
      a[c * n + j] = mulmod(a[c * n + j], ip, p);
      inv[c * n + j] = mulmod(inv[c * n + j], ip, p);
    }
    for (int r = 0; r < n; ++r) {
      if (r == c || a[r * n + c] == 0) continue;
      const u32 f = a[r * n + c];
      for (int j = 0; j < n; ++j) {
        a[r * n + j] = (a[r * n + j] + p - mulmod(f, a[c * n + j], p)) % p;
        inv[r * n + j] = (inv[r * n + j] + p - mulmod(f, inv[c * n + j], p)) % p;
      }
    }
  }
  return true;
}

// Per-call tables in device memory, one block per group (all residues):
// enc [G][K+2][K+1] as given; dec [G][K][K+1] rows 0..K-1 of C_sq^{-1};
// nul [G][K+2] with nul^T C = 0, nul[K+1] = 1; mix [G][K+1][K] = gamma_j*B[j][i].
struct FieldCoef {
  const u32* enc;
  const u32* dec;
  const u32* nul;
  const u32* mix;
};

dk_status upload_field_coefficients(dk_ctx* ctx, const Geom& g, u32 p, const u32* C_host,
                                    const u32* gamma_host, bool want_dec, bool want_mix,
                                    cudaStream_t st, FieldCoef* view) {
  const int K = g.K, K1 = K + 1, E = K + 2, G = g.G;
  const size_t n_enc = (size_t)G * E * K1, n_dec = (size_t)G * K * K1, n_nul = (size_t)G * E,
               n_mix = (size_t)G * K1 * K;
  const size_t total = n_enc + n_dec + n_nul + n_mix;
  if (total * sizeof(u32) > kCoefSlotBytes) return DK_ERR_SHAPE;
  for (size_t i = 0; i < n_enc; ++i)
    if (C_host[i] >= p) return DK_ERR_INVALID_ARG;

  int s = ctx->cur_slot;
  ctx->cur_slot = (s + 1) % kCoefSlots;
  if (ctx->slot_used[s]) DK_CUDA_CHECK(cudaEventSynchronize(ctx->slot_ev[s]));
  u32* h = reinterpret_cast<u32*>(ctx->h_stage + (size_t)s * kCoefSlotBytes);
  u32* d = reinterpret_cast<u32*>(ctx->d_stage + (size_t)s * kCoefSlotBytes);
  u32* h_enc = h;
  u32* h_dec = h_enc + n_enc;
  u32* h_nul = h_dec + n_dec;
  u32* h_mix = h_nul + n_nul;
  memcpy(h_enc, C_host, n_enc * sizeof(u32));
  memset(h_dec, 0, (n_dec + n_nul + n_mix) * sizeof(u32));
  if (want_dec || want_mix) {
    u32 inv[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
    for (int gi = 0; gi < G; ++gi) {
      const u32* Cg = C_host + (size_t)gi * E * K1;
      if (!invert_mod(Cg, K1, p, inv)) return DK_ERR_SINGULAR;
      for (int k = 0; k < K; ++k)
        for (int i = 0; i < K1; ++i) h_dec[((size_t)gi * K + k) * K1 + i] = inv[k * K1 + i];
      // null vector: n[0..K] = -C[K+1] . C_sq^{-1}, n[K+1] = 1.  A zero
      // component would hide a fault in that encoding from the check.
      for (int i = 0; i < K1; ++i) {
        u64 acc = 0;
        for (int k = 0; k < K1; ++k) acc = (acc + (u64)Cg[(size_t)K1 * K1 + k] * inv[k * K1 + i]) % p;
        const u32 ni = (u32)((p - acc) % p);
        if (ni == 0) return DK_ERR_SINGULAR;
        h_nul[(size_t)gi * E + i] = ni;
      }
      h_nul[(size_t)gi * E + K1] = 1;
      if (want_mix) {
        // Eq. 5: B[j][i] = inv[i][j] / gamma[j]; the kernels use gamma[j]*B[j][i]
        for (int j = 0; j < K1; ++j) {
          const u32 gm = gamma_host[(size_t)gi * K1 + j];
          if (gm == 0 || gm >= p) return DK_ERR_INVALID_ARG;
          const u32 gi_inv = invmod(gm, p);
          for (int i = 0; i < K; ++i) {
            const u32 B = mulmod(inv[i * K1 + j], gi_inv, p);
            h_mix[((size_t)gi * K1 + j) * K + i] = mulmod(gm, B, p);
          }
        }
      }
    }
  }
  DK_CUDA_CHECK(cudaMemcpyAsync(d, h, total * sizeof(u32), cudaMemcpyHostToDevice, st));
  DK_CUDA_CHECK(cudaEventRecord(ctx->slot_ev[s], st));
  ctx->slot_used[s] = true;
  view->enc = d;
  view->dec = d + n_enc;
  view->nul = view->dec + n_dec;
  view->mix = view->nul + n_nul;
  return DK_OK;
}

// ---------------------------------------------------------------------------
// elementwise kernels
// ---------------------------------------------------------------------------

// Field(Round(v * scale)), Algorithm 1: floor when the fractional part is
// below one half, floor + 1 otherwise; then the residue in [0, p).  v * scale
// (a power of two) and the fractional part are exact in fp32.
__global__ void __launch_bounds__(256) field_quantize_kernel(const float* __restrict__ v, long long n, float scale,
                                                            u32 p, u32* __restrict__ out) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float t = v[i] * scale;
    const float f = floorf(t);
    const float q = (t - f < 0.5f) ? f : f + 1.0f;
    u32 res = 0;
    if (fabsf(q) < 2.0e9f) {        // the usual case: 32-bit remainder
      int m = (int)q % (int)p;
      if (m < 0) m += (int)p;
      res = (u32)m;
    } else if (fabsf(q) < 4.0e18f) {      // also false for NaN
      long long m = (long long)q % (long long)p;
      if (m < 0) m += p;
      res = (u32)m;
    }
    out[i] = res;
  }
}

// value = centred residue * 2^-shift
__global__ void __launch_bounds__(256) field_dequantize_kernel(const u32* __restrict__ vq, long long n, u32 p,
                                                              double inv_scale, float* __restrict__ out) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const u32 r = vq[i];
    const long long c = (2ull * r > p) ? (long long)r - (long long)p : (long long)r;
    out[i] = (float)((double)c * inv_scale);
  }
}

template <int VEC>
struct Vec;
template <>
struct Vec<1> {
  u32 v[1];
  __device__ __forceinline__ void load(const u32* p) { v[0] = __ldg(p); }
  __device__ __forceinline__ void store(u32* p) const { *p = v[0]; }
};
template <>
struct Vec<4> {
  u32 v[4];
  __device__ __forceinline__ void load(const u32* p) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ void store(u32* p) const {
    *reinterpret_cast<uint4*>(p) = make_uint4(v[0], v[1], v[2], v[3]);
  }
};

// out[g*ROUT + i][e] = sum_{k<RA} T[g][i][k]*a[g*RA + k][e] (+ T[g][i][RA]*b[g][e] when b is given).
// Serves Eq. 1 (a = inputs, b = noise, ROUT = K+2) and the delta mixing of
// Eq. 4 (a = deltas, no b, ROUT = K+1).  RIN = RA + (b ? 1 : 0) <= 9 terms below
// 2^60 each: the sum stays below 2^64.
template <int RIN, int VEC>
__global__ void __launch_bounds__(256) field_mix_rows_kernel(const u32* __restrict__ a, const u32* __restrict__ b,
                                                            const u32* __restrict__ table, u32* __restrict__ out,
                                                            long long n, int rout, Modulus md) {
  __shared__ u32 T[(DK_MAX_K + 2) * (DK_MAX_K + 1)];
  const int g = blockIdx.y;
  const int RA = b ? RIN - 1 : RIN;
  for (int i = threadIdx.x; i < rout * RIN; i += blockDim.x) T[i] = table[(size_t)g * rout * RIN + i];
  __syncthreads();
  const long long nvec = n / VEC;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
    Vec<VEC> src[RIN];
#pragma unroll
    for (int k = 0; k < RIN; ++k) {
      if (k < RA) src[k].load(a + ((long long)g * RA + k) * n + i * VEC);
      else src[k].load(b + (long long)g * n + i * VEC);
    }
    for (int r = 0; r < rout; ++r) {
      u64 acc[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc[v] = 0;
#pragma unroll
      for (int k = 0; k < RIN; ++k) {
        const u32 c = T[r * RIN + k];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] += (u64)c * src[k].v[v];
      }
      Vec<VEC> o;
#pragma unroll
      for (int v = 0; v < VEC; ++v) o.v[v] = reduce_sum(acc[v], md);
      o.store(out + ((long long)g * rout + r) * n + i * VEC);
    }
  }
}

template <int VEC>
dk_status launch_mix_rows(int rin, const u32* a, const u32* b, const u32* table, u32* out, long long n, int rout,
                          int G, Modulus md, int sm_count, cudaStream_t st) {
  long long nvec = n / VEC;
  long long bx = (nvec + 255) / 256;
  const long long cap = (16LL * sm_count + G - 1) / G;
  if (bx > cap) bx = cap;
  if (bx < 1) bx = 1;
  dim3 grid((unsigned)bx, (unsigned)G);
  switch (rin) {
#define DK_CASE(R) \
  case R: field_mix_rows_kernel<R, VEC><<<grid, 256, 0, st>>>(a, b, table, out, n, rout, md); break;
    DK_CASE(1) DK_CASE(2) DK_CASE(3) DK_CASE(4) DK_CASE(5) DK_CASE(6) DK_CASE(7) DK_CASE(8) DK_CASE(9)
#undef DK_CASE
    default: return DK_ERR_SHAPE;
  }
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status mix_rows(int rin, const u32* a, const u32* b, const u32* table, u32* out, long long n, int rout, int G,
                   Modulus md, int sm_count, cudaStream_t st) {
  if (G > 65535) return DK_ERR_SHAPE;
  const bool vec4 = (n % 4) == 0 && ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) |
                                      reinterpret_cast<uintptr_t>(out)) & 15) == 0;
  return vec4 ? launch_mix_rows<4>(rin, a, b, table, out, n, rout, G, md, sm_count, st)
              : launch_mix_rows<1>(rin, a, b, table, out, n, rout, G, md, sm_count, st);
}

// Eq. 2 and the redundant equation in F_p.  One thread decodes VEC output
// positions of one group: it reads the K+2 encoded values, forms
// rho = sum_i nul[i]*ybar_i (mod p), which is zero exactly when the redundant
// equation agrees with the other K+1, decodes y_k = sum_i dec[k][i]*ybar_i
// (+ bias) and writes the centred integer and/or Round(y*2^-l)*2^-l.
// Flagged positions are counted per warp and reported with one atomic each.
struct DecodeParams {
  const u32* ybar;
  const u32* dec;
  const u32* nul;
  const u32* bias;   // residues, [cout], nullable
  int* yq;           // nullable
  float* y;          // nullable
  dk_verdict* v;
  long long n;       // positions per sample
  long long ch_div;  // channel of position e = (e / ch_div) % cout
  int cout;
  double inv_scale;  // 2^-l
  int lbits;         // l
  int kstore;        // decoded rows k >= kstore of a group (noise vectors, Section 4.5) are neither computed nor stored
  Modulus md;
};

template <int K, int VEC>
__global__ void __launch_bounds__(256) field_decode_verify_kernel(DecodeParams p) {
  constexpr int K1 = K + 1, E = K + 2;
  __shared__ u32 D[K * K1];
  __shared__ u32 N[E];
  const int g = blockIdx.y;
  for (int i = threadIdx.x; i < K * K1; i += blockDim.x) D[i] = p.dec[(size_t)g * K * K1 + i];
  for (int i = threadIdx.x; i < E; i += blockDim.x) N[i] = p.nul[(size_t)g * E + i];
  __syncthreads();
  const long long nvec = p.n / VEC;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long first = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long lane0 = first - (threadIdx.x & 31);
  // every lane of a warp runs the same number of rounds (the ballot below is warp-wide)
  for (long long i0 = lane0; i0 < nvec; i0 += stride) {
    const long long i = i0 + (threadIdx.x & 31);
    const bool act = i < nvec;
    unsigned int nbad = 0;
    long long firstbad = 0x7fffffffffffffffLL;
    if (act) {
      Vec<VEC> yb[E];
#pragma unroll
      for (int e = 0; e < E; ++e) yb[e].load(p.ybar + ((long long)g * E + e) * p.n + i * VEC);
      u64 rho[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) rho[v] = 0;
#pragma unroll
      for (int e = 0; e < E; ++e)
#pragma unroll
        for (int v = 0; v < VEC; ++v) rho[v] += (u64)N[e] * yb[e].v[v];
#pragma unroll
      for (int v = VEC - 1; v >= 0; --v)
        if (reduce_sum(rho[v], p.md) != 0) {
          ++nbad;
          firstbad = (long long)g * p.n + i * VEC + v;
        }
#pragma unroll
      for (int k = 0; k < K; ++k) {
        if (k >= p.kstore) continue;
        u64 acc[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = 0;
#pragma unroll
        for (int e = 0; e < K1; ++e) {
          const u32 c = D[k * K1 + e];
#pragma unroll
          for (int v = 0; v < VEC; ++v) acc[v] += (u64)c * yb[e].v[v];
        }
        const long long o = ((long long)g * K + k) * p.n + i * VEC;
        int cq[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          u32 r = reduce_sum(acc[v], p.md);
          if (p.bias) {
            const long long e = i * VEC + v;
            r += __ldg(p.bias + (int)((e / p.ch_div) % p.cout));
            if (r >= p.md.p) r -= p.md.p;
          }
          cq[v] = (2u * r > p.md.p) ? (int)r - (int)p.md.p : (int)r;      // p < 2^30: no overflow
        }
        if (p.yq) {
          if (VEC == 4) *reinterpret_cast<int4*>(p.yq + o) = make_int4(cq[0], cq[1], cq[2], cq[3 % VEC]);
          else p.yq[o] = cq[0];
        }
        if (p.y) {
          float yv[VEC];
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            // Round(c * 2^-l) = floor(c * 2^-l + 1/2) = (c + 2^(l-1)) >> l in integers (arithmetic shift = floor);
            // |c| < 2^29 keeps the sum in range and the quotient, below 2^24 for l >= 6, exact in fp32 for any l
            // once scaled by the power of two (a quotient of more than 24 bits rounds as the product would)
            const int q = p.lbits > 0 ? (cq[v] + (1 << (p.lbits - 1))) >> p.lbits : cq[v];
            yv[v] = __int2float_rn(q) * (float)p.inv_scale;      // (2^-l is a power of two: one rounding, as in fp64)
          }
          if (VEC == 4) *reinterpret_cast<float4*>(p.y + o) = make_float4(yv[0], yv[1], yv[2], yv[3 % VEC]);
          else p.y[o] = yv[0];
        }
      }
    }
    const unsigned int any = __ballot_sync(0xffffffffu, nbad != 0);
    if (any) {
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        nbad += __shfl_xor_sync(0xffffffffu, nbad, s);
        const long long other = __shfl_xor_sync(0xffffffffu, firstbad, s);
        firstbad = other < firstbad ? other : firstbad;
      }
      if ((threadIdx.x & 31) == 0) {
        atomicAdd(&p.v->n_flagged, nbad);
        atomicMin(reinterpret_cast<u64*>(&p.v->first_index), (u64)firstbad);
        atomicExch(&p.v->ok, 0);
        p.v->max_ratio = 1.0f;
      }
    }
  }
}

__global__ void field_verdict_begin_kernel(dk_verdict* v) {
  v->ok = 1;
  v->n_flagged = 0;
  v->first_index = -1;      // all ones: also the identity of the unsigned minimum
  v->max_ratio = 0.f;
  v->status = 0;
}

__global__ void field_add_fault_kernel(u32* ybar, long long index, u32 delta, u32 p) {
  ybar[index] = (u32)(((u64)ybar[index] + delta) % p);
}

template <int VEC>
dk_status launch_decode_t(int K, const DecodeParams& p, int G, int sm_count, cudaStream_t st) {
  long long nvec = p.n / VEC;
  long long bx = (nvec + 255) / 256;
  const long long cap = (16LL * sm_count + G - 1) / G;
  if (bx > cap) bx = cap;
  if (bx < 1) bx = 1;
  dim3 grid((unsigned)bx, (unsigned)G);
  switch (K) {
#define DK_CASE(KK) \
  case KK: field_decode_verify_kernel<KK, VEC><<<grid, 256, 0, st>>>(p); break;
    DK_CASE(1) DK_CASE(2) DK_CASE(3) DK_CASE(4) DK_CASE(5) DK_CASE(6) DK_CASE(7) DK_CASE(8)
#undef DK_CASE
    default: return DK_ERR_SHAPE;
  }
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

// ---------------------------------------------------------------------------
// the contraction <W_q, x_bar> modulo p (implicit GEMM, every geometry/layout)
// ---------------------------------------------------------------------------
constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

struct FwdParams {
  const u32* W;
  const u32* x;
  u32* y;
  int cin, cout, h, w, kw, stride, pad, ho, wo, kc;
  long long N;           // samples * ho * wo
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
  int fold_tiles;        // k-tiles between two reductions
  Modulus md;
};

__global__ void __launch_bounds__(NT) field_fwd_kernel(FwdParams p) {
  __shared__ __align__(16) u32 As[BK][BM + 4];
  __shared__ __align__(16) u32 Bs[BK][BN + 4];
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
    const int mm = t / BK + 16 * i;
    a_ok[i] = (m0 + mm) < p.cout;
    a_off[i] = (long long)(m0 + mm) * p.ws_o;
    const long long n = n0 + mm;
    b_ok[i] = n < p.N;
    const long long nn = b_ok[i] ? n : 0;
    const int ow = (int)(nn % p.wo);
    const long long r = nn / p.wo;
    const int oh = (int)(r % p.ho);
    const long long s = r / p.ho;
    b_base[i] = s * p.n_in;
    b_ih0[i] = oh * p.stride - p.pad;
    b_iw0[i] = ow * p.stride - p.pad;
  }

  u64 acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0;

  int fold = 0;
  for (int k0 = 0; k0 < p.kc; k0 += BK) {
    const int k = k0 + kk;
    const bool kok = k < p.kc;
    const int tap = kok ? k / p.cin : 0;
    const int ci = kok ? k - tap * p.cin : 0;
    const int u = tap / p.kw, v = tap - u * p.kw;
    const long long woff = (long long)ci * p.ws_c + (long long)u * p.ws_u + (long long)v * p.ws_v;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int mm = t / BK + 16 * i;
      As[kk][mm] = (kok && a_ok[i]) ? __ldg(p.W + a_off[i] + woff) : 0u;
      const int ih = b_ih0[i] + u, iw = b_iw0[i] + v;
      const bool ok = kok && b_ok[i] && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
      Bs[kk][mm] = ok ? __ldg(p.x + b_base[i] + (long long)ci * p.xs_c + (long long)ih * p.xs_h +
                              (long long)iw * p.xs_w)
                      : 0u;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < BK; ++q) {
      const uint4 a4 = *reinterpret_cast<const uint4*>(&As[q][ty * 4]);
      const uint4 b4 = *reinterpret_cast<const uint4*>(&Bs[q][tx * 4]);
      const u32 a[4] = {a4.x, a4.y, a4.z, a4.w};
      const u32 b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += (u64)a[i] * b[j];
    }
    __syncthreads();
    if (++fold == p.fold_tiles) {
      fold = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = reduce64(acc[i][j], p.md);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const long long n = n0 + tx * 4 + j;
    if (n >= p.N) continue;
    const int ow = (int)(n % p.wo);
    const long long r = n / p.wo;
    const int oh = (int)(r % p.ho);
    const long long s = r / p.ho;
    u32* yo = p.y + s * p.n_out + (long long)oh * p.ys_h + (long long)ow * p.ys_w;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m < p.cout) yo[(long long)m * p.ys_c] = reduce64(acc[i][j], p.md);
    }
  }
}

// ---------------------------------------------------------------------------
// The same contraction on the integer tensor cores.  A residue below 2^32 is
// four base-256 digits, which are the four bytes of its uint32 as stored, so
// <W_q, x_bar> = sum_{a,b<4} 2^{8(a+b)} * sum_k Wdigit_a[k] * xdigit_b[k]:
// sixteen u8 x u8 -> s32 matrix products (mma.sync m16n8k32), accumulated in
// seven s32 accumulators by weight class a+b and folded modulo p into uint64
// totals before a class can overflow (255^2 * 4 pairs * 4096 terms < 2^31).
// The digit planes are formed in registers by a 4x4 byte transpose of four
// consecutive k-elements; operands sit in shared memory as plain residues.
// ---------------------------------------------------------------------------
constexpr int MMA_BM = 64, MMA_BN = 64, MMA_BK = 32;
constexpr int kMmaFoldTiles = 4096 / MMA_BK;
constexpr int kMmaStageWords = (MMA_BM + MMA_BN) * MMA_BK;     // one pipeline stage: A tile then B tile
constexpr int kMmaStages = 4;
// Warp tile 16 x (8*kMmaNT): 4 x (8/kMmaNT) warps cover the 64 x 64 block tile.  Measured on conv layers of
// 64-512 channels: 4 n-tiles per warp (8 warps, 255 registers) 11-12 T modular MAC/s, 2 n-tiles (16 warps,
// 128 registers) 10-11: the rate does not follow occupancy, the tensor pipe reads 33 % busy in both.
constexpr int kMmaNT = 4;
constexpr int kMmaThreads = 1024 / kMmaNT;
constexpr size_t kMmaSmemBytes = (size_t)kMmaStages * kMmaStageWords * sizeof(u32);

struct RowInfo {        // one output pixel (column of the GEMM) of the block's tile
  long long base;       // offset of its sample in x, or -1 when past the end
  int ih0, iw0;
};

// Word k of row r of a 32-word tile row.  Odd rows swap their two 16-word
// halves, so that the 16-byte fragment reads of a quarter warp (rows r, r+1,
// four chunks each) fall into distinct banks.
__device__ __forceinline__ int tile_word(int r, int k) { return r * MMA_BK + (k ^ ((r & 1) << 4)); }

// Asynchronous global -> shared copy of BYTES (4 or 16); `valid` false writes zeros and reads nothing.
template <int BYTES>
__device__ __forceinline__ void copy_async(u32* smem_dst, const u32* gsrc, bool valid) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  const int n = valid ? BYTES : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;\n" ::"r"(d), "l"(gsrc), "n"(BYTES), "r"(n));
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void copy_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void digit_planes(const uint4 w, u32 (&pl)[4]) {
  const u32 t0 = __byte_perm(w.x, w.y, 0x5140), t1 = __byte_perm(w.z, w.w, 0x5140);
  const u32 u0 = __byte_perm(w.x, w.y, 0x7362), u1 = __byte_perm(w.z, w.w, 0x7362);
  pl[0] = __byte_perm(t0, t1, 0x5410);
  pl[1] = __byte_perm(t0, t1, 0x7632);
  pl[2] = __byte_perm(u0, u1, 0x5410);
  pl[3] = __byte_perm(u0, u1, 0x7632);
}

__device__ __forceinline__ void mma_u8(int (&d)[4], const u32 a0, const u32 a1, const u32 a2, const u32 a3,
                                       const u32 b0, const u32 b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct MmaConsts {
  u32 pow32;   // 2^32 mod p
};

// total = (total + sum_c acc_c * 2^{8c}) mod p for the seven class sums of one output element
__device__ __forceinline__ u32 fold_classes(u32 total, const int (&c)[7], Modulus md, u32 pow32) {
  const u64 lo = (u64)(u32)c[0] + ((u64)(u32)c[1] << 8) + ((u64)(u32)c[2] << 16) + ((u64)(u32)c[3] << 24);
  const u64 hi = (u64)(u32)c[4] + ((u64)(u32)c[5] << 8) + ((u64)(u32)c[6] << 16);     // weight 2^32
  const u64 t = (u64)total + reduce64(lo, md) + (u64)reduce64(hi, md) * pow32;
  return reduce64(t, md);
}

// VEC = 4: channels are contiguous in W and x and cin % 4 == 0, so four
// consecutive k-elements are 16 contiguous bytes of one filter tap; VEC = 1:
// every geometry and layout, one element per copy.
template <int VEC>
__global__ void __launch_bounds__(kMmaThreads, 1) field_fwd_mma_kernel(FwdParams p, MmaConsts mc) {
  extern __shared__ __align__(16) u32 tiles[];      // kMmaStages pipeline stages
  __shared__ RowInfo rows[MMA_BN];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int g = lane >> 2, tig = lane & 3;
  const int wm = warp & 3, wn = warp >> 2;          // warp tile: rows 16*wm.., columns 8*kMmaNT*wn..
  const int m0 = blockIdx.y * MMA_BM;
  const long long n0 = (long long)blockIdx.x * MMA_BN;

  if (t < MMA_BN) {
    const long long n = n0 + t;
    RowInfo ri;
    if (n < p.N) {
      const int ow = (int)(n % p.wo);
      const long long r = n / p.wo;
      const int oh = (int)(r % p.ho);
      ri.base = (r / p.ho) * p.n_in;
      ri.ih0 = oh * p.stride - p.pad;
      ri.iw0 = ow * p.stride - p.pad;
    } else {
      ri.base = -1; ri.ih0 = 0; ri.iw0 = 0;
    }
    rows[t] = ri;
  }
  __syncthreads();

  // loader: a thread copies elements k = kq .. kq+VEC-1 of rows r0 + RSTEP*i of both tiles
  constexpr int CPR = MMA_BK / VEC;              // copies per tile row
  constexpr int RSTEP = kMmaThreads / CPR, NCOPY = MMA_BM / RSTEP;
  const int kq = (t % CPR) * VEC, r0 = t / CPR;
  auto load_tile = [&](int k0, u32* stage) {
    const int k = k0 + kq;
    const bool kok = k < p.kc;
    const int tap = kok ? k / p.cin : 0;
    const int ci = kok ? k - tap * p.cin : 0;
    const int u = tap / p.kw, v = tap - u * p.kw;
    const long long woff = (long long)ci * p.ws_c + (long long)u * p.ws_u + (long long)v * p.ws_v;
    const long long xoff = (long long)ci * p.xs_c;
    u32* as = stage;
    u32* bs = stage + MMA_BM * MMA_BK;
#pragma unroll
    for (int i = 0; i < NCOPY; ++i) {
      const int mm = r0 + RSTEP * i;
      const bool aok = kok && (m0 + mm) < p.cout;
      copy_async<4 * VEC>(as + tile_word(mm, kq), aok ? p.W + (long long)(m0 + mm) * p.ws_o + woff : p.W, aok);
      const RowInfo ri = rows[mm];
      const int ih = ri.ih0 + u, iw = ri.iw0 + v;
      const bool ok = kok && ri.base >= 0 && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
      copy_async<4 * VEC>(bs + tile_word(mm, kq),
                          ok ? p.x + ri.base + xoff + (long long)ih * p.xs_h + (long long)iw * p.xs_w : p.x, ok);
    }
    copy_async_commit();
  };

  int acc[7][kMmaNT][4];       // [weight class][n-tile][fragment register]
  u32 tot[kMmaNT][4];
#pragma unroll
  for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      tot[j][r] = 0;
#pragma unroll
      for (int c = 0; c < 7; ++c) acc[c][j][r] = 0;
    }

  // Multi-stage pipeline with one barrier per k-tile: tiles kt+1 .. kt+S-2 are in
  // flight while tile kt is multiplied; the stage refilled in iteration kt is the
  // one every warp finished reading before it arrived at this iteration's barrier.
  // (A group is committed every iteration, empty past the end, so that
  // "all but the newest S-2 groups" always means "tile kt has landed".)
  const int ntiles = (p.kc + MMA_BK - 1) / MMA_BK;
#pragma unroll
  for (int s = 0; s < kMmaStages - 1; ++s) {
    if (s < ntiles) load_tile(s * MMA_BK, tiles + s * kMmaStageWords);
    else copy_async_commit();
  }
  int fold = 0;
  for (int kt = 0; kt < ntiles; ++kt) {
    u32* stage = tiles + (kt % kMmaStages) * kMmaStageWords;
    copy_async_wait<kMmaStages - 2>();
    __syncthreads();
    {
      const int nt = kt + kMmaStages - 1;
      if (nt < ntiles) load_tile(nt * MMA_BK, tiles + (nt % kMmaStages) * kMmaStageWords);
      else copy_async_commit();
    }
    {
      const u32* as = stage;
      const u32* bs = stage + MMA_BM * MMA_BK;
      u32 a[4][4];       // [fragment register][digit]
      const int ra = wm * 16 + g;      // rows ra and ra + 8 have the same parity
      digit_planes(*reinterpret_cast<const uint4*>(as + tile_word(ra, 4 * tig)), a[0]);
      digit_planes(*reinterpret_cast<const uint4*>(as + tile_word(ra + 8, 4 * tig)), a[1]);
      digit_planes(*reinterpret_cast<const uint4*>(as + tile_word(ra, 16 + 4 * tig)), a[2]);
      digit_planes(*reinterpret_cast<const uint4*>(as + tile_word(ra + 8, 16 + 4 * tig)), a[3]);
#pragma unroll
      for (int j = 0; j < kMmaNT; ++j) {
        u32 b[2][4];
        const int rb = wn * (8 * kMmaNT) + j * 8 + g;
        digit_planes(*reinterpret_cast<const uint4*>(bs + tile_word(rb, 4 * tig)), b[0]);
        digit_planes(*reinterpret_cast<const uint4*>(bs + tile_word(rb, 16 + 4 * tig)), b[1]);
        // digit pairs in an order that keeps two products of one weight class four instructions apart
#pragma unroll
        for (int da = 0; da < 4; ++da)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int db = (i + 4 - da) & 3;
            mma_u8(acc[da + db][j], a[0][da], a[1][da], a[2][da], a[3][da], b[0][db], b[1][db]);
          }
      }
    }
    if (++fold == kMmaFoldTiles) {
      fold = 0;
#pragma unroll
      for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int c[7] = {acc[0][j][r], acc[1][j][r], acc[2][j][r], acc[3][j][r],
                            acc[4][j][r], acc[5][j][r], acc[6][j][r]};
          tot[j][r] = fold_classes(tot[j][r], c, p.md, mc.pow32);
#pragma unroll
          for (int cc = 0; cc < 7; ++cc) acc[cc][j][r] = 0;
        }
    }
  }
  // fragment register r of n-tile j: row g + 8*(r >> 1), column 2*tig + (r & 1)
#pragma unroll
  for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
    for (int cb = 0; cb < 2; ++cb) {
      const long long n = n0 + wn * (8 * kMmaNT) + j * 8 + 2 * tig + cb;
      if (n >= p.N) continue;
      const int ow = (int)(n % p.wo);
      const long long rr = n / p.wo;
      const int oh = (int)(rr % p.ho);
      u32* yo = p.y + (rr / p.ho) * p.n_out + (long long)oh * p.ys_h + (long long)ow * p.ys_w;
#pragma unroll
      for (int rb = 0; rb < 2; ++rb) {
        const int r = rb * 2 + cb;
        const int m = m0 + wm * 16 + g + 8 * rb;
        if (m >= p.cout) continue;
        const int c[7] = {acc[0][j][r], acc[1][j][r], acc[2][j][r], acc[3][j][r],
                          acc[4][j][r], acc[5][j][r], acc[6][j][r]};
        yo[(long long)m * p.ys_c] = fold_classes(tot[j][r], c, p.md, mc.pow32);
      }
    }
}

// ---------------------------------------------------------------------------
// The forward contraction on the tcgen05 integer tensor path.  Same digit
// decomposition as above, but the sixteen u8 x u8 products of a k-step are
// tcgen05.mma.kind::i8 instructions on digit PLANES in shared memory (K-major,
// 128-byte swizzle: one row = 128 contraction elements of one digit), and the
// seven weight-class sums live in tensor memory (7 x 64 columns of s32).
//
//   tile: 128 output channels (TMEM lanes) x 64 pixels, k-tiles of 128 elements
//   16 producer warps: fetch W's digit planes (cp.async), load residues of x
//                (16-byte groups of one filter tap), split them into digit planes,
//                store the planes swizzled; two stages, handed over by mbarriers
//   one thread of a 17th warp: 64 MMAs per k-tile (16 digit pairs x 4 k-steps of 32), commit
//   the producer warps: at the end (and every 64 k-tiles, before a class sum can pass
//                2^31) read the class sums with tcgen05.ld and fold them mod p;
//                between two folds the partial residues wait in the output buffer
// Every mbarrier wait is bounded; on expiry the CTA stops issuing, reports
// DK_ERR_TIMEOUT in *status, still frees its tensor memory and returns.
// ---------------------------------------------------------------------------
namespace tcf {
constexpr int TM = 128, TN = 64, TK = 128;
constexpr int kProducers = 512;                 // 16 warps fill the stages and read the sums
constexpr int kThreads = kProducers + 32;       // + one warp whose first lane issues the products
constexpr int A_PLANE = TM * TK, B_PLANE = TN * TK;              // bytes per digit plane
constexpr int STAGE = 4 * A_PLANE + 4 * B_PLANE;                 // 96 KB
constexpr int kStages = 2;
constexpr size_t kSmem = (size_t)kStages * STAGE + 1024;         // + slack for 1024-byte alignment
constexpr int kFoldTiles = 8192 / TK;                            // 4 pairs * 255^2 * 8192 < 2^31

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned cap) {
  for (unsigned i = 0; i < cap; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void ld8(uint32_t taddr, int (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}
// K-major operand plane, rows of 128 bytes (one swizzle span), 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t plane_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= 2ull << 61;                 // 128-byte swizzle
  return d;
}
}  // namespace tcf

// W as four digit planes, [digit][cout][kcp] bytes with kcp = kc rounded up to the k-tile (zero filled):
// written once per call, so that every CTA fetches its rows of W as ready 16-byte chunks.
__global__ void __launch_bounds__(256) field_w_planes_kernel(const u32* __restrict__ W, int cout, int kc, int kcp,
                                                            uint8_t* __restrict__ planes) {
  const long long chunks = (long long)cout * (kcp / 16);
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += stride) {
    const int m = (int)(i / (kcp / 16));
    const int k0 = (int)(i - (long long)m * (kcp / 16)) * 16;
    u32 pl[4][4];
#pragma unroll
    for (int gq = 0; gq < 4; ++gq) {
      const int k = k0 + gq * 4;
      const uint4 w = k < kc ? __ldg(reinterpret_cast<const uint4*>(W + (long long)m * kc + k))
                             : make_uint4(0u, 0u, 0u, 0u);
      digit_planes(w, pl[gq]);
    }
#pragma unroll
    for (int dg = 0; dg < 4; ++dg)
      *reinterpret_cast<uint4*>(planes + ((long long)dg * cout + m) * kcp + k0) =
          make_uint4(pl[0][dg], pl[1][dg], pl[2][dg], pl[3][dg]);
  }
}

__global__ void __launch_bounds__(tcf::kThreads, 1) field_fwd_tc_kernel(FwdParams p, MmaConsts mc,
                                                                       const uint8_t* __restrict__ wplanes, int kcp,
                                                                       u64* split_acc, int tiles_per_split,
                                                                       int* status, unsigned spin_cap, int withhold) {
  // spin_cap: polls after which a wait gives up; withhold (test hook, -1 = off): thread 0 does not arrive
  // for that k-tile's stage and stops, so every other role's wait runs out
  using namespace tcf;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[kStages];     // a stage's planes are in shared memory (kProducers arrivals)
  __shared__ uint64_t mma_done[kStages];     // the products that read a stage have completed (one commit)
  __shared__ uint32_t tmem_slot[2];          // [0] TMEM base address, [1] abort flag
  __shared__ RowInfo rows[TN];
  __shared__ long long out_off[TN];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int m0 = blockIdx.y * TM;
  const long long n0 = (long long)blockIdx.x * TN;

  if (t == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar + s, kProducers); mbar_init(mma_done + s, 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (t < TN) {
    const long long n = n0 + t;
    RowInfo ri;
    long long oo = -1;
    if (n < p.N) {
      const int ow = (int)(n % p.wo);
      const long long r = n / p.wo;
      const int oh = (int)(r % p.ho);
      const long long smp = r / p.ho;
      ri.base = smp * p.n_in;
      ri.ih0 = oh * p.stride - p.pad;
      ri.iw0 = ow * p.stride - p.pad;
      oo = smp * p.n_out + (long long)oh * p.ys_h + (long long)ow * p.ys_w;
    } else {
      ri.base = -1; ri.ih0 = 0; ri.iw0 = 0;
    }
    rows[t] = ri;
    out_off[t] = oo;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot[0];
  // this CTA's slice of the contraction: k-tiles kt0 .. kt0 + ntiles - 1 (the whole of it unless the launch
  // is split; slices meet as residues in split_acc, a uint64 per output element that the caller cleared)
  const int kt0 = blockIdx.z * tiles_per_split;
  const int ntiles = min(tiles_per_split, (p.kc + TK - 1) / TK - kt0);

  if (warp == kProducers / 32) {
    // ---------------- MMA issuer: one thread ----------------
    if (lane == 0) {
      // S32 accumulator, unsigned 8-bit A and B, both K-major, M = 128; N = 64 columns per weight class.
      // The four digit planes of x lie one after the other in shared memory, so W's digit a against ALL of
      // them is one instruction with N = 256 whose result columns are the classes a .. a+3, which are
      // adjacent in tensor memory too: four instructions per k-step instead of sixteen.  Only the first
      // k-step after a fold, where some of those classes must be overwritten and others added to, is split.
      auto idesc_n = [](int n) {
        return (2u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      };
      bool fresh = true;               // no product since the last fold
      for (int kt = 0; kt < ntiles; ++kt) {
        const int stage = kt & 1;
        if (!mbar_wait(full_bar + stage, (uint32_t)((kt / kStages) & 1), abort_flag, spin_cap)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_u32(smem + (size_t)stage * STAGE), sb = sa + 4 * A_PLANE;
        const uint64_t bdesc = plane_desc(sb);
#pragma unroll
        for (int ks = 0; ks < TK / 32; ++ks) {
          const uint64_t adv = (uint64_t)(ks * 2);       // 32 bytes per k-step, in 16-byte units
#pragma unroll
          for (int da = 0; da < 4; ++da) {
            const uint64_t adesc = plane_desc(sa + da * A_PLANE) + adv;
            const uint32_t d = tmem_base + (uint32_t)(da * TN);
            if (fresh && ks == 0 && da > 0) {
              // classes da .. da+2 have a product already, class da+3 has none
              mma_i8(d, adesc, bdesc + adv, idesc_n(3 * TN), 1u);
              mma_i8(d + 3 * TN, adesc, plane_desc(sb + 3 * B_PLANE) + adv, idesc_n(TN), 0u);
            } else {
              mma_i8(d, adesc, bdesc + adv, idesc_n(4 * TN), (fresh && ks == 0) ? 0u : 1u);
            }
          }
        }
        fresh = false;
        commit(mma_done + stage);
        if (((kt + 1) % kFoldTiles) == 0) fresh = true;      // the producers fold and restart the sums here
      }
    }
  } else {
    // ---------------- producers (and, at a fold, readers of the sums): 16 warps ----------------
    // this thread's part of the result: TMEM lane (output channel) 32*(warp & 3) + lane, columns 16*(warp >> 2) ..
    const int q = warp & 3, h = warp >> 2;
    bool folded = false;           // a partial result is already in y
    bool alive = true;
    for (int kt = 0; alive && kt < ntiles; ++kt) {
      const int stage = kt & 1;
      uint8_t* st = smem + (size_t)stage * STAGE;
      // the products that read this stage two k-tiles ago must have completed
      if (kt >= kStages && !mbar_wait(mma_done + stage, (uint32_t)((kt / kStages - 1) & 1), abort_flag, spin_cap)) {
        alive = false;
        break;
      }
      // units of 16 contraction elements of one row.  A thread's units all sit in the same 16-element
      // column c = t & 7 of the k-tile, so the filter taps of its four 4-element groups are worked out once.
      const int c = t & 7;
      int g_ci[4], g_u[4], g_v[4];
      bool g_ok[4];
      {
        int k = (kt0 + kt) * TK + c * 16;
        int tap = k / p.cin;
        int ci = k - tap * p.cin;
        int u = tap / p.kw, v = tap - u * p.kw;
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
          g_ok[gq] = k < p.kc;
          g_ci[gq] = ci; g_u[gq] = u; g_v[gq] = v;
          k += 4; ci += 4;
          if (ci >= p.cin) {
            ci -= p.cin;
            if (++v == p.kw) { v = 0; ++u; }
          }
        }
      }
      // rows of W: ready digit planes, copied asynchronously chunk by chunk into the swizzled layout
#pragma unroll
      for (int i = 0; i < 4 * TM * 8 / kProducers; ++i) {
        const int idx = t + i * kProducers;            // (digit, row, chunk)
        const int dg = idx / (TM * 8), row = (idx >> 3) & (TM - 1);
        const bool rok = m0 + row < p.cout;
        const uint8_t* src = wplanes + ((long long)dg * p.cout + (rok ? m0 + row : 0)) * kcp + (kt0 + kt) * TK + c * 16;
        const unsigned dst = smem_u32(st + dg * A_PLANE + row * TK + ((c ^ (row & 7)) << 4));
        const int nbytes = rok ? 16 : 0;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(nbytes));
      }
      asm volatile("cp.async.commit_group;\n" ::);
      // pixels of x: one unit of 16 contraction elements per thread
      {
        static_assert(TN * 8 == kProducers, "one x unit per thread");
        const int row = t >> 3;
        const RowInfo ri = rows[row];
        uint4 w[4];
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
          const int ih = ri.ih0 + g_u[gq], iw = ri.iw0 + g_v[gq];
          const bool ok = g_ok[gq] && ri.base >= 0 && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
          w[gq] = ok ? __ldg(reinterpret_cast<const uint4*>(p.x + ri.base + g_ci[gq] + (long long)ih * p.xs_h +
                                                            (long long)iw * p.xs_w))
                     : make_uint4(0u, 0u, 0u, 0u);
        }
        u32 pl[4][4];      // [group of four elements][digit]
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) digit_planes(w[gq], pl[gq]);
        uint8_t* base = st + 4 * A_PLANE + row * TK + ((c ^ (row & 7)) << 4);
#pragma unroll
        for (int dg = 0; dg < 4; ++dg)
          *reinterpret_cast<uint4*>(base + dg * B_PLANE) = make_uint4(pl[0][dg], pl[1][dg], pl[2][dg], pl[3][dg]);
      }
      asm volatile("cp.async.wait_group 0;\n" ::);
      // make the planes visible to the tensor core's (asynchronous-proxy) reads, then hand the stage over
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (t == 0 && kt == withhold) { alive = false; break; }      // test hook: this stage never becomes full
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(full_bar + stage)) : "memory");

      // fold before a class sum can overflow, and at the end
      const bool last = kt + 1 == ntiles;
      if (last || ((kt + 1) % kFoldTiles) == 0) {
        // every product issued so far has completed once the commit of this k-tile has arrived
        // (a commit covers all earlier products of the issuing thread)
        if (!mbar_wait(mma_done + stage, (uint32_t)((kt / kStages) & 1), abort_flag, spin_cap)) {
          alive = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int m = m0 + q * 32 + lane;
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          int cls[7][8];
#pragma unroll
          for (int c = 0; c < 7; ++c)
            ld8(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * TN + h * 16 + cg * 8), cls[c]);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const long long oo = out_off[h * 16 + cg * 8 + j];
            if (oo < 0 || m >= p.cout) continue;
            u32* dst = p.y + oo + (long long)m * p.ys_c;
            const int cc[7] = {cls[0][j], cls[1][j], cls[2][j], cls[3][j], cls[4][j], cls[5][j], cls[6][j]};
            if (split_acc != nullptr) atomicAdd(split_acc + (dst - p.y), (u64)fold_classes(0u, cc, p.md, mc.pow32));
            else *dst = fold_classes(folded ? *dst : 0u, cc, p.md, mc.pow32);
          }
        }
        folded = true;
        // the next arrival on a full barrier orders these reads before the products that overwrite the sums
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      }
    }
  }
  __syncthreads();
  if (*abort_flag) {
    // a bounded wait expired: report, and give products still in flight time to retire
    if (t == 0 && status != nullptr) atomicExch(status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---------------------------------------------------------------------------
// The forward contraction with operands fetched by TMA.  Both operands are digit planes in global memory
// (W_q as [digit][cout][k], written by field_w_planes_kernel; x_bar as [digit][sample][h][w][cin], written by
// field_x_planes_kernel), so a pipeline stage is two bulk tensor copies: 128 rows of W and, for filter tap
// (u,v), the tile's box of 64 output pixels shifted by (u-pad, v-pad), all four digits of each; positions
// outside the image are zero-filled by the TMA unit.  One producer thread, one MMA thread, eight warps that
// read and fold the class sums.  KT = contraction elements per k-tile = bytes per shared-memory row (one
// swizzle span): 128 when cin % 128 == 0 (two stages), else 64 (cin % 64 == 0, four stages).  Stride 1 only.
// The products, the merged N = 256 instruction and the folds are those of field_fwd_tc_kernel above.
// ---------------------------------------------------------------------------
namespace ftm {
constexpr int TM = 128, TN = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;      // producer warp, MMA warp, epilogue warps
constexpr int kFoldK = 8192;                       // contraction elements between folds: 4 pairs * 255^2 * 8192 < 2^31

struct Params {
  int bw, bh, bs;              // the 64 columns of a tile: a box of bw x bh output pixels of bs samples (powers of two)
  int WT, HT;                  // tiles along width and height (sample tile = blockIdx.x / (WT*HT))
  int cblocks;                 // cin / KT
  int kw, pad;
  int ktiles, tiles_per_split; // k-tiles in all and per contraction slice (blockIdx.z)
  int cout, ho, wo, nsamples;
  long long n_out, ys_c, ys_h, ys_w;
  u32* y;
  u64* split_acc;              // nullable: slices add their residues here
  Modulus md;
  u32 pow32;
  int* status;
  unsigned spin_cap;
  int withhold;                // test hook: the producer arms this k-tile's stage, copies nothing and stops (-1 = off)
};
}  // namespace ftm

// Activations as four digit planes, [digit][sample][h][w][c] bytes (the element order of the source).  The
// source holds `rows` samples per group of which the first `used` are copied (rows = used: all of them):
// n = elements written per plane = groups * used * row_elems; row_elems % 16 == 0.
__global__ void __launch_bounds__(256) field_x_planes_kernel(const u32* __restrict__ x, long long n, uint8_t* __restrict__ planes,
                                                            long long row_elems, int rows, int used) {
  const long long chunks = n / 16;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += stride) {
    long long src = i * 16;
    if (rows != used) {
      const long long r = src / row_elems;                 // destination row = group * used + j
      src += (r / used) * (long long)(rows - used) * row_elems;
    }
    u32 pl[4][4];
#pragma unroll
    for (int gq = 0; gq < 4; ++gq)
      digit_planes(__ldg(reinterpret_cast<const uint4*>(x + src) + gq), pl[gq]);
#pragma unroll
    for (int dg = 0; dg < 4; ++dg)
      *reinterpret_cast<uint4*>(planes + (long long)dg * n + i * 16) = make_uint4(pl[0][dg], pl[1][dg], pl[2][dg], pl[3][dg]);
  }
}

template <int KT>
__global__ void __launch_bounds__(ftm::kThreads, 1)
field_fwd_tma_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                     const ftm::Params p) {
  using namespace ftm;
  constexpr int A_PLANE = TM * KT, B_PLANE = TN * KT, STAGE = 4 * (A_PLANE + B_PLANE);
  constexpr int NST = KT == 128 ? 2 : 4;
  constexpr int kFoldTiles = kFoldK / KT;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[NST];       // a stage's two copies have landed (transaction bytes)
  __shared__ uint64_t empty_bar[NST];      // the products that read a stage have completed (one commit)
  __shared__ uint64_t tfull_bar;           // every product up to a fold point has completed (one commit)
  __shared__ uint64_t tempty_bar;          // the class sums have been read (one arrival per epilogue warp)
  __shared__ uint32_t tmem_slot[2];        // [0] TMEM base address, [1] abort flag
  uint8_t* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int m0 = blockIdx.y * TM;
  const int wt = blockIdx.x % p.WT, ht = (blockIdx.x / p.WT) % p.HT, stl = blockIdx.x / (p.WT * p.HT);
  const int x0 = wt * p.bw, y0 = ht * p.bh, s0 = stl * p.bs;
  const int kt0 = blockIdx.z * p.tiles_per_split;
  const int ntiles = min(p.tiles_per_split, p.ktiles - kt0);
  const int nfolds = (ntiles + kFoldTiles - 1) / kFoldTiles;

  if (t == 0) {
    for (int s = 0; s < NST; ++s) { tc::mbar_init(full_bar + s, 1); tc::mbar_init(empty_bar + s, 1); }
    tc::mbar_init(&tfull_bar, 1);
    tc::mbar_init(&tempty_bar, kEpiWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = tmem_slot[0];

  if (warp == 0) {
    // ---------------- TMA producer: one thread ----------------
    if (lane == 0) {
      for (int kt = 0; kt < ntiles; ++kt) {
        const int stage = kt % NST;
        if (kt >= NST && !tc::mbar_wait(empty_bar + stage, (uint32_t)((kt / NST - 1) & 1), abort_flag, p.spin_cap)) break;
        tc::mbar_expect_tx(full_bar + stage, (uint32_t)STAGE);
        if (kt == p.withhold) break;      // test hook: armed, nothing copied
        const int ktg = kt0 + kt;
        const int tap = ktg / p.cblocks, c0 = (ktg - tap * p.cblocks) * KT;
        const int u = tap / p.kw, v = tap - u * p.kw;
        uint8_t* st = smem + (size_t)stage * STAGE;
        tc::tma_load_3d(st, &map_w, full_bar + stage, ktg * KT, m0, 0);
        tc::tma_load_5d(st + 4 * A_PLANE, &map_x, full_bar + stage, c0, x0 + v - p.pad, y0 + u - p.pad, s0, 0);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one thread ----------------
    if (lane == 0) {
      // S32 accumulator, unsigned 8-bit A and B, both K-major, M = 128; W's digit a against all four digit planes
      // of x_bar (adjacent in shared memory) is one instruction with N = 256 whose columns are classes a .. a+3
      auto idesc_n = [](int n) {
        return (2u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      };
      bool fresh = true;               // no product since the last fold
      int fold = 0;
      for (int kt = 0; kt < ntiles; ++kt) {
        const int stage = kt % NST;
        if (fresh && fold > 0) {
          // the class sums of the previous fold must have been read before they are overwritten
          if (!tc::mbar_wait(&tempty_bar, (uint32_t)((fold - 1) & 1), abort_flag, p.spin_cap)) break;
          tc::tc_fence_after();
        }
        if (!tc::mbar_wait(full_bar + stage, (uint32_t)((kt / NST) & 1), abort_flag, p.spin_cap)) break;
        tc::tc_fence_after();
        const uint32_t sa = tc::smem_u32(smem + (size_t)stage * STAGE), sb = sa + 4 * A_PLANE;
        const uint64_t bdesc = tc::make_desc<KT>(sb);
#pragma unroll
        for (int ks = 0; ks < KT / 32; ++ks) {
          const uint64_t adv = (uint64_t)(ks * 2);       // 32 bytes per k-step, in 16-byte units
#pragma unroll
          for (int da = 0; da < 4; ++da) {
            const uint64_t adesc = tc::make_desc<KT>(sa + da * A_PLANE) + adv;
            const uint32_t d = tmem_base + (uint32_t)(da * TN);
            if (fresh && ks == 0 && da > 0) {
              // classes da .. da+2 have a product already, class da+3 has none
              tcf::mma_i8(d, adesc, bdesc + adv, idesc_n(3 * TN), 1u);
              tcf::mma_i8(d + 3 * TN, adesc, tc::make_desc<KT>(sb + 3 * B_PLANE) + adv, idesc_n(TN), 0u);
            } else {
              tcf::mma_i8(d, adesc, bdesc + adv, idesc_n(4 * TN), (fresh && ks == 0) ? 0u : 1u);
            }
          }
        }
        fresh = false;
        tc::tc_commit(empty_bar + stage);
        if (kt + 1 == ntiles || ((kt + 1) % kFoldTiles) == 0) {
          tc::tc_commit(&tfull_bar);      // (a commit covers all earlier products of this thread)
          fresh = true;
          ++fold;
        }
      }
    }
  } else {
    // ---------------- epilogue: eight warps read the class sums at every fold point and fold them ----------------
    // this thread: TMEM lane (output channel) 32*q + lane, columns 32*h .. 32*h+31
    const int q = warp & 3, h = (warp - 2) >> 2;
    const int m = m0 + q * 32 + lane;
    bool alive = true;
    for (int fold = 0; alive && fold < nfolds; ++fold) {
      if (!tc::mbar_wait(&tfull_bar, (uint32_t)(fold & 1), abort_flag, p.spin_cap)) { alive = false; break; }
      tc::tc_fence_after();
#pragma unroll 1
      for (int cg = 0; cg < 4; ++cg) {
        int cls[7][8];
#pragma unroll
        for (int c = 0; c < 7; ++c)
          tcf::ld8(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * TN + h * 32 + cg * 8), cls[c]);
        tc::tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int col = h * 32 + cg * 8 + j;
          const int dx = col % p.bw, dy = (col / p.bw) % p.bh, ds = col / (p.bw * p.bh);
          const int ow = x0 + dx, oh = y0 + dy, smp = s0 + ds;
          if (ow >= p.wo || oh >= p.ho || smp >= p.nsamples || m >= p.cout) continue;
          const long long off = (long long)smp * p.n_out + (long long)oh * p.ys_h + (long long)ow * p.ys_w +
                                (long long)m * p.ys_c;
          const int cc[7] = {cls[0][j], cls[1][j], cls[2][j], cls[3][j], cls[4][j], cls[5][j], cls[6][j]};
          if (p.split_acc != nullptr) atomicAdd(p.split_acc + off, (u64)fold_classes(0u, cc, p.md, p.pow32));
          else p.y[off] = fold_classes(fold > 0 ? p.y[off] : 0u, cc, p.md, p.pow32);
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&tempty_bar);
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a bounded wait expired: report, and give copies and products still in flight time to retire
    if (t == 0 && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  if (warp == 1) {
    tc::tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---------------------------------------------------------------------------
// The weight-gradient contraction on tcgen05 (Eq. 4-6 in F_p):
//   dW[co][tap][ci] = sum_{sample, pixel} dtil[sample][pixel][co] * xbar[sample][pixel + tap - pad][ci]   (mod p)
// M = 128 output channels, N = 64 input channels of one filter tap, the contraction runs over output pixels:
// the contiguous dimension of neither operand, so both digit-plane tiles are MN-major ([pixel][channel] rows of
// 128 and 64 bytes, one swizzle span each), fetched by TMA as boxes of 64 pixels (the box of x_bar shifted by the
// tap; zero fill outside the image).  As in the forward kernels a digit of dtil against all four digit planes
// of x_bar is one N = 256 instruction, and seven class sums live in tensor memory; they are folded every 8192
// contraction elements and at the end, and the residues are added to the uint64 accumulators of dW.
// Grid: (cout tile x channel block x tap, contraction slice).  Stride 1, channels-last, cin and cout % 16 == 0.
// ---------------------------------------------------------------------------
namespace fwg {
constexpr int TM = 128, TN = 64, KP = 64, NST = 4;
constexpr int A_PLANE = KP * TM, B_PLANE = KP * TN, STAGE = 4 * (A_PLANE + B_PLANE);      // 48 KB
constexpr size_t kSmem = (size_t)NST * STAGE + 1024;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kFoldStages = 8192 / KP;

struct Params {
  int bw, bh, bs;              // the 64 pixels of a k-block: bw x bh output pixels of bs samples (powers of two)
  int WT, HT;                  // pixel blocks along width and height (sample block = pb / (WT*HT))
  long long PB;                // pixel blocks in all
  int pb_per_split;
  int MT, cblocks, kw, pad;
  int cout, cin;
  long long ws_o, ws_c, ws_u, ws_v;
  u64* acc;
  Modulus md;
  u32 pow32;
  int* status;
  unsigned spin_cap;
  int withhold;
};

// MN-major operand: rows of ROW bytes (one swizzle span) along the contraction, 8-row groups ROW*8 bytes apart,
// further spans of ROW channels `span_bytes` apart
template <int ROW>
__device__ __forceinline__ uint64_t desc_mn(uint32_t smem_addr, uint32_t span_bytes) {
  constexpr uint64_t layout = ROW == 128 ? 2ull : 4ull;
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)((span_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((ROW * 8) >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= layout << 61;
  return d;
}
}  // namespace fwg

__global__ void __launch_bounds__(fwg::kThreads, 1)
field_wgrad_tma_kernel(const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_x,
                       const fwg::Params p) {
  using namespace fwg;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[NST], empty_bar[NST], tfull_bar, tempty_bar;
  __shared__ uint32_t tmem_slot[2];        // [0] TMEM base address, [1] abort flag
  uint8_t* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int item = blockIdx.x;
  const int mt = item % p.MT, cb = (item / p.MT) % p.cblocks, tap = item / (p.MT * p.cblocks);
  const int m0 = mt * TM, c0 = cb * TN;
  const int u = tap / p.kw, v = tap - u * p.kw;
  const long long pb0 = (long long)blockIdx.y * p.pb_per_split;
  const int nst = (int)min((long long)p.pb_per_split, p.PB - pb0);
  const int nfolds = (nst + kFoldStages - 1) / kFoldStages;

  if (t == 0) {
    for (int s = 0; s < NST; ++s) { tc::mbar_init(full_bar + s, 1); tc::mbar_init(empty_bar + s, 1); }
    tc::mbar_init(&tfull_bar, 1);
    tc::mbar_init(&tempty_bar, kEpiWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = tmem_slot[0];

  if (warp == 0) {
    // ---------------- TMA producer: one thread ----------------
    if (lane == 0) {
      for (int k = 0; k < nst; ++k) {
        const int stage = k % NST;
        if (k >= NST && !tc::mbar_wait(empty_bar + stage, (uint32_t)((k / NST - 1) & 1), abort_flag, p.spin_cap)) break;
        tc::mbar_expect_tx(full_bar + stage, (uint32_t)STAGE);
        if (k == p.withhold) break;      // test hook: armed, nothing copied
        const long long pb = pb0 + k;
        const int wt = (int)(pb % p.WT), ht = (int)((pb / p.WT) % p.HT), sb = (int)(pb / ((long long)p.WT * p.HT));
        const int x0 = wt * p.bw, y0 = ht * p.bh, s0 = sb * p.bs;
        uint8_t* st = smem + (size_t)stage * STAGE;
        tc::tma_load_5d(st, &map_d, full_bar + stage, m0, x0, y0, s0, 0);
        tc::tma_load_5d(st + 4 * A_PLANE, &map_x, full_bar + stage, c0, x0 + v - p.pad, y0 + u - p.pad, s0, 0);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one thread ----------------
    if (lane == 0) {
      // S32 accumulator, unsigned 8-bit A and B, both MN-major, M = 128
      auto idesc_n = [](int n) {
        return (2u << 4) | (0u << 7) | (0u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
               ((uint32_t)(TM >> 4) << 24);
      };
      bool fresh = true;
      int fold = 0;
      for (int k = 0; k < nst; ++k) {
        const int stage = k % NST;
        if (fresh && fold > 0) {
          if (!tc::mbar_wait(&tempty_bar, (uint32_t)((fold - 1) & 1), abort_flag, p.spin_cap)) break;
          tc::tc_fence_after();
        }
        if (!tc::mbar_wait(full_bar + stage, (uint32_t)((k / NST) & 1), abort_flag, p.spin_cap)) break;
        tc::tc_fence_after();
        const uint32_t sa = tc::smem_u32(smem + (size_t)stage * STAGE), sb = sa + 4 * A_PLANE;
#pragma unroll
        for (int ks = 0; ks < KP / 32; ++ks) {
          const uint64_t bdesc = desc_mn<TN>(sb + ks * 32 * TN, B_PLANE);
#pragma unroll
          for (int da = 0; da < 4; ++da) {
            const uint64_t adesc = desc_mn<TM>(sa + da * A_PLANE + ks * 32 * TM, A_PLANE);
            const uint32_t d = tmem_base + (uint32_t)(da * TN);
            if (fresh && ks == 0 && da > 0) {
              // classes da .. da+2 have a product already, class da+3 has none
              tcf::mma_i8(d, adesc, bdesc, idesc_n(3 * TN), 1u);
              tcf::mma_i8(d + 3 * TN, adesc, desc_mn<TN>(sb + 3 * B_PLANE + ks * 32 * TN, B_PLANE), idesc_n(TN), 0u);
            } else {
              tcf::mma_i8(d, adesc, bdesc, idesc_n(4 * TN), (fresh && ks == 0) ? 0u : 1u);
            }
          }
        }
        fresh = false;
        tc::tc_commit(empty_bar + stage);
        if (k + 1 == nst || ((k + 1) % kFoldStages) == 0) {
          tc::tc_commit(&tfull_bar);
          fresh = true;
          ++fold;
        }
      }
    }
  } else {
    // ---------------- epilogue: fold the class sums, add the residues to dW's accumulators ----------------
    const int q = warp & 3, h = (warp - 2) >> 2;
    const int co = m0 + q * 32 + lane;
    bool alive = true;
    for (int fold = 0; alive && fold < nfolds; ++fold) {
      if (!tc::mbar_wait(&tfull_bar, (uint32_t)(fold & 1), abort_flag, p.spin_cap)) { alive = false; break; }
      tc::tc_fence_after();
#pragma unroll 1
      for (int cg = 0; cg < 4; ++cg) {
        int cls[7][8];
#pragma unroll
        for (int c = 0; c < 7; ++c)
          tcf::ld8(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * TN + h * 32 + cg * 8), cls[c]);
        tc::tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int ci = c0 + h * 32 + cg * 8 + j;
          if (co >= p.cout || ci >= p.cin) continue;
          const int cc[7] = {cls[0][j], cls[1][j], cls[2][j], cls[3][j], cls[4][j], cls[5][j], cls[6][j]};
          atomicAdd(p.acc + (long long)co * p.ws_o + (long long)ci * p.ws_c + (long long)u * p.ws_u + (long long)v * p.ws_v,
                    (u64)fold_classes(0u, cc, p.md, p.pow32));
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&tempty_bar);
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (t == 0 && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  if (warp == 1) {
    tc::tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// How many products of two residues may be added to one residue in a uint64.
long long terms_per_reduction(u32 p) {
  const u64 pm = (u64)p - 1;
  return (long long)((~0ull - pm) / (pm * pm));
}

bool aligned16(const void* p);

// the test hook DK_OPT_TEST_WITHHOLD serves one launch
int take_withhold(dk_ctx* ctx) {
  const int w = ctx->opt.v[DK_OPT_TEST_WITHHOLD];
  ctx->opt.v[DK_OPT_TEST_WITHHOLD] = -1;
  return w;
}

// `path` (option DK_OPT_FIELD_PATH): 0 = tensor cores (tcgen05 where the shape allows, else mma.sync),
// 1 = the 64-bit integer-ALU kernels, 2 = mma.sync only (1 and 2 are cross-checks of the default).
// `wplanes` (nullable): device scratch of at least 4 * cout * round_up(kc, 128) bytes for the digit planes of W;
// without it the contraction runs on the mma.sync kernel.
__global__ void field_reduce_kernel(const u64* __restrict__ acc, long long n, Modulus md, u32* __restrict__ out);
int ew_blocks(long long n, int sm_count);

// Slices of the contraction for the tcgen05 kernel: `ctas` output tiles of `ntiles` k-tiles on `sms` SMs.
// Cost of ns slices = rounds of CTAs x (k-tiles per slice + a fixed part of about three k-tiles for set-up,
// the fold and the write-out); slices keep at least four k-tiles.
int field_fwd_slices(long long ctas, int ntiles, int sms) {
  int best = 1;
  double best_cost = 1e300;
  for (int ns = 1; ns <= 16 && ntiles / ns >= 4; ++ns) {
    const long long rounds = (ctas * ns + sms - 1) / sms;
    const double cost = (double)rounds * ((double)((ntiles + ns - 1) / ns) + 3.0) + (ns > 1 ? 1.0 : 0.0);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = ns; }
  }
  return best;
}

// The TMA-fed forward kernel: digit planes of W_q and x_bar written first, then one CTA per (pixel tile,
// 128 output channels, contraction slice).  DK_ERR_UNSUPPORTED: the driver refused a tensor map.
dk_status launch_field_fwd_tma(const dk_ctx* ctx, const Geom& g, const FwdParams& fp, const MmaConsts& mc,
                               const u32* W, const u32* xbar, int nsamples, uint8_t* wplanes, int kcp,
                               uint8_t* xplanes, u64* split_acc, size_t split_bytes, int sm_count, int* status,
                               unsigned spin_cap, int withhold, cudaStream_t st) {
  const int KT = (g.cin % 128) == 0 ? 128 : 64;
  ftm::Params q;
  // the box of 64 output pixels that covers the fewest positions outside the output
  long long best = -1;
  q.bw = q.bh = q.bs = 1;
  for (int bw = 1; bw <= 64; bw *= 2)
    for (int bh = 1; bw * bh <= 64; bh *= 2) {
      const int bs = 64 / (bw * bh);
      const long long cost = (long long)((g.wo + bw - 1) / bw) * bw * ((g.ho + bh - 1) / bh) * bh *
                             ((nsamples + bs - 1) / bs) * bs;
      if (best < 0 || cost < best || (cost == best && bw > q.bw)) { best = cost; q.bw = bw; q.bh = bh; q.bs = bs; }
    }
  q.WT = (g.wo + q.bw - 1) / q.bw;
  q.HT = (g.ho + q.bh - 1) / q.bh;
  const long long tiles = (long long)q.WT * q.HT * ((nsamples + q.bs - 1) / q.bs);
  const int mtiles = (g.cout + ftm::TM - 1) / ftm::TM;
  if (tiles > 2147483647LL || mtiles > 65535) return DK_ERR_SHAPE;
  q.cblocks = g.cin / KT;
  q.kw = g.kw; q.pad = g.pad;
  q.ktiles = g.kh * g.kw * q.cblocks;
  q.cout = g.cout; q.ho = g.ho; q.wo = g.wo; q.nsamples = nsamples;
  q.n_out = g.n_out; q.ys_c = g.ys_c; q.ys_h = g.ys_h; q.ys_w = g.ys_w;
  q.y = fp.y; q.md = fp.md; q.pow32 = mc.pow32;
  q.status = status; q.spin_cap = spin_cap; q.withhold = withhold;
  const long long n_y = (long long)nsamples * g.n_out;
  int ns = field_fwd_slices(tiles * mtiles, q.ktiles, sm_count);
  if (split_acc == nullptr || split_bytes < (size_t)n_y * sizeof(u64)) ns = 1;
  q.tiles_per_split = (q.ktiles + ns - 1) / ns;
  ns = (q.ktiles + q.tiles_per_split - 1) / q.tiles_per_split;
  q.split_acc = ns > 1 ? split_acc : nullptr;

  CUtensorMap map_w, map_x;
  {
    const unsigned long long dims[3] = {(unsigned long long)kcp, (unsigned long long)g.cout, 4ull};
    const unsigned long long str[2] = {(unsigned long long)kcp, (unsigned long long)kcp * g.cout};
    const unsigned int box[3] = {(unsigned)KT, (unsigned)ftm::TM, 4u};
    if (!tc_encode_map_bytes(ctx, &map_w, wplanes, 3, dims, str, box, KT)) return DK_ERR_UNSUPPORTED;
  }
  {
    const unsigned long long n_x = (unsigned long long)nsamples * g.n_in;
    const unsigned long long dims[5] = {(unsigned long long)g.cin, (unsigned long long)g.w, (unsigned long long)g.h,
                                        (unsigned long long)nsamples, 4ull};
    const unsigned long long str[4] = {(unsigned long long)g.cin, (unsigned long long)g.cin * g.w,
                                       (unsigned long long)g.n_in, n_x};
    const unsigned int box[5] = {(unsigned)KT, (unsigned)q.bw, (unsigned)q.bh, (unsigned)q.bs, 4u};
    if (!tc_encode_map_bytes(ctx, &map_x, xplanes, 5, dims, str, box, KT)) return DK_ERR_UNSUPPORTED;
  }
  const long long chunks = (long long)g.cout * (kcp / 16);
  field_w_planes_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(W, g.cout, g.kc, kcp, wplanes);
  DK_CUDA_CHECK(cudaGetLastError());
  const long long nx = (long long)nsamples * g.n_in;
  field_x_planes_kernel<<<ew_blocks(nx / 16, sm_count), 256, 0, st>>>(xbar, nx, xplanes, g.n_in, 1, 1);
  DK_CUDA_CHECK(cudaGetLastError());
  if (ns > 1) DK_CUDA_CHECK(cudaMemsetAsync(split_acc, 0, (size_t)n_y * sizeof(u64), st));
  const dim3 grid((unsigned)tiles, (unsigned)mtiles, (unsigned)ns);
  constexpr size_t kSmem = (size_t)2 * 4 * (ftm::TM + ftm::TN) * 128 + 1024;      // two stages of 128-byte rows = four of 64
  static const bool attr_ok =
      cudaFuncSetAttribute(field_fwd_tma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) == cudaSuccess &&
      cudaFuncSetAttribute(field_fwd_tma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) == cudaSuccess;
  if (!attr_ok) return DK_ERR_CUDA;
  if (KT == 128) field_fwd_tma_kernel<128><<<grid, ftm::kThreads, kSmem, st>>>(map_w, map_x, q);
  else field_fwd_tma_kernel<64><<<grid, ftm::kThreads, kSmem, st>>>(map_w, map_x, q);
  DK_CUDA_CHECK(cudaGetLastError());
  if (ns > 1) {
    field_reduce_kernel<<<ew_blocks(n_y, sm_count), 256, 0, st>>>(split_acc, n_y, fp.md, fp.y);
    DK_CUDA_CHECK(cudaGetLastError());
  }
  return DK_OK;
}

// `wplanes` (nullable): device scratch of at least 4 * cout * round_up(kc, 128) bytes for the digit planes of W;
// without it the contraction runs on the mma.sync kernel.  `split_acc` (nullable, split_bytes): uint64 scratch
// in which slices of the contraction meet when a layer has too few output tiles to fill the device.
dk_status launch_field_fwd(const Geom& g, const u32* W, const u32* xbar, u32* ybar, int nsamples, Modulus md,
                           uint8_t* wplanes, size_t wplanes_bytes, u64* split_acc, size_t split_bytes, int sm_count,
                           int* status, int path, unsigned spin_cap, int withhold, cudaStream_t st,
                           const dk_ctx* ctx = nullptr, uint8_t* xplanes = nullptr, size_t xplanes_bytes = 0) {
  FwdParams p;
  p.W = W; p.x = xbar; p.y = ybar;
  p.cin = g.cin; p.cout = g.cout; p.h = g.h; p.w = g.w; p.kw = g.kw; p.stride = g.stride;
  p.pad = g.pad; p.ho = g.ho; p.wo = g.wo; p.kc = g.kc;
  p.N = (long long)nsamples * g.ho * g.wo;
  p.n_in = g.n_in; p.n_out = g.n_out;
  p.xs_c = g.xs_c; p.xs_h = g.xs_h; p.xs_w = g.xs_w;
  p.ws_o = g.ws_o; p.ws_c = g.ws_c; p.ws_u = g.ws_u; p.ws_v = g.ws_v;
  p.ys_c = g.ys_c; p.ys_h = g.ys_h; p.ys_w = g.ys_w;
  long long ft = terms_per_reduction(md.p) / BK;
  if (ft < 1) return DK_ERR_UNSUPPORTED;
  if (ft > 256) ft = 256;
  p.fold_tiles = (int)ft;
  p.md = md;
  const long long nb = (p.N + BN - 1) / BN;
  if (nb > 2147483647LL) return DK_ERR_SHAPE;
  dim3 grid((unsigned)nb, (unsigned)((g.cout + BM - 1) / BM));
  if (grid.y > 65535) return DK_ERR_SHAPE;
  static_assert(BM == MMA_BM && BN == MMA_BN, "one grid shape serves both kernels");
  if (path == 1) {
    field_fwd_kernel<<<grid, NT, 0, st>>>(p);
  } else {
    MmaConsts mc;
    mc.pow32 = (u32)((1ull << 32) % md.p);
    const bool vec4 = g.xs_c == 1 && g.ws_c == 1 && (g.cin % 4) == 0 && aligned16(W) && aligned16(xbar);
    const int kcp = (g.kc + tcf::TK - 1) / tcf::TK * tcf::TK;
    if (vec4 && path != 2 && wplanes != nullptr && wplanes_bytes >= (size_t)4 * g.cout * kcp) {
      // operands by TMA (path 0 only; option value 3 keeps the kernel that splits x_bar in registers)
      const long long n_x = (long long)nsamples * g.n_in;
      if (path == 0 && ctx != nullptr && xplanes != nullptr && xplanes_bytes >= (size_t)4 * n_x &&
          g.layout == DK_NHWC && g.stride == 1 && (g.cin % 64) == 0 && (n_x % 16) == 0) {
        dk_status ts = launch_field_fwd_tma(ctx, g, p, mc, W, xbar, nsamples, wplanes, kcp, xplanes, split_acc,
                                            split_bytes, sm_count, status, spin_cap, withhold, st);
        if (ts != DK_ERR_UNSUPPORTED) return ts;
      }
      static const bool tc_attr_ok =
          cudaFuncSetAttribute(field_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)tcf::kSmem) == cudaSuccess;
      if (!tc_attr_ok) return DK_ERR_CUDA;
      const long long tnb = (p.N + tcf::TN - 1) / tcf::TN;
      dim3 tgrid((unsigned)tnb, (unsigned)((g.cout + tcf::TM - 1) / tcf::TM));
      const long long chunks = (long long)g.cout * (kcp / 16);
      field_w_planes_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(W, g.cout, g.kc, kcp, wplanes);
      DK_CUDA_CHECK(cudaGetLastError());
      const int ntiles = kcp / tcf::TK;
      const long long n_y = (long long)nsamples * g.n_out;
      int ns = field_fwd_slices((long long)tgrid.x * tgrid.y, ntiles, sm_count);
      if (split_acc == nullptr || split_bytes < (size_t)n_y * sizeof(u64)) ns = 1;
      if (ns > 1) {
        tgrid.z = (unsigned)ns;
        const int tps = (ntiles + ns - 1) / ns;
        tgrid.z = (unsigned)((ntiles + tps - 1) / tps);
        DK_CUDA_CHECK(cudaMemsetAsync(split_acc, 0, (size_t)n_y * sizeof(u64), st));
        field_fwd_tc_kernel<<<tgrid, tcf::kThreads, tcf::kSmem, st>>>(p, mc, wplanes, kcp, split_acc, tps, status, spin_cap, withhold);
        DK_CUDA_CHECK(cudaGetLastError());
        field_reduce_kernel<<<ew_blocks(n_y, sm_count), 256, 0, st>>>(split_acc, n_y, md, ybar);
      } else {
        field_fwd_tc_kernel<<<tgrid, tcf::kThreads, tcf::kSmem, st>>>(p, mc, wplanes, kcp, nullptr, ntiles, status, spin_cap, withhold);
      }
      DK_CUDA_CHECK(cudaGetLastError());
      return DK_OK;
    }
    static const bool attr_ok = [] {
      return cudaFuncSetAttribute(field_fwd_mma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)kMmaSmemBytes) == cudaSuccess &&
             cudaFuncSetAttribute(field_fwd_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)kMmaSmemBytes) == cudaSuccess;
    }();
    if (!attr_ok) return DK_ERR_CUDA;
    if (vec4) field_fwd_mma_kernel<4><<<grid, kMmaThreads, kMmaSmemBytes, st>>>(p, mc);
    else field_fwd_mma_kernel<1><<<grid, kMmaThreads, kMmaSmemBytes, st>>>(p, mc);
  }
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

// ---------------------------------------------------------------------------
// the weight-gradient contraction modulo p
// ---------------------------------------------------------------------------
struct WgParams {
  const u32* d;     // mixed deltas [G*(K+1)][n_out]
  const u32* x;     // encodings, xbar_rows per group
  u64* acc;         // [cout*kc] partial sums of residues, cleared by the caller
  int cin, cout, h, w, kw, stride, pad, ho, wo, kc;
  int K1, xbar_rows, P, PC;   // P = ho*wo pixels, PC = ceil(P/BK)
  long long GP;               // G * PC contraction blocks
  long long per_split;
  int fold_blocks;            // contraction blocks between two reductions (0: after every k-tile)
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
  Modulus md;
};

__global__ void __launch_bounds__(NT) field_wgrad_kernel(WgParams p) {
  __shared__ __align__(16) u32 As[BK][BM + 4];
  __shared__ __align__(16) u32 Bs[BK][BN + 4];
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
  const int tap = b_ok ? kcol / p.cin : 0;
  const int ci = b_ok ? kcol - tap * p.cin : 0;
  const int u = tap / p.kw, v = tap - u * p.kw;
  const long long b_off = (long long)ci * p.xs_c;

  u64 acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0;

  int fold = 0;
  for (long long gp = gp_lo; gp < gp_hi; ++gp) {
    const long long g = gp / p.PC;
    const int pc = (int)(gp - g * p.PC);
    int oh[4], ow[4];
    bool pok[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int pix = pc * BK + t / 64 + 4 * i;
      pok[i] = pix < p.P;
      const int pp = pok[i] ? pix : 0;
      oh[i] = pp / p.wo;
      ow[i] = pp - oh[i] * p.wo;
    }
    for (int j = 0; j < p.K1; ++j) {
      const u32* dj = p.d + (g * p.K1 + j) * p.n_out;
      const u32* xj = p.x + (g * p.xbar_rows + j) * p.n_in;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int pp = t / 64 + 4 * i;
        As[pp][cc] = (pok[i] && a_ok)
                         ? __ldg(dj + a_off + (long long)oh[i] * p.ys_h + (long long)ow[i] * p.ys_w)
                         : 0u;
        const int ih = oh[i] * p.stride + u - p.pad, iw = ow[i] * p.stride + v - p.pad;
        const bool ok = pok[i] && b_ok && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
        Bs[pp][cc] = ok ? __ldg(xj + b_off + (long long)ih * p.xs_h + (long long)iw * p.xs_w) : 0u;
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < BK; ++q) {
        const uint4 a4 = *reinterpret_cast<const uint4*>(&As[q][ty * 4]);
        const uint4 b4 = *reinterpret_cast<const uint4*>(&Bs[q][tx * 4]);
        const u32 a[4] = {a4.x, a4.y, a4.z, a4.w};
        const u32 b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[i][jj] += (u64)a[i] * b[jj];
      }
      __syncthreads();
      if (p.fold_blocks == 0) {      // large p: only one k-tile of products fits between reductions
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[i][jj] = reduce64(acc[i][jj], p.md);
      }
    }
    if (++fold == p.fold_blocks) {
      fold = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) acc[i][jj] = reduce64(acc[i][jj], p.md);
    }
  }
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int kcol2 = kb0 + tx * 4 + jj;
    if (kcol2 >= p.kc) continue;
    const int tap2 = kcol2 / p.cin, ci2 = kcol2 - tap2 * p.cin;
    const int u2 = tap2 / p.kw, v2 = tap2 - u2 * p.kw;
    const long long woff = (long long)ci2 * p.ws_c + (long long)u2 * p.ws_u + (long long)v2 * p.ws_v;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m < p.cout) atomicAdd(p.acc + (long long)m * p.ws_o + woff, (u64)reduce64(acc[i][jj], p.md));
    }
  }
}

// The weight-gradient contraction on the integer tensor cores.  The contraction
// index r runs over (group, encoding, output pixel) flattened; both operands are
// stored with the channel contiguous, so a tile is kept in shared memory as it
// arrives, [r][column], and a thread gathers the four consecutive r of one
// column with four 32-bit reads (row pitch == 2 mod 32 words: conflict-free)
// before the same byte transpose into digit planes as in the forward kernel.
constexpr int WG_LD = MMA_BM + 2;
constexpr int kWgStageWords = 2 * MMA_BK * WG_LD;
constexpr size_t kWgSmemBytes = (size_t)kMmaStages * kWgStageWords * sizeof(u32);

// n / d for 0 <= n < 2^32 by multiplication (Granlund-Montgomery round-up
// method): s = ceil(log2 d), m = floor(2^32 (2^s - d) / d) + 1, q = (mulhi(n, m) + n) >> s.
struct FastDiv {
  u32 m;
  int s;
};
FastDiv make_fastdiv(u32 d) {
  FastDiv f;
  f.s = 0;
  while ((1ull << f.s) < d) ++f.s;
  f.m = (u32)((((1ull << f.s) - d) << 32) / d + 1);
  return f;
}
__device__ __forceinline__ u32 fastdiv(u32 n, FastDiv f) { return (u32)(((u64)__umulhi(n, f.m) + n) >> f.s); }

struct WgMmaParams {
  FastDiv div_P, div_K1, div_wo;
  const u32* d;     // mixed deltas [G*(K+1)][n_out]
  const u32* x;     // encodings, xbar_rows per group
  u64* acc;         // [cout*kc] sums of the slices' residues, cleared by the caller
  int cin, cout, h, w, kw, stride, pad, ho, wo, kc;
  int K1, xbar_rows, P;
  long long R;                // G * (K+1) * P contraction elements
  int tiles_per_split, ntiles;
  long long n_in, n_out;
  long long xs_c, xs_h, xs_w, ws_o, ws_c, ws_u, ws_v, ys_c, ys_h, ys_w;
  Modulus md;
  u32 pow32;
};

__device__ __forceinline__ uint4 gather4(const u32* col) {
  return make_uint4(col[0], col[WG_LD], col[2 * WG_LD], col[3 * WG_LD]);
}

template <int VEC>
__global__ void __launch_bounds__(kMmaThreads, 1) field_wgrad_mma_kernel(WgMmaParams p) {
  extern __shared__ __align__(16) u32 tiles[];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int g = lane >> 2, tig = lane & 3;
  const int wm = warp & 3, wn = warp >> 2;
  const int m0 = blockIdx.y * MMA_BM;
  const int kb0 = blockIdx.x * MMA_BN;
  const int t_lo = blockIdx.z * p.tiles_per_split;
  const int t_hi = min(t_lo + p.tiles_per_split, p.ntiles);

  // loader: VEC columns starting at `col` of the r-rows rr0 + RSTEP*i of both tiles
  constexpr int CPR = MMA_BM / VEC, RSTEP = kMmaThreads / CPR, NCOPY = MMA_BK / RSTEP;
  const int col = (t % CPR) * VEC, rr0 = t / CPR;
  const bool a_ok = (m0 + col) < p.cout;
  const long long a_off = (long long)(m0 + col) * p.ys_c;
  const int kcol = kb0 + col;
  const bool b_ok = kcol < p.kc;
  const int tap = b_ok ? kcol / p.cin : 0;
  const int ci = b_ok ? kcol - tap * p.cin : 0;
  const int u = tap / p.kw, v = tap - u * p.kw;
  const long long b_off = (long long)ci * p.xs_c;
  auto load_tile = [&](int rt, u32* stage) {
    u32* as = stage;
    u32* bs = stage + MMA_BK * WG_LD;
#pragma unroll
    for (int i = 0; i < NCOPY; ++i) {
      const int rr = rr0 + RSTEP * i;
      const u32 r = (u32)rt * MMA_BK + rr;
      const bool rok = r < (u32)p.R;
      const u32 gj = rok ? fastdiv(r, p.div_P) : 0;
      const int pix = rok ? (int)(r - gj * p.P) : 0;
      const long long gg = fastdiv(gj, p.div_K1);
      const int j = (int)(gj - (u32)gg * p.K1);
      const int oh = (int)fastdiv((u32)pix, p.div_wo), ow = pix - oh * p.wo;
      const bool aok = rok && a_ok;
      copy_async<4 * VEC>(as + rr * WG_LD + col,
                          aok ? p.d + (gg * p.K1 + j) * p.n_out + a_off + (long long)oh * p.ys_h + (long long)ow * p.ys_w
                              : p.d, aok);
      const int ih = oh * p.stride + u - p.pad, iw = ow * p.stride + v - p.pad;
      const bool bok = rok && b_ok && ih >= 0 && ih < p.h && iw >= 0 && iw < p.w;
      copy_async<4 * VEC>(bs + rr * WG_LD + col,
                          bok ? p.x + (gg * p.xbar_rows + j) * p.n_in + b_off + (long long)ih * p.xs_h +
                                    (long long)iw * p.xs_w
                              : p.x, bok);
    }
    copy_async_commit();
  };

  int acc[7][kMmaNT][4];
  u32 tot[kMmaNT][4];
#pragma unroll
  for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      tot[j][r] = 0;
#pragma unroll
      for (int c = 0; c < 7; ++c) acc[c][j][r] = 0;
    }

  const int ntiles = t_hi - t_lo;
#pragma unroll
  for (int s = 0; s < kMmaStages - 1; ++s) {
    if (s < ntiles) load_tile(t_lo + s, tiles + s * kWgStageWords);
    else copy_async_commit();
  }
  int fold = 0;
  for (int kt = 0; kt < ntiles; ++kt) {
    const u32* as = tiles + (kt % kMmaStages) * kWgStageWords;
    const u32* bs = as + MMA_BK * WG_LD;
    copy_async_wait<kMmaStages - 2>();
    __syncthreads();
    {
      const int nt = kt + kMmaStages - 1;
      if (nt < ntiles) load_tile(t_lo + nt, tiles + (nt % kMmaStages) * kWgStageWords);
      else copy_async_commit();
    }
    {
      u32 a[4][4];
      const u32* ac = as + (4 * tig) * WG_LD + wm * 16 + g;
      digit_planes(gather4(ac), a[0]);
      digit_planes(gather4(ac + 8), a[1]);
      digit_planes(gather4(ac + 16 * WG_LD), a[2]);
      digit_planes(gather4(ac + 16 * WG_LD + 8), a[3]);
#pragma unroll
      for (int j = 0; j < kMmaNT; ++j) {
        u32 b[2][4];
        const u32* bc = bs + (4 * tig) * WG_LD + wn * (8 * kMmaNT) + j * 8 + g;
        digit_planes(gather4(bc), b[0]);
        digit_planes(gather4(bc + 16 * WG_LD), b[1]);
        // digit pairs in an order that keeps two products of one weight class four instructions apart
#pragma unroll
        for (int da = 0; da < 4; ++da)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int db = (i + 4 - da) & 3;
            mma_u8(acc[da + db][j], a[0][da], a[1][da], a[2][da], a[3][da], b[0][db], b[1][db]);
          }
      }
    }
    if (++fold == kMmaFoldTiles) {
      fold = 0;
#pragma unroll
      for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int c[7] = {acc[0][j][r], acc[1][j][r], acc[2][j][r], acc[3][j][r],
                            acc[4][j][r], acc[5][j][r], acc[6][j][r]};
          tot[j][r] = fold_classes(tot[j][r], c, p.md, p.pow32);
#pragma unroll
          for (int cc = 0; cc < 7; ++cc) acc[cc][j][r] = 0;
        }
    }
  }
#pragma unroll
  for (int j = 0; j < kMmaNT; ++j)
#pragma unroll
    for (int cb = 0; cb < 2; ++cb) {
      const int kcol2 = kb0 + wn * (8 * kMmaNT) + j * 8 + 2 * tig + cb;
      if (kcol2 >= p.kc) continue;
      const int tap2 = kcol2 / p.cin, ci2 = kcol2 - tap2 * p.cin;
      const int u2 = tap2 / p.kw, v2 = tap2 - u2 * p.kw;
      const long long woff = (long long)ci2 * p.ws_c + (long long)u2 * p.ws_u + (long long)v2 * p.ws_v;
#pragma unroll
      for (int rb = 0; rb < 2; ++rb) {
        const int r = rb * 2 + cb;
        const int m = m0 + wm * 16 + g + 8 * rb;
        if (m >= p.cout) continue;
        const int c[7] = {acc[0][j][r], acc[1][j][r], acc[2][j][r], acc[3][j][r],
                          acc[4][j][r], acc[5][j][r], acc[6][j][r]};
        atomicAdd(p.acc + (long long)m * p.ws_o + woff, (u64)fold_classes(tot[j][r], c, p.md, p.pow32));
      }
    }
}

// the slices' residues (at most 65535 of them, each below p) summed in uint64 -> residue
__global__ void __launch_bounds__(256) field_reduce_kernel(const u64* __restrict__ acc, long long n, Modulus md,
                                                          u32* __restrict__ out) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    out[i] = reduce64(acc[i], md);
}

int ew_blocks(long long n, int sm_count) {
  long long b = (n + 255) / 256;
  if (b > 16LL * sm_count) b = 16LL * sm_count;
  return (int)(b < 1 ? 1 : b);
}

// The context's device status word (read and cleared by dk_device_status).
int* field_status_word(dk_ctx* ctx) { return reinterpret_cast<int*>(ctx->d_vstats + kVerifyStatFloats) + 2; }

struct FieldWs {
  size_t wq, wpl, wpl_bytes, xq, xbar, ybar, bq, dtil, acc64, xpl, xpl_bytes, total;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

FieldWs plan_field_ws(const Geom& g) {
  FieldWs w;
  size_t off = 0;
  w.wq = off; off += align_up((size_t)g.cout * g.kc * sizeof(u32), 1024);
  w.wpl_bytes = (size_t)4 * g.cout * ((g.kc + 127) / 128 * 128);      // digit planes of W_q
  w.wpl = off; off += align_up(w.wpl_bytes, 1024);
  w.xq = off; off += align_up((size_t)g.G * g.K * g.n_in * sizeof(u32), 1024);
  w.xbar = off; off += align_up((size_t)g.G * g.E * g.n_in * sizeof(u32), 1024);
  w.ybar = off; off += align_up((size_t)g.G * g.E * g.n_out * sizeof(u32), 1024);
  w.bq = off; off += align_up((size_t)g.cout * sizeof(u32), 1024);
  w.dtil = off; off += align_up((size_t)g.G * (g.K + 1) * g.n_out * sizeof(u32), 1024);
  // digit planes of the encodings (forward) or of the mixed gradients and the encodings (weight gradient)
  w.xpl_bytes = (size_t)4 * g.G * (g.E * g.n_in + (g.K + 1) * g.n_out);
  w.xpl = off; off += align_up(w.xpl_bytes, 1024);
  // last: uint64 accumulators of the weight gradient; the forward kernels' contraction slices meet in whatever
  // follows this offset
  w.acc64 = off; off += align_up((size_t)g.cout * g.kc * sizeof(u64), 1024);
  w.total = off;
  return w;
}

struct Guard {
  int prev;
  bool ok;
  explicit Guard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) return;
    ok = true;
  }
  ~Guard() {
    int cur = -1;
    if (ok && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

dk_status make_modulus(uint32_t p, Modulus* md) {
  if (p >= (1u << 30) || !prime_by_trial_division(p)) return DK_ERR_INVALID_ARG;
  md->p = p;
  md->m = ~0ull / p;      // = floor(2^64 / p): p is odd, so it does not divide 2^64
  md->s = -1;
  md->m32 = 0;
  if (p < (1u << 27)) {
    int s = 0;
    while ((2u << s) <= p) ++s;      // 2^s <= p < 2^(s+1)
    md->s = s;
    md->m32 = (u32)((1ull << (32 + s)) / p);      // in (2^31, 2^32): p is not a power of two
  }
  return DK_OK;
}

dk_status quantize_launch(const float* v, long long n, int scale_bits, u32 p, u32* out, int sm_count,
                          cudaStream_t st) {
  if (n == 0) return DK_OK;
  field_quantize_kernel<<<ew_blocks(n, sm_count), 256, 0, st>>>(v, n, ldexpf(1.0f, scale_bits), p, out);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status decode_verify_launch(dk_ctx* ctx, const Geom& g, int l, const u32* ybar, const FieldCoef& fc,
                               const u32* bias_q, int* yq, float* y, dk_verdict* verdict, Modulus md,
                               cudaStream_t st) {
  {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    field_verdict_begin_kernel<<<1, 1, 0, st>>>(verdict);
    DK_CUDA_CHECK(cudaGetLastError());
  }
  DecodeParams dp;
  dp.ybar = ybar; dp.dec = fc.dec; dp.nul = fc.nul; dp.bias = bias_q; dp.yq = yq; dp.y = y; dp.v = verdict;
  dp.n = g.n_out;
  dp.ch_div = (g.layout == DK_NCHW) ? (long long)g.ho * g.wo : 1;
  dp.cout = g.cout;
  dp.inv_scale = ldexp(1.0, -l);
  dp.lbits = l;
  {      // Section 4.5 relabelling, as in the floating-point calls: at least one row stays
    int n = ctx->opt.v[DK_OPT_NOISE_ROWS];
    if (n > g.K - 1) n = g.K - 1;
    dp.kstore = g.K - (n > 0 ? n : 0);
  }
  dp.md = md;
  const bool vec4 = (g.n_out % 4) == 0 && aligned16(ybar) && aligned16(yq) && aligned16(y);
  ProfScope ps(ctx, DK_KERNEL_DECODE_VERIFY, 1, st);
  return vec4 ? launch_decode_t<4>(g.K, dp, g.G, ctx->sm_count, st)
              : launch_decode_t<1>(g.K, dp, g.G, ctx->sm_count, st);
}

}  // namespace
}  // namespace dk

using namespace dk;

extern "C" {

dk_status dk_field_workspace_bytes(const dk_problem* p, size_t* bytes) {
  if (!bytes) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  *bytes = plan_field_ws(g).total;
  return DK_OK;
}

dk_status dk_field_quantize(dk_ctx* ctx, const float* v, int64_t n, int32_t scale_bits, uint32_t prime,
                            uint32_t* vq, void* stream) {
  if (!ctx || n < 0 || (n > 0 && (!v || !vq)) || scale_bits < 0 || scale_bits > 60) return DK_ERR_INVALID_ARG;
  Modulus md;
  dk_status s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
  return quantize_launch(v, n, scale_bits, prime, vq, ctx->sm_count, st);
}

dk_status dk_field_dequantize(dk_ctx* ctx, const uint32_t* vq, int64_t n, int32_t scale_bits, uint32_t prime,
                              float* v, void* stream) {
  if (!ctx || n < 0 || (n > 0 && (!v || !vq)) || scale_bits < 0 || scale_bits > 60) return DK_ERR_INVALID_ARG;
  Modulus md;
  dk_status s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  if (n == 0) return DK_OK;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
  field_dequantize_kernel<<<ew_blocks(n, ctx->sm_count), 256, 0, st>>>(vq, n, prime, ldexp(1.0, -scale_bits), v);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status dk_field_encode(dk_ctx* ctx, const dk_problem* p, uint32_t prime, const uint32_t* xq,
                          const uint32_t* rq, const uint32_t* C_host, uint32_t* xbar, void* stream) {
  if (!ctx || !xq || !rq || !C_host || !xbar) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  Modulus md;
  s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FieldCoef fc;
  s = upload_field_coefficients(ctx, g, prime, C_host, nullptr, false, false, st, &fc);
  if (s != DK_OK) return s;
  ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
  return mix_rows(g.K + 1, xq, rq, fc.enc, xbar, g.n_in, g.E, g.G, md, ctx->sm_count, st);
}

dk_status dk_field_linear_fwd(dk_ctx* ctx, const dk_problem* p, uint32_t prime, const uint32_t* Wq,
                              const uint32_t* xbar, uint32_t* ybar, void* stream) {
  if (!ctx || !Wq || !xbar || !ybar) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  Modulus md;
  s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
  const FieldWs wp = plan_field_ws(g);
  const bool have_ws = ctx->ws && ctx->ws_bytes >= wp.total;
  return launch_field_fwd(g, Wq, xbar, ybar, g.G * g.E, md,
                          have_ws ? reinterpret_cast<uint8_t*>(static_cast<char*>(ctx->ws) + wp.wpl) : nullptr,
                          have_ws ? wp.wpl_bytes : 0,
                          have_ws ? reinterpret_cast<u64*>(static_cast<char*>(ctx->ws) + wp.acc64) : nullptr,
                          have_ws ? wp.total - wp.acc64 : 0, ctx->sm_count, field_status_word(ctx), ctx->opt.v[DK_OPT_FIELD_PATH], (unsigned)ctx->opt.v[DK_OPT_SPIN_LIMIT],
                          take_withhold(ctx), st, ctx,
                          have_ws ? reinterpret_cast<uint8_t*>(static_cast<char*>(ctx->ws) + wp.xpl) : nullptr,
                          have_ws ? wp.xpl_bytes : 0);
}

dk_status dk_field_decode_verify(dk_ctx* ctx, const dk_problem* p, uint32_t prime, int32_t l,
                                 const uint32_t* ybar, const uint32_t* C_host, const uint32_t* bias_q,
                                 int32_t* yq, float* y, dk_verdict* verdict, void* stream) {
  if (!ctx || !ybar || !C_host || !verdict || (!yq && !y) || l < 0 || l > 30) return DK_ERR_INVALID_ARG;
  if (!aligned16(verdict)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  Modulus md;
  s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FieldCoef fc;
  s = upload_field_coefficients(ctx, g, prime, C_host, nullptr, true, false, st, &fc);
  if (s != DK_OK) return s;
  return decode_verify_launch(ctx, g, l, ybar, fc, bias_q, yq, y, verdict, md, st);
}

dk_status dk_field_masked_linear(dk_ctx* ctx, const dk_problem* p, uint32_t prime, int32_t l, const float* W,
                                 const float* x, const uint32_t* rq, const uint32_t* C_host, const float* bias,
                                 float* y, int32_t* yq, uint32_t* xbar_save, dk_verdict* verdict,
                                 const dk_field_fault* fault, void* stream) {
  if (!ctx || !W || !x || !rq || !C_host || !verdict || (!yq && !y) || l < 0 || l > 30) return DK_ERR_INVALID_ARG;
  if (!aligned16(verdict)) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  Modulus md;
  s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  if (fault) {
    if (fault->group < 0 || fault->group >= g.G || fault->enc < 0 || fault->enc >= g.E ||
        fault->out_index < 0 || fault->out_index >= g.n_out)
      return DK_ERR_INVALID_ARG;
  }
  const FieldWs wp = plan_field_ws(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FieldCoef fc;
  s = upload_field_coefficients(ctx, g, prime, C_host, nullptr, true, false, st, &fc);
  if (s != DK_OK) return s;
  char* ws = static_cast<char*>(ctx->ws);
  u32* Wq = reinterpret_cast<u32*>(ws + wp.wq);
  u32* xq = reinterpret_cast<u32*>(ws + wp.xq);
  u32* xbar = xbar_save ? xbar_save : reinterpret_cast<u32*>(ws + wp.xbar);
  u32* ybar = reinterpret_cast<u32*>(ws + wp.ybar);
  u32* bq = bias ? reinterpret_cast<u32*>(ws + wp.bq) : nullptr;
  {
    // Algorithm 1: W_q = Field(Round(W*2^l)), X_q likewise, b_q with 2l bits
    ProfScope ps(ctx, DK_KERNEL_OTHER, bias ? 3 : 2, st);
    s = quantize_launch(W, (long long)g.cout * g.kc, l, prime, Wq, ctx->sm_count, st);
    if (s == DK_OK) s = quantize_launch(x, (long long)g.G * g.K * g.n_in, l, prime, xq, ctx->sm_count, st);
    if (s == DK_OK && bias) s = quantize_launch(bias, g.cout, 2 * l, prime, bq, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  {
    ProfScope ps(ctx, DK_KERNEL_ENCODE, 1, st);
    s = mix_rows(g.K + 1, xq, rq, fc.enc, xbar, g.n_in, g.E, g.G, md, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  {
    ProfScope ps(ctx, DK_KERNEL_LINEAR_FWD, 1, st);
    s = launch_field_fwd(g, Wq, xbar, ybar, g.G * g.E, md, reinterpret_cast<uint8_t*>(ws + wp.wpl), wp.wpl_bytes,
                         reinterpret_cast<u64*>(ws + wp.acc64), wp.total - wp.acc64, ctx->sm_count,
                         field_status_word(ctx), ctx->opt.v[DK_OPT_FIELD_PATH], (unsigned)ctx->opt.v[DK_OPT_SPIN_LIMIT],
                          take_withhold(ctx), st, ctx, reinterpret_cast<uint8_t*>(ws + wp.xpl), wp.xpl_bytes);
  }
  if (s != DK_OK) return s;
  if (fault) {
    ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
    field_add_fault_kernel<<<1, 1, 0, st>>>(ybar, ((long long)fault->group * g.E + fault->enc) * g.n_out +
                                                      fault->out_index, fault->delta % prime, prime);
    DK_CUDA_CHECK(cudaGetLastError());
  }
  return decode_verify_launch(ctx, g, l, ybar, fc, bq, yq, y, verdict, md, st);
}

dk_status dk_field_linear_bwd_wgrad(dk_ctx* ctx, const dk_problem* p, uint32_t prime, const uint32_t* deltaq,
                                    const uint32_t* xbar, int32_t xbar_rows, const uint32_t* C_host,
                                    const uint32_t* gamma_host, uint32_t* dWq, void* stream) {
  if (!ctx || !deltaq || !xbar || !C_host || !gamma_host || !dWq) return DK_ERR_INVALID_ARG;
  Geom g;
  dk_status s = make_geom(p, &g);
  if (s != DK_OK) return s;
  if (xbar_rows != g.K + 1 && xbar_rows != g.K + 2) return DK_ERR_INVALID_ARG;
  Modulus md;
  s = make_modulus(prime, &md);
  if (s != DK_OK) return s;
  const FieldWs wp = plan_field_ws(g);
  if (!ctx->ws || ctx->ws_bytes < wp.total) return DK_ERR_WORKSPACE;
  Guard dg(ctx->device);
  if (!dg.ok) return DK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FieldCoef fc;
  s = upload_field_coefficients(ctx, g, prime, C_host, gamma_host, true, true, st, &fc);
  if (s != DK_OK) return s;
  char* ws = static_cast<char*>(ctx->ws);
  u32* dtil = reinterpret_cast<u32*>(ws + wp.dtil);
  u64* acc = reinterpret_cast<u64*>(ws + wp.acc64);
  {
    // Eq. 4: delta_bar^(j) = sum_i B[j][i] delta^(i), with gamma_j folded in
    ProfScope ps(ctx, DK_KERNEL_MIX_DELTA, 1, st);
    s = mix_rows(g.K, deltaq, nullptr, fc.mix, dtil, g.n_out, g.K + 1, g.G, md, ctx->sm_count, st);
  }
  if (s != DK_OK) return s;
  const long long n_dw = (long long)g.cout * g.kc;
  const long long tiles = (long long)((g.cout + BM - 1) / BM) * ((g.kc + BN - 1) / BN);
  if ((g.cout + BM - 1) / BM > 65535) return DK_ERR_SHAPE;
  const long long n_d = (long long)g.G * (g.K + 1) * g.n_out, n_xu = (long long)g.G * (g.K + 1) * g.n_in;
  if (ctx->opt.v[DK_OPT_FIELD_PATH] == 0 && g.layout == DK_NHWC && g.stride == 1 && (g.cin % 16) == 0 &&
      (g.cout % 16) == 0 && wp.xpl_bytes >= (size_t)4 * (n_d + n_xu) && aligned16(xbar)) {
    // tcgen05 kernel on digit planes of the mixed gradients and of the K+1 encodings Eq. 4 uses
    uint8_t* dpl = reinterpret_cast<uint8_t*>(ws + wp.xpl);
    uint8_t* xpl = dpl + 4 * n_d;
    fwg::Params q;
    const int S = g.G * (g.K + 1);
    long long best = -1;
    q.bw = q.bh = q.bs = 1;
    for (int bw = 1; bw <= fwg::KP; bw *= 2)
      for (int bh = 1; bw * bh <= fwg::KP; bh *= 2) {
        const int bs = fwg::KP / (bw * bh);
        const long long cost = (long long)((g.wo + bw - 1) / bw) * bw * ((g.ho + bh - 1) / bh) * bh *
                               ((S + bs - 1) / bs) * bs;
        if (best < 0 || cost < best || (cost == best && bw > q.bw)) { best = cost; q.bw = bw; q.bh = bh; q.bs = bs; }
      }
    q.WT = (g.wo + q.bw - 1) / q.bw;
    q.HT = (g.ho + q.bh - 1) / q.bh;
    q.PB = (long long)q.WT * q.HT * ((S + q.bs - 1) / q.bs);
    q.MT = (g.cout + fwg::TM - 1) / fwg::TM;
    q.cblocks = (g.cin + fwg::TN - 1) / fwg::TN;
    q.kw = g.kw; q.pad = g.pad; q.cout = g.cout; q.cin = g.cin;
    q.ws_o = g.ws_o; q.ws_c = g.ws_c; q.ws_u = g.ws_u; q.ws_v = g.ws_v;
    q.acc = acc; q.md = md; q.pow32 = (u32)((1ull << 32) % md.p);
    q.status = field_status_word(ctx); q.spin_cap = (unsigned)ctx->opt.v[DK_OPT_SPIN_LIMIT];
    q.withhold = take_withhold(ctx);
    const long long items = (long long)q.MT * q.cblocks * g.kh * g.kw;
    // contraction slices: about two rounds of CTAs on the device, at least 8 k-blocks each
    long long splits = (2LL * ctx->sm_count + items - 1) / items;
    if (splits > (q.PB + 7) / 8) splits = (q.PB + 7) / 8;
    if (splits > 65535) splits = 65535;
    if (splits < 1) splits = 1;
    q.pb_per_split = (int)((q.PB + splits - 1) / splits);
    splits = (q.PB + q.pb_per_split - 1) / q.pb_per_split;
    CUtensorMap map_d, map_x;
    bool maps_ok;
    {
      const unsigned long long dims[5] = {(unsigned long long)g.cout, (unsigned long long)g.wo, (unsigned long long)g.ho,
                                          (unsigned long long)S, 4ull};
      const unsigned long long str[4] = {(unsigned long long)g.cout, (unsigned long long)g.cout * g.wo,
                                         (unsigned long long)g.n_out, (unsigned long long)n_d};
      const unsigned int box[5] = {(unsigned)fwg::TM, (unsigned)q.bw, (unsigned)q.bh, (unsigned)q.bs, 4u};
      maps_ok = tc_encode_map_bytes(ctx, &map_d, dpl, 5, dims, str, box, 128);
    }
    if (maps_ok) {
      const unsigned long long dims[5] = {(unsigned long long)g.cin, (unsigned long long)g.w, (unsigned long long)g.h,
                                          (unsigned long long)S, 4ull};
      const unsigned long long str[4] = {(unsigned long long)g.cin, (unsigned long long)g.cin * g.w,
                                         (unsigned long long)g.n_in, (unsigned long long)n_xu};
      const unsigned int box[5] = {(unsigned)fwg::TN, (unsigned)q.bw, (unsigned)q.bh, (unsigned)q.bs, 4u};
      maps_ok = tc_encode_map_bytes(ctx, &map_x, xpl, 5, dims, str, box, 64);
    }
    static const bool tma_attr_ok = cudaFuncSetAttribute(field_wgrad_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                         (int)fwg::kSmem) == cudaSuccess;
    if (maps_ok && tma_attr_ok && items <= 2147483647LL) {
      {
        ProfScope ps(ctx, DK_KERNEL_WGRAD, 3, st);
        field_x_planes_kernel<<<ew_blocks(n_d / 16, ctx->sm_count), 256, 0, st>>>(dtil, n_d, dpl, g.n_out, 1, 1);
        DK_CUDA_CHECK(cudaGetLastError());
        field_x_planes_kernel<<<ew_blocks(n_xu / 16, ctx->sm_count), 256, 0, st>>>(xbar, n_xu, xpl, g.n_in, xbar_rows,
                                                                                  g.K + 1);
        DK_CUDA_CHECK(cudaGetLastError());
        DK_CUDA_CHECK(cudaMemsetAsync(acc, 0, (size_t)n_dw * sizeof(u64), st));
        field_wgrad_tma_kernel<<<dim3((unsigned)items, (unsigned)splits), fwg::kThreads, fwg::kSmem, st>>>(map_d, map_x, q);
        DK_CUDA_CHECK(cudaGetLastError());
      }
      ProfScope ps2(ctx, DK_KERNEL_OTHER, 1, st);
      field_reduce_kernel<<<ew_blocks(n_dw, ctx->sm_count), 256, 0, st>>>(acc, n_dw, md, dWq);
      DK_CUDA_CHECK(cudaGetLastError());
      return DK_OK;
    }
  }
  if (ctx->opt.v[DK_OPT_FIELD_PATH] == 1) {
    WgParams wg;
    wg.d = dtil; wg.x = xbar; wg.acc = acc;
    wg.cin = g.cin; wg.cout = g.cout; wg.h = g.h; wg.w = g.w; wg.kw = g.kw; wg.stride = g.stride;
    wg.pad = g.pad; wg.ho = g.ho; wg.wo = g.wo; wg.kc = g.kc;
    wg.K1 = g.K + 1; wg.xbar_rows = xbar_rows;
    wg.P = g.ho * g.wo;
    wg.PC = (wg.P + BK - 1) / BK;
    wg.GP = (long long)g.G * wg.PC;
    wg.n_in = g.n_in; wg.n_out = g.n_out;
    wg.xs_c = g.xs_c; wg.xs_h = g.xs_h; wg.xs_w = g.xs_w;
    wg.ws_o = g.ws_o; wg.ws_c = g.ws_c; wg.ws_u = g.ws_u; wg.ws_v = g.ws_v;
    wg.ys_c = g.ys_c; wg.ys_h = g.ys_h; wg.ys_w = g.ys_w;
    wg.md = md;
    if (terms_per_reduction(prime) < BK) return DK_ERR_UNSUPPORTED;
    long long fb = terms_per_reduction(prime) / ((long long)BK * wg.K1);      // 0: reduce after every k-tile
    if (fb > 64) fb = 64;
    wg.fold_blocks = (int)fb;
    long long splits = (4LL * ctx->sm_count + tiles - 1) / tiles;
    if (splits > wg.GP) splits = wg.GP;
    if (splits > 65535) splits = 65535;
    if (splits < 1) splits = 1;
    wg.per_split = (wg.GP + splits - 1) / splits;
    splits = (wg.GP + wg.per_split - 1) / wg.per_split;
    dim3 grid((unsigned)((g.kc + BN - 1) / BN), (unsigned)((g.cout + BM - 1) / BM), (unsigned)splits);
    ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
    DK_CUDA_CHECK(cudaMemsetAsync(acc, 0, (size_t)n_dw * sizeof(u64), st));
    field_wgrad_kernel<<<grid, NT, 0, st>>>(wg);
    DK_CUDA_CHECK(cudaGetLastError());
  } else {
    WgMmaParams wg;
    wg.d = dtil; wg.x = xbar; wg.acc = acc;
    wg.cin = g.cin; wg.cout = g.cout; wg.h = g.h; wg.w = g.w; wg.kw = g.kw; wg.stride = g.stride;
    wg.pad = g.pad; wg.ho = g.ho; wg.wo = g.wo; wg.kc = g.kc;
    wg.K1 = g.K + 1; wg.xbar_rows = xbar_rows;
    wg.P = g.ho * g.wo;
    wg.R = (long long)g.G * wg.K1 * wg.P;
    const long long nt = (wg.R + MMA_BK - 1) / MMA_BK;
    if (wg.R >= (1LL << 31)) return DK_ERR_SHAPE;
    wg.div_P = make_fastdiv((u32)wg.P);
    wg.div_K1 = make_fastdiv((u32)wg.K1);
    wg.div_wo = make_fastdiv((u32)g.wo);
    wg.ntiles = (int)nt;
    wg.n_in = g.n_in; wg.n_out = g.n_out;
    wg.xs_c = g.xs_c; wg.xs_h = g.xs_h; wg.xs_w = g.xs_w;
    wg.ws_o = g.ws_o; wg.ws_c = g.ws_c; wg.ws_u = g.ws_u; wg.ws_v = g.ws_v;
    wg.ys_c = g.ys_c; wg.ys_h = g.ys_h; wg.ys_w = g.ys_w;
    wg.md = md;
    wg.pow32 = (u32)((1ull << 32) % md.p);
    // slices of the contraction: about two rounds of blocks on the device, at least 8 tiles each
    long long splits = (2LL * ctx->sm_count + tiles - 1) / tiles;
    if (splits > (nt + 7) / 8) splits = (nt + 7) / 8;
    if (splits > 65535) splits = 65535;
    if (splits < 1) splits = 1;
    wg.tiles_per_split = (int)((nt + splits - 1) / splits);
    splits = (nt + wg.tiles_per_split - 1) / wg.tiles_per_split;
    dim3 grid((unsigned)((g.kc + BN - 1) / BN), (unsigned)((g.cout + BM - 1) / BM), (unsigned)splits);
    static const bool attr_ok = [] {
      return cudaFuncSetAttribute(field_wgrad_mma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)kWgSmemBytes) == cudaSuccess &&
             cudaFuncSetAttribute(field_wgrad_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)kWgSmemBytes) == cudaSuccess;
    }();
    if (!attr_ok) return DK_ERR_CUDA;
    const bool vec2 = g.xs_c == 1 && g.ys_c == 1 && (g.cin % 2) == 0 && (g.cout % 2) == 0 &&
                      ((reinterpret_cast<uintptr_t>(dtil) | reinterpret_cast<uintptr_t>(xbar)) & 7) == 0;
    ProfScope ps(ctx, DK_KERNEL_WGRAD, 1, st);
    DK_CUDA_CHECK(cudaMemsetAsync(acc, 0, (size_t)n_dw * sizeof(u64), st));
    if (vec2) field_wgrad_mma_kernel<2><<<grid, kMmaThreads, kWgSmemBytes, st>>>(wg);
    else field_wgrad_mma_kernel<1><<<grid, kMmaThreads, kWgSmemBytes, st>>>(wg);
    DK_CUDA_CHECK(cudaGetLastError());
  }
  ProfScope ps(ctx, DK_KERNEL_OTHER, 1, st);
  field_reduce_kernel<<<ew_blocks(n_dw, ctx->sm_count), 256, 0, st>>>(acc, n_dw, md, dWq);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // extern "C"
