// HBM-bound kernels: encode (Eq. 1), decode + redundant-equation check
// (Eq. 2, Section 4.4), delta mixing (Eq. 4) and the verdict bookkeeping.
//
// All of them stream rows of length n (elements of one sample) with 128-bit
// accesses; a thread owns one 4-element column slice of a whole group, keeps
// the group's coefficients in registers and touches every byte exactly once.
#include "dk_internal.h"
#include "dk_verify.cuh"

namespace dk {
namespace {

constexpr int kThreads = 256;

struct f4 {
  float v[4];
};

template <bool VEC>
__device__ __forceinline__ f4 load4(const float* p, long long e, long long n) {
  f4 o;
  if (VEC) {
    float4 t = __ldg(reinterpret_cast<const float4*>(p + e));
    o.v[0] = t.x; o.v[1] = t.y; o.v[2] = t.z; o.v[3] = t.w;
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) o.v[q] = (e + q < n) ? __ldg(p + e + q) : 0.f;
  }
  return o;
}

template <bool VEC>
__device__ __forceinline__ void store4(float* p, long long e, long long n, const f4& o) {
  if (VEC) {
    *reinterpret_cast<float4*>(p + e) = make_float4(o.v[0], o.v[1], o.v[2], o.v[3]);
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (e + q < n) p[e + q] = o.v[q];
  }
}

// out[g*NOUT + i][e] = sum_{k<NIN} coef[g][i][k] * src_k[e]; the first NX
// sources are rows g*NX.. of `x`, the optional last one is row g of `r`.
template <int NX, bool HAS_R, int NOUT, bool VEC>
__global__ void __launch_bounds__(kThreads)
mix_rows_kernel(const float* __restrict__ x, const float* __restrict__ r,
                const float* __restrict__ coef, float* __restrict__ out, long long n) {
  constexpr int NIN = NX + (HAS_R ? 1 : 0);
  const int g = blockIdx.y;
  float c[NOUT][NIN];
#pragma unroll
  for (int i = 0; i < NOUT; ++i)
#pragma unroll
    for (int k = 0; k < NIN; ++k) c[i][k] = __ldg(coef + ((size_t)g * NOUT + i) * NIN + k);
  const float* xg = x + (size_t)g * NX * n;
  const float* rg = HAS_R ? r + (size_t)g * n : nullptr;
  float* og = out + (size_t)g * NOUT * n;
  const long long nvec = (n + 3) / 4;
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < nvec;
       v += (long long)gridDim.x * kThreads) {
    const long long e = v * 4;
    f4 src[NIN];
#pragma unroll
    for (int k = 0; k < NX; ++k) src[k] = load4<VEC>(xg + (size_t)k * n, e, n);
    if (HAS_R) src[NIN - 1] = load4<VEC>(rg, e, n);
#pragma unroll
    for (int i = 0; i < NOUT; ++i) {
      f4 o;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        // last source (the noise, when present) first, then one FMA per input
        float acc = c[i][NIN - 1] * src[NIN - 1].v[q];
#pragma unroll
        for (int k = 0; k < NIN - 1; ++k) acc = fmaf(c[i][k], src[k].v[q], acc);
        o.v[q] = acc;
      }
      store4<VEC>(og + (size_t)i * n, e, n, o);
    }
  }
}

__global__ void add_fault_kernel(float* ybar, long long idx, float delta) { ybar[idx] += delta; }

// Clears the per-call statistics of the integrity check.
__global__ void verify_begin_kernel(float* stats, int nstats, unsigned int* count) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nstats; i += gridDim.x * blockDim.x)
    stats[i] = 0.f;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    count[0] = 0u;   // suspects appended
    count[1] = 0u;   // status word a producing kernel may raise (DK_ERR_TIMEOUT)
  }
}

// One block of 256 threads: final decision for every candidate, summary into *vd.
__global__ void __launch_bounds__(256)
verify_finalize_kernel(const float* sumsq, const int* maxrho, const unsigned int* count,
                       const Candidate* cand, const float* nul, dk_verdict* vd, int G, int E,
                       long long n_out, float tau) {
  verify_finalize_block((int)threadIdx.x, sumsq, maxrho, count, cand, nul, vd, G, E, n_out, tau);
}

// Per-block merge of the verify statistics: E sums of squares and max |rho|.
template <int E>
__device__ __forceinline__ void stats_merge(const VerifyScratch& vs, int g, float (&sq)[E],
                                            float maxrho) {
  __shared__ float s_sq[kThreads / 32][E + 1];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < E; ++i)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], o);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) maxrho = fmaxf(maxrho, __shfl_xor_sync(0xffffffffu, maxrho, o));
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < E; ++i) s_sq[wid][i] = sq[i];
    s_sq[wid][E] = maxrho;
  }
  __syncthreads();
  if (threadIdx.x < E) {
    float t = 0.f;
    for (int w = 0; w < kThreads / 32; ++w) t += s_sq[w][threadIdx.x];
    if (t != 0.f) atomicAdd(vs.sumsq + (size_t)g * E + threadIdx.x, t);
  } else if (threadIdx.x == E) {
    float t = 0.f;
    for (int w = 0; w < kThreads / 32; ++w) t = fmaxf(t, s_sq[w][E]);
    if (t > 0.f) atomicMax(vs.maxrho + g, __float_as_int(t));
  }
}

template <int K, bool VEC>
__global__ void __launch_bounds__(kThreads)
decode_verify_kernel(const float* __restrict__ ybar, const float* __restrict__ dec,
                     const float* __restrict__ decl, const float* __restrict__ nul,
                     const float* __restrict__ bias, float* __restrict__ y, VerifyScratch vs,
                     long long n, float tau, int cout, long long cdiv, int kstore) {
  constexpr int K1 = K + 1, E = K + 2;
  const int g = blockIdx.y;
  // One fp32 coefficient per term: the fp32 sum's own rounding is as large as
  // what the second float of the coefficient pair (decl) would contribute.
  (void)decl;
  float dh[K][K1], nv[E];
#pragma unroll
  for (int k = 0; k < K; ++k)
#pragma unroll
    for (int i = 0; i < K1; ++i) dh[k][i] = __ldg(dec + ((size_t)g * K + k) * K1 + i);
#pragma unroll
  for (int i = 0; i < E; ++i) nv[i] = __ldg(nul + (size_t)g * E + i);
  const float* yb = ybar + (size_t)g * E * n;
  float* yo = y + (size_t)g * K * n;
  float sq[E];
#pragma unroll
  for (int i = 0; i < E; ++i) sq[i] = 0.f;
  float maxrho = 0.f;
  const float kInf = __int_as_float(0x7f800000);
  const long long nvec = (n + 3) / 4;
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < nvec;
       v += (long long)gridDim.x * kThreads) {
    const long long e = v * 4;
    f4 in[E];
#pragma unroll
    for (int i = 0; i < E; ++i) in[i] = load4<VEC>(yb + (size_t)i * n, e, n);
    f4 b;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      b.v[q] = 0.f;
      if (bias != nullptr && e + q < n) b.v[q] = __ldg(bias + ((e + q) / cdiv) % cout);
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
      if (k >= kstore) continue;      // (a noise vector in the place of a private input: its output is not wanted)
      f4 o;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float acc = dh[k][0] * in[0].v[q];
#pragma unroll
        for (int i = 1; i < K1; ++i) acc = fmaf(dh[k][i], in[i].v[q], acc);
        o.v[q] = acc + b.v[q];
      }
      store4<VEC>(yo + (size_t)k * n, e, n, o);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (e + q < n) {
        float rho = 0.f, sc = 0.f;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          const float val = in[i].v[q];
          rho = fmaf(nv[i], val, rho);
          sc = fmaf(fabsf(nv[i]), fabsf(val), sc);
          if (fabsf(val) < kInf) sq[i] = fmaf(val, val, sq[i]);
        }
        const float ar = fabsf(rho);
        maxrho = fmaxf(maxrho, ar);
        if (!(ar <= tau * sc) || !(sc < kInf)) {
          unsigned int slot = atomicAdd(vs.count, 1u);
          if (slot < kCandCap) {
            Candidate cd;
            cd.index = (long long)g * n + e + q;
            cd.absrho = ar;
            cd.s_e = sc;
            vs.cand[slot] = cd;
          }
        }
      }
    }
  }
  stats_merge<E>(vs, g, sq, maxrho);
}

inline int blocks_for(long long n, int G, int sm_count) {
  long long nvec = (n + 3) / 4;
  long long want = (nvec + kThreads - 1) / kThreads;
  // about 16 blocks per SM over the whole grid, never more than there is work
  long long cap = ((long long)sm_count * 16 + G - 1) / G;
  if (cap < 1) cap = 1;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return (int)want;
}

template <int NX, bool HAS_R, int NOUT>
dk_status launch_mix(const float* x, const float* r, const float* coef, float* out, long long n,
                     int G, int sm_count, cudaStream_t st) {
  dim3 grid(blocks_for(n, G, sm_count), G);
  if (n % 4 == 0)
    mix_rows_kernel<NX, HAS_R, NOUT, true><<<grid, kThreads, 0, st>>>(x, r, coef, out, n);
  else
    mix_rows_kernel<NX, HAS_R, NOUT, false><<<grid, kThreads, 0, st>>>(x, r, coef, out, n);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

template <int K>
dk_status launch_dv(const Geom& g, const float* ybar, const CoefView& cv, const float* bias,
                    float* y, const VerifyScratch& vs, int sm_count, cudaStream_t st) {
  dim3 grid(blocks_for(g.n_out, g.G, sm_count), g.G);
  // channel of element e: (e / cdiv) % cout
  long long cdiv = (g.layout == DK_NCHW && g.kind == DK_CONV2D) ? (long long)g.ho * g.wo : 1;
  if (g.n_out % 4 == 0)
    decode_verify_kernel<K, true><<<grid, kThreads, 0, st>>>(
        ybar, cv.dec, cv.decl, cv.nul, bias, y, vs, g.n_out, g.tol, g.cout, cdiv, g.kstore);
  else
    decode_verify_kernel<K, false><<<grid, kThreads, 0, st>>>(
        ybar, cv.dec, cv.decl, cv.nul, bias, y, vs, g.n_out, g.tol, g.cout, cdiv, g.kstore);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace

#define DK_DISPATCH_K(Kval, CALL)              \
  switch (Kval) {                              \
    case 1: { constexpr int KK = 1; CALL; }    \
    case 2: { constexpr int KK = 2; CALL; }    \
    case 3: { constexpr int KK = 3; CALL; }    \
    case 4: { constexpr int KK = 4; CALL; }    \
    case 5: { constexpr int KK = 5; CALL; }    \
    case 6: { constexpr int KK = 6; CALL; }    \
    case 7: { constexpr int KK = 7; CALL; }    \
    case 8: { constexpr int KK = 8; CALL; }    \
    default: return DK_ERR_SHAPE;              \
  }

dk_status launch_encode(const Geom& g, const float* x, const float* r, const float* enc,
                        float* xbar, int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  DK_DISPATCH_K(g.K, return (launch_mix<KK, true, KK + 2>(x, r, enc, xbar, g.n_in, g.G, sm_count, st)));
}

dk_status launch_mix_delta(const Geom& g, const float* delta, const float* dmix, float* dtil,
                           int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  DK_DISPATCH_K(g.K, return (launch_mix<KK, false, KK + 1>(delta, nullptr, dmix, dtil, g.n_out,
                                                          g.G, sm_count, st)));
}

VerifyScratch verify_scratch(const dk_ctx* ctx, const Geom& g) {
  VerifyScratch vs;
  vs.sumsq = ctx->d_vstats;
  vs.maxrho = reinterpret_cast<int*>(ctx->d_vstats + (size_t)g.G * g.E);
  vs.count = reinterpret_cast<unsigned int*>(ctx->d_vstats + kVerifyStatFloats);
  vs.cand = ctx->d_cand;
  return vs;
}

dk_status launch_verify_begin(const Geom& g, const VerifyScratch& vs, cudaStream_t st) {
  int nstats = g.G * (g.E + 1);
  int blocks = (nstats + 255) / 256;
  if (blocks > 64) blocks = 64;
  verify_begin_kernel<<<blocks, 256, 0, st>>>(vs.sumsq, nstats, vs.count);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status launch_decode_verify(const Geom& g, const float* ybar, const CoefView& cv,
                               const float* bias, float* y, const VerifyScratch& vs,
                               int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  DK_DISPATCH_K(g.K, return (launch_dv<KK>(g, ybar, cv, bias, y, vs, sm_count, st)));
}

dk_status launch_verify_finalize(const Geom& g, const float* nul, const VerifyScratch& vs,
                                 dk_verdict* v, cudaStream_t st) {
  verify_finalize_kernel<<<1, 256, 0, st>>>(vs.sumsq, vs.maxrho, vs.count, vs.cand, nul, v, g.G,
                                            g.E, g.n_out, g.tol);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status launch_add_fault(float* ybar, long long index, float delta, cudaStream_t st) {
  add_fault_kernel<<<1, 1, 0, st>>>(ybar, index, delta);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
