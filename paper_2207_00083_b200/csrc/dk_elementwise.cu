// HBM-bound kernels: encode (Eq. 1), decode + redundant-equation check
// (Eq. 2, Section 4.4), delta mixing (Eq. 4) and the verdict bookkeeping.
//
// All of them stream rows of length n (elements of one sample) with 128-bit
// accesses; a thread owns one 4-element column slice of a whole group, keeps
// the group's coefficients in registers and touches every byte exactly once.
#include "dk_internal.h"

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

__global__ void verdict_init_kernel(dk_verdict* v) {
  v->ok = 1;
  v->n_flagged = 0;
  v->first_index = 0x7fffffffffffffffLL;
  v->max_ratio = 0.f;
  v->status = 0;
}

__global__ void add_fault_kernel(float* ybar, long long idx, float delta) { ybar[idx] += delta; }

// Block-level merge of per-thread verify results into the device verdict;
// the last block to finish turns an untouched first_index into -1.
__device__ void verdict_merge(dk_verdict* vd, unsigned int* counter, unsigned int nflag,
                              long long first, float maxr, unsigned int nblocks) {
  __shared__ unsigned int s_n[32];
  __shared__ long long s_f[32];
  __shared__ float s_r[32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int nw = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    nflag += __shfl_xor_sync(0xffffffffu, nflag, o);
    long long f2 = __shfl_xor_sync(0xffffffffu, first, o);
    first = f2 < first ? f2 : first;
    maxr = fmaxf(maxr, __shfl_xor_sync(0xffffffffu, maxr, o));
  }
  if (lane == 0) { s_n[wid] = nflag; s_f[wid] = first; s_r[wid] = maxr; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < nw; ++w) {
      nflag += s_n[w];
      first = s_f[w] < first ? s_f[w] : first;
      maxr = fmaxf(maxr, s_r[w]);
    }
    if (nflag) {
      atomicAdd(&vd->n_flagged, nflag);
      atomicMin(reinterpret_cast<unsigned long long*>(&vd->first_index), (unsigned long long)first);
      atomicExch(&vd->ok, 0);
    }
    if (maxr > 0.f) atomicMax(reinterpret_cast<int*>(&vd->max_ratio), __float_as_int(maxr));
    __threadfence();
    unsigned int done = atomicAdd(counter, 1u);
    if (done == nblocks - 1) {
      __threadfence();
      unsigned long long fi =
          atomicAdd(reinterpret_cast<unsigned long long*>(&vd->first_index), 0ULL);
      if (fi == 0x7fffffffffffffffULL) vd->first_index = -1;
      *counter = 0;
    }
  }
}

template <int K, bool VEC>
__global__ void __launch_bounds__(kThreads)
decode_verify_kernel(const float* __restrict__ ybar, const float* __restrict__ dec,
                     const float* __restrict__ decl, const float* __restrict__ nul,
                     const float* __restrict__ bias, float* __restrict__ y, dk_verdict* vd,
                     unsigned int* counter, long long n, float tau, int cout, long long cdiv) {
  constexpr int K1 = K + 1, E = K + 2;
  const int g = blockIdx.y;
  float dh[K][K1], dl[K][K1], nv[E];
#pragma unroll
  for (int k = 0; k < K; ++k)
#pragma unroll
    for (int i = 0; i < K1; ++i) {
      dh[k][i] = __ldg(dec + ((size_t)g * K + k) * K1 + i);
      dl[k][i] = __ldg(decl + ((size_t)g * K + k) * K1 + i);
    }
#pragma unroll
  for (int i = 0; i < E; ++i) nv[i] = __ldg(nul + (size_t)g * E + i);
  const float* yb = ybar + (size_t)g * E * n;
  float* yo = y + (size_t)g * K * n;
  unsigned int nflag = 0;
  long long first = 0x7fffffffffffffffLL;
  float maxr = 0.f;
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
      f4 o;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float lo = 0.f, hi = 0.f;
#pragma unroll
        for (int i = 0; i < K1; ++i) {
          lo = fmaf(dl[k][i], in[i].v[q], lo);
          hi = fmaf(dh[k][i], in[i].v[q], hi);
        }
        o.v[q] = (hi + lo) + b.v[q];
      }
      store4<VEC>(yo + (size_t)k * n, e, n, o);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (e + q < n) {
        float rho = 0.f, sc = 0.f;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          rho = fmaf(nv[i], in[i].v[q], rho);
          sc = fmaf(fabsf(nv[i]), fabsf(in[i].v[q]), sc);
        }
        const float ar = fabsf(rho);
        if (!(ar <= tau * sc)) {
          ++nflag;
          long long idx = (long long)g * n + e + q;
          first = idx < first ? idx : first;
        }
        if (sc > 0.f) maxr = fmaxf(maxr, ar / sc);
      }
    }
  }
  verdict_merge(vd, counter, nflag, first, maxr, gridDim.x * gridDim.y);
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
                    float* y, dk_verdict* v, unsigned int* counter, int sm_count,
                    cudaStream_t st) {
  dim3 grid(blocks_for(g.n_out, g.G, sm_count), g.G);
  // channel of element e: (e / cdiv) % cout
  long long cdiv = (g.layout == DK_NCHW && g.kind == DK_CONV2D) ? (long long)g.ho * g.wo : 1;
  if (g.n_out % 4 == 0)
    decode_verify_kernel<K, true><<<grid, kThreads, 0, st>>>(
        ybar, cv.dec, cv.decl, cv.nul, bias, y, v, counter, g.n_out, g.tol, g.cout, cdiv);
  else
    decode_verify_kernel<K, false><<<grid, kThreads, 0, st>>>(
        ybar, cv.dec, cv.decl, cv.nul, bias, y, v, counter, g.n_out, g.tol, g.cout, cdiv);
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

dk_status launch_verdict_init(dk_verdict* v, cudaStream_t st) {
  verdict_init_kernel<<<1, 1, 0, st>>>(v);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status launch_decode_verify(const Geom& g, const float* ybar, const CoefView& cv,
                               const float* bias, float* y, dk_verdict* v,
                               unsigned int* counter, int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  DK_DISPATCH_K(g.K, return (launch_dv<KK>(g, ybar, cv, bias, y, v, counter, sm_count, st)));
}

dk_status launch_add_fault(float* ybar, long long index, float delta, cudaStream_t st) {
  add_fault_kernel<<<1, 1, 0, st>>>(ybar, index, delta);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
