// fp64 variants of the encoder (Eq. 1) and of the decoder + integrity check
// (Eq. 2, Section 4.4) for DK_FP64_SIMT.  With noise a thousand times larger
// than the inputs one fp32 rounding of an encoded value already costs ~1e-4 of
// the decoded result per unit of decoder gain, so in that regime the encodings
// and y_bar are kept as doubles between the three kernels of the fused call.
#include "dk_internal.h"

namespace dk {
namespace {

constexpr int kThreads64 = 256;

// xbar64[g*E+i][e] = sum_k C[g][i][k]*x[g*K+k][e] + C[g][i][K]*r[g][e] in fp64;
// `full32` (nullable) receives the same values rounded to fp32.
template <int K>
__global__ void __launch_bounds__(kThreads64)
encode64_kernel(const float* __restrict__ x, const float* __restrict__ r, const float* __restrict__ enc,
                double* __restrict__ out64, float* __restrict__ full32, long long n) {
  constexpr int K1 = K + 1, E = K + 2;
  const int g = blockIdx.y;
  double c[E][K1];
#pragma unroll
  for (int i = 0; i < E; ++i)
#pragma unroll
    for (int k = 0; k < K1; ++k) c[i][k] = (double)__ldg(enc + ((size_t)g * E + i) * K1 + k);
  const float* xg = x + (size_t)g * K * n;
  const float* rg = r + (size_t)g * n;
  const size_t ob = (size_t)g * E * n;
  for (long long e = (long long)blockIdx.x * kThreads64 + threadIdx.x; e < n;
       e += (long long)gridDim.x * kThreads64) {
    double s[K1];
#pragma unroll
    for (int k = 0; k < K; ++k) s[k] = (double)__ldg(xg + (size_t)k * n + e);
    s[K] = (double)__ldg(rg + e);
#pragma unroll
    for (int i = 0; i < E; ++i) {
      double acc = c[i][K] * s[K];
#pragma unroll
      for (int k = 0; k < K; ++k) acc = fma(c[i][k], s[k], acc);
      out64[ob + (size_t)i * n + e] = acc;
      if (full32 != nullptr) full32[ob + (size_t)i * n + e] = (float)acc;
    }
  }
}

// Decode and residual in fp64 from fp64 y_bar; statistics and suspects as in
// the fp32 kernel (their consumers compare with tolerances far above fp32 ulp).
template <int K>
__global__ void __launch_bounds__(kThreads64)
decode_verify64_kernel(const double* __restrict__ ybar, const float* __restrict__ dec,
                       const float* __restrict__ decl, const float* __restrict__ nul,
                       const float* __restrict__ bias, float* __restrict__ y, VerifyScratch vs,
                       long long n, float tau, int cout, long long cdiv, int kstore) {
  constexpr int K1 = K + 1, E = K + 2;
  __shared__ float s_red[kThreads64 / 32][E + 1];
  const int g = blockIdx.y;
  const double* yb = ybar + (size_t)g * E * n;
  float* yo = y + (size_t)g * K * n;
  float sq[E];
#pragma unroll
  for (int i = 0; i < E; ++i) sq[i] = 0.f;
  float maxrho = 0.f;
  const float kInf = __int_as_float(0x7f800000);
  for (long long e = (long long)blockIdx.x * kThreads64 + threadIdx.x; e < n;
       e += (long long)gridDim.x * kThreads64) {
    double v[E];
#pragma unroll
    for (int i = 0; i < E; ++i) v[i] = yb[(size_t)i * n + e];
    const double b = bias != nullptr ? (double)__ldg(bias + (e / cdiv) % cout) : 0.0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
      if (k >= kstore) continue;      // (a noise vector in the place of a private input)
      double acc = 0.0;
#pragma unroll
      for (int i = 0; i < K1; ++i) {
        const size_t ci = ((size_t)g * K + k) * K1 + i;
        acc = fma((double)__ldg(dec + ci) + (double)__ldg(decl + ci), v[i], acc);
      }
      yo[(size_t)k * n + e] = (float)(acc + b);
    }
    double rho = 0.0, sc = 0.0;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const double n_i = (double)__ldg(nul + (size_t)g * E + i);
      rho = fma(n_i, v[i], rho);
      sc = fma(fabs(n_i), fabs(v[i]), sc);
      const float vf = (float)v[i];
      if (fabsf(vf) < kInf) sq[i] = fmaf(vf, vf, sq[i]);
    }
    const float ar = (float)fabs(rho), scf = (float)sc;
    maxrho = fmaxf(maxrho, ar);
    if (!(ar <= tau * scf) || !(scf < kInf)) {
      unsigned int slot = atomicAdd(vs.count, 1u);
      if (slot < kCandCap) {
        Candidate cd;
        cd.index = (long long)g * n + e;
        cd.absrho = ar;
        cd.s_e = scf;
        vs.cand[slot] = cd;
      }
    }
  }
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < E; ++i)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], o);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) maxrho = fmaxf(maxrho, __shfl_xor_sync(0xffffffffu, maxrho, o));
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < E; ++i) s_red[wid][i] = sq[i];
    s_red[wid][E] = maxrho;
  }
  __syncthreads();
  if (threadIdx.x < E) {
    float t = 0.f;
    for (int w = 0; w < kThreads64 / 32; ++w) t += s_red[w][threadIdx.x];
    if (t != 0.f) atomicAdd(vs.sumsq + (size_t)g * E + threadIdx.x, t);
  } else if (threadIdx.x == E) {
    float t = 0.f;
    for (int w = 0; w < kThreads64 / 32; ++w) t = fmaxf(t, s_red[w][E]);
    if (t > 0.f) atomicMax(vs.maxrho + g, __float_as_int(t));
  }
}

__global__ void add_fault64_kernel(double* ybar, long long idx, float delta) { ybar[idx] += (double)delta; }

inline dim3 grid_for(long long n, int G, int sm_count) {
  long long want = (n + kThreads64 - 1) / kThreads64;
  long long cap = ((long long)sm_count * 16 + G - 1) / G;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return dim3((unsigned)want, (unsigned)G);
}

}  // namespace

#define DK_K_SWITCH(Kval, STMT)                     \
  switch (Kval) {                                   \
    case 1: { constexpr int KK = 1; STMT; } break;  \
    case 2: { constexpr int KK = 2; STMT; } break;  \
    case 3: { constexpr int KK = 3; STMT; } break;  \
    case 4: { constexpr int KK = 4; STMT; } break;  \
    case 5: { constexpr int KK = 5; STMT; } break;  \
    case 6: { constexpr int KK = 6; STMT; } break;  \
    case 7: { constexpr int KK = 7; STMT; } break;  \
    case 8: { constexpr int KK = 8; STMT; } break;  \
    default: return DK_ERR_SHAPE;                   \
  }

dk_status launch_encode64(const Geom& g, const float* x, const float* r, const float* enc, double* out64,
                          float* full32, int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  dim3 grid = grid_for(g.n_in, g.G, sm_count);
  DK_K_SWITCH(g.K, (encode64_kernel<KK><<<grid, kThreads64, 0, st>>>(x, r, enc, out64, full32, g.n_in)));
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status launch_decode_verify64(const Geom& g, const double* ybar, const CoefView& cv, const float* bias,
                                 float* y, const VerifyScratch& vs, int sm_count, cudaStream_t st) {
  if (g.G > 65535) return DK_ERR_SHAPE;
  dim3 grid = grid_for(g.n_out, g.G, sm_count);
  const long long cdiv = (g.layout == DK_NCHW && g.kind == DK_CONV2D) ? (long long)g.ho * g.wo : 1;
  DK_K_SWITCH(g.K, (decode_verify64_kernel<KK><<<grid, kThreads64, 0, st>>>(
                       ybar, cv.dec, cv.decl, cv.nul, bias, y, vs, g.n_out, g.tol, g.cout, cdiv, g.kstore)));
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status launch_add_fault64(double* ybar, long long index, float delta, cudaStream_t st) {
  add_fault64_kernel<<<1, 1, 0, st>>>(ybar, index, delta);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
