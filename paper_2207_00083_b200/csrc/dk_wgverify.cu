// Comparison of two weight gradients decoded from different sets of K+1 of the
// K+2 stored encodings (the redundancy idea of Section 4.4 applied to
// Eq. 4-6).  HBM-bound and small: dW has cout x kc elements.
//   pass 1: sum of squares of the first result (its rms is the normaliser)
//   pass 2: element flagged iff not(|a - b| <= tol * rms); count, smallest
//           flagged index and largest ratio by atomics
//   pass 3: one thread writes the dk_verdict
#include "dk_internal.h"

namespace dk {
namespace {

struct WgCheck {          // 32 bytes of device scratch
  float sumsq;
  unsigned int max_bits;  // bit pattern of the largest |a - b| (non-negative floats order like their bits)
  unsigned int nflag;
  unsigned int pad;
  unsigned long long first;
};

__global__ void __launch_bounds__(256) wg_sumsq_kernel(const float* __restrict__ a, long long n, WgCheck* c) {
  __shared__ float s[8];
  if (blockIdx.x == 0 && threadIdx.x == 0) c->first = ~0ull;
  float acc = 0.f;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float v = a[i];
    if (fabsf(v) < __int_as_float(0x7f800000)) acc = fmaf(v, v, acc);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += s[w];
    if (t != 0.f) atomicAdd(&c->sumsq, t);
  }
}

__global__ void __launch_bounds__(256) wg_compare_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                                         long long n, float tol, WgCheck* c) {
  const float rms = sqrtf(c->sumsq / (float)n);
  const float bound = tol * rms;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float d = fabsf(a[i] - b[i]);
    if (!(d <= bound)) {              // also true for NaN
      atomicAdd(&c->nflag, 1u);
      atomicMin(&c->first, (unsigned long long)i);
    }
    if (d > 0.f && d <= __int_as_float(0x7f800000)) atomicMax(&c->max_bits, __float_as_uint(d));
  }
}

__global__ void wg_verdict_kernel(const WgCheck* c, long long n, const int* status_word, dk_verdict* v) {
  const float rms = sqrtf(c->sumsq / (float)n);
  const int status = status_word ? *status_word : 0;
  v->ok = (c->nflag == 0 && status == 0) ? 1 : 0;
  v->n_flagged = c->nflag;
  v->first_index = c->nflag ? (long long)c->first : -1;
  const float dmax = __uint_as_float(c->max_bits);
  v->max_ratio = rms > 0.f ? dmax / rms : (dmax > 0.f ? __int_as_float(0x7f800000) : 0.f);
  v->status = status;
}

}  // namespace

dk_status launch_wgrad_compare(const float* a, const float* b, long long n, float tol, void* scratch32,
                               const int* status_word, dk_verdict* v, int sm_count, cudaStream_t st) {
  WgCheck* c = static_cast<WgCheck*>(scratch32);
  DK_CUDA_CHECK(cudaMemsetAsync(c, 0, sizeof(WgCheck), st));
  long long blocks = (n + 255) / 256;
  if (blocks > (long long)sm_count * 8) blocks = (long long)sm_count * 8;
  if (blocks < 1) blocks = 1;
  wg_sumsq_kernel<<<(unsigned)blocks, 256, 0, st>>>(a, n, c);
  wg_compare_kernel<<<(unsigned)blocks, 256, 0, st>>>(a, b, n, tol, c);
  wg_verdict_kernel<<<1, 1, 0, st>>>(c, n, status_word, v);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
