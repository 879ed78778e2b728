// Final decisions of the integrity check (section 4.4 reading: an element is
// flagged iff not(|rho| <= tau * max(s_e, s_g))), shared by the one-block
// kernel and by the GEMM kernel whose last CTA runs it in its tail.
#pragma once

#include "dk_internal.h"

namespace dk {

// s_g = sum_i |n_i| * rms(ybar_i) for group g from the accumulated sums of squares.
__device__ __forceinline__ float group_scale(const float* sumsq, const float* nul, long long g,
                                             int E, float inv_n) {
  float s = 0.f;
  for (int i = 0; i < E; ++i) s += fabsf(nul[g * E + i]) * sqrtf(__ldcg(sumsq + g * E + i) * inv_n);
  return s;
}

// Run by exactly 256 threads (tid = 0..255) that can meet at named barrier 1:
// final decision for every candidate, summary into *vd.  The statistics must
// be complete and visible to the caller (they are read past L1, from where
// the other CTAs' atomics put them).
__device__ __forceinline__ void verify_finalize_block(int tid, const float* sumsq, const int* maxrho,
                                                      const unsigned int* count, const Candidate* cand,
                                                      const float* nul, dk_verdict* vd, int G, int E,
                                                      long long n_out, float tau) {
  __shared__ unsigned int s_n[8];
  __shared__ long long s_f[8];
  __shared__ float s_r[8];
  const float inv_n = 1.f / (float)n_out;
  unsigned int nflag = 0;
  long long first = 0x7fffffffffffffffLL;
  float maxr = 0.f;
  for (int g = tid; g < G; g += 256) {
    float sg = group_scale(sumsq, nul, g, E, inv_n);
    float mr = __int_as_float(__ldcg(maxrho + g));
    if (sg > 0.f) maxr = fmaxf(maxr, mr / sg);
  }
  const unsigned int total = __ldcg(count);
  const unsigned int n = total < kCandCap ? total : kCandCap;
  for (unsigned int c = tid; c < n; c += 256) {
    Candidate cd = cand[c];
    long long g = cd.index / n_out;
    float sg = group_scale(sumsq, nul, g, E, inv_n);
    float scale = fmaxf(cd.s_e, sg);
    bool bad = !(cd.absrho <= tau * scale) || !(cd.s_e < __int_as_float(0x7f800000));
    if (bad) {
      ++nflag;
      first = cd.index < first ? cd.index : first;
    }
  }
  const int lane = tid & 31, wid = tid >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    nflag += __shfl_xor_sync(0xffffffffu, nflag, o);
    long long f2 = __shfl_xor_sync(0xffffffffu, first, o);
    first = f2 < first ? f2 : first;
    maxr = fmaxf(maxr, __shfl_xor_sync(0xffffffffu, maxr, o));
  }
  if (lane == 0) { s_n[wid] = nflag; s_f[wid] = first; s_r[wid] = maxr; }
  asm volatile("bar.sync 1, 256;" ::: "memory");
  if (tid == 0) {
    for (int w = 1; w < 8; ++w) {
      nflag += s_n[w];
      first = s_f[w] < first ? s_f[w] : first;
      maxr = fmaxf(maxr, s_r[w]);
    }
    int status = (int)__ldcg(count + 1);   // raised by a producing kernel that gave up: nothing can be trusted
    if (total > kCandCap) {
      // more suspects than the list holds: everything beyond it counts as flagged
      nflag += total - kCandCap;
      if (status == 0) status = DK_ERR_WORKSPACE;
    }
    vd->ok = (nflag == 0 && status == 0) ? 1 : 0;
    vd->n_flagged = nflag;
    vd->first_index = (first != 0x7fffffffffffffffLL) ? first : -1;
    vd->max_ratio = maxr;
    vd->status = status;
  }
}

}  // namespace dk
