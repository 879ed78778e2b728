// The fp64 regime (DK_FP64_SIMT) for pointwise layers, in ONE kernel: Eq. 1 in
// the prologue, the contraction on the fp64 tensor path, Eq. 2 and the
// redundant equation of Section 4.4 in the epilogue.
//
// Why fp64.  With noise a thousand times larger than the inputs and K = 8 the
// encoded outputs must be known to ~1e-10 of their own size for the decoded
// result to be good to 1e-3: every fp32 accumulator (CUDA core or tensor
// memory, whose adds truncate) loses 2^-24 of the running sum per addition,
// which the decoder multiplies by ~1000 * |C^-1|.  Splitting the operands finer
// does not help, the accumulator is what is too short; mma.sync m8n8k4 f64
// accumulates in fp64 and runs at the same 37 TFLOP/s as plain fp64 FMAs on
// this part, with a quarter of the instructions and operand fetches.
//
// Why fused.  A 1x1 convolution reads every input element once per output
// channel block, so encoding inside the kernel costs (K+1)/rows extra FMAs and
// nothing else: the fp64 encodings live in shared memory only (the unfused
// path wrote and re-read them as 8-byte values), y_bar lives in registers, and
// the call moves what it must: K inputs and the noise in, K outputs (and the
// fp32 encodings, when the caller stores them) out.
//
// Tiling.  A CTA owns P = 8*PB pixels of one virtual batch and 16*MT16 output
// channels; each of its warps owns one (16 channels) x (8 pixels x all K+2
// encodings) block: 2 x (K+2) m8n8k4 accumulators.  Column e*8 + j of a warp's
// block is encoding e of its pixel j, so a thread's accumulators hold every
// encoding of its two pixels: decoding and the residual are thread-local.
#include "dk_internal.h"

namespace dk {
namespace {

constexpr int KC = 16;        // contraction elements per chunk
constexpr int S = 20;         // row pitch of the fp64 tiles in doubles: = 4 (mod 16), conflict-free fragment reads
constexpr int kWarps = 4;        // warps per CTA: small CTAs, several per SM, hide each other's load and barrier phases
constexpr int kThreads = 32 * kWarps;

struct F64Params {
  const float* W; const float* x; const float* r; const float* bias;
  float* y; float* xsave;
  const float* enc; const float* dec; const float* decl; const float* nul;
  VerifyScratch vs;
  float tau;
  int cin, cout, npix, G;
  int MT16, PB, tiles_per_g, mtiles;
  long long ntiles;
  int f_group, f_enc;
  long long f_index;          // pixel * cout + channel
  float f_delta;
  int kstore;                 // decoded rows k >= kstore of a group are neither computed nor stored
};

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

// One CTA per tile = (virtual batch, P pixels, 16*MT16 output channels), three CTAs of four warps per SM:
// they cover each other's load and barrier phases.  (A persistent variant that staged the next chunk's
// raw inputs with cp.async measured slower, as did integer-only fp32/fp64 conversions.)
template <int K>
__global__ void __launch_bounds__(kThreads, 3) fused64_kernel(const F64Params p) {
  constexpr int K1 = K + 1, E = K + 2;
  extern __shared__ double smem64[];
  const int P = 8 * p.PB, rows = 16 * p.MT16;
  double* xs = smem64;                              // [E][P][S]   fp64 encodings of the current chunk
  double* ws = xs + (size_t)E * P * S;              // [rows][S]   fp64 weights of the current chunk
  double* cenc = ws + (size_t)rows * S;             // [E][K1]
  double* cdec = cenc + E * K1;                     // [K][K1]
  double* cnul = cdec + K * K1;                     // [E]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gq = lane >> 2, q = lane & 3;
  const int m16 = warp % p.MT16, pb = warp / p.MT16;
  const long long n_in = (long long)p.npix * p.cin, n_out = (long long)p.npix * p.cout;
  int g, pt, mt;
  {
    const long long t = blockIdx.x;
    mt = (int)(t % p.mtiles);
    const long long rest = t / p.mtiles;
    pt = (int)(rest % p.tiles_per_g);
    g = (int)(rest / p.tiles_per_g);
  }
  for (int i = tid; i < E * K1; i += kThreads) cenc[i] = (double)__ldg(p.enc + (size_t)g * E * K1 + i);
  for (int i = tid; i < K * K1; i += kThreads)
    cdec[i] = (double)__ldg(p.dec + (size_t)g * K * K1 + i) + (double)__ldg(p.decl + (size_t)g * K * K1 + i);
  for (int i = tid; i < E; i += kThreads) cnul[i] = (double)__ldg(p.nul + (size_t)g * E + i);

  double acc[2][E][2];
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[mi][e][0] = acc[mi][e][1] = 0.0;

  const float* xg = p.x + (size_t)g * K * n_in;
  const float* rg = p.r + (size_t)g * n_in;
  const bool store_x = p.xsave != nullptr && mt == 0;
  {
    for (int c0 = 0; c0 < p.cin; c0 += KC) {
      __syncthreads();      // the previous chunk's fragments have been read (and the coefficient tables written)
      // rows of W as doubles
      for (int u = tid; u < rows * (KC / 4); u += kThreads) {
        const int row = u >> 2, c4 = (u & 3) * 4;
        float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mt * rows + row < p.cout && c0 + c4 < p.cin)
          w = __ldg(reinterpret_cast<const float4*>(p.W + (size_t)(mt * rows + row) * p.cin + c0 + c4));
        double* d = ws + (size_t)row * S + c4;
        d[0] = (double)w.x; d[1] = (double)w.y; d[2] = (double)w.z; d[3] = (double)w.w;
      }
      // Eq. 1 in fp64: the K+2 encodings of this chunk of the tile's pixels, two channels per thread
      // (wider units would not fit beside the accumulators in the register budget)
      for (int u = tid; u < P * (KC / 2); u += kThreads) {
        const int pix = u >> 3, c2 = (u & 7) * 2;
        const int gp = pt * P + pix;
        const bool ok = gp < p.npix && c0 + c2 < p.cin;
        const size_t off = (size_t)gp * p.cin + c0 + c2;
        float2 s[K1];
#pragma unroll
        for (int k = 0; k < K; ++k)
          s[k] = ok ? __ldg(reinterpret_cast<const float2*>(xg + (size_t)k * n_in + off)) : make_float2(0.f, 0.f);
        s[K] = ok ? __ldg(reinterpret_cast<const float2*>(rg + off)) : make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const double cr = cenc[e * K1 + K];
          double o0 = cr * (double)s[K].x, o1 = cr * (double)s[K].y;
#pragma unroll
          for (int k = 0; k < K; ++k) {
            const double ck = cenc[e * K1 + k];
            o0 = fma(ck, (double)s[k].x, o0);
            o1 = fma(ck, (double)s[k].y, o1);
          }
          *reinterpret_cast<double2*>(xs + ((size_t)e * P + pix) * S + c2) = make_double2(o0, o1);
          if (store_x && ok)
            *reinterpret_cast<float2*>(p.xsave + ((size_t)g * E + e) * n_in + off) = make_float2((float)o0, (float)o1);
        }
      }
      __syncthreads();
      const double* wa = ws + (size_t)(m16 * 16 + gq) * S + q;
      const double* xb = xs + (size_t)(pb * 8 + gq) * S + q;
#pragma unroll
      for (int ks = 0; ks < KC / 4; ++ks) {
        const double a0 = wa[ks * 4], a1 = wa[8 * S + ks * 4];
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const double b = xb[(size_t)e * P * S + ks * 4];
          dmma(acc[0][e], a0, b);
          dmma(acc[1][e], a1, b);
        }
      }
    }
    const int rowbase = mt * rows;

  // ---- epilogue: this thread holds, for rows r0 and r0 + 8 and pixels px and px + 1, all K+2 encoded outputs
  float sq[E];
#pragma unroll
  for (int e = 0; e < E; ++e) sq[e] = 0.f;
  float maxrho = 0.f;
  const float kInf = __int_as_float(0x7f800000);
#pragma unroll
  for (int mi = 0; mi < 2; ++mi) {
    const int row = rowbase + m16 * 16 + mi * 8 + gq;
    const double bd = (p.bias != nullptr && row < p.cout) ? (double)__ldg(p.bias + row) : 0.0;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int gp = pt * P + pb * 8 + 2 * q + j;
      const bool ok = row < p.cout && gp < p.npix;
      const long long oi = (long long)gp * p.cout + row;
      double v[E];
#pragma unroll
      for (int e = 0; e < E; ++e) v[e] = acc[mi][e][j];
      if (ok && g == p.f_group && oi == p.f_index) {
#pragma unroll
        for (int e = 0; e < E; ++e) v[e] += (e == p.f_enc) ? (double)p.f_delta : 0.0;
      }
      if (ok) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
          if (k >= p.kstore) continue;
          double yv = 0.0;
#pragma unroll
          for (int i = 0; i < K1; ++i) yv = fma(cdec[k * K1 + i], v[i], yv);
          p.y[((size_t)g * K + k) * n_out + oi] = (float)(yv + bd);
        }
        double rho = 0.0, sc = 0.0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          rho = fma(cnul[e], v[e], rho);
          sc = fma(fabs(cnul[e]), fabs(v[e]), sc);
          const float vf = (float)v[e];
          if (fabsf(vf) < kInf) sq[e] = fmaf(vf, vf, sq[e]);
        }
        const float ar = (float)fabs(rho), scf = (float)sc;
        maxrho = fmaxf(maxrho, ar);
        if (!(ar <= p.tau * scf) || !(scf < kInf)) {
          const unsigned int slot = atomicAdd(p.vs.count, 1u);
          if (slot < kCandCap) {
            Candidate cd;
            cd.index = (long long)g * n_out + oi;
            cd.absrho = ar;
            cd.s_e = scf;
            p.vs.cand[slot] = cd;
          }
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
    float t = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) t = lane == e ? sq[e] : t;
    if (lane < E && t != 0.f) atomicAdd(p.vs.sumsq + (size_t)g * E + lane, t);
  }
    if (lane == 0 && maxrho > 0.f) atomicMax(p.vs.maxrho + g, __float_as_int(maxrho));
  }
}

// Output-channel blocks of 16 per CTA (a power of two up to the warp count; the other warps take more pixels): the choice that
// minimises padded rows plus the encoding work repeated once per channel block.
int pick_mt16(int cout, int K) {
  int best = kWarps;
  long long best_cost = -1;
  for (int mt = kWarps; mt >= 1; mt >>= 1) {
    const long long blocks = (cout + 16 * mt - 1) / (16 * mt);
    const long long cost = blocks * (16 * mt + K + 1);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = mt; }
  }
  return best;
}

}  // namespace

bool fused64_supported(const Geom& g) {
  return g.kind == DK_CONV2D && g.layout == DK_NHWC && g.kh == 1 && g.kw == 1 && g.stride == 1 && g.pad == 0 &&
         (g.cin % 4) == 0;
}

dk_status launch_fused64(const Geom& g, const float* W, const float* x, const float* r, const CoefView& cv,
                         const float* bias, float* y, float* xsave, const VerifyScratch& vs, const dk_fault* fault,
                         int sm_count, cudaStream_t st) {
  F64Params p;
  p.W = W; p.x = x; p.r = r; p.bias = bias; p.y = y; p.xsave = xsave;
  p.enc = cv.enc; p.dec = cv.dec; p.decl = cv.decl; p.nul = cv.nul;
  p.vs = vs; p.tau = g.tol;
  p.cin = g.cin; p.cout = g.cout; p.npix = g.h * g.w; p.G = g.G;
  p.MT16 = pick_mt16(g.cout, g.K);
  p.PB = kWarps / p.MT16;
  const int P = 8 * p.PB;
  p.tiles_per_g = (p.npix + P - 1) / P;
  const int rows = 16 * p.MT16;
  p.mtiles = (g.cout + rows - 1) / rows;
  p.ntiles = (long long)p.tiles_per_g * g.G * p.mtiles;
  p.f_group = -1; p.f_enc = 0; p.f_index = -1; p.f_delta = 0.f;
  p.kstore = g.kstore;
  if (fault) { p.f_group = fault->group; p.f_enc = fault->enc; p.f_index = fault->out_index; p.f_delta = fault->delta; }
  const int E = g.E, K1 = g.K + 1;
  const size_t smem = ((size_t)E * P * S + (size_t)rows * S + (size_t)E * K1 + (size_t)g.K * K1 + E) * sizeof(double);
  (void)sm_count;
  if (p.ntiles > 0x7fffffffLL) return DK_ERR_SHAPE;
  dim3 grid((unsigned)p.ntiles);
#define DK_F64_CASE(KK)                                                                                    \
  case KK: {                                                                                               \
    if (smem > 48 * 1024)                                                                                  \
      DK_CUDA_CHECK(cudaFuncSetAttribute(fused64_kernel<KK>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                         (int)smem));                                                      \
    fused64_kernel<KK><<<grid, kThreads, smem, st>>>(p);                                                   \
  } break;
  switch (g.K) {
    DK_F64_CASE(1) DK_F64_CASE(2) DK_F64_CASE(3) DK_F64_CASE(4)
    DK_F64_CASE(5) DK_F64_CASE(6) DK_F64_CASE(7) DK_F64_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_F64_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

}  // namespace dk
