// Device side of the tensor-core path: PTX wrappers (TMA, mbarrier, tcgen05)
// and the persistent warp-specialised 3xTF32 implicit-GEMM kernel.
//
// Arithmetic.  Every fp32 operand v is split as v = hi + lo with
// hi = tf32(v), lo = tf32(v - hi) (round to nearest).  The product keeps
// W_hi*x_hi + W_hi*x_lo + W_lo*x_hi and drops W_lo*x_lo (~2^-22 relative).
// The tensor pipe adds into its fp32 accumulator with truncation; measured on
// B200, a contraction of length 4608 accumulated entirely in TMEM is off by
// 3.6e-5 (relative, max norm), which the decoder amplifies ~200x at noise
// sigma 100.  So TMEM only ever accumulates a short chunk of k-blocks; the
// epilogue warps add the chunks into fp32 registers with round-to-nearest.
//
// Tiling.  GEMM M = cout (128 rows of W per CTA tile = 128 TMEM lanes),
// N = encodings x pixels.  One N tile holds P output pixels for ALL K+2
// encodings of the same virtual batch(es): column e*P + p.  A thread of the
// epilogue owns one TMEM lane (one output channel) and half of the pixels,
// and sees every encoding of each of them: decoding and the redundant-equation
// residual are thread-local.  The P pixels are a box bw x bh x bg (columns,
// rows, groups) of the output; for filter tap (u,v) the operand tile is the
// same box of the channels-last input shifted by (u-pad, v-pad), fetched by
// one TMA box per encoding; out-of-image coordinates are zero-filled by the
// TMA unit, which implements the zero padding.
//
// Pipeline.  Persistent CTAs (one per SM): warp 0 issues TMA loads into a ring
// of shared-memory stages, warp 1 issues tcgen05.mma and commits, warps 4-11
// (two warpgroups, which take the registers warpgroup 0 gives up) drain the
// double-buffered TMEM accumulator chunk by chunk.  Every mbarrier
// wait is bounded; on expiry the CTA raises DK_ERR_TIMEOUT in the status
// word, lets in-flight copies land, frees TMEM and returns.
#pragma once

#include <cuda.h>

#include "dk_internal.h"
#include "dk_verify.cuh"

namespace dk {
namespace tc {

constexpr int BM = 128;            // output channels per tile = TMEM lanes
constexpr int kEpiWarps = 8;
constexpr int kThreadsTc = 32 * (4 + kEpiWarps);   // warpgroup 0: TMA, MMA, two idle warps
constexpr int kMaxStages = 8;
constexpr int MODE_YBAR = 0, MODE_DECODE = 1;

// Pixels per encoding in one N tile, by virtual-batch size: (K+2)*P is a legal
// UMMA N (multiple of 16, <= 256) and each epilogue thread keeps (K+2)*P/2
// accumulators in registers.
__host__ __device__ constexpr int tile_pixels(int K) {
  return K == 1 ? 64 : K == 2 ? 48 : (K == 3 || K == 4) ? 32 : 16;
}

struct TcParams {
  // tiling
  int bw, bh, bg;              // box shape of the P pixels (bw a power of two; bh too unless bg = 1)
  int log2_bw, log2_S;         // log2 of bw and of S = bw*bh
  int WT, HT, GT, MT;          // tiles along width, height, groups, cout
  int gt0;                     // first group tile of this launch (a call may be served by several launches, each
                               // covering GT group tiles from gt0 on)
  int ntiles;
  int KB, CB;                  // k-blocks in total and per filter tap
  int chunk;                   // most k-blocks accumulated in TMEM before promotion
  const unsigned char* chunk_tab;   // nullable, G <= kChunkTabMax entries: per virtual batch, the k-blocks (of 32
                               // contraction elements) its coefficients allow; copied to shared memory at start
  int chunk_mul;               // k-blocks per 32 contraction elements
  int ksplit, kb_per_split;    // contraction slices per tile (slices add into `out` with atomics)
  int kw, pad, stride;
  int nstages;
  int nstages_b;               // single-CTA forward kernel: 0 = one ring of stages (W tiles and activations together);
                               // n > 0 = two rings, `nstages` slots for the W tiles and n slots for the activations,
                               // filled by two producer warps (the activations run one k-block further ahead)
  unsigned spin_cap;           // polls after which a wait gives up
  int withhold;                // test hook: the producer arms its n-th stage but issues no copy (-1 = off)
  int hmul;                    // 2: the tile's rows 64-127 are the image row below rows 0-63 (cout <= 64), else 1
  int nprod;                   // 3: W_hi.x_hi + W_hi.x_lo + W_lo.x_hi; 2: W as one TF32 term, W_lo neither loaded nor used
  int b_onebox;                // 1 (tiles of one virtual batch, bg = 1): the encodings of a stage arrive as ONE box over the
                               // encoding dimension per TF32 term instead of one box per encoding
  int gbox;                    // 1 (with b_onebox; tiles of two virtual batches of P/2 pixels): that box spans both
                               // batches, so the tile's columns run batch-major (batch, encoding, pixel) within
                               // each CTA's share instead of (encoding, batch, pixel)
  unsigned int* pace;          // nullable: counter (zero at launch) that keeps the CTAs' walks over the tiles together
  int pace_every;              // tiles between two meetings on that counter
  int lo_inkernel;             // 1: the activations' second TF32 term is not loaded: two warps derive it in shared
                               // memory from the fp32 values the first copy brought (tf32(v - trunc(v)))
  // problem
  int cout, ho, wo, G;
  int kstore;                  // decoded rows k >= kstore of a group (noise vectors, Section 4.5) are neither computed nor stored
  long long n_out;
  // outputs / epilogue inputs
  float* out;                  // MODE_YBAR: ybar [G*E][ho][wo][cout]; MODE_DECODE: y [G*K][ho][wo][cout]
  const float* dec;
  const float* decl;
  const float* nul;
  const float* bias;
  VerifyScratch vs;
  float tau;
  int* status;                 // device word that receives DK_ERR_TIMEOUT
  // MODE_DECODE: when `verdict` is given, the CTA that finishes last takes the
  // final decisions of the check (`done` counts finished CTAs, starts at zero
  // and is left at zero)
  dk_verdict* verdict;
  unsigned int* done;
  // fault injection (MODE_DECODE): group < 0 disables
  int f_group, f_enc, f_co, f_oh, f_ow;
  float f_delta;
};

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the
// barrier did not complete within `cap` polls or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned cap) {
  for (unsigned i = 0; i < cap; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float to_tf32(float v) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
  return __uint_as_float(r);
}

// Shared-memory matrix descriptor of a K-major operand tile whose rows are
// SWZ bytes long (one swizzle span per row), rows packed, 8-row groups SWZ*8
// bytes apart.
template <int SWZ>
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  constexpr uint64_t layout = (SWZ == 128) ? 2ull : (SWZ == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;                             // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)((SWZ * 8) >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
  d |= layout << 61;
  return d;
}

// First accumulator column of encoding e for the `half`-th P/2 pixels of a tile.  `share` = encodings whose
// activations one CTA stages (all of them; half of them in a CTA pair).
template <int P>
__device__ __forceinline__ uint32_t tile_column(int gbox, int share, int e, int half) {
  const int r = e / share, el = e - r * share;
  return (uint32_t)(gbox ? (r * share * 2 + half * share + el) * (P / 2) : e * P + half * (P / 2));
}

// ---------------------------------------------------------------------------
// Epilogue of one tile, from the fp32 sums in registers: stores the encoded
// outputs (MODE_YBAR) or decodes them, evaluates the integrity residual and
// collects the statistics of the check (MODE_DECODE).  Thread (quad, lane)
// owns output channel `co`; `half` selects its PH of the tile's P pixels.
// ---------------------------------------------------------------------------
template <int MODE, int K>
__device__ __forceinline__ void tile_epilogue(const TcParams& p, float (&acc)[K + 2][tile_pixels(K) / 2], int half,
                                              int lane, int co, bool co_ok, int gt, int ht, int wt) {
  constexpr int E = K + 2, K1 = K + 1;
  constexpr int PH = tile_pixels(K) / 2;
  const int S = p.bw * p.bh;                    // pixels of one group inside the tile
  // position of this thread's j-th pixel; false when it lies outside the tensor
  auto locate = [&](int j, int& g, int& oh, int& ow) -> bool {
    const int pix = half * PH + j;
    // (S and bw are powers of two; a box of one group may have any height)
    const int gl = p.bg == 1 ? 0 : pix >> p.log2_S, rem = p.bg == 1 ? pix : pix & (S - 1);
    g = gt * p.bg + gl;
    oh = ht * p.bh + (rem >> p.log2_bw);
    ow = wt * p.bw + (rem & (p.bw - 1));
    return g < p.G && oh < p.ho && ow < p.wo;                  // warp-uniform
  };

  // A tile that lies inside one group (every convolution whose image has at
  // least P pixels) takes a branch-free walk over its pixels: the epilogue
  // warps are few, so their speed depends on independent instructions from
  // different pixels being in flight together.  Offsets fit 32 bits (n_out
  // is checked on the host).
  // The same walk serves a tile of several groups whose groups hold at least
  // PH pixels each (S and PH are powers of two): this thread's PH pixels then
  // lie in one group, `g1`.  A group past the last one leaves every pixel
  // invalid; its coefficients are read from the last group and not used.
  const bool one_group = S >= PH;
  const int g1raw = gt * p.bg + ((half * PH) >> p.log2_S);
  const bool g1_ok = g1raw < p.G;
  const int g1 = g1_ok ? g1raw : p.G - 1;
  const int oh0 = ht * p.bh, ow0 = wt * p.bw;
  auto pixel = [&](int j, int& off) -> bool {      // one_group only
    const int pix = p.bg == 1 ? half * PH + j : (half * PH + j) & (S - 1);
    const int oh = oh0 + (pix >> p.log2_bw), ow = ow0 + (pix & (p.bw - 1));
    off = (oh * p.wo + ow) * p.cout;
    return oh < p.ho && ow < p.wo && g1_ok;
  };

  if (MODE == MODE_YBAR) {
    if (one_group) {
      float* base = p.out + ((size_t)g1 * E) * p.n_out + co;
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        int off;
        const bool ok = pixel(j, off) && co_ok;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          float* dst = base + (size_t)e * p.n_out + off;
          if (ok) {
            if (p.ksplit > 1) atomicAdd(dst, acc[e][j]);   // `out` was cleared
            else *dst = acc[e][j];
          }
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        int g, oh, ow;
        if (locate(j, g, oh, ow) && co_ok) {
          float* dst = p.out + ((size_t)g * E) * p.n_out + ((size_t)oh * p.wo + ow) * p.cout + co;
#pragma unroll
          for (int e = 0; e < E; ++e) {
            if (p.ksplit > 1) atomicAdd(dst + (size_t)e * p.n_out, acc[e][j]);   // `out` was cleared
            else dst[(size_t)e * p.n_out] = acc[e][j];
          }
        }
      }
    }
  } else {
    if (p.f_group >= 0 && co == p.f_co) {      // fault hook: one element of one encoding
      // (the per-encoding addend is formed first so that the accumulators
      // are only ever indexed with compile-time constants)
      float fd[E];
#pragma unroll
      for (int e = 0; e < E; ++e) fd[e] = (e == p.f_enc) ? p.f_delta : 0.f;
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        int g, oh, ow;
        const bool hit = locate(j, g, oh, ow) && g == p.f_group && oh == p.f_oh && ow == p.f_ow;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e][j] += hit ? fd[e] : 0.f;
      }
    }
    if (one_group) {
      const int g = g1;
      const float bias_co = (p.bias != nullptr && co_ok) ? __ldg(p.bias + co) : 0.f;
      // Offsets and validity of this thread's pixels, once; sums of pixels outside
      // the tensor (or of a channel past cout) are cleared so that the passes
      // below need no further selects.  The instruction count of this epilogue
      // is what bounds layers with a short contraction, so each pass is kept to
      // the arithmetic it cannot avoid.
      int off[PH];
      uint32_t okm = 0;
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        const bool ok = pixel(j, off[j]) && co_ok;
        okm |= (uint32_t)ok << j;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e][j] = ok ? acc[e][j] : 0.f;
      }
      // decoded rows (Eq. 2).  One fp32 coefficient per term: the fp32 sums'
      // own rounding is as large as the second float of the coefficient pair
      // would contribute.
#pragma unroll
      for (int k = 0; k < K; ++k) {
        if (k >= p.kstore) continue;
        float ck[K1];
#pragma unroll
        for (int i = 0; i < K1; ++i) ck[i] = __ldg(p.dec + ((size_t)g * K + k) * K1 + i);
        float* base = p.out + ((size_t)g * K + k) * p.n_out + co;
#pragma unroll
        for (int j = 0; j < PH; ++j) {
          float yv = ck[0] * acc[0][j];
#pragma unroll
          for (int i = 1; i < K1; ++i) yv = fmaf(ck[i], acc[i][j], yv);
          if ((okm >> j) & 1u) base[off[j]] = yv + bias_co;
        }
      }
      // integrity residual, statistics and candidates
      float nv[E], sq[E];
#pragma unroll
      for (int e = 0; e < E; ++e) { nv[e] = __ldg(p.nul + (size_t)g * E + e); sq[e] = 0.f; }
      const float kInf = __int_as_float(0x7f800000);
      float maxrho = 0.f;
      uint32_t bad = 0;
      auto residual = [&](int j, float& ar, float& sc) {
        float rho = 0.f;
        sc = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          rho = fmaf(nv[e], acc[e][j], rho);
          sc = fmaf(fabsf(nv[e]), fabsf(acc[e][j]), sc);
        }
        ar = fabsf(rho);
      };
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        float ar, sc;
        residual(j, ar, sc);
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const float vf = fabsf(acc[e][j]) < kInf ? acc[e][j] : 0.f;     // non-finite values stay out of the rms
          sq[e] = fmaf(vf, vf, sq[e]);
        }
        maxrho = fmaxf(maxrho, ar);
        bad |= (uint32_t)(!(ar <= p.tau * sc) || !(sc < kInf)) << j;
      }
      if (bad != 0u) {       // rare: append the candidates
#pragma unroll
        for (int j = 0; j < PH; ++j)
          if ((bad >> j) & 1u) {
            float ar, sc;
            residual(j, ar, sc);
            unsigned int slot = atomicAdd(p.vs.count, 1u);
            if (slot < kCandCap) {
              Candidate cd;
              cd.index = (long long)g * p.n_out + off[j] + co;
              cd.absrho = ar;
              cd.s_e = sc;
              p.vs.cand[slot] = cd;
            }
          }
      }
      // warp sums of the E statistics and the maximum, the butterflies interleaved
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int e = 0; e < E; ++e) sq[e] += __shfl_xor_sync(0xffffffffu, sq[e], o);
        maxrho = fmaxf(maxrho, __shfl_xor_sync(0xffffffffu, maxrho, o));
      }
      {      // lane e adds statistic e
        float t = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) t = lane == e ? sq[e] : t;
        if (lane < E && t != 0.f) atomicAdd(p.vs.sumsq + (size_t)g * E + lane, t);
      }
      if (lane == 0 && maxrho > 0.f) atomicMax(p.vs.maxrho + g, __float_as_int(maxrho));
    } else {
      // The epilogue walks the pixels once per decoded row and once for the
      // integrity residual, so that only one row of coefficients is live at a
      // time; a row is re-read only when the group changes, and a tile of a
      // convolution usually lies inside one group.
      const float bias_co = (p.bias != nullptr && co_ok) ? __ldg(p.bias + co) : 0.f;
#pragma unroll
      for (int k = 0; k < K; ++k) {
        if (k >= p.kstore) continue;
        int cg = -1;
        float ch[K1], cl[K1];
#pragma unroll
        for (int j = 0; j < PH; ++j) {
          int g, oh, ow;
          if (!locate(j, g, oh, ow)) continue;
          if (g != cg) {
            const float* gh = p.dec + ((size_t)g * K + k) * K1;
            const float* gl = p.decl + ((size_t)g * K + k) * K1;
#pragma unroll
            for (int i = 0; i < K1; ++i) { ch[i] = __ldg(gh + i); cl[i] = __ldg(gl + i); }
            cg = g;
          }
          float hi = 0.f, lo = 0.f;
#pragma unroll
          for (int i = 0; i < K1; ++i) {
            lo = fmaf(cl[i], acc[i][j], lo);
            hi = fmaf(ch[i], acc[i][j], hi);
          }
          if (co_ok)
            p.out[((size_t)g * K + k) * p.n_out + ((size_t)oh * p.wo + ow) * p.cout + co] = (hi + lo) + bias_co;
        }
      }
      // integrity residual, statistics and candidates
      float sq[E], nv[E];
#pragma unroll
      for (int e = 0; e < E; ++e) sq[e] = 0.f;
      float maxrho = 0.f;
      int cur_g = -1, cg = -1;
      auto flush_stats = [&](int g) {
        if (g < 0) return;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          float s = sq[e];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if (lane == 0 && s != 0.f) atomicAdd(p.vs.sumsq + (size_t)g * E + e, s);
          sq[e] = 0.f;
        }
        float m = maxrho;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0 && m > 0.f) atomicMax(p.vs.maxrho + g, __float_as_int(m));
        maxrho = 0.f;
      };
      const float kInf = __int_as_float(0x7f800000);
#pragma unroll
      for (int j = 0; j < PH; ++j) {
        int g, oh, ow;
        const bool in_range = locate(j, g, oh, ow);
        if (g != cur_g) {      // warp-uniform: g depends on the tile and the pixel only
          flush_stats(cur_g);
          cur_g = (g < p.G) ? g : -1;
        }
        if (!in_range) continue;
        if (g != cg) {
#pragma unroll
          for (int e = 0; e < E; ++e) nv[e] = __ldg(p.nul + (size_t)g * E + e);
          cg = g;
        }
        float rho = 0.f, sc = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const float v = co_ok ? acc[e][j] : 0.f;
          rho = fmaf(nv[e], v, rho);
          sc = fmaf(fabsf(nv[e]), fabsf(v), sc);
          if (fabsf(v) < kInf) sq[e] = fmaf(v, v, sq[e]);
        }
        const float ar = fabsf(rho);
        maxrho = fmaxf(maxrho, ar);
        if (co_ok && (!(ar <= p.tau * sc) || !(sc < kInf))) {
          unsigned int slot = atomicAdd(p.vs.count, 1u);
          if (slot < kCandCap) {
            Candidate cd;
            cd.index = (long long)g * p.n_out + ((long long)oh * p.wo + ow) * p.cout + co;
            cd.absrho = ar;
            cd.s_e = sc;
            p.vs.cand[slot] = cd;
          }
        }
      }
      flush_stats(cur_g);
    }
  }
}
// ---------------------------------------------------------------------------
// After its last tile a CTA's 256 epilogue threads (tid 0..255) come here.  The
// CTA that arrives last has every statistic of the integrity check in front of
// it and writes the verdict, which saves the separate one-block launch.
// `alive` = false: this warp's wait expired; the status is raised before the
// count so that whoever decides sees it.
// ---------------------------------------------------------------------------
// k-blocks a tile accumulates in tensor memory between promotions: the accumulator truncates when it adds, and
// the decoder multiplies that error by the amplification of the tile's coefficient sets, so ill-conditioned
// virtual batches take shorter chunks (table from the host, see upload_coefficients).  `tab` = the table in shared
// memory; t = tile index.
constexpr int kChunkTabMax = 1024;
__device__ __forceinline__ void load_chunk_tab(const TcParams& p, unsigned char* tab) {
  if (p.chunk_tab == nullptr) return;
  for (int i = threadIdx.x; i < p.G && i < kChunkTabMax; i += blockDim.x) tab[i] = __ldg(p.chunk_tab + i);
}
__device__ __forceinline__ int tile_chunk(const TcParams& p, const unsigned char* tab, int t) {
  if (p.chunk_tab == nullptr) return p.chunk;
  const int gt = p.gt0 + (t / p.MT) / (p.WT * p.HT);
  const int g0 = gt * p.bg, g1 = min(p.G, g0 + p.bg);
  int c = p.chunk;
  for (int g = g0; g < g1; ++g) c = min(c, (int)tab[g] * p.chunk_mul);
  return max(c, 1);
}

template <int MODE, int K>
__device__ __forceinline__ void tail_finalize(const TcParams& p, int tid, bool alive, volatile int* last_flag) {
  if (MODE != MODE_DECODE || p.verdict == nullptr) return;
  if (!alive && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
  __threadfence();
  asm volatile("bar.sync 1, 256;" ::: "memory");
  if (tid == 0) *last_flag = (atomicAdd(p.done, 1u) == gridDim.x - 1) ? 1 : 0;
  asm volatile("bar.sync 1, 256;" ::: "memory");
  if (*last_flag) {
    __threadfence();
    verify_finalize_block(tid, p.vs.sumsq, p.vs.maxrho, p.vs.count, p.vs.cand, p.nul, p.verdict, p.G, K + 2,
                          p.n_out, p.tau);
    if (tid == 0) *p.done = 0u;
  }
}

// ---------------------------------------------------------------------------
// the GEMM kernel
// ---------------------------------------------------------------------------
template <int BK, int MODE, int K>
__global__ void __launch_bounds__(kThreadsTc, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
              const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
              const TcParams p) {
  constexpr int E = K + 2;
  constexpr int P = tile_pixels(K), PH = P / 2;
  constexpr int BN = E * P;
  constexpr int SWZ = BK * 4;
  constexpr int A_BYTES = BM * BK * 4;
  constexpr int B_BYTES = BN * BK * 4;
  constexpr int STAGE_BYTES = 2 * (A_BYTES + B_BYTES);
  static_assert(BN % 16 == 0 && BN <= 256 && PH % 8 == 0, "illegal tile");
  extern __shared__ unsigned char smem_raw[];
  __shared__ unsigned char s_chunk[kChunkTabMax];      // chunk lengths per virtual batch (see tile_chunk)
  load_chunk_tab(p, s_chunk);
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  // One ring: stage s = [W_hi][W_lo][x_hi][x_lo] at s * STAGE_BYTES.  Two rings: the W tiles' slots first, then the
  // activations' slots.
  const bool split = p.nstages_b > 0;
  unsigned char* const b_base = split ? smem + (size_t)p.nstages * 2 * A_BYTES : smem + 2 * A_BYTES;
  const size_t a_pitch = split ? (size_t)2 * A_BYTES : (size_t)STAGE_BYTES;
  const size_t b_pitch = split ? (size_t)2 * B_BYTES : (size_t)STAGE_BYTES;
  unsigned char* ctrl = split ? b_base + (size_t)p.nstages_b * 2 * B_BYTES : smem + (size_t)p.nstages * STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctrl);
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tfull_bar = empty_bar + kMaxStages;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint64_t* ready_bar = tempty_bar + 2;        // a stage's second term has been derived (one arrival per converter warp)
  uint64_t* bfull_bar = ready_bar + kMaxStages;      // the activations' ring, when there are two
  uint64_t* bempty_bar = bfull_bar + kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bempty_bar + kMaxStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nwork = p.ntiles * p.ksplit;     // work item = (tile, contraction slice)

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.nstages; ++s) {
      mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); mbar_init(ready_bar + s, 2);
    }
    for (int s = 0; s < p.nstages_b; ++s) { mbar_init(bfull_bar + s, 1); mbar_init(bempty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Register re-partitioning.  The CTA's register pool is fixed at launch
  // (168 per thread x 384 threads for this launch bound); setmaxnreg.inc BLOCKS
  // until the pool can serve it, so the two requests below must fit the pool.
  static_assert(40 * 128 + 232 * 256 <= 168 * kThreadsTc, "setmaxnreg budget exceeds the CTA's register pool");
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
  if (warp == 0 || (warp == 2 && split)) {
    // ---------------- TMA producer(s) ----------------
    // The whole warp runs the loop: lane 0 waits for the slot and arms its barrier, then one lane per copy
    // issues it, so that the copies of a k-block go out side by side.  One ring: warp 0 fetches everything.
    // Two rings: warp 0 fetches the W tiles into theirs, warp 2 the activations into theirs.
    {
      const bool do_a = warp == 0, do_b = !split || warp == 2;
      uint64_t* const fbar = (split && warp == 2) ? bfull_bar : full_bar;
      uint64_t* const ebar = (split && warp == 2) ? bempty_bar : empty_bar;
      const int nst = (split && warp == 2) ? p.nstages_b : p.nstages;
      const uint32_t tx = (do_a ? (uint32_t)(p.nprod == 2 ? A_BYTES : 2 * A_BYTES) : 0u) +
                          (do_b ? (uint32_t)(p.lo_inkernel ? B_BYTES : 2 * B_BYTES) : 0u);
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool alive = true;
      int round = 0;
      for (int w = blockIdx.x; alive && w < nwork; w += gridDim.x, ++round) {
        // Pace.  The CTAs walk the tiles side by side (tile = CTA + round * grid), so the tiles in flight are
        // neighbours in the image and share their halo rows through L2 -- while the CTAs stay together.  Over
        // hundreds of rounds they drift apart and the halo is fetched from DRAM again (measured on a 224 x 224
        // layer: 1.02 x the operands' bytes with 42 rounds, 1.55 x with 339).  So every pace_every rounds a CTA
        // goes on only when all have issued the loads of the round before, or after a bounded wait: a hint,
        // never a condition for progress.  (A CTA that waits here has a tile left, so every CTA had one in the
        // round before and has counted.)
        if (p.pace != nullptr && do_a && lane == 0 && round > 0 && round % p.pace_every == 0) {
          const unsigned int target = (unsigned int)(round / p.pace_every) * gridDim.x;
          for (int spin = 0; spin < 4096 && *reinterpret_cast<volatile unsigned int*>(p.pace) < target; ++spin)
            __nanosleep(64);
        }
        const int t = w / p.ksplit, ks = w - t * p.ksplit;
        const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
        const int mt = t % p.MT;
        int nt = t / p.MT;
        const int wt = nt % p.WT; nt /= p.WT;
        const int ht = nt % p.HT;
        const int gt = p.gt0 + nt / p.HT;
        const int x0 = wt * p.bw * p.stride - p.pad, y0 = ht * p.bh * p.hmul * p.stride - p.pad;     // input position of tap (0,0)
        const int g0 = gt * p.bg, m0 = mt * BM;
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          int ok = 1;
          if (lane == 0) {
            ok = mbar_wait(ebar + stage, phase ^ 1u, abort_flag, p.spin_cap) ? 1 : 0;
            if (ok) mbar_expect_tx(fbar + stage, tx);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) { alive = false; break; }
          if (do_a && issued++ == p.withhold) { alive = false; break; }      // test hook: armed, nothing copied
          const int tap = kb / p.CB, c0 = (kb - tap * p.CB) * BK;
          const int u = tap / p.kw, v = tap - u * p.kw;
          unsigned char* sta = smem + (size_t)stage * a_pitch;
          unsigned char* stb = b_base + (size_t)stage * b_pitch;
          constexpr int SUB = P * BK * 4;
          if (lane == 0) {
            if (do_a) tma_load_3d(sta, &map_a_hi, fbar + stage, c0, tap, m0);
          } else if (lane == 1) {
            if (do_a && p.nprod == 3) tma_load_3d(sta + A_BYTES, &map_a_lo, fbar + stage, c0, tap, m0);
          } else if (!do_b) {
          } else if (p.b_onebox) {
            // (same bytes at the same places as the E boxes below: with one group per tile the encoding is the
            // slowest dimension of the stage either way; fewer copies measured 4-7 % faster)
            if (lane == 2) tma_load_5d(stb, &map_b_hi, fbar + stage, c0, x0 + v, y0 + u, 0, g0);
            else if (lane == 3 && !p.lo_inkernel)
              tma_load_5d(stb + B_BYTES, &map_b_lo, fbar + stage, c0, x0 + v, y0 + u, 0, g0);
          } else if (lane < 2 + 2 * E) {
            const int e = (lane - 2) >> 1;
            if ((lane & 1) == 0)
              tma_load_5d(stb + e * SUB, &map_b_hi, fbar + stage, c0, x0 + v, y0 + u, e, g0);
            else if (!p.lo_inkernel)
              tma_load_5d(stb + B_BYTES + e * SUB, &map_b_lo, fbar + stage, c0, x0 + v, y0 + u, e, g0);
          }
          __syncwarp();
          if (++stage == nst) { stage = 0; phase ^= 1u; }
        }
        // (the last round before a meeting: this CTA's loads of it are out)
        if (p.pace != nullptr && alive && do_a && lane == 0 && (round + 1) % p.pace_every == 0) atomicAdd(p.pace, 1u);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                 ((uint32_t)(BM >> 4) << 24);
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      uint32_t acc_it = 0;     // chunks issued so far (all tiles)
      bool alive = true;
      for (int w = blockIdx.x; alive && w < nwork; w += gridDim.x) {
        const int ks = w % p.ksplit;
        const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
        const int chunk = tile_chunk(p, s_chunk, w / p.ksplit);
        const int nchunks = (kb_hi - kb_lo + chunk - 1) / chunk;
        for (int ci = 0; alive && ci < nchunks; ++ci, ++acc_it) {
          const uint32_t buf = acc_it & 1u, aphase = (acc_it >> 1) & 1u;
          if (!mbar_wait(tempty_bar + buf, aphase ^ 1u, abort_flag, p.spin_cap)) { alive = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * 256u;
          const int kb_beg = kb_lo + ci * chunk, kb_end = min(kb_hi, kb_beg + chunk);
          for (int kb = kb_beg; kb < kb_end; ++kb) {
            if (!mbar_wait(full_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
            if (split && !mbar_wait(bfull_bar + stage_b, phase_b, abort_flag, p.spin_cap)) { alive = false; break; }
            tc_fence_after();
            const uint32_t sta = smem_u32(smem + (size_t)stage * a_pitch);
            const uint32_t stb = smem_u32(b_base + (size_t)(split ? stage_b : stage) * b_pitch);
            const uint64_t a_hi = make_desc<SWZ>(sta), a_lo = make_desc<SWZ>(sta + A_BYTES);
            const uint64_t b_hi = make_desc<SWZ>(stb);
            const uint64_t b_lo = make_desc<SWZ>(stb + B_BYTES);
            const bool first = kb == kb_beg;
            // the products that need only what the copies brought go first; the one with the activations' second
            // term follows, after the converter warps have derived it (when they do)
#pragma unroll
            for (int kk = 0; kk < BK / 8; ++kk) {
              const uint64_t adv = (uint64_t)(kk * 2);     // 32 bytes per k-step, in 16-byte units
              tc_mma_tf32(d_tmem, a_hi + adv, b_hi + adv, idesc, (first && kk == 0) ? 0u : 1u);
              if (p.nprod == 3) tc_mma_tf32(d_tmem, a_lo + adv, b_hi + adv, idesc, 1u);
            }
            if (p.lo_inkernel) {
              if (!mbar_wait(ready_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
              tc_fence_after();
            }
#pragma unroll
            for (int kk = 0; kk < BK / 8; ++kk) {
              const uint64_t adv = (uint64_t)(kk * 2);
              tc_mma_tf32(d_tmem, a_hi + adv, b_lo + adv, idesc, 1u);
            }
            tc_commit(empty_bar + stage);
            if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
            if (split) {
              tc_commit(bempty_bar + stage_b);
              if (++stage_b == p.nstages_b) { stage_b = 0; phase_b ^= 1u; }
            }
          }
          if (alive) tc_commit(tfull_bar + buf);
        }
      }
    }
  } else if (p.lo_inkernel) {
    // ---------------- converters: warps 2 and 3 ----------------
    // second TF32 term of the stage's activations, element by element in place of the copy that used to bring
    // it (the swizzled position of an element is the same in both halves of the stage)
    const int ctid = (int)threadIdx.x - 64;
    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;
    for (int w = blockIdx.x; alive && w < nwork; w += gridDim.x) {
      const int ks = w % p.ksplit;
      const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        if (!mbar_wait(full_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
        const float4* src = reinterpret_cast<const float4*>(b_base + (size_t)stage * b_pitch);
        float4* dst = reinterpret_cast<float4*>(b_base + (size_t)stage * b_pitch + B_BYTES);
#pragma unroll 4
        for (int i = ctid; i < B_BYTES / 16; i += 64) {
          const float4 v = src[i];
          float4 l;
          l.x = to_tf32(v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u));
          l.y = to_tf32(v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u));
          l.z = to_tf32(v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u));
          l.w = to_tf32(v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u));
          dst[i] = l;
        }
        // make the stores visible to the tensor core's (asynchronous-proxy) reads, then hand the stage over
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(ready_bar + stage);
        if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
    // ---------------- epilogue: warps 4..11 ----------------
    const int quad = warp & 3;                    // TMEM lane quadrant this warp may read
    const int half = (warp - 4) >> 2;             // which half of the tile's pixels
    uint32_t acc_it = 0;
    bool alive = true;
    float acc[E][PH];
    for (int w = blockIdx.x; alive && w < nwork; w += gridDim.x) {
      const int t = w / p.ksplit, ks = w - t * p.ksplit;
      const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
      const int chunk = tile_chunk(p, s_chunk, t);
      const int nchunks = (kb_hi - kb_lo + chunk - 1) / chunk;
      const int mt = t % p.MT;
      int nt = t / p.MT;
      const int wt = nt % p.WT; nt /= p.WT;
      const int ht = nt % p.HT;
      const int gt = p.gt0 + nt / p.HT;
      // (two-row tiles: lanes 64-127 hold the same output channels for the image row below)
      const int co = p.hmul == 2 ? (quad & 1) * 32 + lane : mt * BM + quad * 32 + lane;
      const int ht_e = p.hmul == 2 ? 2 * ht + (quad >> 1) : ht;
      const bool co_ok = co < p.cout;

      // ---- sum the chunks of this tile in registers (round to nearest) ----
      for (int ci = 0; ci < nchunks; ++ci, ++acc_it) {
        const uint32_t buf = acc_it & 1u, aphase = (acc_it >> 1) & 1u;
        if (!mbar_wait(tfull_bar + buf, aphase, abort_flag, p.spin_cap)) { alive = false; break; }
        tc_fence_after();
        const uint32_t tbase = tmem_base + buf * 256u + ((uint32_t)(quad * 32) << 16);
        constexpr int EB = 2;      // encodings per round trip to tensor memory
#pragma unroll
        for (int e0 = 0; e0 < E; e0 += EB) {
          float tmp[EB][PH];
#pragma unroll
          for (int de = 0; de < EB; ++de)
            if (e0 + de < E) {
              const uint32_t col = tile_column<P>(p.gbox, E, e0 + de, half);
#pragma unroll
              for (int c = 0; c < PH; c += 8) tc_ld8(tbase + col + (uint32_t)c, &tmp[de][c]);
            }
          tc_wait_ld();
#pragma unroll
          for (int de = 0; de < EB; ++de)
            if (e0 + de < E) {
#pragma unroll
              for (int j = 0; j < PH; ++j)
                acc[e0 + de][j] = (ci == 0) ? tmp[de][j] : acc[e0 + de][j] + tmp[de][j];
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar + buf);
      }
      if (!alive) break;

      tile_epilogue<MODE, K>(p, acc, half, lane, co, co_ok, gt, ht_e, wt);
    }
    tail_finalize<MODE, K>(p, (int)threadIdx.x - 128, alive, abort_flag + 1);
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a bounded wait expired: report, give copies still in flight time to land
    if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace tc
}  // namespace dk
