// Host side of the tensor-core path: tensor maps, tile planning, launches, and
// the HBM-bound pre-passes that write the TF32 hi/lo split operands.
#include <cuda.h>

#include <new>

#include "dk_internal.h"
#include "dk_tc_kernel.cuh"
#include "dk_tc_pair.cuh"
#include "dk_tc_wgrad.cuh"

namespace dk {
namespace {

using namespace tc;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct TcState {
  EncodeTiledFn encode;
  int smem_optin;
  int device;
  Options* opt;             // the context's options (dk_set_option)
};

// What the launch of one kernel instantiation needs to know about it, looked
// up once per device instead of on every call (each query costs microseconds
// of host time, which small layers cannot hide).
constexpr int kMaxDevices = 64;
struct KernelCache {
  int regs[kMaxDevices];          // registers per thread, 0 = not queried yet
  size_t smem[kMaxDevices];       // dynamic shared memory limit already set
  int pairs[kMaxDevices];         // resident CTA pairs, 0 = not queried yet
};

// Checks the register pool the kernel's setmaxnreg split relies on and raises
// the dynamic shared memory limit to `smem` when it is not there yet.
template <typename Kern>
dk_status prepare_kernel(Kern kern, KernelCache& kc, int dev, size_t smem) {
  if (dev < 0 || dev >= kMaxDevices) return DK_ERR_UNSUPPORTED;
  if (kc.regs[dev] == 0) {
    cudaFuncAttributes fa;
    DK_CUDA_CHECK(cudaFuncGetAttributes(&fa, kern));
    kc.regs[dev] = fa.numRegs;
  }
  // The kernels re-partition registers between their warpgroups and would wait
  // forever if the pool they were launched with were smaller than they assume.
  if (kc.regs[dev] * kThreadsTc < 40 * 128 + 232 * 256) return DK_ERR_UNSUPPORTED;
  if (kc.smem[dev] < smem) {
    DK_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kc.smem[dev] = smem;
  }
  return DK_OK;
}

// CTA pairs of `kern` that can be resident together (a GPC with an odd number
// of SMs leaves one out), at most sm_count / 2.
template <typename Kern>
int resident_pairs(Kern kern, KernelCache& kc, int dev, size_t smem, int sm_count, bool cluster_attr) {
  if (kc.pairs[dev] == 0) {
    int pairs = sm_count / 2;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(kThreadsTc);
    cfg.dynamicSmemBytes = smem;
    if (cluster_attr) { cfg.attrs = &attr; cfg.numAttrs = 1; }
    int active = 0;
    if (cudaOccupancyMaxActiveClusters(&active, kern, &cfg) == cudaSuccess && active > 0 && active < pairs)
      pairs = active;
    else
      (void)cudaGetLastError();
    kc.pairs[dev] = pairs;
  }
  return kc.pairs[dev];
}

constexpr int kSwz128Atom32 = 1128;

// k-block of the forward kernel: 32 fp32 (128-byte rows, fewer and larger
// stages) or 16 (64-byte rows, twice as many stages in the same shared memory)
int fwd_bk(const TcState* ts) { return ts->opt->v[DK_OPT_TC_BK] == 16 ? 16 : 32; }

// ---------------------------------------------------------------------------
// HBM-bound pre-passes: TF32 hi/lo split, alone or fused with the encoder
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
split_tf32_kernel(const float4* __restrict__ src, float4* __restrict__ hi, float4* __restrict__ lo, long long n4,
                  int raw) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    float4 v = __ldg(src + i), h, l;
    if (raw) {
      // only the second term; the reader takes src itself as the first (the tensor core ignores the 13 low
      // mantissa bits of a TF32 operand, i.e. it sees trunc(src))
      l.x = to_tf32(v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u));
      l.y = to_tf32(v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u));
      l.z = to_tf32(v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u));
      l.w = to_tf32(v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u));
      lo[i] = l;
      continue;
    }
    h.x = to_tf32(v.x); l.x = to_tf32(v.x - h.x);
    h.y = to_tf32(v.y); l.y = to_tf32(v.y - h.y);
    h.z = to_tf32(v.z); l.z = to_tf32(v.z - h.z);
    h.w = to_tf32(v.w); l.w = to_tf32(v.w - h.w);
    hi[i] = h;
    lo[i] = l;
  }
}

// Eq. 1 with the split fused in: reads the K inputs and the noise once,
// writes the K+2 encodings as hi/lo pairs (and in full when `full` is given).
template <int K>
__global__ void __launch_bounds__(256)
encode_split_kernel(const float* __restrict__ x, const float* __restrict__ r, const float* __restrict__ enc,
                    float* __restrict__ full, float* __restrict__ hi, float* __restrict__ lo, long long n) {
  constexpr int K1 = K + 1, E = K + 2;
  const int g = blockIdx.y;
  float c[E][K1];
#pragma unroll
  for (int i = 0; i < E; ++i)
#pragma unroll
    for (int k = 0; k < K1; ++k) c[i][k] = __ldg(enc + ((size_t)g * E + i) * K1 + k);
  const float* xg = x + (size_t)g * K * n;
  const float* rg = r + (size_t)g * n;
  const size_t ob = (size_t)g * E * n;
  const long long n4 = n / 4;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += (long long)gridDim.x * blockDim.x) {
    float4 s[K1];
#pragma unroll
    for (int k = 0; k < K; ++k) s[k] = __ldg(reinterpret_cast<const float4*>(xg + (size_t)k * n) + q);
    s[K] = __ldg(reinterpret_cast<const float4*>(rg) + q);
#pragma unroll
    for (int i = 0; i < E; ++i) {
      float4 o, h, l;
      o.x = c[i][K] * s[K].x; o.y = c[i][K] * s[K].y; o.z = c[i][K] * s[K].z; o.w = c[i][K] * s[K].w;
#pragma unroll
      for (int k = 0; k < K; ++k) {
        o.x = fmaf(c[i][k], s[k].x, o.x); o.y = fmaf(c[i][k], s[k].y, o.y);
        o.z = fmaf(c[i][k], s[k].z, o.z); o.w = fmaf(c[i][k], s[k].w, o.w);
      }
      h.x = to_tf32(o.x); l.x = to_tf32(o.x - h.x);
      h.y = to_tf32(o.y); l.y = to_tf32(o.y - h.y);
      h.z = to_tf32(o.z); l.z = to_tf32(o.z - h.z);
      h.w = to_tf32(o.w); l.w = to_tf32(o.w - h.w);
      const size_t off = ob + (size_t)i * n;
      if (full != nullptr) reinterpret_cast<float4*>(full + off)[q] = o;
      reinterpret_cast<float4*>(hi + off)[q] = h;
      reinterpret_cast<float4*>(lo + off)[q] = l;
    }
  }
}

// ---------------------------------------------------------------------------
// tile planning
// ---------------------------------------------------------------------------
struct Tiling {
  int P, bw, bh, bg, WT, HT, GT, MT, ntiles, KB, CB, nstages, BN;
  int nstages_b;           // single-CTA kernel: slots of a separate ring for the activations (0: one ring)
  size_t smem_one_ring;    // dynamic shared memory of the one-ring layout (the kernel derives the second term itself)
  bool mpack;              // two output rows of the image in one 128-row tile (cout <= 64)
  bool pair;               // tiles of 256 output channels on CTA pairs
  size_t smem_bytes;
};

// Tiles whose activations arrive as one box over the encodings per TF32 term: those of one virtual batch, and
// those of two batches of P/2 pixels (the box then spans both, see TcParams::gbox)
bool onebox_tiles(const Tiling& t) { return t.bg == 1 || (t.bg == 2 && t.bw * t.bh * 2 == t.P); }

template <int BK>
bool plan_tiling(const Geom& g, int smem_optin, Tiling* t, bool pair = false) {
  const int E = g.E;
  const int P = tile_pixels(g.K);
  // Box shape bw x bh x bg with bw*bh*bg = P (bw, bh powers of two): the one
  // that covers the fewest out-of-range positions, weighted by what its
  // epilogue and copies cost; ties go to wider rows.
  t->P = P;
  t->bw = t->bh = t->bg = 1;
  long long best = -1;
  for (int bw = 1; bw <= P; bw *= 2)
    for (int bh = 1; bw * bh <= P; ++bh) {
      if (P % (bw * bh)) continue;
      const int bg = P / (bw * bh);
      if (bg > 256) continue;
      // (a height that is no power of two, e.g. 16 x 3 of the 48 pixels at K = 2, only for boxes of one virtual
      // batch: the epilogue's walk over several batches splits pixel indices with shifts and masks)
      if ((bh & (bh - 1)) != 0 && bg != 1) continue;
      long long cost = (long long)((g.wo + bw - 1) / bw) * bw * ((g.ho + bh - 1) / bh) * bh *
                       ((g.G + bg - 1) / bg) * bg * 64;
      // (measured on 28x28 and 14x14 images: a tile whose epilogue threads each span several groups runs ~30 %
      // longer than one with 12 % of its positions out of range; per-encoding boxes cost a few per cent)
      if (bw * bh < P / 2) cost += cost * 5 / 16;
      else if (bg > 1) cost += cost / 32;
      if (best < 0 || cost < best || (cost == best && (bw > t->bw || (bw == t->bw && bh > t->bh)))) {
        best = cost; t->bw = bw; t->bh = bh; t->bg = bg;
      }
    }
  if (best < 0) return false;
  t->mpack = g.mpack != 0 && !pair;
  if (t->mpack) { t->bw = P; t->bh = 1; t->bg = 1; }      // a row segment of P pixels; the tile holds two such rows
  t->WT = (g.wo + t->bw - 1) / t->bw;
  t->HT = t->mpack ? (g.ho + 1) / 2 : (g.ho + t->bh - 1) / t->bh;
  t->GT = (g.G + t->bg - 1) / t->bg;
  t->pair = pair;
  t->MT = pair ? (g.cout + BM2 - 1) / BM2 : (g.cout + BM - 1) / BM;
  long long nt = (long long)t->WT * t->HT * t->GT * t->MT;
  if (nt > 0x7fffffffLL) return false;
  t->ntiles = (int)nt;
  t->CB = (g.cin + BK - 1) / BK;
  t->KB = t->CB * (t->mpack ? g.kh + 1 : g.kh) * g.kw;
  t->BN = E * P;
  // a CTA of a pair stages its own 128 rows of W and half of the activation rows
  const size_t stage = 2 * ((size_t)BM * BK * 4 + (size_t)(pair ? t->BN / 2 : t->BN) * BK * 4);
  const size_t ctrl = 1024 + 512;   // alignment slack + barriers
  const size_t fixed = 1024 + 64;   // the kernels' static shared memory (table of chunk lengths)
  int ns = (int)(((size_t)smem_optin - ctrl - fixed) / stage);
  if (ns > kMaxStages) ns = kMaxStages;
  if (ns < 2) return false;
  t->nstages = ns;
  t->smem_bytes = (size_t)ns * stage + ctrl;
  t->smem_one_ring = t->smem_bytes;
  t->nstages_b = 0;
  if (!pair) {
    // Two rings: the W tiles keep `ns` slots, the activations (the larger part of a k-block) get one more when it
    // fits: their copies then run a k-block further ahead.  Measured with a three-slot ring for everything
    // (possible in the two-product mode only): 27-30 % faster kernels than with two slots; the one- and
    // two-slot hand-over is what the single-CTA kernel loses against its tensor and copy floors.
    const size_t a2 = 2 * (size_t)BM * BK * 4, b2 = 2 * (size_t)t->BN * BK * 4;
    int nb = ns + 1;
    if (nb <= kMaxStages && (size_t)ns * a2 + (size_t)nb * b2 + ctrl + fixed <= (size_t)smem_optin) {
      t->nstages_b = nb;
      t->smem_bytes = (size_t)ns * a2 + (size_t)nb * b2 + ctrl;
    }
  }
  return true;
}

bool encode_map(const TcState* ts, CUtensorMap* m, const void* base, int rank, const cuuint64_t* dims,
                const cuuint64_t* strides_bytes, const cuuint32_t* box, int swz_bytes, int step_wh = 1) {
  // step_wh > 1: every step_wh-th column and row (dimensions 1 and 2), the input
  // positions a strided convolution reads; such a box spans box*step_wh positions
  cuuint32_t estr[5] = {1, (cuuint32_t)step_wh, (cuuint32_t)step_wh, 1, 1};
  if (rank < 3) estr[1] = estr[2] = 1;
  // swz_bytes: 32/64/128 = 16-byte chunks swizzled within that span (K-major
  // operands); kSwz128Atom32 = 32-byte chunks within 128 bytes, the only layout
  // the tensor core accepts for MN-major 32-bit operands
  CUtensorMapSwizzle sw = swz_bytes == kSwz128Atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                          : swz_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (swz_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  CUresult r = ts->encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<void*>(base), dims,
                          strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor maps of the forward kernels: W as [cout][tap][cin] with a box of 128
// output channels x one tap x BK channels; the encoded activations as
// [G][E][h][w][cin] with one box of the tile's pixels per encoding.
template <int BK>
bool encode_fwd_maps(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                     const float* xb_hi, const float* xb_lo, CUtensorMap* ma_hi, CUtensorMap* ma_lo,
                     CUtensorMap* mb_hi, CUtensorMap* mb_lo) {
  // (two-row tiles: the pre-pass laid the weights out as 128 rows x (kh+1)*kw taps, see tc_fwd_prepass)
  const int taps = tl.mpack ? (g.kh + 1) * g.kw : g.kh * g.kw;
  {
    cuuint64_t dims[3] = {(cuuint64_t)g.cin, (cuuint64_t)taps, (cuuint64_t)(tl.mpack ? BM : g.cout)};
    cuuint64_t str[2] = {(cuuint64_t)g.cin * 4, (cuuint64_t)g.cin * taps * 4};
    cuuint32_t box[3] = {(cuuint32_t)BK, 1, (cuuint32_t)BM};
    if (!encode_map(ts, ma_hi, w_hi, 3, dims, str, box, BK * 4) ||
        !encode_map(ts, ma_lo, w_lo, 3, dims, str, box, BK * 4))
      return false;
  }
  {
    cuuint64_t dims[5] = {(cuuint64_t)g.cin, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.E, (cuuint64_t)g.G};
    cuuint64_t str[4] = {(cuuint64_t)g.cin * 4, (cuuint64_t)g.cin * g.w * 4, (cuuint64_t)g.n_in * 4,
                         (cuuint64_t)g.n_in * g.E * 4};
    // (tiles of one virtual batch fetch all their encodings, or a CTA pair's half of them, as one box)
    const cuuint32_t ebox = onebox_tiles(tl) ? (cuuint32_t)(tl.pair ? g.E / 2 : g.E) : 1u;
    cuuint32_t box[5] = {(cuuint32_t)BK, (cuuint32_t)(tl.bw * g.stride), (cuuint32_t)(tl.bh * g.stride), ebox,
                         (cuuint32_t)tl.bg};
    if (!encode_map(ts, mb_hi, xb_hi, 5, dims, str, box, BK * 4, g.stride) ||
        !encode_map(ts, mb_lo, xb_lo, 5, dims, str, box, BK * 4, g.stride))
      return false;
  }
  return true;
}

template <int BK, int MODE, int K>
dk_status launch_one(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                     const float* xb_hi, const float* xb_lo, TcParams& prm, int sm_count, cudaStream_t st) {
  CUtensorMap ma_hi, ma_lo, mb_hi, mb_lo;
  if (xb_lo == nullptr) xb_lo = xb_hi;      // (the kernel derives the second term: that map is not used)
  if (!encode_fwd_maps<BK>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, &ma_hi, &ma_lo, &mb_hi, &mb_lo)) return DK_ERR_CUDA;
  auto kern = tc_fwd_kernel<BK, MODE, K>;
  static KernelCache kc = {};
  if (dk_status e = prepare_kernel(kern, kc, ts->device, tl.smem_bytes)) return e;
  const long long nwork = (long long)tl.ntiles * prm.ksplit;
  int grid = nwork < sm_count ? (int)nwork : sm_count;
  kern<<<grid, kThreadsTc, tl.smem_bytes, st>>>(ma_hi, ma_lo, mb_hi, mb_lo, prm);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

// CTA-pair kernel (even K only): grid = 2 x the number of resident pairs
template <int MODE, int K>
dk_status launch_pair_one(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                          const float* xb_hi, const float* xb_lo, TcParams& prm, int sm_count, cudaStream_t st) {
  if constexpr (K % 2 != 0) {
    return DK_ERR_UNSUPPORTED;
  } else {
    CUtensorMap ma_hi, ma_lo, mb_hi, mb_lo;
    if (!encode_fwd_maps<32>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, &ma_hi, &ma_lo, &mb_hi, &mb_lo)) return DK_ERR_CUDA;
    auto kern = tc_fwd_pair_kernel<MODE, K>;
    static KernelCache kc = {};
    if (dk_status e = prepare_kernel(kern, kc, ts->device, tl.smem_bytes)) return e;
    const long long nwork = (long long)tl.ntiles * prm.ksplit;
    int pairs = resident_pairs(kern, kc, ts->device, tl.smem_bytes, sm_count, false);
    if (nwork < pairs) pairs = (int)nwork;
    kern<<<2 * pairs, kThreadsTc, tl.smem_bytes, st>>>(ma_hi, ma_lo, mb_hi, mb_lo, prm);
    DK_CUDA_CHECK(cudaGetLastError());
    return DK_OK;
  }
}

template <int BK, int MODE>
dk_status launch_k(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                   const float* xb_hi, const float* xb_lo, TcParams& prm, int sm_count, cudaStream_t st) {
  switch (g.K) {
    case 1: return launch_one<BK, MODE, 1>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 2: return launch_one<BK, MODE, 2>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 3: return launch_one<BK, MODE, 3>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 4: return launch_one<BK, MODE, 4>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 5: return launch_one<BK, MODE, 5>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 6: return launch_one<BK, MODE, 6>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 7: return launch_one<BK, MODE, 7>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 8: return launch_one<BK, MODE, 8>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
  }
  return DK_ERR_SHAPE;
}

void fill_params(const TcState* ts, const Geom& g, const Tiling& tl, TcParams* p) {
  p->bw = tl.bw; p->bh = tl.bh; p->bg = tl.bg;
  p->log2_bw = 0; while ((1 << p->log2_bw) < tl.bw) ++p->log2_bw;
  p->log2_S = 0; while ((1 << p->log2_S) < tl.bw * tl.bh) ++p->log2_S;
  p->WT = tl.WT; p->HT = tl.HT; p->GT = tl.GT; p->MT = tl.MT;
  p->gt0 = 0;
  p->ntiles = tl.ntiles; p->KB = tl.KB; p->CB = tl.CB;
  // 32-wide k-blocks accumulated in TMEM between promotions (the error grows ~linearly with it)
  p->chunk = ts->opt->v[DK_OPT_TC_CHUNK] * (32 / fwd_bk(ts));
  p->chunk_tab = nullptr; p->chunk_mul = 32 / fwd_bk(ts);
  p->spin_cap = (unsigned)ts->opt->v[DK_OPT_SPIN_LIMIT];
  p->withhold = ts->opt->v[DK_OPT_TEST_WITHHOLD];
  p->nprod = g.nprod == 2 ? 2 : 3;
  p->lo_inkernel = 0;
  p->pace = nullptr; p->pace_every = 1;
  p->nstages_b = ts->opt->v[DK_OPT_TC_SPLIT_RING] ? tl.nstages_b : 0;
  p->b_onebox = onebox_tiles(tl) ? 1 : 0;
  p->gbox = p->b_onebox && tl.bg == 2 ? 1 : 0;
  p->hmul = tl.mpack ? 2 : 1;
  ts->opt->v[DK_OPT_TEST_WITHHOLD] = -1;      // the hook serves one launch
  p->ksplit = 1;
  p->kb_per_split = tl.KB;
  p->kw = g.kw; p->pad = g.pad; p->stride = g.stride; p->nstages = tl.nstages;
  p->cout = g.cout; p->ho = g.ho; p->wo = g.wo; p->G = g.G;
  p->kstore = g.kstore;
  p->n_out = g.n_out;
  p->out = nullptr; p->dec = p->decl = p->nul = p->bias = nullptr;
  p->vs.sumsq = nullptr; p->vs.maxrho = nullptr; p->vs.count = nullptr; p->vs.cand = nullptr;
  p->tau = g.tol;
  p->status = nullptr;
  p->verdict = nullptr; p->done = nullptr;
  p->f_group = -1; p->f_enc = p->f_co = p->f_oh = p->f_ow = 0;
  p->f_delta = 0.f;
}

// CTA pairs serve layers with more than 128 output channels and an even
// number of encodings (option DK_OPT_TC_PAIR switches them off)
bool use_pair(const TcState* ts, const Geom& g) {
  return ts->opt->v[DK_OPT_TC_PAIR] && fwd_bk(ts) == 32 && g.cout > BM && (g.E % 2) == 0;
}

bool plan_fwd(const TcState* ts, const Geom& g, Tiling* t) {
  const int smem_optin = ts->smem_optin;
  if (use_pair(ts, g) && plan_tiling<32>(g, smem_optin, t, true)) return true;
  return fwd_bk(ts) == 16 ? plan_tiling<16>(g, smem_optin, t) : plan_tiling<32>(g, smem_optin, t);
}

template <int MODE>
dk_status launch_pair(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                      const float* xb_hi, const float* xb_lo, TcParams& prm, int sm_count, cudaStream_t st) {
  switch (g.K) {
    case 2: return launch_pair_one<MODE, 2>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 4: return launch_pair_one<MODE, 4>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 6: return launch_pair_one<MODE, 6>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
    case 8: return launch_pair_one<MODE, 8>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
  }
  return DK_ERR_UNSUPPORTED;
}

template <int MODE>
dk_status launch_bk(const TcState* ts, const Geom& g, const Tiling& tl, const float* w_hi, const float* w_lo,
                    const float* xb_hi, const float* xb_lo, TcParams& prm, int sm_count, cudaStream_t st) {
  if (tl.pair) return launch_pair<MODE>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
  return fwd_bk(ts) == 16 ? launch_k<16, MODE>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st)
                        : launch_k<32, MODE>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, sm_count, st);
}

}  // namespace

dk_status tc_init(dk_ctx* ctx) {
  TcState* ts = new (std::nothrow) TcState();
  if (!ts) return DK_ERR_CUDA;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    delete ts;
    return DK_ERR_CUDA;
  }
  ts->encode = reinterpret_cast<EncodeTiledFn>(fn);
  int optin = 0;
  if (cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) != cudaSuccess) {
    delete ts;
    return DK_ERR_CUDA;
  }
  ts->smem_optin = optin;
  ts->device = ctx->device;
  ts->opt = &ctx->opt;
  ctx->tc_state = ts;
  return DK_OK;
}

// Tiled tensor map over bytes (the digit planes of the finite-field kernels): swz_bytes = 64 or 128.
bool tc_encode_map_bytes(const dk_ctx* ctx, CUtensorMap* m, const void* base, int rank, const unsigned long long* dims,
                         const unsigned long long* strides_bytes, const unsigned int* box, int swz_bytes) {
  const TcState* ts = static_cast<const TcState*>(ctx->tc_state);
  if (!ts || rank < 1 || rank > 5) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
  CUresult r = ts->encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swz_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int tc_smem_optin(const dk_ctx* ctx) {
  return ctx->tc_state ? static_cast<TcState*>(ctx->tc_state)->smem_optin : 0;
}

void tc_destroy(dk_ctx* ctx) {
  delete static_cast<TcState*>(ctx->tc_state);
  ctx->tc_state = nullptr;
}

bool tc_mpack_eligible(const Geom& g) {
  if (g.kind != DK_CONV2D || g.layout != DK_NHWC || g.precision != DK_TF32X3) return false;
  if (g.cout > 64 || g.kh < 2 || g.stride != 1 || (g.cin % 4) != 0) return false;
  const int P = tile_pixels(g.K);
  return (P & (P - 1)) == 0;      // the row segment of P pixels must be a power of two
}

bool tc_fwd_supported(const dk_ctx* ctx, const Geom& g) {
  if (g.precision != DK_TF32X3 || ctx->tc_state == nullptr) return false;
  if (g.layout != DK_NHWC || g.stride < 1 || g.stride > 4 || (g.cin % 4) != 0) return false;
  if (g.n_out >= (1LL << 31)) return false;     // the epilogue keeps pixel offsets in 32 bits
  Tiling tl;
  return plan_fwd(static_cast<TcState*>(ctx->tc_state), g, &tl);
}

dk_status tc_split(const float* src, float* hi, float* lo, long long n, int sm_count, cudaStream_t st, int raw) {
  if ((raw != 0) != (hi == nullptr)) return DK_ERR_INVALID_ARG;
  if (n % 4) return DK_ERR_SHAPE;
  long long n4 = n / 4;
  long long blocks = (n4 + 255) / 256;
  if (blocks > (long long)sm_count * 16) blocks = (long long)sm_count * 16;
  if (blocks < 1) blocks = 1;
  split_tf32_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(src),
                                                      reinterpret_cast<float4*>(hi), reinterpret_cast<float4*>(lo), n4, raw);
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

dk_status tc_encode_split(const Geom& g, const float* x, const float* r, const float* enc, float* full,
                          float* hi, float* lo, int sm_count, cudaStream_t st) {
  if (g.n_in % 4 || g.G > 65535) return DK_ERR_SHAPE;
  long long n4 = g.n_in / 4;
  long long want = (n4 + 255) / 256;
  long long cap = ((long long)sm_count * 16 + g.G - 1) / g.G;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  dim3 grid((unsigned)want, (unsigned)g.G);
#define DK_ENC_CASE(KK) \
  case KK: encode_split_kernel<KK><<<grid, 256, 0, st>>>(x, r, enc, full, hi, lo, g.n_in); break;
  switch (g.K) {
    DK_ENC_CASE(1) DK_ENC_CASE(2) DK_ENC_CASE(3) DK_ENC_CASE(4)
    DK_ENC_CASE(5) DK_ENC_CASE(6) DK_ENC_CASE(7) DK_ENC_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_ENC_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

// Contraction slices for problems with fewer tiles than SMs.  Work items are
// dealt round-robin to the resident CTAs (or pairs), so a slice count costs
// rounds x (k-blocks per slice + a fixed per-item part: pipeline fill, epilogue
// atomics), plus, for any count above one, the launches of the unfused path
// (y_bar cleared, decode in a second kernel).  The cheapest count wins; slices
// keep at least 8 k-blocks.  All figures in units of one k-block's time.
int tc_fwd_ksplit(const dk_ctx* ctx, const Geom& g) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  Tiling tl;
  if (!ts || !plan_fwd(ts, g, &tl)) return 1;
  const int units = tl.pair ? ctx->sm_count / 2 : ctx->sm_count;     // CTAs or CTA pairs that run together
  if (tl.ntiles >= units) return 1;
  const int unit_kb = 32 / fwd_bk(ts);           // k-blocks per 32 contraction elements
  const int cap = tl.KB / (8 * unit_kb);
  const long long kItem = 6 * unit_kb, kUnfused = 20 * unit_kb;
  int best = 1;
  long long best_cost = (long long)((tl.ntiles + units - 1) / units) * (tl.KB + kItem);
  for (int c = 2; c <= cap; ++c) {
    const int per = (tl.KB + c - 1) / c;
    const int eff = (tl.KB + per - 1) / per;
    if (eff != c) continue;                      // same slices as a smaller count
    const long long items = (long long)tl.ntiles * eff;
    const long long rounds = (items + units - 1) / units;
    const long long cost = rounds * (per + kItem) + kUnfused;
    if (cost < best_cost) { best_cost = cost; best = c; }
  }
  return best;
}

// Whether the forward kernel that serves g derives the activations' second TF32 term itself (then nobody writes
// or reads that array): option DK_OPT_TC_LO_INKERNEL, and a kernel that has the converter warps.
bool tc_fwd_lo_inkernel(const dk_ctx* ctx, const Geom& g) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  Tiling tl;
  if (!ts || !ctx->opt.v[DK_OPT_TC_LO_INKERNEL] || !ctx->opt.v[DK_OPT_XBAR_HI] || !plan_fwd(ts, g, &tl)) return false;
  // option value 1: every forward kernel; 2: CTA pairs only (four stages hide the derivation, two do not)
  return ctx->opt.v[DK_OPT_TC_LO_INKERNEL] == 1 || tl.pair;
}

bool tc_fwd_group_tiles(const dk_ctx* ctx, const Geom& g, int* GT, int* bg, long long* rounds) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  Tiling tl;
  if (!ts || !plan_fwd(ts, g, &tl)) return false;
  const int units = tl.pair ? ctx->sm_count / 2 : ctx->sm_count;
  *GT = tl.GT; *bg = tl.bg;
  *rounds = (tl.ntiles + units - 1) / units;
  return true;
}

// Pace of the forward kernels (see tc_fwd_kernel): only when every CTA (pair) walks several meetings' worth of whole
// tiles.  The counter is the word three after the status word, cleared on the stream before the launch.
static dk_status arm_pace(const dk_ctx* ctx, const Tiling& tl, TcParams* prm, int* status_word, cudaStream_t st) {
  const int every = ctx->opt.v[DK_OPT_TC_PACE];
  const int units = tl.pair ? ctx->sm_count / 2 : ctx->sm_count;
  if (every > 0 && status_word != nullptr && prm->ksplit == 1 && tl.ntiles / units >= 2 * every) {
    prm->pace = reinterpret_cast<unsigned int*>(status_word) + 3;
    prm->pace_every = every;
    DK_CUDA_CHECK(cudaMemsetAsync(prm->pace, 0, sizeof(unsigned int), st));
  }
  return DK_OK;
}

dk_status tc_linear_fwd(dk_ctx* ctx, const Geom& g, const float* w_hi, const float* w_lo, const float* xb_hi,
                        const float* xb_lo, float* ybar, int ksplit, bool ybar_cleared, int* status_word,
                        cudaStream_t st, int chunk_cap, bool lo_inkernel) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  Tiling tl;
  if (!plan_fwd(ts, g, &tl)) return DK_ERR_UNSUPPORTED;
  TcParams prm;
  fill_params(ts, g, tl, &prm);
  if (ksplit > 1) {
    prm.kb_per_split = (tl.KB + ksplit - 1) / ksplit;
    prm.ksplit = (tl.KB + prm.kb_per_split - 1) / prm.kb_per_split;
    if (!ybar_cleared)
      DK_CUDA_CHECK(cudaMemsetAsync(ybar, 0, (size_t)g.G * g.E * g.n_out * sizeof(float), st));
  }
  prm.out = ybar;
  if (chunk_cap > 0 && prm.chunk > chunk_cap * (32 / fwd_bk(ts))) prm.chunk = chunk_cap * (32 / fwd_bk(ts));
  prm.lo_inkernel = lo_inkernel ? 1 : 0;
  if (lo_inkernel) prm.nstages_b = 0;      // (the converter warps work on the one-ring layout)
  prm.status = status_word;
  if (dk_status e = arm_pace(ctx, tl, &prm, status_word, st)) return e;
  return launch_bk<MODE_YBAR>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, ctx->sm_count, st);
}

dk_status tc_masked_fwd(dk_ctx* ctx, const Geom& g, const float* w_hi, const float* w_lo, const float* xb_hi,
                        const float* xb_lo, const CoefView& cv, const float* bias, float* y,
                        const VerifyScratch& vs, int* status_word, const dk_fault* fault, dk_verdict* verdict,
                        cudaStream_t st, int gt_lo, int gt_cnt, bool lo_inkernel) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  Tiling tl;
  if (!plan_fwd(ts, g, &tl)) return DK_ERR_UNSUPPORTED;
  if (gt_cnt >= 0) {
    // this launch covers group tiles [gt_lo, gt_lo + gt_cnt) only
    if (gt_lo < 0 || gt_cnt < 1 || gt_lo + gt_cnt > tl.GT) return DK_ERR_INVALID_ARG;
    tl.ntiles = tl.WT * tl.HT * gt_cnt * tl.MT;
    tl.GT = gt_cnt;
  }
  TcParams prm;
  fill_params(ts, g, tl, &prm);
  if (gt_cnt >= 0) prm.gt0 = gt_lo;
  prm.lo_inkernel = lo_inkernel ? 1 : 0;
  if (lo_inkernel) prm.nstages_b = 0;      // (the converter warps work on the one-ring layout)
  prm.out = y;
  prm.dec = cv.dec; prm.decl = cv.decl; prm.nul = cv.nul; prm.bias = bias;
  // ill-conditioned coefficient sets take shorter chunks (see upload_coefficients): per virtual batch where the
  // kernels' table holds them all, else the worst one's for the whole call
  if (cv.chunk_tab != nullptr && g.G <= kChunkTabMax) {
    if (cv.chunk_cap * (32 / fwd_bk(ts)) < prm.chunk) prm.chunk_tab = cv.chunk_tab;      // (else no group needs less)
  } else if (cv.chunk_cap > 0 && prm.chunk > cv.chunk_cap * (32 / fwd_bk(ts))) prm.chunk = cv.chunk_cap * (32 / fwd_bk(ts));
  prm.vs = vs;
  prm.status = status_word;
  prm.verdict = verdict;
  prm.done = vs.count + 3;      // fourth word after the statistics: zero between calls
  if (fault) {
    prm.f_group = fault->group;
    prm.f_enc = fault->enc;
    long long pix = fault->out_index / g.cout;
    prm.f_co = (int)(fault->out_index - pix * g.cout);
    prm.f_oh = (int)(pix / g.wo);
    prm.f_ow = (int)(pix - (long long)prm.f_oh * g.wo);
    prm.f_delta = fault->delta;
  }
  if (dk_status e = arm_pace(ctx, tl, &prm, status_word, st)) return e;
  return launch_bk<MODE_DECODE>(ts, g, tl, w_hi, w_lo, xb_hi, xb_lo, prm, ctx->sm_count, st);
}

// ---------------------------------------------------------------------------
// weight gradient
// ---------------------------------------------------------------------------
namespace {


// dtil[g*(K+1)+j] = sum_i dmix[g][j][i] * delta[g*K+i], written as a TF32 hi/lo pair (Eq. 4).
template <int K>
__global__ void __launch_bounds__(256)
mix_split_kernel(const float* __restrict__ delta, const float* __restrict__ dmix, float* __restrict__ hi,
                 float* __restrict__ lo, long long n) {
  constexpr int K1 = K + 1;
  const int g = blockIdx.y;
  float c[K1][K];
#pragma unroll
  for (int j = 0; j < K1; ++j)
#pragma unroll
    for (int i = 0; i < K; ++i) c[j][i] = __ldg(dmix + ((size_t)g * K1 + j) * K + i);
  const float* dg = delta + (size_t)g * K * n;
  const size_t ob = (size_t)g * K1 * n;
  const long long n4 = n / 4;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += (long long)gridDim.x * blockDim.x) {
    float4 s[K];
#pragma unroll
    for (int i = 0; i < K; ++i) s[i] = __ldg(reinterpret_cast<const float4*>(dg + (size_t)i * n) + q);
#pragma unroll
    for (int j = 0; j < K1; ++j) {
      float4 o, h, l;
      o.x = c[j][K - 1] * s[K - 1].x; o.y = c[j][K - 1] * s[K - 1].y;
      o.z = c[j][K - 1] * s[K - 1].z; o.w = c[j][K - 1] * s[K - 1].w;
#pragma unroll
      for (int i = 0; i < K - 1; ++i) {
        o.x = fmaf(c[j][i], s[i].x, o.x); o.y = fmaf(c[j][i], s[i].y, o.y);
        o.z = fmaf(c[j][i], s[i].z, o.z); o.w = fmaf(c[j][i], s[i].w, o.w);
      }
      h.x = to_tf32(o.x); l.x = to_tf32(o.x - h.x);
      h.y = to_tf32(o.y); l.y = to_tf32(o.y - h.y);
      h.z = to_tf32(o.z); l.z = to_tf32(o.z - h.z);
      h.w = to_tf32(o.w); l.w = to_tf32(o.w - h.w);
      const size_t off = ob + (size_t)j * n;
      reinterpret_cast<float4*>(hi + off)[q] = h;
      reinterpret_cast<float4*>(lo + off)[q] = l;
    }
  }
}

struct WgPlan {
  WgTcParams prm;
  int BN;
  bool pair;               // 256 output channels per work item on CTA pairs
  size_t smem_bytes;
};

bool plan_wgrad(const Options& opt, const Geom& g, int smem_optin, int sm_count, WgPlan* w, int gt_lo = 0,
                int gt_cnt = -1) {
  WgTcParams& p = w->prm;
  const int P = kWgPix;
  long long best = -1;
  p.bw = p.bh = p.bg = 1;
  for (int bw = 1; bw <= P; bw *= 2)
    for (int bh = 1; bw * bh <= P; bh *= 2) {
      const int bg = P / (bw * bh);
      const long long cost = (long long)((g.wo + bw - 1) / bw) * bw * ((g.ho + bh - 1) / bh) * bh *
                             ((g.G + bg - 1) / bg) * bg;
      if (best < 0 || cost < best || (cost == best && (bw > p.bw || (bw == p.bw && bh > p.bh)))) {
        best = cost; p.bw = bw; p.bh = bh; p.bg = bg;
      }
    }
  // Layers with at most 64 output channels (3-wide filters, stride 1): rows 0-63 of the tile hold the
  // gradients of an even image row, rows 64-127 those of the odd row below it, so one box of encodings at
  // vertical offset dy serves filter row dy for the even rows and dy-1 for the odd ones: kh+1 items over
  // half the image rows instead of kh half-used items over all of them.
  // Taken when its padded pixel count x (kh+1) is below the plain tiling's x kh.
  p.mpack = (opt.v[DK_OPT_TC_MPACK] && g.kind == DK_CONV2D && g.cout <= 64 && g.cin <= 64 && g.kw == 3 && g.kh >= 2 &&
             g.stride == 1 && opt.v[DK_OPT_WG_PACK]) ? 1 : 0;
  if (p.mpack) {
    const long long two_row = (long long)((g.wo + P - 1) / P) * P * ((g.ho + 1) / 2) * g.G * (g.kh + 1);
    if (two_row >= best * g.kh) p.mpack = 0;
  }
  if (p.mpack) { p.bw = P; p.bh = 1; p.bg = 1; }
  p.WT = (g.wo + p.bw - 1) / p.bw;
  p.HT = p.mpack ? (g.ho + 1) / 2 : (g.ho + p.bh - 1) / p.bh;
  p.GT = (g.G + p.bg - 1) / p.bg;
  if ((long long)p.WT * p.HT * p.GT > 0x3fffffffLL) return false;
  p.pb0 = 0;
  if (gt_cnt >= 0) {
    // this launch covers group tiles [gt_lo, gt_lo + gt_cnt) only
    if (gt_lo < 0 || gt_cnt < 1 || gt_lo + gt_cnt > p.GT) return false;
    p.pb0 = gt_lo * p.WT * p.HT;
    p.GT = gt_cnt;
  }
  p.PB = p.WT * p.HT * p.GT;
  p.K1 = g.K + 1;
  // N tile = tpn tap slots of cb channels.  Few input channels would make a
  // narrow tile (N = 64 or 128 re-reads the 128 rows of dtil from shared memory
  // once per 64 or 128 columns); putting several filter taps side by side keeps
  // N at 192 or 256.
  p.taps = g.kh * g.kw;
  const int pack_on = opt.v[DK_OPT_WG_PACK];
  if (g.cin <= 64) {
    p.cb = 64;
    p.tpn = !pack_on || p.taps == 1 ? 1 : (p.taps % 3 == 0 || p.taps < 4 ? (p.taps < 3 ? p.taps : 3) : 4);
  } else if (g.cin <= 128) {
    p.cb = 128;
    p.tpn = !pack_on || p.taps == 1 ? 1 : 2;
  } else {
    p.cb = 256;
    p.tpn = 1;
  }
  if (p.mpack) p.tpn = g.kw;
  w->BN = p.cb * p.tpn;
  p.TG = p.mpack ? g.kh + 1 : (p.taps + p.tpn - 1) / p.tpn;
  const int pair_on = opt.v[DK_OPT_WG_PAIR];
  w->pair = pair_on && g.cout > BM;
  p.MT = w->pair ? (g.cout + BM2 - 1) / BM2 : (g.cout + BM - 1) / BM;
  const int units = w->pair ? sm_count / 2 : sm_count;     // CTAs or CTA pairs that run together
  p.NB = (g.cin + p.cb - 1) / p.cb;
  const long long base = (long long)p.MT * p.NB * p.TG;
  // Slices of the pixel-block range per tile.  Work items are dealt round-robin to
  // the resident CTAs (or pairs), so a slice count costs rounds x (k-blocks per
  // slice + a fixed per-item part: pipeline fill and the cout x cin reductions
  // into dW), in units of one k-block's time.  The cheapest count (at most 64
  // slices) wins, the smaller one on ties.
  long long max_split = p.PB < 64 ? p.PB : 64;
  if (max_split < 1) max_split = 1;
  const long long kItem = 10;
  long long nsplit = 1, best_cost = -1;
  for (long long c = 1; c <= max_split; ++c) {
    const long long per = (p.PB + c - 1) / c;
    const long long eff_split = (p.PB + per - 1) / per;
    if (eff_split != c) continue;               // same slices as a smaller count
    const long long items_c = base * eff_split;
    const long long rounds = (items_c + units - 1) / units;
    const long long cost = rounds * (per * p.K1 + kItem);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; nsplit = c; }
  }
  p.pb_per_split = (int)((p.PB + nsplit - 1) / nsplit);
  p.nsplit = (p.PB + p.pb_per_split - 1) / p.pb_per_split;
  const long long items = base * p.nsplit;
  if (items > 0x7fffffffLL) return false;
  p.nitems = (int)items;
  p.kw = g.kw; p.pad = g.pad; p.stride = g.stride;
  p.chunk = opt.v[DK_OPT_WG_CHUNK];      // k-blocks accumulated in TMEM between promotions
  p.spin_cap = (unsigned)opt.v[DK_OPT_SPIN_LIMIT];
  p.withhold = -1;
  p.cout = g.cout; p.cin = g.cin;
  const size_t stage = 2 * ((size_t)(BM / 32) * kWgBox + (size_t)((w->pair ? w->BN / 2 : w->BN) / 32) * kWgBox);
  const size_t ctrl = 1024 + 512;
  int ns = (int)(((size_t)smem_optin - ctrl) / stage);
  if (ns > kMaxStages) ns = kMaxStages;
  if (ns < 2) return false;
  p.nstages = ns;
  p.nstages_b = 0;
  w->smem_bytes = (size_t)ns * stage + ctrl;
  if (!w->pair && opt.v[DK_OPT_TC_SPLIT_RING]) {
    // two rings (see the forward kernel's plan): one more slot for the encodings when that fits, else one more
    // for the gradients
    const size_t a2 = 2 * (size_t)(BM / 32) * kWgBox, b2 = 2 * (size_t)(w->BN / 32) * kWgBox;
    if ((size_t)ns * a2 + (size_t)(ns + 1) * b2 + ctrl <= (size_t)smem_optin && ns + 1 <= kMaxStages) {
      p.nstages_b = ns + 1;
      w->smem_bytes = (size_t)ns * a2 + (size_t)(ns + 1) * b2 + ctrl;
    } else if ((size_t)(ns + 1) * a2 + (size_t)ns * b2 + ctrl <= (size_t)smem_optin && ns + 1 <= kMaxStages) {
      p.nstages = ns + 1;
      p.nstages_b = ns;
      w->smem_bytes = (size_t)(ns + 1) * a2 + (size_t)ns * b2 + ctrl;
    }
  }
  return true;
}

template <int BN, bool PAIR>
dk_status launch_wgrad(const WgPlan& w, const CUtensorMap& md_hi, const CUtensorMap& md_lo,
                       const CUtensorMap& mx_hi, const CUtensorMap& mx_lo, int dev, int sm_count, cudaStream_t st) {
  auto kern = tc_wgrad_kernel<BN, PAIR>;
  static KernelCache kc = {};
  if (dk_status e = prepare_kernel(kern, kc, dev, w.smem_bytes)) return e;
  if (!PAIR) {
    int grid = w.prm.nitems < sm_count ? w.prm.nitems : sm_count;
    kern<<<grid, kThreadsTc, w.smem_bytes, st>>>(md_hi, md_lo, mx_hi, mx_lo, w.prm);
    DK_CUDA_CHECK(cudaGetLastError());
    return DK_OK;
  }
  // clusters of two CTAs; as many pairs as can be resident together
  int pairs = resident_pairs(kern, kc, dev, w.smem_bytes, sm_count, true);
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreadsTc);
  cfg.dynamicSmemBytes = w.smem_bytes;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (w.prm.nitems < pairs) pairs = w.prm.nitems;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  DK_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kern, md_hi, md_lo, mx_hi, mx_lo, w.prm));
  return DK_OK;
}

}  // namespace

bool tc_wgrad_supported(const dk_ctx* ctx, const Geom& g) {
  if (g.precision != DK_TF32X3 || ctx->tc_state == nullptr) return false;
  if (g.layout != DK_NHWC || g.stride < 1 || g.stride > 4 || (g.cin % 4) != 0 || (g.cout % 4) != 0) return false;
  WgPlan w;
  return plan_wgrad(ctx->opt, g, static_cast<TcState*>(ctx->tc_state)->smem_optin, ctx->sm_count, &w);
}

bool tc_stem_supported(const dk_ctx* ctx, const Geom& g) {
  if (ctx->opt.v[DK_OPT_TC_STEM] == 0 || g.kind != DK_CONV2D || g.layout != DK_NHWC || g.precision != DK_TF32X3) return false;
  if ((g.cin % 4) == 0 || g.kc > 256 || (g.cout % 4) != 0) return false;
  const Geom s = tc_stem_gemm_geom(g);
  return tc_fwd_supported(ctx, s);
}

dk_status tc_mix_split(const Geom& g, const float* delta, const float* dmix, float* hi, float* lo,
                       int sm_count, cudaStream_t st) {
  if (g.n_out % 4 || g.G > 65535) return DK_ERR_SHAPE;
  long long n4 = g.n_out / 4;
  long long want = (n4 + 255) / 256;
  long long cap = ((long long)sm_count * 16 + g.G - 1) / g.G;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  dim3 grid((unsigned)want, (unsigned)g.G);
#define DK_MIX_CASE(KK) \
  case KK: mix_split_kernel<KK><<<grid, 256, 0, st>>>(delta, dmix, hi, lo, g.n_out); break;
  switch (g.K) {
    DK_MIX_CASE(1) DK_MIX_CASE(2) DK_MIX_CASE(3) DK_MIX_CASE(4)
    DK_MIX_CASE(5) DK_MIX_CASE(6) DK_MIX_CASE(7) DK_MIX_CASE(8)
    default: return DK_ERR_SHAPE;
  }
#undef DK_MIX_CASE
  DK_CUDA_CHECK(cudaGetLastError());
  return DK_OK;
}

bool tc_wgrad_group_tiles(const dk_ctx* ctx, const Geom& g, int* GT, int* bg, long long* rounds) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  WgPlan w;
  if (!ts || !plan_wgrad(ctx->opt, g, ts->smem_optin, ctx->sm_count, &w)) return false;
  const int units = w.pair ? ctx->sm_count / 2 : ctx->sm_count;
  *GT = w.prm.GT; *bg = w.prm.bg;
  *rounds = (w.prm.nitems + units - 1) / units;
  return true;
}

dk_status tc_wgrad(dk_ctx* ctx, const Geom& g, const float* dt_hi, const float* dt_lo, const float* xb_hi,
                   const float* xb_lo, int xbar_rows, float scale, float* dW, int* status_word,
                   cudaStream_t st, int gt_lo, int gt_cnt) {
  TcState* ts = static_cast<TcState*>(ctx->tc_state);
  WgPlan w;
  if (!plan_wgrad(ctx->opt, g, ts->smem_optin, ctx->sm_count, &w, gt_lo, gt_cnt)) return DK_ERR_UNSUPPORTED;
  w.prm.withhold = ctx->opt.v[DK_OPT_TEST_WITHHOLD];
  ctx->opt.v[DK_OPT_TEST_WITHHOLD] = -1;      // the hook serves one launch
  w.prm.scale = scale;
  w.prm.dW = dW;
  w.prm.status = status_word;
  // the pace counter (the word after the status word) only when CTAs take several rounds of items
  {
    const int units = w.pair ? ctx->sm_count / 2 : ctx->sm_count;
    w.prm.pace = nullptr;
    // (long items only: with short ones the wait costs more than the shared reads save; fc6 measured 17 % slower)
    if (ctx->opt.v[DK_OPT_WG_PACE] && w.prm.nitems > units && (long long)w.prm.pb_per_split * w.prm.K1 >= 128) {
      w.prm.pace = reinterpret_cast<unsigned int*>(status_word) + 2;
      DK_CUDA_CHECK(cudaMemsetAsync(w.prm.pace, 0, sizeof(unsigned int), st));
    }
  }
  CUtensorMap md_hi, md_lo, mx_hi, mx_lo;
  {
    cuuint64_t dims[5] = {(cuuint64_t)g.cout, (cuuint64_t)g.wo, (cuuint64_t)g.ho, (cuuint64_t)(g.K + 1),
                          (cuuint64_t)g.G};
    cuuint64_t str[4] = {(cuuint64_t)g.cout * 4, (cuuint64_t)g.cout * g.wo * 4, (cuuint64_t)g.n_out * 4,
                         (cuuint64_t)g.n_out * (g.K + 1) * 4};
    cuuint32_t box[5] = {32, (cuuint32_t)w.prm.bw, (cuuint32_t)w.prm.bh, 1, (cuuint32_t)w.prm.bg};
    if (!encode_map(ts, &md_hi, dt_hi, 5, dims, str, box, kSwz128Atom32) ||
        !encode_map(ts, &md_lo, dt_lo, 5, dims, str, box, kSwz128Atom32))
      return DK_ERR_CUDA;
  }
  {
    cuuint64_t dims[5] = {(cuuint64_t)g.cin, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)xbar_rows,
                          (cuuint64_t)g.G};
    cuuint64_t str[4] = {(cuuint64_t)g.cin * 4, (cuuint64_t)g.cin * g.w * 4, (cuuint64_t)g.n_in * 4,
                         (cuuint64_t)g.n_in * xbar_rows * 4};
    cuuint32_t box[5] = {32, (cuuint32_t)(w.prm.bw * g.stride), (cuuint32_t)(w.prm.bh * g.stride), 1,
                         (cuuint32_t)w.prm.bg};
    if (!encode_map(ts, &mx_hi, xb_hi, 5, dims, str, box, kSwz128Atom32, g.stride) ||
        !encode_map(ts, &mx_lo, xb_lo, 5, dims, str, box, kSwz128Atom32, g.stride))
      return DK_ERR_CUDA;
  }
  switch (w.BN) {
    case 64: return w.pair ? launch_wgrad<64, true>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st)
                           : launch_wgrad<64, false>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st);
    case 192: return w.pair ? launch_wgrad<192, true>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st)
                            : launch_wgrad<192, false>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st);
    case 128: return w.pair ? launch_wgrad<128, true>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st)
                            : launch_wgrad<128, false>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st);
    default: return w.pair ? launch_wgrad<256, true>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st)
                           : launch_wgrad<256, false>(w, md_hi, md_lo, mx_hi, mx_lo, ctx->device, ctx->sm_count, st);
  }
}

}  // namespace dk
