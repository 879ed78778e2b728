// Weight-gradient product of Eq. 4/6 on the tensor cores:
//   dW[co][tap][ci] = scale * sum_{g, j<=K, pixel} dtil[g,j][pixel][co] * xbar[g,j][pixel + tap - pad][ci]
// with dtil[g,j] = sum_i gamma_j B[j][i] delta[g,i] mixed beforehand.
//
// GEMM view: M = cout (128 per tile), N = a block of input channels of one
// filter tap, contraction = (virtual batch, encoding, output pixel).  Both
// operands are channels-last tensors, i.e. contiguous along M / N and strided
// along the contraction: they are fetched by TMA as [32 pixels][32 channels]
// boxes (128-byte rows, 32-byte chunks swizzled within the row) and fed to
// tcgen05.mma as MN-major operands.  Same 3xTF32 split and the same pipeline as the forward kernel.
//
// Accuracy.  The K+1 encodings of a pixel block are consecutive k-blocks, so
// the masking noise cancels every K+1 k-blocks and partial sums return to the
// scale of the signal.  TMEM accumulates `chunk` k-blocks only (the tensor pipe
// truncates when it adds into the accumulator); the epilogue warps sum the
// chunks in registers with round-to-nearest.
//
// Parallelism.  Work item = (cout tile, tap, channel block, contraction
// slice); persistent CTAs walk the items and add their slice into dW with
// fp32 atomics (dW is cleared first).
//
// PAIR = true runs the same pipeline on clusters of two CTAs with
// tcgen05 cta_group::2 (see dk_tc_pair.cuh): a pair owns 256 output channels,
// each CTA stages its own 128 columns of dtil and half of the channel block
// of xbar, the leader issues the MMAs for both.
#pragma once

#include "dk_tc_pair.cuh"

namespace dk {
namespace tc {

constexpr int kWgPix = 32;                 // contraction elements (pixels) per k-block
constexpr int kWgBox = kWgPix * 128;       // bytes of one [32 pixels][32 channels] box

struct WgTcParams {
  int bw, bh, bg;              // box shape of the 32 pixels: columns, rows, groups
  int WT, HT, GT;              // pixel blocks along width, height, groups
  int PB;                      // pixel blocks of this launch
  int pb0;                     // its first pixel block (a call may be served by several launches over ranges of groups)
  int K1;                      // encodings used (K+1)
  int MT, NB, taps;            // cout tiles, channel blocks, filter taps
  int cb, tpn, TG;             // channels per tap slot, tap slots per N tile (BN = cb*tpn), tap groups
  int nsplit, pb_per_split;    // contraction slices
  int nitems;                  // MT*NB*taps*nsplit
  int kw, pad, stride;
  int nstages, chunk;
  int nstages_b;               // single-CTA kernel: 0 = one ring of stages; n > 0 = two rings, `nstages` slots for the
                               // gradients and n for the encodings, filled by two producer warps
  unsigned spin_cap;           // polls after which a wait gives up
  int withhold;                // test hook: the producer arms its n-th stage but issues no copy (-1 = off)
  int mpack;                   // cout <= 64: rows 64-127 of the tile are the gradients one image row below rows 0-63
  int cout, cin;
  float scale;
  float* dW;                   // [cout][taps][cin]
  int* status;
  unsigned int* pace;          // nullable: counter (zero at launch) with which the CTAs start their rounds of work items together
};

// Shared-memory descriptor of an MN-major 32-bit operand: [k][32 floats] boxes
// of 128-byte rows whose 32-byte chunks are swizzled with a period of 4 rows
// (the only MN-major layout the tensor core takes for 32-bit elements);
// 4-row groups 512 bytes apart along k, column blocks `block_bytes` apart
// along M/N.
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr, uint32_t block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)((block_bytes >> 4) & 0x3FFF) << 16;   // leading byte offset: next 32-channel block
  d |= (uint64_t)(512 >> 4) << 32;                      // stride byte offset: next 4 pixels
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)1 << 61;                               // 128-byte span, 32-byte swizzle atom
  return d;
}

template <int BN, bool PAIR>
__global__ void __launch_bounds__(kThreadsTc, 1)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap map_d_hi, const __grid_constant__ CUtensorMap map_d_lo,
                const __grid_constant__ CUtensorMap map_x_hi, const __grid_constant__ CUtensorMap map_x_lo,
                const WgTcParams p) {
  constexpr int NH = BN / 2;                     // accumulators per epilogue thread
  constexpr int A_BYTES = (BM / 32) * kWgBox;    // 16 KiB
  constexpr int BNL = PAIR ? BN / 2 : BN;        // channels of xbar this CTA stages
  constexpr int B_BYTES = (BNL / 32) * kWgBox;
  constexpr int STAGE_BYTES = 2 * (A_BYTES + B_BYTES);
  constexpr int MROWS = PAIR ? 2 * BM : BM;      // output channels of a work item
  static_assert(BN % 64 == 0 && BN <= 256, "illegal channel block");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  // One ring: stage s = [d_hi][d_lo][x_hi][x_lo] at s * STAGE_BYTES.  Two rings (single CTA only): the gradients'
  // slots first, then the encodings' slots.
  const bool split = !PAIR && p.nstages_b > 0;
  unsigned char* const b_base = split ? smem + (size_t)p.nstages * 2 * A_BYTES : smem + 2 * A_BYTES;
  const size_t a_pitch = split ? (size_t)2 * A_BYTES : (size_t)STAGE_BYTES;
  const size_t b_pitch = split ? (size_t)2 * B_BYTES : (size_t)STAGE_BYTES;
  unsigned char* ctrl = split ? b_base + (size_t)p.nstages_b * 2 * B_BYTES : smem + (size_t)p.nstages * STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctrl);
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tfull_bar = empty_bar + kMaxStages;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint64_t* bfull_bar = tempty_bar + 2;              // the encodings' ring, when there are two
  uint64_t* bempty_bar = bfull_bar + kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bempty_bar + kMaxStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int first_item = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int item_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.nstages; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int s = 0; s < (split ? p.nstages_b : 0); ++s) { mbar_init(bfull_bar + s, 1); mbar_init(bempty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar + b, 1);
      mbar_init(tempty_bar + b, PAIR ? 2 * kEpiWarps : kEpiWarps);     // a pair's chunks are released on the leader
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(512u)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(512u)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // item -> (mt, nb, tap group, slice); k-blocks of an item = pixel blocks of its slice x K1 encodings.
  // The N tile of an item is tpn slots of cb channels: slot t holds channels
  // [nb*cb, nb*cb + cb) of filter tap tg*tpn + t (layers with few input channels
  // put several taps side by side so that the tile stays wide).
  auto item_range = [&](int item, int& mt, int& nb, int& tg, int& pb_lo, int& pb_hi) {
    mt = item % p.MT;
    int r = item / p.MT;
    nb = r % p.NB; r /= p.NB;
    tg = r % p.TG;
    const int s = r / p.TG;
    pb_lo = s * p.pb_per_split;
    pb_hi = min(p.PB, pb_lo + p.pb_per_split);
  };

  static_assert(40 * 128 + 232 * 256 <= 168 * kThreadsTc, "setmaxnreg budget exceeds the CTA's register pool");
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
    if (warp == 0 || (warp == 2 && split)) {
      // ---------------- TMA producer(s) ----------------
      // (two rings: warp 0 fetches the gradients into theirs, warp 2 the encodings into theirs)
      // whole warp: lane 0 arms the stage, then each lane issues its share of
      // the 2*(BM+BN)/32 box copies so that they go out side by side
      const bool do_a = warp == 0, do_b = !split || warp == 2;
      uint64_t* const fbar = (split && warp == 2) ? bfull_bar : full_bar;
      uint64_t* const ebar = (split && warp == 2) ? bempty_bar : empty_bar;
      const int nst = (split && warp == 2) ? p.nstages_b : p.nstages;
      const uint32_t tx = (uint32_t)(PAIR ? 2 : 1) * ((do_a ? 2u * A_BYTES : 0u) + (do_b ? 2u * B_BYTES : 0u));
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool alive = true;
      constexpr int NBOX = 2 * (BM / 32) + 2 * (BNL / 32);
      static_assert(NBOX <= 32, "one box per lane");
      int round = 0;
      for (int item = first_item; alive && item < p.nitems; item += item_step, ++round) {
        // Pace.  The items that run at the same time are the filter taps (and channel blocks) of the same few
        // slices of the contraction: they read the same gradients and, shifted, the same encodings, once from
        // DRAM and then from L2 -- as long as they stay close in time.  CTAs that drift apart over several rounds
        // of items lose that (measured: DRAM traffic of three passes over the operands where one would do), so a
        // CTA starts round r only when all have issued the loads of round r-1, or after a bounded wait: this is
        // a hint, never a condition for progress.
        if (p.pace != nullptr && round > 0 && lane == 0 && rank == 0 && do_a) {
          const unsigned int target = (unsigned int)round * (unsigned int)item_step;
          for (int spin = 0; spin < 4096 && *reinterpret_cast<volatile unsigned int*>(p.pace) < target; ++spin)
            __nanosleep(128);
        }
        int mt, nb, tg, pb_lo, pb_hi;
        item_range(item, mt, nb, tg, pb_lo, pb_hi);
        const int m0 = mt * MROWS + (int)rank * BM;
        // this lane's box of x_bar: 32 channels of one tap slot (a slot past the
        // last tap reads from beyond the channel range, i.e. zeros)
        int bx_c = 0, bx_u = 0, bx_v = 0;
        if (lane >= 2 * (BM / 32) && lane < NBOX) {
          const int gb = (int)rank * (PAIR ? BNL / 32 : 0) + ((lane - 2 * (BM / 32)) >> 1);
          const int slot = (gb * 32) / p.cb;
          if (p.mpack) {
            // two-row tiles: the item is a vertical offset dy = tg (0..kh), its slots the kw taps of a filter
            // row; rows 0-63 (even image rows) pair the box with tap row dy, rows 64-127 (the odd row below) with tap row dy-1
            bx_c = nb * p.cb + (gb * 32 - slot * p.cb);
            bx_u = tg;
            bx_v = slot;
          } else {
            const int tap = tg * p.tpn + slot;
            bx_c = tap < p.taps ? nb * p.cb + (gb * 32 - slot * p.cb) : p.cin;
            const int tt = tap < p.taps ? tap : 0;
            bx_u = tt / p.kw;
            bx_v = tt - bx_u * p.kw;
          }
        }
        for (int pb = pb_lo; alive && pb < pb_hi; ++pb) {
          int r = p.pb0 + pb;
          const int wt = r % p.WT; r /= p.WT;
          const int ht = r % p.HT;
          const int gt = r / p.HT;
          const int x0 = wt * p.bw, y0 = p.mpack ? 2 * ht : ht * p.bh, g0 = gt * p.bg;      // (two-row tiles step two image rows)
          for (int j = 0; j < p.K1; ++j) {
            int ok = 1;
            if (lane == 0) {
              ok = mbar_wait(ebar + stage, phase ^ 1u, abort_flag, p.spin_cap) ? 1 : 0;
              // the bytes of both CTAs of a pair are counted on the leader's barrier
              if (ok && rank == 0) mbar_expect_tx(fbar + stage, tx);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) { alive = false; break; }
            if (do_a && issued++ == p.withhold) { alive = false; break; }      // test hook: armed, nothing copied
            unsigned char* sta = smem + (size_t)stage * a_pitch;
            unsigned char* stb = b_base + (size_t)stage * b_pitch;
            const uint32_t pbar = PAIR ? mapa_shared(smem_u32(full_bar + stage), 0u) : 0u;
            auto load = [&](void* dst, const CUtensorMap* map, int c0, int c1, int c2) {
              if constexpr (PAIR) tma_pair_load_5d(dst, map, pbar, c0, c1, c2, j, g0);
              else tma_load_5d(dst, map, fbar + stage, c0, c1, c2, j, g0);
            };
            if (lane < 2 * (BM / 32)) {
              const int cb = lane >> 1;
              // two-row tiles: channel blocks 2 and 3 are channels 0..63 of the gradients one row below
              const int ch = (p.mpack && cb >= 2) ? (cb - 2) * 32 : m0 + cb * 32;
              const int yy = (p.mpack && cb >= 2) ? y0 + 1 : y0;
              if (!do_a) {
              } else if ((lane & 1) == 0) load(sta + cb * kWgBox, &map_d_hi, ch, x0, yy);
              else load(sta + A_BYTES + cb * kWgBox, &map_d_lo, ch, x0, yy);
            } else if (lane < NBOX && do_b) {
              const int q = lane - 2 * (BM / 32);
              const int cb = q >> 1;
              const int xi = x0 * p.stride + bx_v - p.pad, yi = y0 * p.stride + bx_u - p.pad;   // input position
              if ((q & 1) == 0) load(stb + cb * kWgBox, &map_x_hi, bx_c, xi, yi);
              else load(stb + B_BYTES + cb * kWgBox, &map_x_lo, bx_c, xi, yi);
            }
            __syncwarp();
            if (++stage == nst) { stage = 0; phase ^= 1u; }
          }
        }
        if (p.pace != nullptr && alive && lane == 0 && rank == 0 && do_a) atomicAdd(p.pace, 1u);
      }
    } else if (warp == 1 && lane == 0 && rank == 0) {
      // ---------------- MMA issuer (of a pair: the leader only) ----------------
      constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) |
                                 ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(MROWS >> 4) << 24);
      auto mma = [&](uint32_t d, uint64_t a, uint64_t b, uint32_t acc) {
        if constexpr (PAIR) tc_pair_mma_tf32(d, a, b, idesc, acc);
        else tc_mma_tf32(d, a, b, idesc, acc);
      };
      auto commit = [&](uint64_t* bar) {
        if constexpr (PAIR) tc_pair_commit(bar);
        else tc_commit(bar);
      };
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      uint32_t acc_it = 0;
      bool alive = true;
      for (int item = first_item; alive && item < p.nitems; item += item_step) {
        int mt, nb, tg, pb_lo, pb_hi;
        item_range(item, mt, nb, tg, pb_lo, pb_hi);
        const int KB = (pb_hi - pb_lo) * p.K1;
        const int nchunks = (KB + p.chunk - 1) / p.chunk;
        for (int ci = 0; alive && ci < nchunks; ++ci, ++acc_it) {
          const uint32_t buf = acc_it & 1u, aphase = (acc_it >> 1) & 1u;
          if (!mbar_wait(tempty_bar + buf, aphase ^ 1u, abort_flag, p.spin_cap)) { alive = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * 256u;
          const int kb_end = min(KB, (ci + 1) * p.chunk);
          for (int kb = ci * p.chunk; kb < kb_end; ++kb) {
            if (!mbar_wait(full_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
            if (split && !mbar_wait(bfull_bar + stage_b, phase_b, abort_flag, p.spin_cap)) { alive = false; break; }
            tc_fence_after();
            const uint32_t sta = smem_u32(smem + (size_t)stage * a_pitch);
            const uint32_t stb = smem_u32(b_base + (size_t)(split ? stage_b : stage) * b_pitch);
            const uint64_t a_hi = make_desc_mn(sta, kWgBox), a_lo = make_desc_mn(sta + A_BYTES, kWgBox);
            const uint64_t b_hi = make_desc_mn(stb, kWgBox);
            const uint64_t b_lo = make_desc_mn(stb + B_BYTES, kWgBox);
            const bool first = kb == ci * p.chunk;
#pragma unroll
            for (int kk = 0; kk < kWgPix / 8; ++kk) {
              const uint64_t adv = (uint64_t)(kk * (1024 >> 4));   // 8 pixels = one 1024-byte row group
              mma(d_tmem, a_hi + adv, b_hi + adv, (first && kk == 0) ? 0u : 1u);
              mma(d_tmem, a_hi + adv, b_lo + adv, 1u);
              mma(d_tmem, a_lo + adv, b_hi + adv, 1u);
            }
            commit(empty_bar + stage);
            if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
            if (split) {
              commit(bempty_bar + stage_b);
              if (++stage_b == p.nstages_b) { stage_b = 0; phase_b ^= 1u; }
            }
          }
          if (alive) commit(tfull_bar + buf);
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
    // ---------------- epilogue: warps 4..11 ----------------
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    uint32_t acc_it = 0;
    bool alive = true;
    float acc[NH];
    for (int item = first_item; alive && item < p.nitems; item += item_step) {
      int mt, nb, tg, pb_lo, pb_hi;
      item_range(item, mt, nb, tg, pb_lo, pb_hi);
      const int KB = (pb_hi - pb_lo) * p.K1;
      const int nchunks = (KB + p.chunk - 1) / p.chunk;
      for (int ci = 0; ci < nchunks; ++ci, ++acc_it) {
        const uint32_t buf = acc_it & 1u, aphase = (acc_it >> 1) & 1u;
        if (!mbar_wait(tfull_bar + buf, aphase, abort_flag, p.spin_cap)) { alive = false; break; }
        tc_fence_after();
        const uint32_t tbase = tmem_base + buf * 256u + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * NH);
        // columns per round trip to tensor memory: as many as the registers hold beside the NH running sums (a
        // chunk is promoted in NH / TS round trips, and with short chunks their latency is what the tensor
        // pipe ends up waiting for)
        constexpr int TS = NH > 96 ? 16 : NH;      // (128 sums leave room for 16)
#pragma unroll
        for (int c0 = 0; c0 < NH; c0 += TS) {
          float tmp[TS];
#pragma unroll
          for (int c = 0; c < TS; c += 8) tc_ld8(tbase + (uint32_t)(c0 + c), &tmp[c]);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < TS; ++c) acc[c0 + c] = (ci == 0) ? tmp[c] : acc[c0 + c] + tmp[c];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (PAIR) mbar_arrive_cluster(mapa_shared(smem_u32(tempty_bar + buf), 0u));
          else mbar_arrive(tempty_bar + buf);
        }
      }
      if (!alive) break;
      // two-row tiles: lanes 64-127 hold the same output channels, paired with the filter row one up
      const int co = p.mpack ? (quad & 1) * 32 + lane : mt * MROWS + (int)rank * BM + quad * 32 + lane;
      const int urow = p.mpack ? tg - (quad >> 1) : 0;      // filter row of this lane's products (two-row tiles)
      if (co < p.cout && nchunks > 0 && (!p.mpack || (urow >= 0 && urow * p.kw < p.taps))) {
        float* row = p.dW + (size_t)co * p.taps * p.cin;
        // 16-byte vector reductions: cin % 4 == 0 and cb % 4 == 0 keep every group
        // of four inside one tap slot, wholly inside or outside the channel range,
        // and its address 16-byte aligned
#pragma unroll
        for (int c = 0; c < NH; c += 4) {
          const int col = half * NH + c;
          const int slot = col / p.cb;
          const int tap = p.mpack ? urow * p.kw + slot : tg * p.tpn + slot;
          const int ch = nb * p.cb + (col - slot * p.cb);
          if (tap < p.taps && ch < p.cin)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(row + (size_t)tap * p.cin + ch),
                         "f"(p.scale * acc[c]), "f"(p.scale * acc[c + 1]), "f"(p.scale * acc[c + 2]),
                         "f"(p.scale * acc[c + 3])
                         : "memory");
        }
      }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  if constexpr (PAIR) cluster_sync_all();     // neither CTA frees TMEM or exits while its peer may still use the pair's resources
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace tc
}  // namespace dk
