// Forward 3xTF32 implicit-GEMM kernel on CTA pairs (tcgen05 cta_group::2).
//
// Why pairs.  With one CTA per tile the kernel moves 80 KB from L2 into shared
// memory per k-block (128 rows of W and (K+2)*P activation rows, each as a
// hi/lo pair); measured on B200 the MMA thread then waits for data ~40 % of
// the time with the tensor pipe ~55 % busy.  A pair of CTAs on neighbouring
// SMs computes a 256 x N tile with ONE instruction stream: each CTA stages its
// own 128 rows of W but only HALF of the activation rows, and the tensor cores
// of the two SMs share the halves.  Per SM that is 56 KB per k-block instead
// of 80 KB, for the same flops, and four stages fit instead of two.
//
// Roles.  In both CTAs warp 0 loads this CTA's operands (the byte counts of
// both CTAs arrive on the barrier of the leader, CTA rank 0 of the pair).
// Warp 1 of the leader issues every MMA and signals, with multicast commits,
// the "stage free" and "accumulator chunk ready" barriers of both CTAs.
// Warps 4-11 of each CTA drain that CTA's 128 TMEM lanes exactly as in the
// single-CTA kernel and release the chunk on the leader's barrier.
//
// All waits are bounded; a CTA whose wait expires raises the abort flag,
// reports DK_ERR_TIMEOUT, and both CTAs still meet at the closing cluster
// barrier before TMEM is freed.
#pragma once

#include "dk_tc_kernel.cuh"

namespace dk {
namespace tc {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
// shared::cluster address of `local` (a shared::cta address) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// bounded wait on a local barrier that the peer CTA's threads arrive on too (their writes to their own
// shared memory, which the pair's tensor-core instruction reads, must be visible: cluster scope)
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned cap) {
  for (unsigned i = 0; i < cap; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// TMA loads of a CTA pair: the data lands in the issuing CTA's shared memory,
// the bytes are counted on the barrier at cluster address `bar` (the leader's).
__device__ __forceinline__ void tma_pair_load_3d(void* dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_5d(void* dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tc_pair_mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives, once the MMAs issued so far have completed, on the barrier at this
// shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void tc_pair_commit(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(smem_u32(bar)), "h"(mask)
      : "memory");
}

constexpr int BM2 = 2 * BM;     // output channels of a pair tile

template <int MODE, int K>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsTc, 1)
tc_fwd_pair_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                   const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                   const TcParams p) {
  constexpr int BK = 32;
  constexpr int E = K + 2, EH = E / 2;
  constexpr int P = tile_pixels(K), PH = P / 2;
  constexpr int BN = E * P;
  constexpr int SWZ = BK * 4;
  constexpr int A_BYTES = BM * BK * 4;            // this CTA's 128 rows of W
  constexpr int SUB = P * BK * 4;                 // one encoding's pixels
  constexpr int B_BYTES = EH * SUB;               // this CTA's half of the activation rows
  constexpr int STAGE_BYTES = 2 * (A_BYTES + B_BYTES);
  static_assert(E % 2 == 0, "the pair kernel splits the encodings in two halves");
  static_assert(BN % 16 == 0 && BN <= 256 && PH % 8 == 0, "illegal tile");
  extern __shared__ unsigned char smem_raw[];
  __shared__ unsigned char s_chunk[kChunkTabMax];      // chunk lengths per virtual batch (see tile_chunk)
  load_chunk_tab(p, s_chunk);
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  unsigned char* ctrl = smem + (size_t)p.nstages * STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctrl);     // used in the leader only
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tfull_bar = empty_bar + kMaxStages;
  uint64_t* tempty_bar = tfull_bar + 2;                       // used in the leader only
  // with the second TF32 term derived in the kernel: a CTA's own activation box has landed (transaction bytes),
  // and, in the leader, both CTAs' converter warps have derived the second term of a stage (4 arrivals)
  uint64_t* bfull_bar = tempty_bar + 2;
  uint64_t* ready_bar = bfull_bar + kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ready_bar + kMaxStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int nwork = p.ntiles * p.ksplit;     // work item = (pair tile, contraction slice)

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.nstages; ++s) {
      mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); mbar_init(bfull_bar + s, 1); mbar_init(ready_bar + s, 4);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, 2 * kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {      // one warp of each CTA of the pair takes part in the allocation
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();      // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  static_assert(40 * 128 + 232 * 256 <= 168 * kThreadsTc, "setmaxnreg budget exceeds the CTA's register pool");
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    int stage = 0, issued = 0;
    uint32_t phase = 0;
    bool alive = true;
    int round = 0;
    for (int w = pair; alive && w < nwork; w += npairs, ++round) {
      // pace (see tc_fwd_kernel): the leaders meet every pace_every rounds; the peer's copies follow within the ring
      if (p.pace != nullptr && rank == 0 && lane == 0 && round > 0 && round % p.pace_every == 0) {
        const unsigned int target = (unsigned int)(round / p.pace_every) * (unsigned int)npairs;
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
      const int x0 = wt * p.bw * p.stride - p.pad, y0 = ht * p.bh * p.stride - p.pad, g0 = gt * p.bg;
      const int m0 = mt * BM2 + (int)rank * BM;
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag, p.spin_cap) ? 1 : 0;
          if (ok && rank == 0)
            mbar_expect_tx(full_bar + stage, (uint32_t)(2 * (STAGE_BYTES - (p.nprod == 2 ? A_BYTES : 0) -
                                                             (p.lo_inkernel ? 2 * B_BYTES : 0))));
          if (ok && p.lo_inkernel) mbar_expect_tx(bfull_bar + stage, (uint32_t)B_BYTES);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { alive = false; break; }
        if (issued++ == p.withhold) { alive = false; break; }      // test hook: armed, nothing copied
        const int tap = kb / p.CB, c0 = (kb - tap * p.CB) * BK;
        const int u = tap / p.kw, v = tap - u * p.kw;
        unsigned char* st = smem + (size_t)stage * STAGE_BYTES;
        const uint32_t bar = mapa_shared(smem_u32(full_bar + stage), 0u);
        if (lane == 0) {
          tma_pair_load_3d(st, &map_a_hi, bar, c0, tap, m0);
        } else if (lane == 1) {
          if (p.nprod == 3) tma_pair_load_3d(st + A_BYTES, &map_a_lo, bar, c0, tap, m0);
        } else if (p.b_onebox) {
          // one box over this CTA's half of the encodings per TF32 term (see tc_fwd_kernel)
          if (lane == 2) {
            // (second term derived here: the box is counted on this CTA's own barrier, for its converter warps)
            const uint32_t bbar = p.lo_inkernel ? mapa_shared(smem_u32(bfull_bar + stage), rank) : bar;
            tma_pair_load_5d(st + 2 * A_BYTES, &map_b_hi, bbar, c0, x0 + v, y0 + u, (int)rank * EH, g0);
          } else if (lane == 3 && !p.lo_inkernel) {
            tma_pair_load_5d(st + 2 * A_BYTES + B_BYTES, &map_b_lo, bar, c0, x0 + v, y0 + u, (int)rank * EH, g0);
          }
        } else if (lane < 2 + 2 * EH) {
          const int i = (lane - 2) >> 1;
          const int e = (int)rank * EH + i;
          // (second term derived here: the boxes are counted on this CTA's own barrier, and none is fetched for
          // the second term; the transaction bytes each barrier expects are set accordingly above)
          if ((lane & 1) == 0)
            tma_pair_load_5d(st + 2 * A_BYTES + i * SUB, &map_b_hi,
                             p.lo_inkernel ? mapa_shared(smem_u32(bfull_bar + stage), rank) : bar, c0, x0 + v, y0 + u, e,
                             g0);
          else if (!p.lo_inkernel)
            tma_pair_load_5d(st + 2 * A_BYTES + B_BYTES + i * SUB, &map_b_lo, bar, c0, x0 + v, y0 + u, e, g0);
        }
        __syncwarp();
        if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
      }
      if (p.pace != nullptr && alive && rank == 0 && lane == 0 && (round + 1) % p.pace_every == 0) atomicAdd(p.pace, 1u);
    }
  } else if (warp == 1 && rank == 0) {
    // ---------------- MMA issuer (leader only) ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                 ((uint32_t)(BM2 >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t acc_it = 0;
      bool alive = true;
      for (int w = pair; alive && w < nwork; w += npairs) {
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
            // (both CTAs' activation boxes have landed and their second terms are derived)
            if (p.lo_inkernel && !mbar_wait_cluster(ready_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
            tc_fence_after();
            const uint32_t st = smem_u32(smem + (size_t)stage * STAGE_BYTES);
            const uint64_t a_hi = make_desc<SWZ>(st), a_lo = make_desc<SWZ>(st + A_BYTES);
            const uint64_t b_hi = make_desc<SWZ>(st + 2 * A_BYTES);
            const uint64_t b_lo = make_desc<SWZ>(st + 2 * A_BYTES + B_BYTES);
            const bool first = kb == kb_beg;
#pragma unroll
            for (int kk = 0; kk < BK / 8; ++kk) {
              const uint64_t adv = (uint64_t)(kk * 2);     // 32 bytes per k-step, in 16-byte units
              tc_pair_mma_tf32(d_tmem, a_hi + adv, b_hi + adv, idesc, (first && kk == 0) ? 0u : 1u);
              tc_pair_mma_tf32(d_tmem, a_hi + adv, b_lo + adv, idesc, 1u);
              if (p.nprod == 3) tc_pair_mma_tf32(d_tmem, a_lo + adv, b_hi + adv, idesc, 1u);
            }
            tc_pair_commit(empty_bar + stage);
            if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
          }
          if (alive) tc_pair_commit(tfull_bar + buf);
        }
      }
    }
  } else if (p.lo_inkernel && warp >= 2) {
    // ---------------- converters: warps 2 and 3 of both CTAs ----------------
    // second TF32 term of this CTA's half of the stage's activations (see tc_fwd_kernel); done is reported to
    // the leader, whose MMA thread issues for both CTAs
    const int ctid = (int)threadIdx.x - 64;
    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;
    for (int w = pair; alive && w < nwork; w += npairs) {
      const int ks = w % p.ksplit;
      const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        if (!mbar_wait(bfull_bar + stage, phase, abort_flag, p.spin_cap)) { alive = false; break; }
        const float4* src = reinterpret_cast<const float4*>(smem + (size_t)stage * STAGE_BYTES + 2 * A_BYTES);
        float4* dst = reinterpret_cast<float4*>(smem + (size_t)stage * STAGE_BYTES + 2 * A_BYTES + B_BYTES);
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
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(ready_bar + stage), 0u));
        if (++stage == p.nstages) { stage = 0; phase ^= 1u; }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
    // ---------------- epilogue: warps 4..11 of both CTAs ----------------
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    uint32_t acc_it = 0;
    bool alive = true;
    float acc[E][PH];
    for (int w = pair; alive && w < nwork; w += npairs) {
      const int t = w / p.ksplit, ks = w - t * p.ksplit;
      const int kb_lo = ks * p.kb_per_split, kb_hi = min(p.KB, kb_lo + p.kb_per_split);
      const int chunk = tile_chunk(p, s_chunk, t);
      const int nchunks = (kb_hi - kb_lo + chunk - 1) / chunk;
      const int mt = t % p.MT;
      int nt = t / p.MT;
      const int wt = nt % p.WT; nt /= p.WT;
      const int ht = nt % p.HT;
      const int gt = p.gt0 + nt / p.HT;
      const int co = mt * BM2 + (int)rank * BM + quad * 32 + lane;
      const bool co_ok = co < p.cout;

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
              const uint32_t col = tile_column<P>(p.gbox, EH, e0 + de, half);
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
        if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(tempty_bar + buf), 0u));
      }
      if (!alive) break;
      tile_epilogue<MODE, K>(p, acc, half, lane, co, co_ok, gt, ht, wt);
    }
    tail_finalize<MODE, K>(p, (int)threadIdx.x - 128, alive, abort_flag + 1);
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, (int)DK_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(16384);
    __syncthreads();
  }
  cluster_sync_all();      // neither CTA frees TMEM or exits while its peer may still use the pair's resources
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace tc
}  // namespace dk
