// tcgen05 path with CTA pairs (cta_group::2, sm_100a only) for shapes whose operand traffic,
// not the output write-back, limits a single-CTA tile (long K, tensor-bound FP16).
//
// Two CTAs of a cluster compute one 256(out-feature) x tile_t(token) tile of Y^T:
//   * CTA rank r keeps W rows [o0 + 128 r, o0 + 128 r + 128) (its half of the MMA M dimension)
//     and HALF of the X tile, tokens [t0 + r*tile_t/2, ...): the pair's tensor cores read the
//     other half of X straight from the peer's shared memory, so every CTA loads 1/2 of the X
//     bytes per unit of MMA work.  No TMA multicast: each CTA issues plain tiled loads for
//     its own shared memory, only the completion is counted on the leader's mbarrier.
//   * rank 0 (leader) issues tcgen05.cp / tcgen05.mma[.sp] with .cta_group::2; tcgen05.commit
//     with cluster multicast releases ring stages and publishes accumulators in both CTAs.
//   * each CTA drains its own 128 TMEM lanes x tile_t columns through the same TMA-store
//     epilogue as the single-CTA kernel; the peer's epilogue warps release the accumulator
//     buffer with remote arrives on the leader's mbarrier.
// Streaming operands only (no residency, no split-K, no decode); other cases use the
// single-CTA kernel.  All waits are bounded polls; the two CTAs meet at a cluster barrier
// before tensor memory is freed, so neither can exit while the other still targets it.
#include <atomic>
#include <cstdlib>

#include "nm_umma_common.cuh"

namespace nm {
namespace {

constexpr int kEpiWarps2 = 8;
constexpr int kThreads2 = 32 * (2 + kEpiWarps2);
constexpr uint32_t kPatchBytes2 = 4096;
constexpr size_t kMaxSmem2 = 227 * 1024;
constexpr uint32_t kMaxAcc2 = 2;

struct PairParams {
  int T, O;
  int tile_t;               // tokens per pair tile = MMA N (multiple of 32, <= 256)
  int stages;
  int acc_bufs;
  int tiles_o2;             // 256-row out-feature tiles
  int n_items;
  int total_ksteps;
  int w_fresh;              // the weight image is written by the launch just before: no W load ahead of the grid-dependency wait
  int out_f16;
  int out_i8;               // requantising epilogue (scale / bias / ReLU / saturate to int8)
  const float* epi_scale; const int32_t* epi_bias; int epi_relu;
  uint32_t tmem_cols;
  uint32_t spin_limit;      // polls after which a bounded wait gives up
  unsigned long long* trace;   // phase stamps (trace builds only; nullptr otherwise)
  int dbg;                     // trace builds only, bits: 1 = no MMAs are issued, 2 = no output is stored, 4 = the ring is loaded once and reused (timing experiments; wrong results)
  uint32_t* status;
};

// arrive on an mbarrier that may live in the peer CTA.  CTA-scope semantics on purpose: the
// arrival only tells the MMA warp that this warp's tcgen05.ld of the accumulator are done
// (ordered by tcgen05.fence::before_thread_sync); no generic-proxy data is handed over, and a
// cluster-scope release costs a memory fence of 1-2 us behind the CTA's in-flight stores.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tiled load into this CTA's shared memory; completion bytes go to an mbarrier of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
// commit of the pair's outstanding MMAs, arriving on the same-offset mbarrier of both CTAs
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
               "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tc_cp_128x128b_pair(uint32_t taddr, uint64_t sdesc) {
  asm volatile("{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
               "@e tcgen05.cp.cta_group::2.128x128b [%0], %1;\n\t}" ::"r"(taddr), "l"(sdesc) : "memory");
}
template <int DT>
__device__ __forceinline__ void tc_mma_dense_pair(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  if (DT == NM_I8) {
    asm volatile("{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "@e tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
  } else {
    asm volatile("{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "@e tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
  }
}
template <int DT>
__device__ __forceinline__ void tc_mma_sparse_pair(uint32_t d, uint64_t a, uint64_t b, uint32_t meta,
                                                   uint32_t idesc, uint32_t acc) {
  if (DT == NM_I8) {
    asm volatile("{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "@e tcgen05.mma.sp.cta_group::2.kind::i8 [%0], %1, %2, [%3], %4, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(meta), "r"(idesc), "r"(acc) : "memory");
  } else {
    asm volatile("{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "@e tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(meta), "r"(idesc), "r"(acc) : "memory");
  }
}

template <int DT, bool SP>
__host__ __device__ constexpr uint32_t meta_bytes2() { return SP ? (DT == NM_I8 ? 4096u : 2048u) : 0u; }
// per CTA and K step: 128 rows x 128 B of W values (+ metadata), then this CTA's half of the X tile
template <int DT, bool SP>
__host__ __device__ inline uint32_t stage_bytes2(int tile_t) {
  return 16384u + meta_bytes2<DT, SP>() + (SP ? 2u : 1u) * (uint32_t)(tile_t / 2) * 128u;
}
__host__ __device__ inline uint32_t tail_bytes2(int stages) {
  return kEpiWarps2 * kPatchBytes2 + 16u * (uint32_t)stages + 8u * 2u * kMaxAcc2 + 16u;
}

// ------------------------------------------------------------------ the pair kernel
template <int DT, bool SP>
__global__ void __launch_bounds__(kThreads2, 1)
nm_umma_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmM, const __grid_constant__ CUtensorMap tmY,
                    const PairParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sbytes = stage_bytes2<DT, SP>(p.tile_t);
  const uint32_t half_rows = (uint32_t)p.tile_t / 2u;
  const uint32_t b_atom_bytes = half_rows * 128u;
  const uint32_t ring_bytes = (uint32_t)p.stages * sbytes;
  const uint32_t patches = smem_base + ring_bytes;
  const uint32_t bars = patches + kEpiWarps2 * kPatchBytes2;
  const uint32_t bar_full = bars, bar_empty = bars + 8u * p.stages;
  const uint32_t bar_tfull = bars + 16u * p.stages, bar_tempty = bar_tfull + 8u * kMaxAcc2;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      gen_base + ring_bytes + kEpiWarps2 * kPatchBytes2 + 16u * p.stages + 8u * 2u * kMaxAcc2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const WaitCtx wctx{abort_flag, p.status, p.spin_limit};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();            // 0 = leader (issues the MMAs), 1 = peer
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    NM_STAMP(p.trace, 0);
    pdl_launch_dependents();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    prefetch_tensormap(&tmY);
    if (SP) prefetch_tensormap(&tmM);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);                 // the leader's arrive.expect_tx; bytes come from both CTAs
      mbar_init(bar_empty + 8u * s, 1);                // multicast commit of the leader's MMAs
    }
    for (int b = 0; b < (int)kMaxAcc2; ++b) {
      mbar_init(bar_tfull + 8u * b, 1);                // multicast commit: accumulator ready in both CTAs
      mbar_init(bar_tempty + 8u * b, 2 * kEpiWarps2);  // leader's copy is used: epilogue warps of both CTAs
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();                                  // barriers of both CTAs exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) NM_STAMP(p.trace, 1);
  const uint32_t tmem_meta = tmem_base + (uint32_t)(p.acc_bufs * p.tile_t);
  const int my_count = (p.n_items > pair) ? (p.n_items - 1 - pair) / n_pairs + 1 : 0;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs): own W rows, own half of the token tile
      // W tiles of the first ring-full of K steps are requested before the grid-dependency wait
      // (the packed weight never depends on the previous kernel); X only after it.
      // (they are requested by warp 1, which has nothing else to do yet: this thread goes straight to the
      // wait, so a CTA that starts after the previous grid has finished asks for X at once)
      const int pre = (my_count > 0 && !p.w_fresh) ? min(p.stages, p.total_ksteps) : 0;
      pdl_wait_prior_grid();
      NM_STAMP(p.trace, 2);
      NM_STAMP_VAL(p.trace, 12, my_count);
      bool ok = true, wrapped = false;
      // ring position kept incrementally (stage s, phase parity ph): no divisions in a lone thread
      uint32_t s = 0, ph = 0, sa = smem_base, armed = 0;
      [[maybe_unused]] long long cyc_empty = 0;     // trace builds: cycles spent waiting for a free stage
      for (int n = 0; n < my_count && ok; ++n) {
        const int item = pair + n * n_pairs;
        const int o0 = (item % p.tiles_o2) * 256 + (int)rank * 128;
        // A ragged last token tile is multiplied over its occupied 32-token chunks only (N = n_eff):
        // the two CTAs then hold the first and the second n_eff / 2 token rows of it.
        const int tile0 = (item / p.tiles_o2) * p.tile_t;
        int t0 = tile0 + (int)rank * (int)half_rows;
        if (p.T - tile0 < p.tile_t) t0 = tile0 + (int)rank * (((p.T - tile0 + 31) & ~31) >> 1);
        for (int ks = 0; ks < p.total_ksteps; ++ks) {
#ifdef NM_HAS_DBG
          if ((p.dbg & 4) && armed >= (uint32_t)p.stages) { n = my_count; break; }   // the ring is filled once and reused
#endif
          if (wrapped) {
            NM_WAIT_TIMED(cyc_empty, ok = mbar_wait(bar_empty + 8u * s, ph ^ 1u, wctx, 1));
            if (!ok) break;
          }
          const uint32_t full_leader = map_to_cta(bar_full + 8u * s, 0u);
          const uint32_t sm = sa + 16384u;
          const uint32_t sb = sm + meta_bytes2<DT, SP>();
          const bool w_prefetched = (n == 0 && ks < pre);
          if (rank == 0u && !w_prefetched) mbar_expect_tx(bar_full + 8u * s, 2u * sbytes);
          if (!w_prefetched) tma_load_2d_pair(sa, &tmA, full_leader, ks * 128, o0);
          if (SP) {
            tma_load_2d_pair(sb, &tmB, full_leader, ks * 256, t0);
            tma_load_2d_pair(sb + b_atom_bytes, &tmB, full_leader, ks * 256 + 128, t0);
          } else {
            tma_load_2d_pair(sb, &tmB, full_leader, ks * 128, t0);
          }
          if (SP && !w_prefetched) {
            const int blocks_per_step = (int)(meta_bytes2<DT, SP>() / 2048u);      // metadata map: one row per 2 KB block
            tma_load_2d_pair(sm, &tmM, full_leader, 0, ((o0 / kTileO) * p.total_ksteps + ks) * blocks_per_step);
          }
          ++armed;
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; wrapped = true; sa = smem_base; } else { sa += sbytes; }
        }
      }
      NM_STAMP_VAL(p.trace, 15, cyc_empty);
      // Before the pair leaves, every copy its producers issued must have landed (a CTA on the abort
      // path gives up its shared memory).  The full barriers live in the leader and count the bytes
      // of both CTAs, so the leader waits (bounded) for the latest use of every armed stage; the peer
      // cannot leave before the leader because of the cluster barrier at the end of the kernel.
      if (rank == 0u) {
        if (armed < (uint32_t)pre) armed = (uint32_t)pre;
        const uint32_t ns = armed < (uint32_t)p.stages ? armed : (uint32_t)p.stages;
        for (uint32_t d = 0; d < ns; ++d)
          mbar_wait_quiet(bar_full + 8u * ((armed - 1u - d) % (uint32_t)p.stages),
                          ((armed - 1u - d) / (uint32_t)p.stages) & 1u, p.spin_limit >> 2);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // Weight prefetch ahead of the grid-dependency wait (both CTAs, each its own W rows): the W
      // tiles and metadata of the first ring-full of K steps; the leader arms the barriers with the
      // byte count of the whole stage of both CTAs, the producers add the X tiles after their wait.
      const int pre = (my_count > 0 && !p.w_fresh) ? min(p.stages, p.total_ksteps) : 0;
      for (int i = 0; i < pre; ++i) {
        const int o0p = (pair % p.tiles_o2) * 256 + (int)rank * 128;
        const uint32_t full_leader = map_to_cta(bar_full + 8u * (uint32_t)i, 0u);
        const uint32_t sa = smem_base + (uint32_t)i * sbytes;
        if (rank == 0u) mbar_expect_tx(bar_full + 8u * (uint32_t)i, 2u * sbytes);
        tma_load_2d_pair(sa, &tmA, full_leader, i * 128, o0p);
        if (SP) tma_load_2d_pair(sa + 16384u, &tmM, full_leader, 0,
                                 ((o0p / kTileO) * p.total_ksteps + i) * (int)(meta_bytes2<DT, SP>() / 2048u));
      }
      // the X boxes of those K steps are pulled towards L2 (a hint, no data is consumed), so that
      // the first real loads after the wait do not pay the HBM latency
      for (int i = 0; i < pre; ++i) {
        const int tile0p = (pair / p.tiles_o2) * p.tile_t, n_leftp = p.T - tile0p;
        const int t0p = tile0p + (int)rank * ((n_leftp >= p.tile_t ? p.tile_t : ((n_leftp + 31) & ~31)) / 2);
        if (SP) {
          tma_prefetch_l2_2d(&tmB, i * 256, t0p);
          tma_prefetch_l2_2d(&tmB, i * 256 + 128, t0p);
        } else {
          tma_prefetch_l2_2d(&tmB, i * 128, t0p);
        }
      }
    }
    __syncwarp();
    if (rank == 0u) {
      // ---------------- MMA issuer (leader only): M = 256 across the pair, N = tile_t.  The whole
      // warp walks the loop in lockstep; the tcgen05 wrappers elect the lane that issues.
      uint32_t idesc = ((uint32_t)(p.tile_t >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      idesc |= (DT == NM_I8) ? ((2u << 4) | (1u << 7) | (1u << 10)) : (1u << 4);
      if (SP) idesc |= 1u << 2;
      bool ok = true;
      // This thread alone paces the pair's tensor cores: ring position advanced incrementally, one
      // descriptor per operand and K step, constant offsets for the four MMAs.
      uint32_t s = 0, ph = 0, sa = smem_base;
      // token-tile index of this pair's items, advanced without a division per item
      const int step_t = n_pairs / p.tiles_o2, step_o = n_pairs % p.tiles_o2;
      int t_idx = pair / p.tiles_o2, o_idx = pair % p.tiles_o2;
      [[maybe_unused]] long long cyc_full = 0, cyc_tempty = 0;      // trace builds: cycles spent inside the two waits of this warp
      pdl_wait_prior_grid();      // keeps the previous grid's run time out of the bounded waits below
      for (int n = 0; n < my_count && ok; ++n) {
        const uint32_t buf = (uint32_t)n % (uint32_t)p.acc_bufs, use = (uint32_t)n / (uint32_t)p.acc_bufs;
        if (use >= 1u) {       // both CTAs' epilogues must have drained this accumulator buffer
          NM_WAIT_TIMED(cyc_tempty, ok = mbar_wait(bar_tempty + 8u * buf, (use - 1u) & 1u, wctx, 4));
          ok = __all_sync(0xffffffffu, ok);        // every lane polls; also re-converges the warp after the poll loop
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem_base + buf * (uint32_t)p.tile_t;
        const int n_left = p.T - t_idx * p.tile_t;
        const uint32_t idesc_n = n_left >= p.tile_t ? idesc : ((idesc & ~(0x3fu << 17)) | ((uint32_t)((n_left + 31) >> 5) << 19));
        t_idx += step_t; o_idx += step_o;
        if (o_idx >= p.tiles_o2) { o_idx -= p.tiles_o2; ++t_idx; }
        for (int ks = 0; ks < p.total_ksteps; ++ks) {
#ifdef NM_HAS_DBG
          if (!((p.dbg & 4) && (n > 0 || ks >= p.stages)))      // 4 = no loads after the first ring-full: the MMAs run alone
#endif
          NM_WAIT_TIMED(cyc_full, ok = mbar_wait(bar_full + 8u * s, ph, wctx, 2));
          ok = __all_sync(0xffffffffu, ok);        // every lane polls; also re-converges the warp after the poll loop
          if (!ok) break;
          tc_fence_after();
          if (n == 0 && ks == 0 && lane == 0) NM_STAMP(p.trace, 3);
          const uint32_t sm = sa + 16384u;
          const uint32_t sb = sm + meta_bytes2<DT, SP>();
          const uint32_t meta_cols = tmem_meta + s * 8u;
#ifdef NM_HAS_DBG
          if (p.dbg & 1) { tc_commit_pair(bar_empty + 8u * s); if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; sa = smem_base; } else { sa += sbytes; } continue; }
#endif
          if (SP) {
            tc_cp_128x128b_pair(meta_cols, desc_meta(sm));
            if (DT == NM_I8) tc_cp_128x128b_pair(meta_cols + 4u, desc_meta(sm + 2048u));
          }
          // start-address fields count 16-byte units: +2 per 32 B of K (A, dense B), +4 per 64 B
          const uint64_t da0 = desc_sw128(sa), db0 = desc_sw128(sb);
          const uint64_t db1 = SP ? desc_sw128(sb + b_atom_bytes) : 0ull;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t acc = (ks > 0 || j > 0) ? 1u : 0u;
            const uint64_t da = da0 + (uint64_t)(2 * j);
            if (SP) {
              const uint64_t db = ((j >> 1) ? db1 : db0) + (uint64_t)(4 * (j & 1));
              if (DT == NM_I8) tc_mma_sparse_pair<DT>(d_tmem, da, db, meta_cols + 2u * j, idesc_n, acc);
              else tc_mma_sparse_pair<DT>(d_tmem, da, db, meta_cols + (uint32_t)(j & 2), idesc_n | (uint32_t)(j & 1), acc);
            } else {
              tc_mma_dense_pair<DT>(d_tmem, da, db0 + (uint64_t)(2 * j), idesc_n, acc);
            }
          }
          tc_commit_pair(bar_empty + 8u * s);          // frees stage s in both CTAs
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; sa = smem_base; } else { sa += sbytes; }
        }
        if (!ok) break;
        tc_commit_pair(bar_tfull + 8u * buf);          // accumulator ready in both CTAs
        if (lane == 0) { if (n == 0) NM_STAMP(p.trace, 4); if (n + 1 == my_count) NM_STAMP(p.trace, 5); }
      }
      if (lane == 0) { NM_STAMP_VAL(p.trace, 13, cyc_full); NM_STAMP_VAL(p.trace, 14, cyc_tempty); }
    }
  } else {
    // ---------------- epilogue warps (both CTAs): own 128 out-feature rows, all tile_t tokens
    const int e = warp - 2, q = warp & 3, h = e >> 2;
    const uint32_t patch = patches + (uint32_t)e * kPatchBytes2;
    const int ob = (DT == NM_F16 && p.out_f16) ? 2 : ((DT == NM_I8 && p.out_i8) ? 1 : 4);
    [[maybe_unused]] long long cyc_tfull = 0;      // trace builds: cycles spent waiting for an accumulator
    pdl_wait_prior_grid();
    for (int n = 0; n < my_count; ++n) {
      const int item = pair + n * n_pairs;
      const int o0 = (item % p.tiles_o2) * 256 + (int)rank * 128;
      const int t0 = (item / p.tiles_o2) * p.tile_t;
      const uint32_t buf = (uint32_t)n % (uint32_t)p.acc_bufs, use = (uint32_t)n / (uint32_t)p.acc_bufs;
      uint32_t ok = 1;
      if (lane == 0) NM_WAIT_TIMED(cyc_tfull, ok = mbar_wait(bar_tfull + 8u * buf, use & 1u, wctx, 3) ? 1u : 0u);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      if (n == 0 && e == 0 && lane == 0) NM_STAMP(p.trace, 6);
      const int o_base = o0 + q * 32;
      float q_scale = 1.0f;
      const float q_lo = p.epi_relu ? 0.0f : -128.0f;
      int32_t q_bias = 0;
      if (ob == 1 && o_base + lane < p.O) {
        q_scale = __ldg(p.epi_scale + o_base + lane);
        if (p.epi_bias) q_bias = __ldg(p.epi_bias + o_base + lane);
      }
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)p.tile_t;
      // the two warps of a quadrant swap the even / odd 32-column chunks from tile to tile, so an
      // odd chunk count (tile_t = 96, 160, 224) loads them equally over time
      for (int cc = (h ^ (n & 1)) * 32; cc < p.tile_t; cc += 64) {
        const int t = t0 + cc;
        if (t >= p.T) break;
        uint32_t r[32];
#ifdef NM_HAS_DBG
        if (p.dbg & 2) continue;
#endif
        if (lane == 0) tma_store_wait_read();
        __syncwarp();
        tc_ld_32x32(lane_addr + (uint32_t)cc, r);
        if (ob == 4) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(patch + (uint32_t)j * 128u + (uint32_t)lane * 4u), "r"(r[j]) : "memory");
        } else if (ob == 2) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const unsigned short hbits = __half_as_ushort(__float2half_rn(__uint_as_float(r[j])));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(patch + (uint32_t)j * 64u + (uint32_t)lane * 2u), "h"(hbits) : "memory");
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t qv = requant_low_byte(r[j], q_scale, q_bias, q_lo);     // st.shared.u8 keeps the low byte
            asm volatile("st.shared.u8 [%0], %1;" ::"r"(patch + (uint32_t)j * 32u + (uint32_t)lane), "r"(qv) : "memory");
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && o_base < p.O) tma_store_2d(&tmY, patch, o_base * ob, t);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(bar_tempty + 8u * buf, 0u));   // the leader's MMA warp waits for both CTAs
      if (e == 0 && lane == 0) { if (n == 0) NM_STAMP(p.trace, 7); if (n + 1 == my_count) NM_STAMP(p.trace, 8); }
    }
    // the staging patches must outlive the stores' reads of them; the writes complete with the grid
    if (lane == 0) tma_store_wait_read();
    if (e == 0 && lane == 0) { NM_STAMP(p.trace, 9); NM_STAMP_VAL(p.trace, 11, cyc_tfull); }
  }

  // neither CTA may free tensor memory or exit while its partner can still signal or read it
  tc_fence_before();
  cluster_sync_all();
  if (threadIdx.x == 0) NM_STAMP(p.trace, 10);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------ host side
template <int DT, bool SP>
nm_status launch_pair(const SpmmArgs& a, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmM,
                      const CUtensorMap& tmY, PairParams& p) {
  auto smem_need = [&](int stages) { return 1024 + (size_t)stages * stage_bytes2<DT, SP>(p.tile_t) + tail_bytes2(stages); };
  while (p.stages > 1 && smem_need(p.stages) > kMaxSmem2) --p.stages;
  if (smem_need(p.stages) > kMaxSmem2) return NM_ERR_UNSUPPORTED;
  const uint32_t meta_cols = SP ? 8u * (uint32_t)p.stages : 0u;
  p.acc_bufs = (int)((512u - meta_cols) / (uint32_t)p.tile_t);
  if (p.acc_bufs > (int)kMaxAcc2) p.acc_bufs = (int)kMaxAcc2;
  if (p.acc_bufs < 1) p.acc_bufs = 1;
  p.tmem_cols = pow2_cols((uint32_t)(p.acc_bufs * p.tile_t) + meta_cols);
  if (p.tmem_cols > 512) return NM_ERR_INVALID_ARG;
  // the attribute belongs to the (function, device) pair: remember per device
  static std::atomic<uint64_t> configured{0};
  const int slot = device_slot();
  if (slot == 63 || !((configured.load(std::memory_order_relaxed) >> slot) & 1ull)) {
    if (cudaFuncSetAttribute(nm_umma_pair_kernel<DT, SP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem2) != cudaSuccess)
      return NM_ERR_CUDA;
    configured.fetch_or(1ull << slot, std::memory_order_relaxed);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * (sm_count() / 2)));
  cfg.blockDim = dim3(kThreads2);
  cfg.dynamicSmemBytes = smem_need(p.stages);
  cfg.stream = static_cast<cudaStream_t>(a.stream);
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // The tile list is static per pair, so every pair must be resident at once: ask how many
  // clusters of this footprint the device can hold (GPC boundaries may leave an SM unpaired).
  // (one entry: a stream of calls normally alternates between few footprints on one device; a
  // concurrent caller that races on it only repeats the query)
  static std::atomic<uint64_t> cache_word{0};       // dev (8 bits) | smem bytes (24 bits) | pairs (16 bits), 0 = empty
  const uint64_t key = ((uint64_t)(slot & 0xff) << 40) | ((uint64_t)(cfg.dynamicSmemBytes & 0xffffff) << 16);
  uint64_t cw = cache_word.load(std::memory_order_relaxed);
  int max_pairs = 0;
  if (slot != 63 && cw != 0 && (cw & ~0xffffull) == key) {
    max_pairs = (int)(cw & 0xffff);
  } else {
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, nm_umma_pair_kernel<DT, SP>, &cfg) != cudaSuccess || n < 1) {
      cudaGetLastError();
      return NM_ERR_CUDA;
    }
    max_pairs = n > 0xffff ? 0xffff : n;
    cache_word.store(key | (uint64_t)max_pairs, std::memory_order_relaxed);
  }
  const int pairs = p.n_items < max_pairs ? p.n_items : max_pairs;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.numAttrs = 2;
  if (cudaLaunchKernelEx(&cfg, nm_umma_pair_kernel<DT, SP>, tmA, tmB, tmM, tmY, p) != cudaSuccess) {
    cudaGetLastError();
    return NM_ERR_CUDA;
  }
  count_launch();
  return NM_OK;
}

}  // namespace

// Runs the plan on CTA pairs when it can (*handled = true); otherwise leaves the call to the
// single-CTA kernel (*handled = false): split-K, operand residency, the decode path, outputs
// that TMA cannot address, or fewer than 129 out-features.
nm_status launch_umma_pair(const SpmmArgs& a, bool* handled) {
  *handled = false;
  const nm_weight* w = a.w;
  const nm_plan& pl = a.plan;
  const bool sp = pl.path == NM_PATH_UMMA_SP24;
  if (pl.path != NM_PATH_UMMA_SP24 && pl.path != NM_PATH_UMMA_DENSE) return NM_OK;
  if (pl.split_k > 1 || pl.resident != NM_RES_NONE || w->O <= kTileO) return NM_OK;
  if (pl.tile_t < 32 || pl.tile_t > 256 || pl.tile_t % 32 != 0 || pl.stages < 1 || pl.stages > 8) return NM_OK;
  const int eb = elem_bytes(w->dtype), ob = out_bytes(a.od);
  if ((reinterpret_cast<uintptr_t>(a.Y) & 15) || ((uint64_t)a.ldy * ob) % 16 != 0) return NM_OK;
  if ((reinterpret_cast<uintptr_t>(a.X) & 15) || ((uint64_t)a.ldx * eb) % 16 != 0) return NM_ERR_ALIGN;

  const uint8_t* base = static_cast<const uint8_t*>(w->dev_base);
  const void* a_ptr;
  uint64_t a_row_bytes, a_pitch;
  if (sp) {
    if (!(w->images & NM_IMG_HW24)) return NM_ERR_UNSUPPORTED;
    a_ptr = base + w->off_hw24_values;
    a_row_bytes = (uint64_t)((w->K + 3) / 4) * 2 * eb;
    a_pitch = w->hw24_row_bytes;
  } else if (w->n == w->m) {
    a_ptr = base + w->off_canonical + 64;
    a_row_bytes = (uint64_t)w->K * eb;
    a_pitch = round_up(a_row_bytes, 16);
  } else {
    if (!(w->images & NM_IMG_DENSE)) return NM_ERR_UNSUPPORTED;
    a_ptr = base + w->off_dense;
    a_row_bytes = (uint64_t)w->K * eb;
    a_pitch = w->dense_row_bytes;
  }
  PairParams p{};
  p.T = a.T; p.O = w->O; p.tile_t = pl.tile_t; p.stages = pl.stages;
  p.total_ksteps = (int)((a_row_bytes + 127) / 128);
  p.out_f16 = a.od == NM_OUT_F16;
  p.out_i8 = a.od == NM_OUT_I8;
  p.epi_scale = a.epi.scale_dev; p.epi_bias = a.epi.bias_dev; p.epi_relu = a.epi.relu;
  if (p.out_i8 && !p.epi_scale) return NM_ERR_INVALID_ARG;
  p.status = a.status;
  p.spin_limit = kSpinLimit;
  p.trace = trace_buffer();
#ifdef NM_HAS_DBG
  { const char* e = getenv("NM_DBG"); p.dbg = e ? atoi(e) : 0; }
#endif
  p.w_fresh = a.w_fresh ? 1 : 0;
  p.tiles_o2 = ceil_div(w->O, 256);
  const int64_t items = (int64_t)p.tiles_o2 * ceil_div(a.T, pl.tile_t);
  if (items > 0x7fffffff) return NM_OK;
  p.n_items = (int)items;
  const uint32_t mb = sp ? (w->dtype == NM_I8 ? 4096u : 2048u) : 0u;
  if (sp && (uint64_t)w->hw24_meta_kblocks * kMetaBlockBytes != (uint64_t)p.total_ksteps * mb) return NM_OK;

  CUtensorMap tmA, tmB, tmM, tmY;
  if (!make_map(&tmA, a_ptr, a_row_bytes, (uint64_t)w->O, a_pitch, 128u, kTileO, true)) return NM_ERR_CUDA;
  if (!make_map(&tmB, a.X, (uint64_t)w->K * eb, (uint64_t)a.T, (uint64_t)a.ldx * eb, 128u, (uint32_t)pl.tile_t / 2u, true))
    return NM_ERR_CUDA;
  if (sp) {
    // the metadata blocks as a 2-D tensor of 2 KB rows: one box = the blocks of one K step
    const uint64_t n_blocks = (uint64_t)ceil_div(w->O, kTileO) * w->hw24_meta_kblocks;
    if (!make_meta_map(&tmM, base + w->off_hw24_meta, n_blocks, mb / 2048u)) return NM_ERR_CUDA;
  } else {
    tmM = tmB;
  }
  if (!make_map(&tmY, a.Y, (uint64_t)w->O * ob, (uint64_t)a.T, (uint64_t)a.ldy * ob, 32u * ob, 32u, false)) return NM_ERR_CUDA;

  *handled = true;
  if (w->dtype == NM_I8) return sp ? launch_pair<NM_I8, true>(a, tmA, tmB, tmM, tmY, p) : launch_pair<NM_I8, false>(a, tmA, tmB, tmM, tmY, p);
  return sp ? launch_pair<NM_F16, true>(a, tmA, tmB, tmM, tmY, p) : launch_pair<NM_F16, false>(a, tmA, tmB, tmM, tmY, p);
}

}  // namespace nm
