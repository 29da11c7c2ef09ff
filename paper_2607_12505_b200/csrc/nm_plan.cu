// Shape-adaptive launch planner (Section 4.3, "Adaptive Parallelism").  Pure host code.
//
// The paper's rule has two parts: "parallelism priority" -- raise splitK until the grid
// has enough blocks to occupy every SM -- and "controlled reduction" -- splitK comes from
// a small discrete set aligned to the MMA K step, and shrinks again when K is short or
// the partial-sum traffic would dominate.  Here a block is one 128 x tile_t output tile
// (x one K slice); the K step is 128 B of the A operand per row.
#include <cuda_runtime.h>

#include "nm_internal.h"

namespace nm {

static int pick_path(int n, int m, uint32_t images, int row_bytes) {
  // one dense K step holds the whole row: the dense MMA wins when both images exist
  const bool short_k = row_bytes <= 128 && (n == m || (images & NM_IMG_DENSE));
  if ((images & NM_IMG_HW24) && !short_k) return NM_PATH_UMMA_SP24;
  if (n == m || (images & NM_IMG_DENSE)) return NM_PATH_UMMA_DENSE;
  // Only the canonical image exists.  Decoding it on chip repeats the work for every token tile that
  // meets the W tile (measured 2-17x slower than a pre-arranged dense image); writing the dense rows
  // once into the workspace and running the dense path on that copy costs one small extra launch.
  return NM_PATH_UMMA_EXPAND;
}

nm_status plan_shape(int T, int O, int K, int n, int m, int dt, int od, uint32_t images, int n_sms, nm_plan* out) {
  if (!out || T < 1) return NM_ERR_INVALID_ARG;
  CanonGeom g;
  nm_status st = canon_geom(O, K, n, m, dt, &g);
  if (st != NM_OK) return st;
  if (dt == NM_I8 ? (od != NM_OUT_I32 && od != NM_OUT_I8) : (od != NM_OUT_F32 && od != NM_OUT_F16)) return NM_ERR_INVALID_ARG;
  if (n_sms <= 0) n_sms = kDefaultSMs;
  nm_plan p{};
  p.path = pick_path(n, m, images, K * g.eb);
  p.cta_group = 1;
  p.split_k = 1;
  p.issuers = 1;
  p.tile_o = kTileO;
  if (p.path == NM_PATH_SIMT) {
    p.image = NM_IMG_CANONICAL;
    p.tile_t = 8; p.stages = 1;
    *out = p;
    return NM_OK;
  }
  const bool sp = p.path == NM_PATH_UMMA_SP24;
  p.image = sp ? NM_IMG_HW24 : ((n == m || p.path == NM_PATH_UMMA_DECODE || p.path == NM_PATH_UMMA_EXPAND) ? NM_IMG_CANONICAL : NM_IMG_DENSE);
  const int eb = g.eb;
  // K steps: 128 B of A per row and step (compressed bytes on the sparse path).
  const int a_row_bytes = sp ? ((K + 3) / 4) * 2 * eb : K * eb;
  const int ksteps = ceil_div(a_row_bytes, 128);

  // ---- choose (CTA group, token tile, split-K) by a small makespan model fitted on B200.
  // The paper's rule (Section 4.3) is kept as the structure of the search: split-K comes from a
  // small discrete set aligned to the MMA K step and is only admitted while it buys parallelism
  // (more work items than one round of the grid would leave SMs idle) and each slice keeps two K
  // steps; "reduction dominates" is the merge term of the model.  The model itself:
  //   * a persistent grid of U units (SMs, or SM pairs) walks ceil(items / U) rounds;
  //   * one item costs the largest of its load time (operand bytes per CTA at ~80 B/ns), its
  //     store time (tile bytes at ~55 B/ns per SM) and its MMA time (dense-equivalent ops at the
  //     measured per-SM tensor rate of its kind), plus 7-16 % of the other two (imperfect
  //     overlap) and a hand-off between tiles;
  //   * a launch pays ~3 us of pipeline ramp (0.6 us more for CTA pairs), a split-K launch a ~1.5 us merge pass plus the
  //     partial-sum traffic.
  const double kPortBytesPerUs = 80e3, kStoreBytesPerUs = 55e3, kRampUs = 3.0, kPairRampUs = 0.56, kMergeUs = 1.5;
  const double kOverlap[2] = {0.089, 0.163}, kHandoffUs[2] = {0.11, 0.40};
  // a K step cannot be issued faster than its tensor-core instructions leave the one issuing
  // thread (4 MMAs, a commit, and 1-2 metadata copies on the sparse path)
  const double kStepIssueUs[2] = {0.233, 0.344};
  // a second issuing warp (even / odd K steps into two accumulators) brings that to 57 %
  const double kTwoIssuerFactor = 0.57;
  // dense-equivalent ops per microsecond and SM: [sparse][pair]
  const double kMmaRateI8[2][2] = {{19.5e6, 19.5e6}, {30e6, 37e6}};
  const double kMmaRateF16[2][2] = {{10.5e6, 10.5e6}, {15e6, 20e6}};
  const uint32_t a_part = 16384u + (sp ? (dt == NM_I8 ? 4096u : 2048u) : 0u);
  const int t_cap = T < 224 ? (int)round_up((uint64_t)T, 32) : 256;
  const bool pairs_ok = p.path != NM_PATH_UMMA_DECODE && O > kTileO && n_sms >= 2;
  const double in_bytes = (double)T * K * eb + (double)O * a_row_bytes;
  double best_cost = -1.0;
  int best_cg = 1, best_t = 128, best_split = 1, best_issuers = 1;
  for (int cg = 1; cg <= (pairs_ok ? 2 : 1); ++cg) {
    const int units = cg == 1 ? n_sms : n_sms / 2;
    for (int cand = 32; cand <= 256; cand += 32) {
      if (cand > t_cap) break;
      if (cand < 64 && t_cap >= 64 && T > 256) continue;  // 32-token tiles only for small token counts
      // Dense-MMA CTA pairs: two 256-token accumulators fill tensor memory exactly (no metadata columns)
      // and a 256-token tile moves the fewest operand bytes per MMA; on every shape swept the pair kernel
      // was fastest there (3-14 % ahead of the 160-224 tokens the cost terms below would pick).
      if (cg == 2 && !sp && T >= 512 && cand != 256) continue;
      // the last token tile is multiplied over its occupied 32-token chunks only
      const int rag_tokens = T % cand, rag_n = (rag_tokens + 31) / 32 * 32;
      for (int s = 1; s <= kMaxSplitK; s *= 2) {
        if (s > 1 && (cg == 2 || p.path == NM_PATH_UMMA_DECODE)) break;
        if (s > 1 && ksteps / s < 2) break;
        const long per_t_tile = (long)ceil_div(O, kTileO * cg) * s;
        const long items = per_t_tile * ceil_div(T, cand);
        if (s > 1 && items / s >= units) break;            // already a full round without splitting
        if (s > 1 && (double)s * T * O * 4.0 > 2.0 * in_bytes) break;     // partial sums would dominate the traffic
        const long rounds = (items + units - 1) / units;
        if (cg == 2 && rounds < 2) continue;               // a single round of pairs loses to single CTAs (measured)
        const int steps = ceil_div(ksteps, s);
        const int meta_cols = sp ? 64 : 0;
        for (int iss = 1; iss <= 2; ++iss) {
          // two issuers: single-CTA tcgen05 paths with streaming operands, and two accumulators of
          // the tile must fit in tensor memory next to the metadata
          if (iss == 2 && (cg == 2 || p.path == NM_PATH_UMMA_DECODE || 2 * cand + meta_cols > 512)) break;
          // time of one work item whose MMAs span n tokens (the tile, or the ragged remainder)
          auto item_us = [&](int n) {
            const double b_part = (sp ? 2.0 : 1.0) * n * 128.0 / cg;          // X bytes per K step and CTA
            const double store_b = (double)kTileO * n * (s > 1 ? 4.0 : (double)out_bytes(od));
            const double load_us = steps * (a_part + b_part) / kPortBytesPerUs;
            const double store_us = store_b / kStoreBytesPerUs;
            const double k_logical = (double)steps * 128.0 / eb * (sp ? 2.0 : 1.0);
            const double mma_math_us = 2.0 * kTileO * n * k_logical / (dt == NM_I8 ? kMmaRateI8 : kMmaRateF16)[sp ? 1 : 0][cg - 1];
            const double issue_us = steps * kStepIssueUs[sp ? 1 : 0] * (iss == 2 ? kTwoIssuerFactor : 1.0);
            const double mma_us = mma_math_us > issue_us ? mma_math_us : issue_us;
            const double longest = load_us > store_us ? (load_us > mma_us ? load_us : mma_us) : (store_us > mma_us ? store_us : mma_us);
            double item = longest + kOverlap[cg - 1] * (load_us + store_us + mma_us - longest) + kHandoffUs[cg - 1];
            if (cg == 2 && 2 * cand + meta_cols > 512) item *= 1.12;   // no room for a second accumulator buffer in tensor memory
            if (iss == 2 && 4 * cand + meta_cols > 512)               // two issuers, one buffer: the write-back does not overlap
              item = (load_us > mma_us ? load_us : mma_us) + store_us + kHandoffUs[0];
            return item;
          };
          // Makespan of the persistent grid: unit u takes items u, u + units, ...; the items of the
          // ragged token tile come last.  The busiest unit is the first one, or the first one past
          // the end of the full items or of all items in their last rounds.
          const double full_us = item_us(cand), rag_us = rag_tokens ? item_us(rag_n) : 0.0;
          const long n_full = per_t_tile * (T / cand);
          auto unit_us = [&](long u) {
            const long f = n_full > u ? (n_full - 1 - u) / units + 1 : 0;
            const long a = items > u ? (items - 1 - u) / units + 1 : 0;
            return f * full_us + (a - f) * rag_us;
          };
          double busiest = unit_us(0);
          const long edges[2] = {n_full % units, items % units};
          for (long e : edges)
            if (e > 0 && unit_us(e) > busiest) busiest = unit_us(e);
          double cost = kRampUs + (cg == 2 ? kPairRampUs : 0.0) + busiest;      // clusters start and meet more slowly
          // a last 256-row pair tile that is at most half full multiplies padding that single CTAs skip
          // (measured on DeiT-S fc2, O = 384: the pair's lead over single CTAs turns into a 9 % loss)
          if (cg == 2 && (256 - O % 256) % 256 >= 128) cost *= 1.0 + 0.3 * ((double)ceil_div(O, 256) * 256.0 / O - 1.0);
          if (s > 1) cost += kMergeUs + 2.0 * s * T * (double)O * 4.0 / 10e6;   // partials are written and re-read through L2
          if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_cg = cg; best_t = cand; best_split = s; best_issuers = iss; }
        }
      }
    }
  }
  const int tile_t = best_t, split = best_split;
  p.tile_t = tile_t;
  p.cta_group = best_cg;
  p.split_k = split;
  p.issuers = best_issuers;
  // The on-chip merge (NM_MERGE_CLUSTER) is left to the caller: timed alone it beats the workspace
  // merge by ~0.9 us while all clusters are resident at once, but a cluster launch does not overlap
  // its neighbours in a stream the way the two dependent launches of the workspace merge do, and
  // inside a stack of different layers it measured 0.3-0.9 us slower per split layer.
  p.merge = NM_MERGE_WORKSPACE;
  // the decode path keeps the decoded W tile resident so it is decoded once per run of tiles
  p.resident = p.path == NM_PATH_UMMA_DECODE ? NM_RES_W : NM_RES_NONE;
  p.stages = 8;                         // upper bound: the launchers trim the ring to the shared memory they have
  p.workspace_bytes = splitk_workspace_bytes(T, O, tile_t, split);
  if (p.path == NM_PATH_UMMA_EXPAND) p.workspace_bytes += expand_workspace_bytes(O, K, eb);   // the dense copy sits at the head

  // Roofline estimate (us): max of HBM time at 6.4 TB/s and tensor time at the nominal
  // dense int8 4.5 / fp16 2.25 Pop/s (x2 on the sparse path).
  const double bytes = in_bytes + (double)T * O * out_bytes(od);
  const double ops = 2.0 * T * (double)O * K;
  const double peak = (dt == NM_I8 ? 4.5e15 : 2.25e15) * (sp ? 2.0 : 1.0);
  const double t_hbm = bytes / 6.4e12, t_mma = ops / peak;
  p.predicted_us = (float)(1e6 * (t_hbm > t_mma ? t_hbm : t_mma));
  if (best_cost > p.predicted_us) p.predicted_us = (float)best_cost;
  *out = p;
  return NM_OK;
}

}  // namespace nm

extern "C" nm_status nm_plan_shape(int T, int O, int K, int n, int m, nm_dtype dt, nm_out_dtype od,
                                   uint32_t images, int n_sms, nm_plan* out) {
  return nm::plan_shape(T, O, K, n, m, dt, od, images, n_sms, out);
}

extern "C" nm_status nm_plan_create(int T, const nm_weight* w, nm_out_dtype od, int device, nm_plan* out) {
  if (!w || w->magic != nm::kWeightMagic) return NM_ERR_INVALID_ARG;
  int sms = nm::kDefaultSMs;
  if (device >= 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return NM_ERR_CUDA;
  }
  return nm::plan_shape(T, w->O, w->K, w->n, w->m, w->dtype, od, w->images, sms, out);
}
