// tcgen05 paths (sm_100a only): a persistent, warp-specialised GEMM kernel.
//
// One CTA per SM walks a static list of work items (output tile x K slice).  A tile is
// 128 out-features x tile_t tokens of Y^T = W_tile * X_tile^T:
//   * W is the MMA A operand (M = 128 out-features), X the B operand (N = tile_t tokens);
//     only A may be sparse, so the accumulator in tensor memory is Y transposed:
//     TMEM lane = out-feature, TMEM column = token.
//   * warp 0 / lane 0 : TMA producer.  Tiled loads (128-byte swizzle, no multicast) of the
//                       W and X K-step tiles plus one bulk copy of the 2:4 metadata block
//                       into a ring of shared-memory stages.
//   * warp 1 / lane 0 : MMA issuer.  tcgen05.cp metadata smem->TMEM, four tcgen05.mma[.sp]
//                       per 128-byte K step, tcgen05.commit recycles the stage; the
//                       accumulator is double-buffered in TMEM so the next tile's MMAs run
//                       while the previous tile drains.
//   * warps 2..9      : epilogue.  tcgen05.ld (32 lanes x 32 columns) -> transposed into a
//                       per-warp shared-memory patch -> TMA store of a 32-token x
//                       32-out-feature box of Y (full 128-byte lines, clipped at the T and
//                       O tails).  Writing Y is the dominant byte stream of these GEMMs, so
//                       the epilogue never waits for loads or MMAs of its own tile.
// This is the B200 form of the paper's micro-dense dataflow (Section 4.2): all sparsity
// handling happens in the load stage, compute is MMA only; for patterns that are 2:4-clean
// the sparse tensor core performs the per-row activation gather itself.
// Split-K (Section 4.3): a work item owns a slice of the K steps and writes its raw 32-bit
// partial tile to the workspace with the same epilogue; a second, grid-wide kernel sums the
// slices in order 0..s-1 into Y ("merged only in the final stage").  No CTA ever waits for
// another, and the result is deterministic for fp32 as well.
// Decode path (third template flag): instead of a TMA load of a pre-arranged W image, four
// decode warps read the canonical packed image (values + b-bit in-window positions, the
// paper's B_pack), one thread per out-feature row with 128-bit loads, and materialise only the
// kept values into a zero-filled, swizzled K-major tile in shared memory -- the micro-dense
// tile of Section 4.2 -- which the dense tcgen05.mma then consumes.  With W resident the tile
// is decoded once per run of token tiles.
// Every wait is a bounded mbarrier poll; on expiry the CTA records NM_ERR_TIMEOUT in the
// status word, raises a CTA-wide abort flag that every role polls, frees its tensor memory
// and returns.
#include <atomic>
#include <cstdlib>

#include "nm_umma_common.cuh"

namespace nm {
namespace {

constexpr int kEpiWarps = 8;                       // two warps per 32-lane TMEM quadrant
constexpr int kThreads = 32 * (2 + kEpiWarps);     // producer warp + MMA warp + epilogue warps
constexpr int kDecWarps = 8;                       // decode path only: two threads per out-feature row
constexpr int kThreadsDec = kThreads + 32 * kDecWarps;
constexpr uint32_t kPatchBytes = 4096;             // staging patch: 32 tokens x 32 out-features x 4 B
constexpr uint32_t kMaxAcc = 2;                    // most TMEM accumulator buffers a CTA rotates through
constexpr uint32_t kPatchBufs = 1;                 // patches per epilogue warp (TMA stores in flight)
constexpr int kMmasPerStep = 4;         // 128 B of A per row = 4 MMA K steps of 32 B
constexpr size_t kMaxSmem = 227 * 1024;  // dynamic shared memory limit per CTA

enum { kEpiTma = 0, kEpiDirect = 1, kEpiSplit = 2 };

struct UmmaParams {
  const uint8_t* meta;      // hw24 metadata blocks (sparse path)
  int meta_kblocks;         // blocks along K per 128-row tile
  void* Y; int64_t ldy;
  int T, O;
  int tile_t;               // tokens per tile (multiple of 32, <= 256)
  int stages;               // shared-memory ring depth
  int issuers;              // 1, or 2: a second warp issues the odd K steps of a tile into a second accumulator
  int acc_bufs;             // TMEM accumulator buffers (2 when 2*tile_t + metadata fit in 512 columns)
  int tiles_o, n_items;     // out-feature tiles; work items = tiles * split_k
  int total_ksteps;         // K steps of 128 B of A per row
  int ksteps_main;          // K remap (NM_PATH_UMMA_REMAP48): K steps from this one on read the gathered third-chunk
                            // activations through the second X map (>= total_ksteps: no remap)
  int ksteps_per_split, split_k;
  int out_f16;              // fp16 path: 1 = convert to half on store
  int out_i8;               // int8 path with requantising epilogue: 1 = scale / bias / ReLU / saturate to int8
  const float* epi_scale; const int32_t* epi_bias; int epi_relu;
  int epi_mode;             // kEpiTma / kEpiDirect / kEpiSplit
  int resident;             // NM_RES_*: which operand stays in shared memory across tiles
  int tiles_t;              // token tiles
  uint32_t res_bytes;       // bytes of the resident region (all K steps of the resident operand)
  uint32_t tmem_cols;       // power of two >= accumulators + metadata columns
  uint32_t* partial;        // split-K: [split][t_pad][O] raw 32-bit partials
  int w_fresh;              // the weight image is written by the launch just before: no W load ahead of the grid-dependency wait
  int cluster_merge;        // split-K: the K slices of a tile are the CTAs of one cluster and meet on chip
  uint32_t recv_bytes;      // ... bytes of shared memory that receive the other slices' partials
  int t_pad;                // split-K: token rows per slice (tiles_t * tile_t)
  uint32_t spin_limit;      // polls after which a bounded wait gives up
  int diag_stall;           // diagnostic (NM_PLAN_DIAG_STALL): CTA 0 arms its first K step for 16 bytes that never come
  unsigned long long* trace;   // phase stamps (trace builds only; nullptr otherwise)
  int dbg;                     // trace builds only: 1 = no MMAs are issued, 2 = no output is stored, 3 = both (timing experiments)
  uint32_t* status;
  // decode path: the canonical image (values + bit-packed positions)
  const uint8_t* canon_vals; const uint8_t* canon_idx;
  uint64_t val_row_bytes, idx_row_bytes;
  int n, m, b, G, K;
};

template <int DT, bool SP>
__host__ __device__ constexpr uint32_t meta_bytes_per_step() {
  return SP ? (DT == NM_I8 ? 4096u : 2048u) : 0u;
}
// Per K step: the A part (128 rows x 128 B of W values + the 2:4 metadata block) and the B
// part (tile_t rows x 128 B of X, two such atoms on the sparse path where 128 B of
// compressed A span 256 B of X).
template <int DT, bool SP>
__host__ __device__ inline uint32_t a_part_bytes() { return 16384u + meta_bytes_per_step<DT, SP>(); }
template <int DT, bool SP>
__host__ __device__ inline uint32_t b_part_bytes(int tile_t) { return (SP ? 2u : 1u) * (uint32_t)tile_t * 128u; }
// bytes of one ring stage (what streams) and of one resident slot (what stays), per K step
template <int DT, bool SP>
__host__ __device__ inline uint32_t stage_bytes(int tile_t, int resident) {
  return (resident == NM_RES_X ? 0u : b_part_bytes<DT, SP>(tile_t)) + (resident == NM_RES_W ? 0u : a_part_bytes<DT, SP>());
}
template <int DT, bool SP>
__host__ __device__ inline uint32_t res_slot_bytes(int tile_t, int resident) {
  return resident == NM_RES_X ? b_part_bytes<DT, SP>(tile_t) : (resident == NM_RES_W ? a_part_bytes<DT, SP>() : 0u);
}
// shared memory after the operand regions: staging patches, then barriers and three words
__host__ __device__ inline uint32_t tail_bytes(int stages, uint32_t recv_bytes = 0u) {
  return kEpiWarps * kPatchBufs * kPatchBytes + recv_bytes + 16u * (uint32_t)stages + 8u * (2u * kMaxAcc + 3u) + 16u;
}
// On-chip split-K merge: the tile is cut into units of (32 out-features) x (32 tokens); unit u
// belongs to the CTA of rank u % split, which receives the unit from every other rank.
__host__ __device__ inline uint32_t cluster_recv_bytes(int tile_t, int split) {
  const uint32_t units = 4u * (uint32_t)(tile_t / 32);
  return ((units + (uint32_t)split - 1u) / (uint32_t)split) * (uint32_t)(split - 1) * kPatchBytes;
}

struct ItemCoord {
  int o0, t0, ks_begin, nsteps, z;
  int key;           // identifies the resident operand this item needs
};
// Work items of one CTA: item(n) = first + n * stride, n < count.  Streaming mode strides over
// the grid with out-feature tiles varying fastest (concurrent CTAs share X rows in L2); the
// resident modes give every CTA one contiguous run so the resident operand changes rarely.
struct ItemRange { int first, stride, count; };
__device__ __forceinline__ ItemRange my_items(const UmmaParams& p) {
  ItemRange r;
  if (p.resident == NM_RES_NONE) {
    r.first = blockIdx.x; r.stride = gridDim.x;
    r.count = (p.n_items > (int)blockIdx.x) ? (p.n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  } else {
    const int per = p.n_items / (int)gridDim.x, rem = p.n_items % (int)gridDim.x;
    r.first = (int)blockIdx.x * per + min((int)blockIdx.x, rem);
    r.stride = 1;
    r.count = per + ((int)blockIdx.x < rem ? 1 : 0);
  }
  return r;
}
__device__ __forceinline__ ItemCoord decode_item(const UmmaParams& p, int item) {
  ItemCoord c;
  c.z = item % p.split_k;
  const int tile = item / p.split_k;
  int ot, tt;
  if (p.resident == NM_RES_W) { ot = tile / p.tiles_t; tt = tile % p.tiles_t; }   // token tiles fastest
  else { tt = tile / p.tiles_o; ot = tile % p.tiles_o; }                            // out-feature tiles fastest
  c.o0 = ot * kTileO;
  c.t0 = tt * p.tile_t;
  c.key = p.resident == NM_RES_W ? ot : tt;
  c.ks_begin = c.z * p.ksteps_per_split;
  c.nsteps = min(p.total_ksteps, c.ks_begin + p.ksteps_per_split) - c.ks_begin;
  return c;
}

// The items of one CTA in order, without the divisions of decode_item per item: in streaming mode
// the CTA strides over the item list, so K slice, out-feature tile and token tile advance by
// constants with carries.  (The lone threads that load and issue pay ~0.3 us per item for the four
// divisions otherwise; only the issuing thread, which paces the tile loop, uses it.)  Resident
// modes walk short contiguous runs and keep decode_item.
struct ItemWalker {
  int z, ot, tt, dz, dot, dtt, item, stride;
  bool fast;
  __device__ __forceinline__ void init(const UmmaParams& p, const ItemRange& R) {
    item = R.first; stride = R.stride;
    fast = p.resident == NM_RES_NONE && R.count > 1;      // a single item is cheaper to decode directly
    if (fast) {
      z = item % p.split_k;
      const int tile = item / p.split_k;
      tt = tile / p.tiles_o; ot = tile % p.tiles_o;
      dz = stride % p.split_k;
      const int dtile = stride / p.split_k;
      dtt = dtile / p.tiles_o; dot = dtile % p.tiles_o;
    }
  }
  __device__ __forceinline__ ItemCoord get(const UmmaParams& p) const {
    if (!fast) return decode_item(p, item);
    ItemCoord c;
    c.z = z;
    c.o0 = ot * kTileO;
    c.t0 = tt * p.tile_t;
    c.key = tt;
    c.ks_begin = z * p.ksteps_per_split;
    c.nsteps = min(p.total_ksteps, c.ks_begin + p.ksteps_per_split) - c.ks_begin;
    return c;
  }
  __device__ __forceinline__ void next(const UmmaParams& p) {
    item += stride;
    if (fast) {
      z += dz;
      int carry = 0;
      if (z >= p.split_k) { z -= p.split_k; carry = 1; }
      ot += dot + carry;
      tt += dtt;
      if (ot >= p.tiles_o) { ot -= p.tiles_o; ++tt; }
    }
  }
};

// r += the same 32 columns of the second accumulator of the buffer (two-issuer mode)
template <int DT>
__device__ __forceinline__ void add_second_acc(uint32_t (&r)[32], uint32_t taddr) {
  uint32_t r2[32];
  tc_ld_32x32(taddr, r2);
#pragma unroll
  for (int j = 0; j < 32; ++j)
    r[j] = (DT == NM_I8) ? r[j] + r2[j] : __float_as_uint(__fadd_rn(__uint_as_float(r[j]), __uint_as_float(r2[j])));
}

// ------------------------------------------------------------------ micro-dense decode
// One thread materialises the weights of its out-feature row for one K step (128 B of dense
// A) into the swizzled K-major tile at `tile`.  The row's packed bytes for the step -- kept
// values and their b-bit in-window positions -- are fetched up front with independent 128-bit
// loads (all in flight together), then each N:M group is assembled in registers (value j is
// shifted to the byte its position names) and written with one store per 8 bytes, zeros
// included, so no separate clearing pass is needed.
template <int DT>
__device__ __forceinline__ void decode_row_kstep(const UmmaParams& p, uint32_t tile, int r, int row, int ks, int half) {
  constexpr int eb = (DT == NM_I8) ? 1 : 2;
  constexpr int kElemsPerStep = 128 / eb;
  const uint32_t row_base = tile + (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u;
  const uint32_t sw = (uint32_t)(r & 7);
  const int gb = p.m * eb;                                   // bytes of one group in the dense row
  const int groups_per_step = kElemsPerStep / p.m;
  const int g0 = ks * groups_per_step;
  const int g_valid = (row < p.O) ? max(0, min(p.G - g0, groups_per_step)) : 0;

  // ---- fetch: aligned 16-byte windows over the value bytes and the position bits of the step
  // Window sizes: a K step is 128 bytes of the dense row, i.e. at most 128 kept values of one
  // byte (n = m) or 64 of two, so at most 128 value bytes plus 15 bytes of window misalignment
  // = 143 -> 9 loads of 16; its position bits are at most 128 * 4 / 8 = 64 bytes (m = 16, n = 15,
  // one-byte values) plus 15 -> 79 -> 5 loads, 6 issued.  A field that ends in the last fetched
  // word still forms `two` from the word after it, so the index buffer keeps one spare, zeroed word.
  uint32_t vbuf[36], ibuf[25];
  ibuf[24] = 0u;
  const size_t v_begin = (size_t)g0 * p.n * eb, v_end = v_begin + (size_t)g_valid * p.n * eb;
  const size_t i_begin = ((size_t)g0 * p.n * p.b) >> 3, i_end = (((size_t)(g0 + g_valid) * p.n * p.b) + 7) >> 3;
  const size_t v_win = v_begin & ~(size_t)15, i_win = i_begin & ~(size_t)15;
  if (g_valid > 0) {
    const uint8_t* vrow = p.canon_vals + (size_t)row * p.val_row_bytes;     // rows are 16-byte aligned and padded
    const uint8_t* irow = p.canon_idx + (size_t)row * p.idx_row_bytes;
#pragma unroll
    for (int q = 0; q < 9; ++q) {
      if (v_win + 16u * q < v_end) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(vrow + v_win) + q);
        vbuf[4 * q] = t.x; vbuf[4 * q + 1] = t.y; vbuf[4 * q + 2] = t.z; vbuf[4 * q + 3] = t.w;
      }
    }
#pragma unroll
    for (int q = 0; q < 6; ++q) {
      if (p.b && i_win + 16u * q < i_end) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(irow + i_win) + q);
        ibuf[4 * q] = t.x; ibuf[4 * q + 1] = t.y; ibuf[4 * q + 2] = t.z; ibuf[4 * q + 3] = t.w;
      }
    }
  }
  const uint32_t bmask = (1u << p.b) - 1u;
  const uint32_t vmask = eb == 1 ? 0xffu : 0xffffu;

  // ---- assemble and store group by group; the two threads of a row take alternate halves
  const int gi_begin = half * (groups_per_step / 2), gi_end = half ? groups_per_step : groups_per_step / 2;
#pragma unroll 2
  for (int gi = gi_begin; gi < gi_end; ++gi) {
    unsigned long long gw[4] = {0ull, 0ull, 0ull, 0ull};
    if (gi < g_valid) {
#pragma unroll 4
      for (int j = 0; j < p.n; ++j) {
        const size_t slot = (size_t)(g0 + gi) * p.n + j;
        const uint32_t vb = (uint32_t)(slot * eb - v_win);                       // byte inside the value window
        const unsigned long long v = (vbuf[vb >> 2] >> (8u * (vb & 3u))) & vmask;
        uint32_t pos = (uint32_t)j;
        if (p.b) {
          const uint32_t bp = (uint32_t)(slot * p.b - i_win * 8);                // bit inside the position window
          const unsigned long long two = ((unsigned long long)ibuf[(bp >> 5) + 1] << 32) | ibuf[bp >> 5];
          pos = (uint32_t)(two >> (bp & 31u)) & bmask;
        }
        const uint32_t off = pos * eb;                                           // byte inside the group
#pragma unroll
        for (int w = 0; w < 4; ++w) gw[w] |= ((off >> 3) == (uint32_t)w) ? (v << (8u * (off & 7u))) : 0ull;
      }
    }
    const uint32_t byte0 = (uint32_t)(gi * gb);                                  // byte inside the 128-byte row
    if (gb >= 8) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        if (w * 8 < gb) {
          const uint32_t bo = byte0 + 8u * w;
          asm volatile("st.shared.b64 [%0], %1;" ::"r"(row_base + (((bo >> 4) ^ sw) << 4) + (bo & 15u)), "l"(gw[w]) : "memory");
        }
      }
    } else if (gb == 4) {
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(row_base + (((byte0 >> 4) ^ sw) << 4) + (byte0 & 15u)), "r"((uint32_t)gw[0]) : "memory");
    } else {
      asm volatile("st.shared.b16 [%0], %1;" ::"r"(row_base + (((byte0 >> 4) ^ sw) << 4) + (byte0 & 15u)), "h"((unsigned short)gw[0]) : "memory");
    }
  }
}

// ------------------------------------------------------------------ the kernel
template <int DT, bool SP, bool DEC, bool DUAL, bool CLU>
__global__ void __launch_bounds__(DEC ? kThreadsDec : kThreads + 32, 1)      // the decode warps only exist in the DEC variants
nm_umma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmY, const UmmaParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sbytes = stage_bytes<DT, SP>(p.tile_t, p.resident);
  const uint32_t slot_bytes = res_slot_bytes<DT, SP>(p.tile_t, p.resident);
  const uint32_t b_tile_bytes = (uint32_t)p.tile_t * 128u;
  const uint32_t ring_base = smem_base + p.res_bytes;              // resident region first, then the ring
  const uint32_t ring_bytes = (uint32_t)p.stages * sbytes;
  const uint32_t patches = ring_base + ring_bytes;
  const uint32_t recv_base = patches + kEpiWarps * kPatchBufs * kPatchBytes;
  const uint32_t bars = recv_base + p.recv_bytes;
  const uint32_t bar_full = bars, bar_empty = bars + 8u * p.stages;
  const uint32_t bar_tfull = bars + 16u * p.stages, bar_tempty = bar_tfull + 8u * kMaxAcc;
  const uint32_t bar_rfull = bar_tempty + 8u * kMaxAcc, bar_rempty = bar_rfull + 8u, bar_recv = bar_rempty + 8u;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      gen_base + p.res_bytes + ring_bytes + kEpiWarps * kPatchBufs * kPatchBytes + p.recv_bytes + 16u * p.stages + 8u * (2u * kMaxAcc + 3u));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const WaitCtx wctx{abort_flag, p.status, p.spin_limit};
  // where the A part (W values, then metadata) and the B part (X) of K step ks / ring stage s live
  const uint32_t a_off_in_stage = p.resident == NM_RES_X ? 0u : b_part_bytes<DT, SP>(p.tile_t);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    NM_STAMP(p.trace, 0);
    pdl_launch_dependents();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    if (SP && p.ksteps_main < p.total_ksteps) prefetch_tensormap(&tmB2);
    if (p.epi_mode == kEpiTma) prefetch_tensormap(&tmY);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(bar_full + 8u * s, (DEC && p.resident != NM_RES_W) ? 1 + kDecWarps : 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int b = 0; b < (int)kMaxAcc; ++b) {
      mbar_init(bar_tfull + 8u * b, DUAL ? 2u : 1u);           // one commit per issuing thread
      mbar_init(bar_tempty + 8u * b, kEpiWarps);
    }
    mbar_init(bar_rfull, (DEC && p.resident == NM_RES_W) ? kDecWarps : 1);
    mbar_init(bar_rempty, 1);
    mbar_init(bar_recv, 1);
    if (CLU) {
      // bytes this CTA will receive: every unit it owns (and that holds tokens < T), from every other rank
      const ItemCoord c = decode_item(p, (int)blockIdx.x);
      const uint32_t rank = cluster_cta_rank();
      uint32_t owned = 0;
      for (uint32_t u = 0; u < 4u * (uint32_t)(p.tile_t / 32); ++u)
        if (u % (uint32_t)p.split_k == rank && c.t0 + (int)(u >> 2) * 32 < p.T) ++owned;
      if (owned) mbar_expect_tx(bar_recv, owned * (uint32_t)(p.split_k - 1) * kPatchBytes);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  if (CLU) cluster_sync_all();     // every CTA's receive barrier is armed before anyone sends
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) NM_STAMP(p.trace, 1);
  const uint32_t acc_cols = (DUAL ? 2u : 1u) * (uint32_t)p.tile_t;          // columns of one accumulator buffer
  const uint32_t tmem_meta = tmem_base + (uint32_t)p.acc_bufs * acc_cols;    // metadata columns follow the accumulators

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer
      const ItemRange R = my_items(p);
      // The packed weight never depends on the kernel that runs just before this one, so the
      // W tiles (and metadata) of the first ring-full of K steps are requested before the
      // grid-dependency wait: in a stack of small-batch layers the weight fetch of layer i+1
      // overlaps layer i.  X is only touched after the wait.
      int pre = 0;
      if (p.resident == NM_RES_NONE && !DEC && !p.w_fresh && !p.diag_stall && R.count > 0) {
        const ItemCoord c0 = decode_item(p, R.first);
        const uint8_t* meta0 = SP ? p.meta + ((size_t)(c0.o0 / kTileO) * p.meta_kblocks) * kMetaBlockBytes : nullptr;
        pre = min(p.stages, c0.nsteps);
        for (int i = 0; i < pre; ++i) {
          const uint32_t full = bar_full + 8u * (uint32_t)i;
          const uint32_t sa = ring_base + (uint32_t)i * sbytes + a_off_in_stage;
          mbar_expect_tx(full, sbytes);
          tma_load_2d(sa, &tmA, full, (c0.ks_begin + i) * 128, c0.o0);
          if (SP) bulk_load(sa + 16384u, meta0 + (size_t)(c0.ks_begin + i) * meta_bytes_per_step<DT, SP>(),
                            meta_bytes_per_step<DT, SP>(), full);
        }
        // and the X boxes of those K steps are pulled towards L2 (a hint, no data is consumed), so
        // that the first real loads after the wait do not pay the HBM latency
        for (int i = 0; i < pre; ++i) {
          if (SP) {
            const int ks = c0.ks_begin + i;
            const bool ovf = ks >= p.ksteps_main;
            const CUtensorMap* bm = ovf ? &tmB2 : &tmB;
            const int kx = (ovf ? ks - p.ksteps_main : ks) * 256;
            tma_prefetch_l2_2d(bm, kx, c0.t0);
            tma_prefetch_l2_2d(bm, kx + 128, c0.t0);
          } else {
            tma_prefetch_l2_2d(&tmB, (c0.ks_begin + i) * 128, c0.t0);
          }
        }
      }
      pdl_wait_prior_grid();      // X (and the workspace) may be written by the previous kernel
      NM_STAMP(p.trace, 2);
      NM_STAMP_VAL(p.trace, 12, R.count);
      uint32_t rloads = 0, s = 0, ph = 0, st = ring_base;
      uint32_t armed = 0;          // ring stages armed so far (K steps whose loads were issued)
      [[maybe_unused]] long long cyc_empty = 0;     // trace builds: cycles spent waiting for a free stage
      bool wrapped = false;
      int prev_key = -1;
      bool ok = true;
      for (int n = 0; n < R.count && ok; ++n) {
        const ItemCoord c = decode_item(p, R.first + n * R.stride);
        const uint8_t* meta_src = SP ? p.meta + ((size_t)(c.o0 / kTileO) * p.meta_kblocks) * kMetaBlockBytes : nullptr;
        if (p.resident != NM_RES_NONE && c.key != prev_key && !(DEC && p.resident == NM_RES_W)) {
          // (re)load the resident operand, all K steps, once the MMAs that read the old one retired
          if (rloads >= 1u) {
            ok = mbar_wait(bar_rempty, (rloads - 1u) & 1u, wctx, 7);
            if (!ok) break;
          }
          mbar_expect_tx(bar_rfull, p.res_bytes);
          for (int ks = 0; ks < p.total_ksteps; ++ks) {
            const uint32_t slot = smem_base + (uint32_t)ks * slot_bytes;
            if (p.resident == NM_RES_X) {
              if (SP) {
                tma_load_2d(slot, &tmB, bar_rfull, ks * 256, c.t0);
                tma_load_2d(slot + b_tile_bytes, &tmB, bar_rfull, ks * 256 + 128, c.t0);
              } else {
                tma_load_2d(slot, &tmB, bar_rfull, ks * 128, c.t0);
              }
            } else {
              tma_load_2d(slot, &tmA, bar_rfull, ks * 128, c.o0);
              if (SP) bulk_load(slot + 16384u, meta_src + (size_t)ks * meta_bytes_per_step<DT, SP>(),
                                meta_bytes_per_step<DT, SP>(), bar_rfull);
            }
          }
          ++rloads;
          prev_key = c.key;
        }
        for (int i = 0; i < c.nsteps; ++i) {
          // ring position kept incrementally (s = g mod stages, ph = parity of g / stages): a lone
          // thread pays full latency for every integer division in its loop
          const bool w_prefetched = (n == 0 && i < pre);       // its W part is already in flight
          if (wrapped) {
            NM_WAIT_TIMED(cyc_empty, ok = mbar_wait(bar_empty + 8u * s, ph ^ 1u, wctx, 1));
            if (!ok) break;
          }
          const uint32_t full = bar_full + 8u * s;
          const int ks = c.ks_begin + i;
          // Diagnostic stall: the first K step of CTA 0 expects 16 bytes more than are sent.  Every
          // copy that was issued lands; the barrier never completes, the issuing warp's bounded wait
          // runs out and the CTA leaves through its abort path with nothing in flight.
          const uint32_t extra = (p.diag_stall && blockIdx.x == 0 && n == 0 && i == 0) ? 16u : 0u;
          if (!w_prefetched)
            mbar_expect_tx(full, ((DEC && p.resident != NM_RES_W) ? sbytes - 16384u : sbytes) + extra);   // decoded A is not a TMA transfer
          if (p.resident != NM_RES_X) {            // B part streams
            if (SP) {
              // under the K remap the K steps of the third chunks read their activations from the gathered copy
              const bool ovf = ks >= p.ksteps_main;
              const CUtensorMap* bm = ovf ? &tmB2 : &tmB;
              const int kx = (ovf ? ks - p.ksteps_main : ks) * 256;
              tma_load_2d(st, bm, full, kx, c.t0);
              tma_load_2d(st + b_tile_bytes, bm, full, kx + 128, c.t0);
            } else {
              tma_load_2d(st, &tmB, full, ks * 128, c.t0);
            }
          }
          if (p.resident != NM_RES_W && !DEC && !w_prefetched) {    // A part streams
            const uint32_t sa = st + a_off_in_stage;
            tma_load_2d(sa, &tmA, full, ks * 128, c.o0);
            if (SP) bulk_load(sa + 16384u, meta_src + (size_t)ks * meta_bytes_per_step<DT, SP>(),
                              meta_bytes_per_step<DT, SP>(), full);
          }
          ++armed;
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; wrapped = true; st = ring_base; } else { st += sbytes; }
        }
      }
      NM_STAMP_VAL(p.trace, 15, cyc_empty);
      // Before this thread leaves, every copy it issued must have landed: a CTA that takes the abort
      // path gives up its shared memory while such a copy could still be writing to it.  Each stage's
      // barrier completes when the bytes of its latest use have arrived (no later use can complete:
      // this thread arms them), so a bounded wait on that phase of every armed stage is enough.  On
      // the normal path the MMAs have consumed every stage and the waits return at once.
      {
        if (armed < (uint32_t)pre) armed = (uint32_t)pre;
        const uint32_t ns = armed < (uint32_t)p.stages ? armed : (uint32_t)p.stages;
        for (uint32_t d = 0; d < ns; ++d) {
          const uint32_t last_use = (armed - 1u - d) / (uint32_t)p.stages;        // use count of stage (armed-1-d) % stages
          mbar_wait_quiet(bar_full + 8u * ((armed - 1u - d) % (uint32_t)p.stages), last_use & 1u, p.spin_limit >> 2);
        }
        if (p.resident != NM_RES_NONE && rloads >= 1u) mbar_wait_quiet(bar_rfull, (rloads - 1u) & 1u, p.spin_limit >> 2);
      }
    }
  } else if (warp == 1 || (DUAL && warp == 2 + kEpiWarps)) {
    // With two issuers (DUAL, streaming operands only) warp 1 issues the even K steps of
    // every tile into the first accumulator of the buffer and the extra warp the odd K steps into
    // the second; the epilogue adds the two.  One thread cannot issue tensor-core instructions
    // faster than ~45-60 cycles each, which bounds small tiles; two threads nearly double that, and
    // the fixed even/odd split keeps the summation order (and FP32 results) reproducible.
    const uint32_t which = warp == 1 ? 0u : 1u;
    {
      // ---------------- MMA issuer: the whole warp walks the loop in lockstep; the tcgen05 wrappers
      // elect the one lane that issues (see nm_umma_common.cuh), every lane polls the barriers.
      // instruction descriptor: D format (F32=1 / S32=2) at bit 4, A/B format at bits 7/10
      // (signed int8 = 1, f16 = 0), both operands K-major, N>>3 at bit 17, M>>4 at bit 24,
      // sparse flag at bit 2, metadata half selector (id2) at bits 0-1.
      uint32_t idesc = ((uint32_t)(p.tile_t >> 3) << 17) | ((uint32_t)(kTileO >> 4) << 24);
      idesc |= (DT == NM_I8) ? ((2u << 4) | (1u << 7) | (1u << 10)) : (1u << 4);
      if (SP) idesc |= 1u << 2;
      const ItemRange R = my_items(p);
      // This warp alone paces the tensor core: the ring position is advanced incrementally (no
      // divisions), one descriptor per operand is built per K step and the four MMAs offset it by
      // constants.
      uint32_t rloads = 0, s = 0, ph = 0, st = ring_base;
      const bool res_w = p.resident == NM_RES_W, res_x = p.resident == NM_RES_X;
      int prev_key = -1;
      bool ok = true;
      ItemWalker walk;
      walk.init(p, R);
      [[maybe_unused]] long long cyc_full = 0, cyc_tempty = 0;      // trace builds: cycles spent inside the two waits of this warp
      // The producer is parked behind the previous grid of the stream until that grid has finished;
      // waiting here too keeps that time out of this warp's bounded waits (it costs nothing once the
      // producer is through).
      pdl_wait_prior_grid();
      for (int n = 0; n < R.count && ok; ++n, walk.next(p)) {
        const uint32_t li = (uint32_t)n;
        const ItemCoord c = walk.get(p);
        const uint32_t buf = p.acc_bufs == 2 ? (li & 1u) : 0u, use = p.acc_bufs == 2 ? (li >> 1) : li;     // acc_bufs is 1 or 2
        if (p.resident != NM_RES_NONE && c.key != prev_key) {
          ok = mbar_wait(bar_rfull, rloads & 1u, wctx, 8);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          ++rloads;
          prev_key = c.key;
        }
        if (use >= 1u) {     // the epilogue must have drained this accumulator buffer
          NM_WAIT_TIMED(cyc_tempty, ok = mbar_wait(bar_tempty + 8u * buf, (use - 1u) & 1u, wctx, 4));
          ok = __all_sync(0xffffffffu, ok);        // every lane polls; also re-converges the warp after the poll loop
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem_base + buf * acc_cols + which * (uint32_t)p.tile_t;
        // the last token tile is usually ragged: its MMAs only span the 32-token chunks that hold tokens
        const int n_left = p.T - c.t0;
        const uint32_t n_eff = n_left >= p.tile_t ? (uint32_t)p.tile_t : (uint32_t)((n_left + 31) & ~31);
        const uint32_t idesc_n = (idesc & ~(0x3fu << 17)) | ((n_eff >> 3) << 17);
        for (int i = 0; i < c.nsteps; ++i) {
          if (DUAL && ((uint32_t)i & 1u) != which) {                  // the other issuer's K step
            if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; st = ring_base; } else { st += sbytes; }
            continue;
          }
          NM_WAIT_TIMED(cyc_full, ok = mbar_wait(bar_full + 8u * s, ph, wctx, 2));
          ok = __all_sync(0xffffffffu, ok);        // every lane polls; also re-converges the warp after the poll loop
          if (!ok) break;
          tc_fence_after();
          if (n == 0 && i == (int)which && lane == 0 && which == 0u) NM_STAMP(p.trace, 3);
          const int ks = c.ks_begin + i;
          const uint32_t slot = smem_base + (uint32_t)ks * slot_bytes;
          const uint32_t sa = res_w ? slot : st + a_off_in_stage;
          const uint32_t sb = res_x ? slot : st;
          // metadata columns follow the copy of the metadata they hold: ring stage or K step
          const uint32_t meta_cols = tmem_meta + (res_w ? (uint32_t)ks : s) * 8u;
#ifdef NM_HAS_DBG
          if (p.dbg & 1) { tc_commit(bar_empty + 8u * s); if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; st = ring_base; } else { st += sbytes; } continue; }
#endif
          if (SP) {
            const uint32_t sm = sa + 16384u;
            tc_cp_128x128b(meta_cols, desc_meta(sm));
            if (DT == NM_I8) tc_cp_128x128b(meta_cols + 4u, desc_meta(sm + 2048u));
          }
          // descriptors: the start-address field counts 16-byte units, so a K advance of 32 B (A,
          // dense B) adds 2 and one of 64 B (B under a sparse A) adds 4; no field can carry
          const uint64_t da0 = desc_sw128(sa), db0 = desc_sw128(sb);
          const uint64_t db1 = SP ? desc_sw128(sb + b_tile_bytes) : 0ull;
#pragma unroll
          for (int j = 0; j < kMmasPerStep; ++j) {
            const uint32_t acc = (i >= (DUAL ? 2 : 1) || j > 0) ? 1u : 0u;   // first K step of this accumulator overwrites
            const uint64_t da = da0 + (uint64_t)(2 * j);
            if (SP) {
              // 32 B of compressed A pair with 64 B of B: two MMAs per 128-byte B atom
              const uint64_t db = ((j >> 1) ? db1 : db0) + (uint64_t)(4 * (j & 1));
              if (DT == NM_I8) {
                tc_mma_sparse<DT>(d_tmem, da, db, meta_cols + 2u * j, idesc_n, acc);
              } else {
                tc_mma_sparse<DT>(d_tmem, da, db, meta_cols + (uint32_t)(j & 2), idesc_n | (uint32_t)(j & 1), acc);
              }
            } else {
              tc_mma_dense<DT>(d_tmem, da, db0 + (uint64_t)(2 * j), idesc_n, acc);
            }
          }
          tc_commit(bar_empty + 8u * s);       // stage reusable once these MMAs retire
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; st = ring_base; } else { st += sbytes; }
        }
        if (!ok) break;
        tc_commit(bar_tfull + 8u * buf);
        if (lane == 0 && which == 0u) { if (n == 0) NM_STAMP(p.trace, 4); if (n + 1 == R.count) NM_STAMP(p.trace, 5); }
        if (p.resident != NM_RES_NONE) {
          // last tile on this resident operand: let the producer overwrite it once the MMAs retire
          const bool last_on_key = (n + 1 >= R.count) || decode_item(p, R.first + (n + 1) * R.stride).key != c.key;
          if (last_on_key) tc_commit(bar_rempty);
        }
      }
      if (lane == 0 && which == 0u) { NM_STAMP_VAL(p.trace, 13, cyc_full); NM_STAMP_VAL(p.trace, 14, cyc_tempty); }
    }
  } else if (warp < 2 + kEpiWarps) {
    // ---------------- epilogue warps: quadrant q = TMEM lanes 32q..32q+31 (fixed by warp id),
    // half h picks the even or odd 32-column chunks of the tile
    const int e = warp - 2, q = warp & 3, h = e >> 2;
    const uint32_t patch0 = patches + (uint32_t)e * kPatchBufs * kPatchBytes;
    uint32_t pbuf = 0;
    // split-K slices are stored raw (32-bit), whatever the output dtype
    const bool ws_split = p.split_k > 1 && !CLU;
    const int ob = (DT == NM_F16 && p.out_f16 && !ws_split) ? 2 : ((DT == NM_I8 && p.out_i8 && !ws_split) ? 1 : 4);
    const uint32_t crank = CLU ? cluster_cta_rank() : 0u;
    const ItemRange R = my_items(p);
    [[maybe_unused]] long long cyc_tfull = 0;      // trace builds: cycles spent waiting for an accumulator
    pdl_wait_prior_grid();        // Y / workspace may still be in use by the previous kernel
    for (int n = 0; n < R.count; ++n) {
      const uint32_t li = (uint32_t)n;
      const ItemCoord c = decode_item(p, R.first + n * R.stride);
      const uint32_t buf = p.acc_bufs == 2 ? (li & 1u) : 0u, use = p.acc_bufs == 2 ? (li >> 1) : li;     // acc_bufs is 1 or 2
      uint32_t ok = 1;
      if (lane == 0) NM_WAIT_TIMED(cyc_tfull, ok = mbar_wait(bar_tfull + 8u * buf, use & 1u, wctx, 3) ? 1u : 0u);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      if (n == 0 && e == 0 && lane == 0) NM_STAMP(p.trace, 6);
      const int o_base = c.o0 + q * 32;
      const int o = o_base + lane;
      float q_scale = 1.0f;
      const float q_lo = p.epi_relu ? 0.0f : -128.0f;
      int32_t q_bias = 0;
      if (ob == 1 && o < p.O) {
        q_scale = __ldg(p.epi_scale + o);
        if (p.epi_bias) q_bias = __ldg(p.epi_bias + o);
      }
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * acc_cols;
      const bool add_odd = DUAL && c.nsteps >= 2;                 // the second accumulator holds the odd K steps
      // the two warps of a quadrant swap the even / odd 32-column chunks from tile to tile, so an
      // odd chunk count (tile_t = 96, 160, 224) loads them equally over time
      for (int cc = (h ^ (n & 1)) * 32; cc < p.tile_t; cc += 64) {
        const int t = c.t0 + cc;
        if (t >= p.T) break;
#ifdef NM_HAS_DBG
        if (p.dbg & 2) continue;
#endif
        uint32_t r[32];
        if (CLU) {
          // Split-K met on chip (Section 4.3: partial sums are merged only in the final stage).
          // Every rank holds this unit's partial; the owner adds the others' to its own in rank order.
          tc_ld_32x32(lane_addr + (uint32_t)cc, r);
          if (add_odd) add_second_acc<DT>(r, lane_addr + (uint32_t)p.tile_t + (uint32_t)cc);
          const uint32_t u = (uint32_t)(cc >> 5) * 4u + (uint32_t)q, split = (uint32_t)p.split_k;
          const uint32_t owner = u % split, slot0 = recv_base + (u / split) * (split - 1u) * kPatchBytes;
          if (owner != crank) {
            // one unit per warp in this mode (tile_t <= 64): the patch is written once and stays
            // untouched until the cluster barrier at the end of the kernel
#pragma unroll
            for (int j = 0; j < 32; ++j)
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(patch0 + (uint32_t)j * 128u + (uint32_t)lane * 4u), "r"(r[j]) : "memory");
            fence_async_smem();
            __syncwarp();
            if (lane == 0)
              bulk_copy_to_cta(map_to_cta(slot0 + (crank < owner ? crank : crank - 1u) * kPatchBytes, owner), patch0, kPatchBytes,
                               map_to_cta(bar_recv, owner));
            continue;
          }
          const bool got = mbar_wait(bar_recv, 0u, wctx, 11);
          if (!__all_sync(0xffffffffu, got)) break;
          // own partial first, then the other ranks' in rank order: a fixed order for every unit
          for (uint32_t z = 0; z + 1u < split; ++z) {
            const uint32_t src = slot0 + z * kPatchBytes + (uint32_t)lane * 4u;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              uint32_t v;
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(src + (uint32_t)j * 128u) : "memory");
              r[j] = (DT == NM_I8) ? r[j] + v : __float_as_uint(__fadd_rn(__uint_as_float(r[j]), __uint_as_float(v)));
            }
          }
        }
        if (p.epi_mode == kEpiTma) {
          const uint32_t patch = patch0 + pbuf * kPatchBytes;
          pbuf = (pbuf + 1u) % kPatchBufs;
          if (lane == 0) tma_store_wait_read();      // the previous box has left the patch
          __syncwarp();
          if (!CLU) {
            tc_ld_32x32(lane_addr + (uint32_t)cc, r);
            if (add_odd) add_second_acc<DT>(r, lane_addr + (uint32_t)p.tile_t + (uint32_t)cc);
          }
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
          if (lane == 0 && o_base < p.O) tma_store_2d(&tmY, patch, o_base * ob, (ws_split ? c.z * p.t_pad : 0) + t);
        } else {
          if (!CLU) {
            tc_ld_32x32(lane_addr + (uint32_t)cc, r);
            if (add_odd) add_second_acc<DT>(r, lane_addr + (uint32_t)p.tile_t + (uint32_t)cc);
          }
          if (o < p.O) {
            if (p.epi_mode == kEpiSplit) {
              uint32_t* dst = p.partial + ((size_t)c.z * p.t_pad + (size_t)t) * p.O + o;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (t + j < p.T) dst[(size_t)j * p.O] = r[j];
            } else if (ob == 1) {
              int8_t* dst = static_cast<int8_t*>(p.Y) + (size_t)t * p.ldy + o;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (t + j < p.T) dst[(size_t)j * p.ldy] = (int8_t)requant_to_i8(r[j], q_scale, q_bias, p.epi_relu);
            } else if (ob == 2) {
              __half* dst = static_cast<__half*>(p.Y) + (size_t)t * p.ldy + o;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (t + j < p.T) dst[(size_t)j * p.ldy] = __float2half_rn(__uint_as_float(r[j]));
            } else {
              uint32_t* dst = static_cast<uint32_t*>(p.Y) + (size_t)t * p.ldy + o;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (t + j < p.T) dst[(size_t)j * p.ldy] = r[j];
            }
          }
        }
      }
      // this warp no longer needs the accumulator buffer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * buf);
      if (e == 0 && lane == 0) { if (n == 0) NM_STAMP(p.trace, 7); if (n + 1 == R.count) NM_STAMP(p.trace, 8); }

    }
    // the staging patches must outlive the stores' reads of them; the writes themselves complete
    // with the grid, which is what a dependent launch waits for
    if (p.epi_mode == kEpiTma && lane == 0) tma_store_wait_read();
    if (e == 0 && lane == 0) { NM_STAMP(p.trace, 9); NM_STAMP_VAL(p.trace, 11, cyc_tfull); }
  } else if (DEC) {
    // ---------------- decode warps: thread r of 128 owns out-feature row o0 + r of the tile
    const int dt_id = (warp - (2 + kEpiWarps)) * 32 + lane;      // 0..255
    const int r = dt_id & 127, half = dt_id >> 7;
    const ItemRange R = my_items(p);
    uint32_t g = 0, rfills = 0;
    int prev_key = -1;
    bool ok = true;
    // The packed weight never depends on the previous grid, so decoding could start at once; but the
    // stages these warps wait for are freed by MMAs that need X, which the producer only loads after
    // the previous grid: waiting here keeps that grid's run time out of the bounded waits below.
    pdl_wait_prior_grid();
    for (int n = 0; n < R.count && ok; ++n) {
      const ItemCoord c = decode_item(p, R.first + n * R.stride);
      if (p.resident == NM_RES_W) {
        if (c.key != prev_key) {
          // decode the whole W tile once for this run of token tiles
          if (rfills >= 1u) {
            ok = mbar_wait(bar_rempty, (rfills - 1u) & 1u, wctx, 9);
            if (!ok) break;
          }
          for (int ks = 0; ks < p.total_ksteps; ++ks)
            decode_row_kstep<DT>(p, smem_base + (uint32_t)ks * slot_bytes, r, c.o0 + r, ks, half);
          fence_async_smem();          // generic-proxy writes must be visible to the MMA (async proxy)
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_rfull);
          ++rfills;
          prev_key = c.key;
        }
        continue;
      }
      for (int i = 0; i < c.nsteps; ++i, ++g) {
        const uint32_t s = g % (uint32_t)p.stages, nuse = g / (uint32_t)p.stages;
        if (nuse >= 1u) {
          ok = mbar_wait(bar_empty + 8u * s, (nuse - 1u) & 1u, wctx, 10);
          if (!ok) break;
        }
        decode_row_kstep<DT>(p, ring_base + s * sbytes + a_off_in_stage, r, c.o0 + r, c.ks_begin + i, half);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_full + 8u * s);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  // no CTA of a cluster leaves while a peer may still write into its shared memory or while its
  // own patches are being read by a copy towards a peer
  if (CLU) cluster_sync_all();
  if (threadIdx.x == 0) NM_STAMP(p.trace, 10);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------ split-K merge
// Y[t,o] = sum_z partial[z][t][o], slices added in order (Section 4.3: partial sums are merged
// only in the final stage).  One thread per 4 consecutive out-features when O % 4 == 0.
template <int DT, int VEC>
__global__ void __launch_bounds__(256)
nm_splitk_merge_kernel(const uint32_t* __restrict__ partial, void* __restrict__ Y, int T, int O, int64_t ldy,
                       int split_k, size_t slice_elems, int out_f16, int out_i8, const float* __restrict__ epi_scale,
                       const int32_t* __restrict__ epi_bias, int epi_relu) {
  pdl_launch_dependents();
  pdl_wait_prior_grid();          // the partial tiles come from the kernel launched just before
  const int ov = O / VEC;
  const size_t total = (size_t)T * ov;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / ov), o = (int)(i % ov) * VEC;
    uint32_t acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0u;
    for (int z = 0; z < split_k; ++z) {
      const uint32_t* src = partial + (size_t)z * slice_elems + (size_t)t * O + o;
      uint32_t val[VEC];
      if (VEC == 4) {
        const uint4 q = __ldcg(reinterpret_cast<const uint4*>(src));
        val[0] = q.x; val[1] = q.y; val[2] = q.z; val[3] = q.w;
      } else {
        val[0] = __ldcg(src);
      }
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        if (DT == NM_I8) acc[v] += val[v];
        else acc[v] = __float_as_uint(__uint_as_float(acc[v]) + __uint_as_float(val[v]));
      }
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const size_t yo = (size_t)t * ldy + o + v;
      if (DT == NM_F16 && out_f16) static_cast<__half*>(Y)[yo] = __float2half_rn(__uint_as_float(acc[v]));
      else if (DT == NM_I8 && out_i8)
        static_cast<int8_t*>(Y)[yo] = (int8_t)requant_to_i8(acc[v], __ldg(epi_scale + o + v), epi_bias ? __ldg(epi_bias + o + v) : 0, epi_relu);
      else static_cast<uint32_t*>(Y)[yo] = acc[v];
    }
  }
}

template <int DT>
nm_status launch_merge(const SpmmArgs& a, const UmmaParams& p) {
  cudaLaunchConfig_t cfg = {};
  const bool vec = (p.O % 4) == 0;
  const size_t total = (size_t)p.T * (vec ? p.O / 4 : p.O);
  size_t blocks = (total + 255) / 256;
  const size_t cap = (size_t)sm_count() * 8;
  cfg.gridDim = dim3((unsigned)(blocks < cap ? blocks : cap));
  cfg.blockDim = dim3(256);
  cfg.stream = static_cast<cudaStream_t>(a.stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const size_t slice = (size_t)p.t_pad * p.O;
  const cudaError_t e = vec
      ? cudaLaunchKernelEx(&cfg, nm_splitk_merge_kernel<DT, 4>, (const uint32_t*)p.partial, p.Y, p.T, p.O, p.ldy, p.split_k, slice, p.out_f16, p.out_i8, p.epi_scale, p.epi_bias, p.epi_relu)
      : cudaLaunchKernelEx(&cfg, nm_splitk_merge_kernel<DT, 1>, (const uint32_t*)p.partial, p.Y, p.T, p.O, p.ldy, p.split_k, slice, p.out_f16, p.out_i8, p.epi_scale, p.epi_bias, p.epi_relu);
  if (e != cudaSuccess) { cudaGetLastError(); return NM_ERR_CUDA; }
  count_launch();
  return NM_OK;
}

// one instantiation of the kernel: shared-memory opt-in once per device, then the launch
template <int DT, bool SP, bool DEC, bool DUAL, bool CLU>
nm_status launch_variant(const cudaLaunchConfig_t& cfg, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                         const CUtensorMap& tmY, const UmmaParams& p) {
  static std::atomic<uint64_t> configured{0};        // the attribute belongs to the (function, device) pair
  const int slot = device_slot();
  if (slot == 63 || !((configured.load(std::memory_order_relaxed) >> slot) & 1ull)) {
    if (cudaFuncSetAttribute(nm_umma_kernel<DT, SP, DEC, DUAL, CLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem) != cudaSuccess)
      return NM_ERR_CUDA;
    configured.fetch_or(1ull << slot, std::memory_order_relaxed);
  }
  if (cudaLaunchKernelEx(&cfg, nm_umma_kernel<DT, SP, DEC, DUAL, CLU>, tmA, tmB, tmB2, tmY, p) != cudaSuccess) {
    cudaGetLastError();
    return NM_ERR_CUDA;
  }
  return NM_OK;
}

template <int DT, bool SP, bool DEC>
nm_status launch_one(const SpmmArgs& a, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const CUtensorMap& tmY,
                     UmmaParams& p) {
  // Residency is a request: it needs every K step of the resident operand plus at least two
  // ring stages in shared memory, the metadata of a resident W in 64 TMEM columns, and no
  // split-K; otherwise both operands stream.
  auto smem_need = [&](int resident, int stages) {
    return 1024 + (size_t)p.total_ksteps * res_slot_bytes<DT, SP>(p.tile_t, resident) +
           (size_t)stages * stage_bytes<DT, SP>(p.tile_t, resident) + tail_bytes(stages, p.recv_bytes);
  };
  if (p.cluster_merge && (DEC || p.resident != NM_RES_NONE || p.tile_t > 64 || p.split_k > 8)) return NM_ERR_INVALID_ARG;
  p.recv_bytes = p.cluster_merge ? cluster_recv_bytes(p.tile_t, p.split_k) : 0u;
  // the persistent grid; with the on-chip merge every CTA owns exactly one (tile, K slice)
  const int grid = p.cluster_merge ? p.n_items : (p.n_items < sm_count() ? p.n_items : sm_count());
  if (p.resident != NM_RES_NONE) {
    const bool meta_ok = !(SP && p.resident == NM_RES_W && p.total_ksteps > 8);
    if (p.split_k > 1 || !meta_ok || smem_need(p.resident, 2) > kMaxSmem) p.resident = NM_RES_NONE;
  }
  // A CTA that issues fewer K steps in its whole life than the ring has stages never reuses a
  // stage: the extra stages would only hold shared memory (and metadata columns) that the CTAs
  // of the next launch, which may start early under programmatic dependent launch, could use.
  if (p.resident == NM_RES_NONE) {
    const int64_t life_steps = (int64_t)ceil_div(p.n_items, grid) * p.ksteps_per_split;
    if (life_steps < p.stages) p.stages = (int)(life_steps < 1 ? 1 : life_steps);
  }
  // the ring depth is an upper bound: shrink it until the CTA fits in shared memory
  while (p.stages > 1 && smem_need(p.resident, p.stages) > kMaxSmem) --p.stages;
  if (smem_need(p.resident, p.stages) > kMaxSmem) return NM_ERR_UNSUPPORTED;
  p.res_bytes = (uint32_t)p.total_ksteps * res_slot_bytes<DT, SP>(p.tile_t, p.resident);
  const uint32_t meta_cols = SP ? 8u * (uint32_t)(p.resident == NM_RES_W ? p.total_ksteps : p.stages) : 0u;
  if (p.issuers == 2 && (DEC || p.resident != NM_RES_NONE || p.stages < 2 || 2u * (uint32_t)p.tile_t + meta_cols > 512u)) p.issuers = 1;
  p.acc_bufs = (int)((512u - meta_cols) / (uint32_t)(p.issuers * p.tile_t));
  if (p.acc_bufs > (int)kMaxAcc) p.acc_bufs = (int)kMaxAcc;
  // a CTA that runs a single work item never rotates: one buffer, and half the tensor memory stays
  // free for a CTA of the next launch that shares the SM under programmatic dependent launch
  if (ceil_div(p.n_items, grid) <= 1) p.acc_bufs = 1;
  // An issuer waits on a ring stage by phase parity, which is only unambiguous while it cannot be
  // two uses of that stage ahead of the producer.  The issuer of the odd K steps observes no
  // barrier of the steps it skips; what bounds its lead is the accumulator hand-off (it can be
  // acc_bufs tiles ahead of the other issuer), so the ring must be deeper than that.
  if (p.issuers == 2 && p.acc_bufs > p.stages - 1) p.acc_bufs = p.stages - 1;
  if (p.acc_bufs < 1) p.acc_bufs = 1;
  p.tmem_cols = pow2_cols((uint32_t)(p.acc_bufs * p.issuers * p.tile_t) + meta_cols);
  if (p.tmem_cols > 512) return NM_ERR_INVALID_ARG;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(DEC ? kThreadsDec : (p.issuers == 2 ? kThreads + 32 : kThreads));
  cfg.dynamicSmemBytes = smem_need(p.resident, p.stages);
  cfg.stream = static_cast<cudaStream_t>(a.stream);
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.cluster_merge) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.split_k;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  nm_status lst;
  if (!DEC && p.cluster_merge)
    lst = p.issuers == 2 ? launch_variant<DT, SP, false, true, true>(cfg, tmA, tmB, tmB2, tmY, p)
                         : launch_variant<DT, SP, false, false, true>(cfg, tmA, tmB, tmB2, tmY, p);
  else
    lst = (!DEC && p.issuers == 2) ? launch_variant<DT, SP, false, true, false>(cfg, tmA, tmB, tmB2, tmY, p)
                                   : launch_variant<DT, SP, DEC, false, false>(cfg, tmA, tmB, tmB2, tmY, p);
  if (lst != NM_OK) return lst;
  count_launch();
  return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace

uint64_t splitk_workspace_bytes(int T, int O, int tile_t, int split_k) {
  if (split_k <= 1) return 0;
  // one raw 32-bit slice per K split, token rows padded to whole tiles so that a tile's
  // store never crosses into the next slice
  const uint64_t t_pad = (uint64_t)ceil_div(T, tile_t) * tile_t;
  return (uint64_t)split_k * t_pad * O * 4;
}

nm_status launch_umma(const SpmmArgs& a) {
  const nm_weight* w = a.w;
  const nm_plan& pl = a.plan;
  const bool sp = pl.path == NM_PATH_UMMA_SP24;
  const bool dec = pl.path == NM_PATH_UMMA_DECODE && w->n != w->m;   // dense rows need no decoding
  const int eb = elem_bytes(w->dtype);
  if (pl.tile_t < 32 || pl.tile_t > 256 || pl.tile_t % 32 != 0 || pl.stages < 1 || pl.stages > 8)
    return NM_ERR_INVALID_ARG;
  if (pl.split_k < 1 || pl.split_k > kMaxSplitK) return NM_ERR_INVALID_ARG;

  const uint8_t* base = static_cast<const uint8_t*>(w->dev_base);
  const void* a_ptr = nullptr;
  uint64_t a_row_bytes, a_pitch = 0;
  if (sp) {
    if (!(w->images & NM_IMG_HW24)) return NM_ERR_UNSUPPORTED;
    a_ptr = base + w->off_hw24_values;
    a_row_bytes = (uint64_t)((w->K + 3) / 4) * 2 * eb;
    a_pitch = w->hw24_row_bytes;
  } else if (w->n == w->m) {
    a_ptr = base + w->off_canonical + 64;                 // dense rows are the canonical values
    a_row_bytes = (uint64_t)w->K * eb;
    a_pitch = round_up(a_row_bytes, 16);
  } else if (dec) {
    a_row_bytes = (uint64_t)w->K * eb;                    // the decoded tile has dense geometry
  } else {
    if (!(w->images & NM_IMG_DENSE)) return NM_ERR_UNSUPPORTED;
    a_ptr = base + w->off_dense;
    a_row_bytes = (uint64_t)w->K * eb;
    a_pitch = w->dense_row_bytes;
  }
  if ((reinterpret_cast<uintptr_t>(a.X) & 15) || ((uint64_t)a.ldx * eb) % 16 != 0) return NM_ERR_ALIGN;

  UmmaParams p{};
  p.meta = sp ? base + w->off_hw24_meta : nullptr;
  p.meta_kblocks = w->hw24_meta_kblocks;
  p.Y = a.Y; p.ldy = a.ldy; p.T = a.T; p.O = w->O;
  p.tile_t = pl.tile_t; p.stages = pl.stages;
  p.issuers = pl.issuers == 2 ? 2 : 1;
  p.w_fresh = a.w_fresh ? 1 : 0;
  p.total_ksteps = (int)((a_row_bytes + 127) / 128);
  p.ksteps_main = a.X_ovf ? a.ksteps_main : 0x7fffffff;
  if (a.X_ovf && (!sp || pl.split_k > 1 || pl.resident != NM_RES_NONE)) return NM_ERR_INVALID_ARG;
  int split = pl.split_k < p.total_ksteps ? pl.split_k : p.total_ksteps;
  p.ksteps_per_split = ceil_div(p.total_ksteps, split);
  split = ceil_div(p.total_ksteps, p.ksteps_per_split);         // no empty slice
  p.split_k = split;
  p.out_f16 = a.od == NM_OUT_F16;
  p.out_i8 = a.od == NM_OUT_I8;
  p.epi_scale = a.epi.scale_dev; p.epi_bias = a.epi.bias_dev; p.epi_relu = a.epi.relu;
  if (p.out_i8 && !p.epi_scale) return NM_ERR_INVALID_ARG;
  p.status = a.status;
  // diagnostic stall (see NM_PLAN_DIAG_STALL in nm.h): a short poll budget so that the stalled wait
  // runs out in milliseconds
  p.diag_stall = (pl.reserved & NM_PLAN_DIAG_STALL) ? 1 : 0;
  p.spin_limit = p.diag_stall ? (1u << 14) : kSpinLimit;
  p.trace = trace_buffer();
#ifdef NM_HAS_DBG
  { const char* e = getenv("NM_DBG"); p.dbg = e ? atoi(e) : 0; }
#endif
  if (dec) {
    CanonGeom g;
    nm_status gs = canon_geom(w->O, w->K, w->n, w->m, w->dtype, &g);
    if (gs != NM_OK) return gs;
    p.canon_vals = base + w->off_canonical + 64;
    p.canon_idx = p.canon_vals + (uint64_t)g.O * g.val_row_bytes;
    p.val_row_bytes = g.val_row_bytes; p.idx_row_bytes = g.idx_row_bytes;
    p.n = g.n; p.m = g.m; p.b = g.b; p.G = g.G; p.K = g.K;
  }
  p.tiles_o = ceil_div(w->O, kTileO);
  p.tiles_t = ceil_div(a.T, pl.tile_t);
  p.resident = (pl.resident == NM_RES_X || pl.resident == NM_RES_W) ? pl.resident : NM_RES_NONE;
  const int64_t tiles = (int64_t)p.tiles_o * ceil_div(a.T, pl.tile_t);
  if (tiles * split > 0x7fffffff) return NM_ERR_UNSUPPORTED;
  p.n_items = (int)(tiles * split);

  const int ob = out_bytes(a.od);
  const void* y_base = a.Y;
  uint64_t y_row_bytes = (uint64_t)w->O * ob, y_rows = (uint64_t)a.T, y_pitch = (uint64_t)a.ldy * ob;
  uint32_t y_box_bytes = 32u * ob;
  p.cluster_merge = (split > 1 && pl.merge == NM_MERGE_CLUSTER) ? 1 : 0;
  if (split > 1 && !p.cluster_merge) {
    const uint64_t need = splitk_workspace_bytes(a.T, w->O, pl.tile_t, split);
    if (!a.workspace || a.workspace_bytes < need) return NM_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(a.workspace) & 15) return NM_ERR_ALIGN;
    p.partial = static_cast<uint32_t*>(a.workspace);
    p.t_pad = p.tiles_t * pl.tile_t;
    y_base = a.workspace;                        // the main kernel's epilogue targets the slices
    y_row_bytes = (uint64_t)w->O * 4; y_rows = (uint64_t)split * p.t_pad; y_pitch = y_row_bytes;
    y_box_bytes = 128u;
  }
  const bool y_tma_ok = !(reinterpret_cast<uintptr_t>(y_base) & 15) && y_pitch % 16 == 0;
  p.epi_mode = y_tma_ok ? kEpiTma : ((split > 1 && !p.cluster_merge) ? kEpiSplit : kEpiDirect);

  CUtensorMap tmA, tmB, tmB2, tmY;
  if (!dec && !make_map(&tmA, a_ptr, a_row_bytes, (uint64_t)w->O, a_pitch, 128u, kTileO, true)) return NM_ERR_CUDA;
  // under the K remap X keeps its own K columns (bytes beyond them read as zero: the padding of the main range)
  // and the second map covers the gathered third-chunk activations
  const uint64_t x_row_bytes = (uint64_t)(a.X_ovf ? a.k_x : w->K) * eb;
  if (!make_map(&tmB, a.X, x_row_bytes, (uint64_t)a.T, (uint64_t)a.ldx * eb, 128u, (uint32_t)pl.tile_t, true))
    return NM_ERR_CUDA;
  if (a.X_ovf) {
    if (!make_map(&tmB2, a.X_ovf, (uint64_t)a.k_ovf * eb, (uint64_t)a.T, (uint64_t)a.ld_ovf * eb, 128u, (uint32_t)pl.tile_t, true))
      return NM_ERR_CUDA;
  } else {
    tmB2 = tmB;
  }
  if (dec) tmA = tmB;      // the decode path never loads W through TMA
  if (p.epi_mode == kEpiTma) {
    if (!make_map(&tmY, y_base, y_row_bytes, y_rows, y_pitch, y_box_bytes, 32u, false)) return NM_ERR_CUDA;
  } else {
    tmY = tmB;      // unused by the kernel in the other epilogue modes
  }

  nm_status st;
  if (w->dtype == NM_I8) {
    st = sp ? launch_one<NM_I8, true, false>(a, tmA, tmB, tmB2, tmY, p)
            : (dec ? launch_one<NM_I8, false, true>(a, tmA, tmB, tmB2, tmY, p) : launch_one<NM_I8, false, false>(a, tmA, tmB, tmB2, tmY, p));
  } else {
    st = sp ? launch_one<NM_F16, true, false>(a, tmA, tmB, tmB2, tmY, p)
            : (dec ? launch_one<NM_F16, false, true>(a, tmA, tmB, tmB2, tmY, p) : launch_one<NM_F16, false, false>(a, tmA, tmB, tmB2, tmY, p));
  }
  if (st != NM_OK || split <= 1 || p.cluster_merge) return st;
  return w->dtype == NM_I8 ? launch_merge<NM_I8>(a, p) : launch_merge<NM_F16>(a, p);
}

}  // namespace nm
