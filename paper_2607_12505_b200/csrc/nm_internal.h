// Internal declarations shared by the translation units of libnm_b200.so.
// Nothing here is part of the ABI (see include/nm.h).
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "nm.h"

namespace nm {

constexpr uint32_t kWeightMagic = 0x44574d4eu;   // "NMWD"
constexpr int kTileO = 128;                      // MMA M: out-features per CTA tile
constexpr int kMetaBlockBytes = 2048;            // 128 rows x 16 B of 2:4 metadata
constexpr int kMaxSplitK = 16;
constexpr int kDefaultSMs = 148;

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int elem_bytes(int dt) { return dt == NM_I8 ? 1 : 2; }
inline int out_bytes(int od) { return od == NM_OUT_F16 ? 2 : (od == NM_OUT_I8 ? 1 : 4); }
inline int ceil_log2(int m) { int b = 0; while ((1 << b) < m) ++b; return b; }

// ---- canonical format geometry ------------------------------------------------------
struct CanonGeom {
  int O, K, n, m, G, b, eb;
  uint64_t val_row_bytes, idx_row_bytes, bytes;
};
nm_status canon_geom(int O, int K, int n, int m, int dt, CanonGeom* g);

// ---- layout of the whole packed device buffer ---------------------------------------
struct PackLayout {
  CanonGeom canon;
  uint32_t images;
  uint64_t off_canonical, off_hw24_values, off_hw24_meta, off_dense;
  uint64_t hw24_row_bytes, dense_row_bytes;
  int hw24_meta_kblocks;        // 2 KB blocks along K per 128-row tile
  uint64_t hw24_meta_bytes;
  // three-chunk K remap image (NM_IMG_REMAP48): a 2:4 image of W' [O x remap_k]
  uint64_t off_remap_values, off_remap_meta, remap_row_bytes, remap_meta_bytes;
  int remap_meta_kblocks, remap_k, remap_k_main;
  uint64_t bytes;
};
nm_status pack_layout(int O, int K, int n, int m, int dt, uint32_t images, PackLayout* L);

// Host packers (nm_format.cu).  `W` row-major with pitch ldw elements.
nm_status build_canonical(const void* W, int64_t ldw, const CanonGeom& g, int dt, uint8_t* out,
                          int64_t* bad_row, int64_t* bad_group);
bool is_24_clean(const void* W, int64_t ldw, int O, int K, int dt);
void build_hw24(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L,
                uint8_t* values, uint8_t* meta);
void build_dense(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L, uint8_t* dense);
nm_status decode_canonical(const uint8_t* canon, size_t bytes, void* W, int64_t ldw);
// NM_IMG_REMAP48: true when every aligned group of 8 k holds at most 4 nonzeros (K % 8 == 0)
bool is_48_remappable(const void* W, int64_t ldw, int O, int K, int dt);
void build_remap48(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L, uint8_t* values, uint8_t* meta);

// ---- kernel launchers (nm_kernels_*.cu) ----------------------------------------------
struct SpmmArgs {
  const void* X; int64_t ldx; int T;
  const nm_weight* w;
  nm_plan plan;
  void* Y; int64_t ldy; int od;
  void* workspace; size_t workspace_bytes;
  uint32_t* status;
  void* stream;
  nm_epilogue epi;         // scale_dev == nullptr: no epilogue
  // NM_PATH_UMMA_REMAP48: K steps below ksteps_main read X, the others the gathered third-chunk activations
  const void* X_ovf = nullptr; int64_t ld_ovf = 0; int k_x = 0, k_ovf = 0, ksteps_main = 0;
  bool w_fresh = false;    // the weight image is written by the launch just before (no load ahead of the grid-dependency wait)
};
// NM_PATH_UMMA_EXPAND: bytes of the dense copy at the head of the workspace (256-byte multiple)
uint64_t expand_workspace_bytes(int O, int K, int eb);
// enqueues the expansion of the canonical image into `dst` (rows of round_up(K*eb,16) bytes)
nm_status launch_expand(const nm_weight* w, void* dst, void* stream);
// NM_PATH_UMMA_REMAP48: bytes of the gathered activations at the head of the workspace, and the gather itself
// (dst[t, 4g + j] = X[t, 8g + {0,1,4,5}[j]], rows of round_up(K/2*eb, 16) bytes)
uint64_t remap_workspace_bytes(int T, int K, int eb);
nm_status launch_remap_gather(const void* X, int64_t ldx, int T, int K, int dt, void* dst, void* stream);
nm_status launch_simt(const SpmmArgs& a);
nm_status launch_umma(const SpmmArgs& a);
nm_status launch_umma_pair(const SpmmArgs& a, bool* handled);   // cta_group::2 variant; may decline
void count_launch(int n = 1);
// trace builds (-DNM_TRACE) only: the buffer the next launches stamp their phases into (nullptr: none)
unsigned long long* trace_buffer();

// Bytes of split-K scratch a plan needs: one raw 32-bit slice [t_pad x O] per K split (t_pad =
// token rows rounded up to whole tiles).  The merge pass reads only rows t < T and columns o < O
// of every slice, all of which the same call's GEMM kernel writes first: nothing has to be zeroed.
uint64_t splitk_workspace_bytes(int T, int O, int tile_t, int split_k);

}  // namespace nm
