// Host-side packers: dense pruned W -> canonical packed format and the device images
// the kernels read (Section 4.2, "Weight Packing").  Pure host code; no device memory here.
#include <cstring>

#include "nm_internal.h"

namespace nm {

nm_status canon_geom(int O, int K, int n, int m, int dt, CanonGeom* g) {
  if (O < 1 || K < 1 || n < 1 || m < 1 || n > m) return NM_ERR_INVALID_ARG;
  if (dt != NM_I8 && dt != NM_F16) return NM_ERR_INVALID_ARG;
  if (m > 16 || (m & (m - 1)) != 0) return NM_ERR_SHAPE;       // m in {1,2,4,8,16}
  if (K % m != 0 || K >= 131072) return NM_ERR_SHAPE;          // int32 accumulation bound
  g->O = O; g->K = K; g->n = n; g->m = m; g->G = K / m;
  g->b = (n == m) ? 0 : ceil_log2(m);
  g->eb = elem_bytes(dt);
  g->val_row_bytes = round_up((uint64_t)g->G * n * g->eb, 16);
  g->idx_row_bytes = g->b ? round_up(((uint64_t)g->G * n * g->b + 7) / 8, 16) : 0;
  g->bytes = 64 + (uint64_t)O * (g->val_row_bytes + g->idx_row_bytes);
  return NM_OK;
}

nm_status pack_layout(int O, int K, int n, int m, int dt, uint32_t images, PackLayout* L) {
  nm_status st = canon_geom(O, K, n, m, dt, &L->canon);
  if (st != NM_OK) return st;
  const int eb = L->canon.eb;
  L->images = images | NM_IMG_CANONICAL;
  uint64_t off = 0;
  L->off_canonical = off;
  off = round_up(off + L->canon.bytes, 256);
  L->off_hw24_values = L->off_hw24_meta = L->off_dense = 0;
  L->hw24_row_bytes = L->dense_row_bytes = 0;
  L->hw24_meta_kblocks = 0;
  L->hw24_meta_bytes = 0;
  if (images & NM_IMG_HW24) {
    const uint64_t chunks = ((uint64_t)K + 3) / 4;
    L->hw24_row_bytes = round_up(chunks * 2 * eb, 16);
    L->off_hw24_values = off;
    off = round_up(off + (uint64_t)O * L->hw24_row_bytes, 256);
    // One K step of the sparse kernel covers 128 B of compressed A per row: 256 logical k
    // (int8, two 2 KB metadata blocks) or 128 logical k (fp16, one block).
    L->hw24_meta_kblocks = (dt == NM_I8) ? 2 * ceil_div(K, 256) : ceil_div(K, 128);
    L->hw24_meta_bytes = (uint64_t)ceil_div(O, kTileO) * L->hw24_meta_kblocks * kMetaBlockBytes;
    L->off_hw24_meta = off;
    off = round_up(off + L->hw24_meta_bytes, 256);
  }
  if ((images & NM_IMG_DENSE) && n != m) {
    L->dense_row_bytes = round_up((uint64_t)K * eb, 16);
    L->off_dense = off;
    off = round_up(off + (uint64_t)O * L->dense_row_bytes, 256);
  }
  L->off_remap_values = L->off_remap_meta = L->remap_row_bytes = L->remap_meta_bytes = 0;
  L->remap_meta_kblocks = L->remap_k = L->remap_k_main = 0;
  if ((images & NM_IMG_REMAP48) && n != m && K % 8 == 0) {
    // W' = [W without the moved elements | zero padding to a whole K step | third chunks (K/2 columns)]
    const int step_elems = 256 / eb;                       // logical k of one sparse K step (256 B of activations)
    L->remap_k_main = ceil_div(K, step_elems) * step_elems;
    L->remap_k = L->remap_k_main + K / 2;
    L->remap_row_bytes = round_up((uint64_t)(L->remap_k / 4) * 2 * eb, 16);
    L->off_remap_values = off;
    off = round_up(off + (uint64_t)O * L->remap_row_bytes, 256);
    L->remap_meta_kblocks = (dt == NM_I8) ? 2 * ceil_div(L->remap_k, 256) : ceil_div(L->remap_k, 128);
    L->remap_meta_bytes = (uint64_t)ceil_div(O, kTileO) * L->remap_meta_kblocks * kMetaBlockBytes;
    L->off_remap_meta = off;
    off = round_up(off + L->remap_meta_bytes, 256);
  }
  L->bytes = off;
  return NM_OK;
}

static inline bool elem_is_zero(const void* W, int dt, int64_t i) {
  if (dt == NM_I8) return static_cast<const int8_t*>(W)[i] == 0;
  return (static_cast<const uint16_t*>(W)[i] & 0x7fffu) == 0;
}

nm_status build_canonical(const void* W, int64_t ldw, const CanonGeom& g, int dt, uint8_t* out,
                          int64_t* bad_row, int64_t* bad_group) {
  std::memset(out, 0, g.bytes);
  std::memcpy(out, "NMW1", 4);
  uint32_t* h32 = reinterpret_cast<uint32_t*>(out);
  h32[1] = 1; h32[2] = (uint32_t)dt;
  int32_t* hi = reinterpret_cast<int32_t*>(out);
  hi[3] = g.O; hi[4] = g.K; hi[5] = g.n; hi[6] = g.m; hi[7] = g.G; hi[8] = g.b;
  uint64_t* h64 = reinterpret_cast<uint64_t*>(out);
  h64[5] = g.val_row_bytes; h64[6] = g.idx_row_bytes;
  uint8_t* vals = out + 64;
  uint8_t* idx = vals + (uint64_t)g.O * g.val_row_bytes;
  for (int o = 0; o < g.O; ++o) {
    uint8_t* vrow = vals + (uint64_t)o * g.val_row_bytes;
    uint8_t* irow = idx + (uint64_t)o * g.idx_row_bytes;
    uint64_t slot = 0;
    for (int gi = 0; gi < g.G; ++gi) {
      const int64_t base = (int64_t)o * ldw + (int64_t)gi * g.m;
      uint32_t keep = 0;
      int cnt = 0;
      for (int p = 0; p < g.m; ++p)
        if (!elem_is_zero(W, dt, base + p)) { keep |= 1u << p; ++cnt; }
      if (cnt > g.n) {
        if (bad_row) *bad_row = o;
        if (bad_group) *bad_group = gi;
        return NM_ERR_NOT_NM;
      }
      for (int p = 0; p < g.m && cnt < g.n; ++p)
        if (!(keep & (1u << p))) { keep |= 1u << p; ++cnt; }
      for (int p = 0; p < g.m; ++p) {
        if (!(keep & (1u << p))) continue;
        if (dt == NM_I8) {
          reinterpret_cast<int8_t*>(vrow)[slot] = static_cast<const int8_t*>(W)[base + p];
        } else {
          uint16_t v = static_cast<const uint16_t*>(W)[base + p];
          reinterpret_cast<uint16_t*>(vrow)[slot] = (v & 0x7fffu) ? v : (uint16_t)0;
        }
        if (g.b) {
          const uint64_t bit = slot * g.b;
          const uint32_t sh = (uint32_t)(bit & 7);
          const uint32_t v = (uint32_t)p << sh;            // b <= 4, so at most two bytes
          irow[bit >> 3] |= (uint8_t)v;
          if (sh + g.b > 8) irow[(bit >> 3) + 1] |= (uint8_t)(v >> 8);
        }
        ++slot;
      }
    }
  }
  return NM_OK;
}

bool is_24_clean(const void* W, int64_t ldw, int O, int K, int dt) {
  for (int o = 0; o < O; ++o)
    for (int c = 0; c < (K + 3) / 4; ++c) {
      int cnt = 0;
      for (int p = 0; p < 4 && c * 4 + p < K; ++p)
        cnt += !elem_is_zero(W, dt, (int64_t)o * ldw + c * 4 + p);
      if (cnt > 2) return false;
    }
  return true;
}

// Byte offset and bit shift of the metadata nibble of 4-chunk `c` (0..31) of row `r`
// (0..127) inside one 2 KB metadata block, in the order tcgen05.cp.128x128b followed by
// tcgen05.mma.sp expects.  8-bit kinds: row-major rows of 16 B.  16-bit kinds: rows r and
// r+8 share 32-bit words, and the two 16-k halves of every 32-k step sit 128 B apart.
static inline void meta_nibble_pos(int dt, int r, int c, uint32_t* byte, uint32_t* shift) {
  if (dt == NM_I8) {
    *byte = (uint32_t)r * 16 + (uint32_t)c / 2;
    *shift = (c & 1) * 4;
    return;
  }
  const int k = c * 4;
  const int k0 = k & 15, k1 = (k >> 4) & 1, k2 = k >> 5;
  const int m0 = r & 7, m1 = (r >> 3) & 1, m2 = r >> 4;
  *byte = (uint32_t)(m0 * 16 + m1 * 2 + m2 * 256 + k1 * 128 + k2 * 4 + k0 / 8);
  *shift = (uint32_t)(k0 & 7);
}

void build_hw24(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L,
                uint8_t* values, uint8_t* meta) {
  const int eb = elem_bytes(dt);
  std::memset(values, 0, (size_t)O * L.hw24_row_bytes);
  std::memset(meta, 0x44, L.hw24_meta_bytes);          // positions (0,1): valid everywhere
  const int chunks = (K + 3) / 4;
  const int chunks_per_block = 128 / 4;
  for (int o = 0; o < O; ++o) {
    uint8_t* vrow = values + (uint64_t)o * L.hw24_row_bytes;
    const int ot = o / kTileO, r = o % kTileO;
    for (int c = 0; c < chunks; ++c) {
      int pos[2], np = 0;
      uint32_t keep = 0;
      for (int p = 0; p < 4 && c * 4 + p < K; ++p)
        if (!elem_is_zero(W, dt, (int64_t)o * ldw + c * 4 + p)) keep |= 1u << p;
      int cnt = __builtin_popcount(keep);
      for (int p = 0; p < 4 && cnt < 2; ++p)
        if (!(keep & (1u << p))) { keep |= 1u << p; ++cnt; }
      for (int p = 0; p < 4; ++p)
        if ((keep & (1u << p)) && np < 2) pos[np++] = p;
      for (int j = 0; j < 2; ++j) {
        const int k = c * 4 + pos[j];
        if (dt == NM_I8) {
          reinterpret_cast<int8_t*>(vrow)[c * 2 + j] =
              (k < K) ? static_cast<const int8_t*>(W)[(int64_t)o * ldw + k] : (int8_t)0;
        } else {
          uint16_t v = (k < K) ? static_cast<const uint16_t*>(W)[(int64_t)o * ldw + k] : (uint16_t)0;
          reinterpret_cast<uint16_t*>(vrow)[c * 2 + j] = (v & 0x7fffu) ? v : (uint16_t)0;
        }
      }
      const int kb = c / chunks_per_block, cc = c % chunks_per_block;
      uint8_t* blk = meta + ((uint64_t)ot * L.hw24_meta_kblocks + kb) * kMetaBlockBytes;
      uint32_t byte, shift;
      meta_nibble_pos(dt, r, cc, &byte, &shift);
      const uint8_t nib = (uint8_t)(pos[0] | (pos[1] << 2));
      blk[byte] = (uint8_t)((blk[byte] & ~(0xFu << shift)) | (nib << shift));
    }
  }
  (void)eb;
}

bool is_48_remappable(const void* W, int64_t ldw, int O, int K, int dt) {
  if (K % 8 != 0) return false;
  for (int o = 0; o < O; ++o)
    for (int g = 0; g < K / 8; ++g) {
      int cnt = 0;
      for (int p = 0; p < 8; ++p) cnt += !elem_is_zero(W, dt, (int64_t)o * ldw + g * 8 + p);
      if (cnt > 4) return false;
    }
  return true;
}

// Three-chunk K remap (NM_PATH_UMMA_REMAP48).  For every row and group of 8 k: a 4-chunk that holds
// more than two nonzeros hands the excess to the group's third chunk, taking it from its first two
// positions (k+0, k+1 of the first chunk; k+4, k+5 of the second), which are the ones the third chunk
// repeats; any three of four positions include one of the first two, all four include both, and a
// group with at most 4 nonzeros has an excess of at most two.  The remapped row is then 2:4-clean and
// is packed by the ordinary 2:4 packer.
void build_remap48(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L, uint8_t* values, uint8_t* meta) {
  const int eb = elem_bytes(dt);
  const int Kr = L.remap_k, Km = L.remap_k_main;
  std::vector<uint8_t> Wr((size_t)O * Kr * eb, 0);
  auto get = [&](int o, int k) -> uint16_t {
    return dt == NM_I8 ? (uint16_t)(uint8_t)static_cast<const int8_t*>(W)[(int64_t)o * ldw + k]
                       : static_cast<const uint16_t*>(W)[(int64_t)o * ldw + k];
  };
  auto put = [&](int o, int k, uint16_t v) {
    if (dt == NM_I8) Wr[(size_t)o * Kr + k] = (uint8_t)v;
    else reinterpret_cast<uint16_t*>(Wr.data())[(size_t)o * Kr + k] = v;
  };
  for (int o = 0; o < O; ++o)
    for (int g = 0; g < K / 8; ++g)
      for (int half = 0; half < 2; ++half) {
        const int k0 = g * 8 + half * 4;
        int nz = 0;
        for (int p = 0; p < 4; ++p) nz += !elem_is_zero(W, dt, (int64_t)o * ldw + k0 + p);
        int excess = nz > 2 ? nz - 2 : 0;
        for (int p = 0; p < 4; ++p) {
          const bool zero = elem_is_zero(W, dt, (int64_t)o * ldw + k0 + p);
          if (!zero && excess > 0 && p < 2) {          // moved to the third chunk: slot 2*half + p
            put(o, Km + g * 4 + half * 2 + p, get(o, k0 + p));
            --excess;
          } else if (!zero) {
            put(o, k0 + p, get(o, k0 + p));
          }
        }
      }
  PackLayout T = L;                                    // the 2:4 packer reads its geometry from these fields
  T.hw24_row_bytes = L.remap_row_bytes;
  T.hw24_meta_kblocks = L.remap_meta_kblocks;
  T.hw24_meta_bytes = L.remap_meta_bytes;
  build_hw24(Wr.data(), Kr, O, Kr, dt, T, values, meta);
}

void build_dense(const void* W, int64_t ldw, int O, int K, int dt, const PackLayout& L, uint8_t* dense) {
  const int eb = elem_bytes(dt);
  std::memset(dense, 0, (size_t)O * L.dense_row_bytes);
  for (int o = 0; o < O; ++o) {
    uint8_t* row = dense + (uint64_t)o * L.dense_row_bytes;
    std::memcpy(row, static_cast<const uint8_t*>(W) + (int64_t)o * ldw * eb, (size_t)K * eb);
    if (dt == NM_F16) {
      uint16_t* r16 = reinterpret_cast<uint16_t*>(row);
      for (int k = 0; k < K; ++k)
        if ((r16[k] & 0x7fffu) == 0) r16[k] = 0;
    }
  }
}

nm_status decode_canonical(const uint8_t* canon, size_t bytes, void* W, int64_t ldw) {
  if (bytes < 64 || std::memcmp(canon, "NMW1", 4) != 0) return NM_ERR_INVALID_ARG;
  const int32_t* hi = reinterpret_cast<const int32_t*>(canon);
  const uint64_t* h64 = reinterpret_cast<const uint64_t*>(canon);
  const int dt = hi[2], O = hi[3], K = hi[4], n = hi[5], m = hi[6], G = hi[7], b = hi[8];
  const uint64_t vr = h64[5], ir = h64[6];
  if (bytes < 64 + (uint64_t)O * (vr + ir)) return NM_ERR_INVALID_ARG;
  const uint8_t* vals = canon + 64;
  const uint8_t* idx = vals + (uint64_t)O * vr;
  const int eb = elem_bytes(dt);
  for (int o = 0; o < O; ++o) {
    std::memset(static_cast<uint8_t*>(W) + (int64_t)o * ldw * eb, 0, (size_t)K * eb);
    const uint8_t* vrow = vals + (uint64_t)o * vr;
    const uint8_t* irow = idx + (uint64_t)o * ir;
    for (int s = 0; s < G * n; ++s) {
      int p = s % n;
      if (b) {
        const uint64_t bit = (uint64_t)s * b;
        uint32_t w = irow[bit >> 3];
        if ((bit & 7) + b > 8) w |= (uint32_t)irow[(bit >> 3) + 1] << 8;
        p = (int)((w >> (bit & 7)) & ((1u << b) - 1));
      }
      const int64_t dst = (int64_t)o * ldw + (int64_t)(s / n) * m + p;
      if (dt == NM_I8) static_cast<int8_t*>(W)[dst] = reinterpret_cast<const int8_t*>(vrow)[s];
      else static_cast<uint16_t*>(W)[dst] = reinterpret_cast<const uint16_t*>(vrow)[s];
    }
  }
  return NM_OK;
}

}  // namespace nm
