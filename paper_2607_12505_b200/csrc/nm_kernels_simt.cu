// CUDA-core path over the canonical packed image: any n:m, any shape, no alignment
// rules.  It is the catch-all behind the tcgen05 paths (odd pitches, weights with no
// tensor-core image) and the on-device cross-check for them; it is not tuned.
// Each thread owns one out-feature o and kSimtRows token rows; the X rows of the block
// sit in shared memory, the thread walks the packed slots of its weight row
// (Section 4.2: value and in-window position are decoded together, slot by slot).
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nm_internal.h"

namespace nm {
namespace {

constexpr int kSimtRows = 8;       // token rows per block
constexpr int kSimtThreads = 128;  // out-features per block
constexpr int kSimtKChunk = 2048;  // k elements staged per pass (multiple of every m)

template <typename TIn> struct Acc;
template <> struct Acc<int8_t> { using type = int32_t; };
template <> struct Acc<__half> { using type = float; };

__device__ __forceinline__ int32_t mac(int32_t acc, int8_t x, int8_t w) { return acc + (int32_t)x * (int32_t)w; }
__device__ __forceinline__ float mac(float acc, __half x, __half w) {
  return fmaf(__half2float(x), __half2float(w), acc);
}

template <typename TIn>
__global__ void __launch_bounds__(kSimtThreads)
nm_simt_kernel(const TIn* __restrict__ X, int64_t ldx, int T, const uint8_t* __restrict__ vals,
               uint64_t val_row_bytes, const uint8_t* __restrict__ idx, uint64_t idx_row_bytes,
               int O, int K, int n, int m, int b, void* __restrict__ Y, int64_t ldy, int od,
               const float* __restrict__ epi_scale, const int32_t* __restrict__ epi_bias, int epi_relu) {
  using TAcc = typename Acc<TIn>::type;
  __shared__ TIn xs[kSimtRows][kSimtKChunk];
  const int o = blockIdx.x * kSimtThreads + threadIdx.x;
  const int64_t t0 = (int64_t)blockIdx.y * kSimtRows;
  TAcc acc[kSimtRows];
#pragma unroll
  for (int r = 0; r < kSimtRows; ++r) acc[r] = TAcc(0);
  const TIn* vrow = reinterpret_cast<const TIn*>(vals + (uint64_t)(o < O ? o : 0) * val_row_bytes);
  const uint8_t* irow = idx + (uint64_t)(o < O ? o : 0) * idx_row_bytes;
  const uint32_t bmask = (1u << b) - 1u;

  for (int kc = 0; kc < K; kc += kSimtKChunk) {
    const int klen = min(kSimtKChunk, K - kc);
    for (int i = threadIdx.x; i < kSimtRows * klen; i += kSimtThreads) {
      const int r = i / klen, k = i - r * klen;
      const int64_t t = t0 + r;
      xs[r][k] = (t < T) ? X[t * ldx + kc + k] : TIn(0);
    }
    __syncthreads();
    if (o < O) {
      const int g0 = kc / m, g1 = (kc + klen) / m;
      for (int g = g0; g < g1; ++g) {
        const int kbase = g * m - kc;
        for (int j = 0; j < n; ++j) {
          const int64_t s = (int64_t)g * n + j;
          int p = j;
          if (b) {
            const uint64_t bit = (uint64_t)s * b;
            uint32_t w = irow[bit >> 3];
            if ((bit & 7) + b > 8) w |= (uint32_t)irow[(bit >> 3) + 1] << 8;
            p = (int)((w >> (bit & 7)) & bmask);
          }
          const TIn v = vrow[s];
#pragma unroll
          for (int r = 0; r < kSimtRows; ++r) acc[r] = mac(acc[r], xs[r][kbase + p], v);
        }
      }
    }
    __syncthreads();
  }
  if (o >= O) return;
#pragma unroll
  for (int r = 0; r < kSimtRows; ++r) {
    const int64_t t = t0 + r;
    if (t >= T) break;
    if (od == NM_OUT_F16) {
      reinterpret_cast<__half*>(Y)[t * ldy + o] = __float2half_rn((float)acc[r]);
    } else if (od == NM_OUT_I8) {
      // requantising epilogue: int32 add, int32 -> fp32 (RN), one fp32 multiply, ReLU, RN-even, saturate
      const int32_t a32 = (int32_t)((uint32_t)(int32_t)acc[r] + (uint32_t)(epi_bias ? epi_bias[o] : 0));
      float v = __fmul_rn(__int2float_rn(a32), epi_scale[o]);
      if (epi_relu) v = fmaxf(v, 0.0f);
      reinterpret_cast<int8_t*>(Y)[t * ldy + o] = (int8_t)max(-128, min(127, __float2int_rn(v)));
    } else {
      reinterpret_cast<TAcc*>(Y)[t * ldy + o] = acc[r];
    }
  }
}


// Expansion of the canonical image into zero-filled dense rows (NM_PATH_UMMA_EXPAND): one thread
// per N:M group reads its n values and b-bit positions, assembles the m elements of the group in
// registers (value j shifted to the byte its position names) and writes them with 8-byte stores.
// The packed weight never depends on the launch before this one, so it is read ahead of the
// grid-dependency wait; the scratch copy may still be read by that launch (a previous layer's
// GEMM), so it is written after it.
template <int EB>
__global__ void __launch_bounds__(256)
nm_expand_kernel(const uint8_t* __restrict__ vals, uint64_t val_row_bytes, const uint8_t* __restrict__ idx,
                 uint64_t idx_row_bytes, int O, int G, int n, int m, int b, uint8_t* __restrict__ dst, uint64_t dst_pitch) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t bmask = (1u << b) - 1u;
  const int64_t total = (int64_t)O * G;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;        // one group per thread
  unsigned long long gw[4] = {0ull, 0ull, 0ull, 0ull};                    // up to 16 elements of 2 bytes
  int o = 0, g = 0;
  if (i < total) {
    o = (int)(i / G); g = (int)(i % G);
    const uint8_t* vrow = vals + (uint64_t)o * val_row_bytes;
    const uint8_t* irow = idx + (uint64_t)o * idx_row_bytes;
    for (int j = 0; j < n; ++j) {
      const int64_t s = (int64_t)g * n + j;
      uint32_t pos = (uint32_t)j;
      if (b) {
        const int64_t bit = s * b;
        uint32_t two = (uint32_t)__ldg(irow + (bit >> 3));
        if ((int)(bit & 7) + b > 8) two |= (uint32_t)__ldg(irow + (bit >> 3) + 1) << 8;      // the field straddles a byte
        pos = (two >> (bit & 7)) & bmask;
      }
      unsigned long long v = EB == 1 ? (unsigned long long)__ldg(vrow + s)
                                     : (unsigned long long)__ldg(reinterpret_cast<const unsigned short*>(vrow) + s);
      const uint32_t off = pos * EB;                                       // byte inside the group
#pragma unroll
      for (int w = 0; w < 4; ++w) gw[w] |= ((off >> 3) == (uint32_t)w) ? (v << (8u * (off & 7u))) : 0ull;
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (i < total) {
    const int gb = m * EB;                                                 // bytes of one group: 2 ... 32
    uint8_t* out = dst + (uint64_t)o * dst_pitch + (uint64_t)g * gb;
    if (gb >= 8) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w * 8 < gb) reinterpret_cast<unsigned long long*>(out)[w] = gw[w];
    } else if (gb == 4) {
      *reinterpret_cast<uint32_t*>(out) = (uint32_t)gw[0];
    } else {
      *reinterpret_cast<unsigned short*>(out) = (unsigned short)gw[0];
    }
  }
}
}  // namespace

nm_status launch_simt(const SpmmArgs& a) {
  const nm_weight* w = a.w;
  CanonGeom g;
  nm_status st = canon_geom(w->O, w->K, w->n, w->m, w->dtype, &g);
  if (st != NM_OK) return st;
  const uint8_t* canon = static_cast<const uint8_t*>(w->dev_base) + w->off_canonical;
  const uint8_t* vals = canon + 64;
  const uint8_t* idx = vals + (uint64_t)g.O * g.val_row_bytes;
  const int64_t row_blocks = ((int64_t)a.T + kSimtRows - 1) / kSimtRows;
  if (row_blocks > 65535) {
    // grid.y limit: walk the token rows in slabs
    const int slab = 65535 * kSimtRows;
    for (int64_t t0 = 0; t0 < a.T; t0 += slab) {
      SpmmArgs sub = a;
      const int eb = elem_bytes(w->dtype);
      sub.X = static_cast<const uint8_t*>(a.X) + t0 * a.ldx * eb;
      sub.Y = static_cast<uint8_t*>(a.Y) + t0 * a.ldy * out_bytes(a.od);
      sub.T = (int)((a.T - t0 < slab) ? (a.T - t0) : slab);
      st = launch_simt(sub);
      if (st != NM_OK) return st;
    }
    return NM_OK;
  }
  dim3 grid((unsigned)ceil_div(g.O, kSimtThreads), (unsigned)row_blocks);
  cudaStream_t s = static_cast<cudaStream_t>(a.stream);
  if (w->dtype == NM_I8) {
    nm_simt_kernel<int8_t><<<grid, kSimtThreads, 0, s>>>(
        static_cast<const int8_t*>(a.X), a.ldx, a.T, vals, g.val_row_bytes, idx, g.idx_row_bytes,
        g.O, g.K, g.n, g.m, g.b, a.Y, a.ldy, a.od, a.epi.scale_dev, a.epi.bias_dev, a.epi.relu);
  } else {
    nm_simt_kernel<__half><<<grid, kSimtThreads, 0, s>>>(
        static_cast<const __half*>(a.X), a.ldx, a.T, vals, g.val_row_bytes, idx, g.idx_row_bytes,
        g.O, g.K, g.n, g.m, g.b, a.Y, a.ldy, a.od, nullptr, nullptr, 0);
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace nm

namespace nm {

uint64_t expand_workspace_bytes(int O, int K, int eb) {
  return round_up((uint64_t)O * round_up((uint64_t)K * eb, 16), 256);
}

// Gather of the third-chunk activations of the 4:8 K remap (NM_PATH_UMMA_REMAP48): for every token row
// and group of 8 k, the elements k+0, k+1, k+4, k+5.  One thread per group: one 8- or 16-byte load,
// one 4- or 8-byte store.  X may come from the launch before, so it is read after the dependency wait.
template <int EB>
__global__ void __launch_bounds__(256)
nm_remap_gather_kernel(const uint8_t* __restrict__ X, int64_t x_pitch, int T, int G8, uint8_t* __restrict__ dst, int64_t dst_pitch) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t total = (int64_t)T * G8;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / G8), g = (int)(i % G8);
    if (EB == 1) {
      const uint2 v = *reinterpret_cast<const uint2*>(X + (int64_t)t * x_pitch + (int64_t)g * 8);
      *reinterpret_cast<uint32_t*>(dst + (int64_t)t * dst_pitch + (int64_t)g * 4) = (v.x & 0xffffu) | (v.y << 16);
    } else {
      const uint4 v = *reinterpret_cast<const uint4*>(X + (int64_t)t * x_pitch + (int64_t)g * 16);
      *reinterpret_cast<uint2*>(dst + (int64_t)t * dst_pitch + (int64_t)g * 8) = make_uint2(v.x, v.z);
    }
  }
}

uint64_t remap_workspace_bytes(int T, int K, int eb) {
  return round_up((uint64_t)T * round_up((uint64_t)(K / 2) * eb, 16), 256);
}

nm_status launch_remap_gather(const void* X, int64_t ldx, int T, int K, int dt, void* dst, void* stream) {
  const int eb = elem_bytes(dt);
  const int G8 = K / 8;
  const int64_t total = (int64_t)T * G8;
  cudaLaunchConfig_t cfg = {};
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  cfg.gridDim = dim3((unsigned)(blocks < 1 ? 1 : blocks));
  cfg.blockDim = dim3(256);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int64_t x_pitch = ldx * eb, d_pitch = (int64_t)round_up((uint64_t)(K / 2) * eb, 16);
  const cudaError_t e = dt == NM_I8
      ? cudaLaunchKernelEx(&cfg, nm_remap_gather_kernel<1>, static_cast<const uint8_t*>(X), x_pitch, T, G8, static_cast<uint8_t*>(dst), d_pitch)
      : cudaLaunchKernelEx(&cfg, nm_remap_gather_kernel<2>, static_cast<const uint8_t*>(X), x_pitch, T, G8, static_cast<uint8_t*>(dst), d_pitch);
  if (e != cudaSuccess) { cudaGetLastError(); return NM_ERR_CUDA; }
  count_launch();
  return NM_OK;
}

nm_status launch_expand(const nm_weight* w, void* dst, void* stream) {
  CanonGeom g;
  nm_status st = canon_geom(w->O, w->K, w->n, w->m, w->dtype, &g);
  if (st != NM_OK) return st;
  const uint8_t* vals = static_cast<const uint8_t*>(w->dev_base) + w->off_canonical + 64;
  const uint8_t* idx = vals + (uint64_t)g.O * g.val_row_bytes;
  const uint64_t pitch = round_up((uint64_t)g.K * g.eb, 16);
  const int64_t total = (int64_t)g.O * g.G;
  cudaLaunchConfig_t cfg = {};
  const int64_t blocks = (total + 255) / 256;                              // one group per thread
  if (blocks > 0x7fffffff) return NM_ERR_UNSUPPORTED;
  cfg.gridDim = dim3((unsigned)(blocks < 1 ? 1 : blocks));
  cfg.blockDim = dim3(256);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = w->dtype == NM_I8
      ? cudaLaunchKernelEx(&cfg, nm_expand_kernel<1>, vals, g.val_row_bytes, idx, g.idx_row_bytes, g.O, g.G, g.n, g.m, g.b, static_cast<uint8_t*>(dst), pitch)
      : cudaLaunchKernelEx(&cfg, nm_expand_kernel<2>, vals, g.val_row_bytes, idx, g.idx_row_bytes, g.O, g.G, g.n, g.m, g.b, static_cast<uint8_t*>(dst), pitch);
  if (e != cudaSuccess) { cudaGetLastError(); return NM_ERR_CUDA; }
  count_launch();
  return NM_OK;
}

}  // namespace nm
