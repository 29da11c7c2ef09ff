// Copy-engine probes for sm_100a (harness only): what one thread pays to issue the asynchronous
// instructions the kernels are built from, how long a tiled TMA load takes to land, and how many
// bytes per nanosecond an SM can pull from L2 / HBM through a ring of TMA loads.
//   part 1 (one thread, cycles): mbarrier arrive, try_wait on a completed phase, expect_tx,
//           cp.async.bulk.tensor issue back to back, time until the first / all of 6 boxes land
//   part 2 (steady-state ring, one issuing thread per CTA, division-free loop): bytes per ns per SM
//           for several box heights, boxes per stage, ring depths, buffer sizes, on 1 / 148 CTAs
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <vector>

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t c) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(c) : "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t b) { asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(b) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar, uint32_t par) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(par) : "memory");
  return ok;
}
// bounded: gives up after 2^22 polls
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t par) {
  for (uint32_t i = 0; i < (1u << 22); ++i) if (mbar_try(bar, par)) return true;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

__global__ void __launch_bounds__(128, 1) issue_cost_kernel(const __grid_constant__ CUtensorMap tm, long long* outg) {
  extern __shared__ uint8_t smem_raw[];
  long long* out = outg + blockIdx.x * 16;
  const int yoff = blockIdx.x * 96;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + 6 * 32768;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 16; ++s) mbar_init(bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    long long t0, t1, t2, t3;
    const int N = 64;
    t0 = clock64();
    for (int i = 0; i < N; ++i) mbar_arrive(bars + 8 * (8 + (i & 7)));
    t1 = clock64(); out[0] = (t1 - t0) / N;
    uint32_t acc = 0;
    t0 = clock64();
    for (int i = 0; i < N; ++i) acc += mbar_try(bars + 8 * (8 + (i & 7)), 1u);
    t1 = clock64(); out[1] = (t1 - t0) / N; out[15] = acc;
    // cold pass (descriptor and data not yet on chip), then the measured warm pass
    for (int pass = 0; pass < 2; ++pass) {
      t0 = clock64();
      for (int i = 0; i < 6; ++i) { mbar_expect_tx(bars + 8 * i, 8192); tma_load_2d(base + i * 32768, &tm, bars + 8 * i, 0, yoff + i * 64); }
      t1 = clock64();
      bool ok = mbar_wait(bars, pass);
      t2 = clock64();
      for (int i = 1; i < 6 && ok; ++i) ok = mbar_wait(bars + 8 * i, pass);
      t3 = clock64();
      out[2 + 3 * pass] = (t1 - t0) / 6; out[3 + 3 * pass] = ok ? t2 - t0 : -1; out[4 + 3 * pass] = ok ? t3 - t0 : -1;
    }
    t0 = clock64();
    for (int i = 0; i < 6; ++i) mbar_expect_tx(bars + 8 * (1 + i), 16);
    t1 = clock64(); out[8] = (t1 - t0) / 6;
  }
}

template <int S>
__global__ void __launch_bounds__(128, 1) ring_kernel(const __grid_constant__ CUtensorMap tm, unsigned long long* outg, int iters, int box_rows,
                                                      int boxes, int ymax, int xboxes) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bb = box_rows * 128, sb = bb * boxes;
  const uint32_t bars = base + S * sb;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) mbar_init(bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    int y = (blockIdx.x * 37) % ymax, xb = 0;
    auto issue = [&](uint32_t s) {
      mbar_expect_tx(bars + 8 * s, sb);
      for (int l = 0; l < boxes; ++l) { tma_load_2d(base + s * sb + l * bb, &tm, bars + 8 * s, xb * 128, y * box_rows); if (++xb == xboxes) xb = 0; }
      y += 13; if (y >= ymax) y -= ymax;
    };
    for (int s = 0; s < S - 1; ++s) issue(s);
    uint32_t si = S - 1, sw = 0, ph = 0;
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool ok = true;
    for (int it = 0; it < iters && ok; ++it) {
      issue(si);
      if (++si == S) si = 0;
      ok = mbar_wait(bars + 8 * sw, ph);
      if (++sw == S) { sw = 0; ph ^= 1u; }
    }
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    outg[blockIdx.x * 2] = t0; outg[blockIdx.x * 2 + 1] = ok ? t1 : 0;
  }
}

// part 3: the operand pattern of a GEMM (T x K activations, O x K weights, 128-byte K slices, out-feature tiles varying
// fastest over the CTAs, so weight boxes are shared by ~1/6 of the CTAs and activation boxes by 6) in a ring whose
// producer thread waits for a consumer warp (all lanes poll the full barrier, lane 0 releases the stage), as the
// GEMM kernels do.  `extra` dependent integer instructions per stage show what the producer's own instruction time costs.
template <int S>
__global__ void __launch_bounds__(128, 1) gemm_ring_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                           unsigned long long* outg, int items, int tiles_o, int ksteps, int tile_t, int extra, int cextra) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bbytes = (uint32_t)tile_t * 128u, abytes = 16384u, sb = bbytes + abytes;
  const uint32_t full = base + S * sb, empty = full + 8 * S;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2 * S; ++s) mbar_init(full + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool ok = true, wrapped = false;
    uint32_t s = 0, ph = 0, v = 1; long steps = 0;
    for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
      const int o0 = (item % tiles_o) * 128, t0r = (item / tiles_o) * tile_t;
      for (int ks = 0; ks < ksteps; ++ks) {
        if (wrapped) { ok = mbar_wait(empty + 8 * s, ph ^ 1u); if (!ok) break; }
        const uint32_t st = base + s * sb;
        mbar_expect_tx(full + 8 * s, sb);
        tma_load_2d(st, &tmB, full + 8 * s, ks * 128, t0r);
        tma_load_2d(st + bbytes, &tmA, full + 8 * s, ks * 128, o0);
        for (int q = 0; q < extra; ++q) asm volatile("mad.lo.u32 %0, %0, %0, %1;" : "+r"(v) : "r"(q));
        ++steps;
        if (++s == S) { s = 0; ph ^= 1u; wrapped = true; }
      }
    }
    for (int d = 0; d < S && ok; ++d)      // let the last loads land before the CTA gives up its shared memory
      if (steps > d) { const long g = steps - 1 - d; ok = mbar_wait(full + 8 * (uint32_t)(g % S), (uint32_t)((g / S) & 1)); }
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    outg[blockIdx.x * 3] = t0; outg[blockIdx.x * 3 + 1] = (ok && v != 0x7fffffffu) ? t1 : 0; outg[blockIdx.x * 3 + 2] = (unsigned long long)steps;
  } else if (threadIdx.x >= 32 && threadIdx.x < 64) {
    const int lane = threadIdx.x & 31;
    uint32_t s = 0, ph = 0, v = 1; bool ok = true;
    for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
      for (int ks = 0; ks < ksteps; ++ks) {
        ok = mbar_wait(full + 8 * s, ph);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        for (int q = 0; q < cextra; ++q) asm volatile("mad.lo.u32 %0, %0, %0, %1;" : "+r"(v) : "r"(q));      // stands for the consumer's own work
        if (lane == 0 && v != 0x7fffffffu) mbar_arrive(empty + 8 * s);
        __syncwarp();
        if (++s == S) { s = 0; ph ^= 1u; }
      }
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool make_map(EncodeTiledFn enc, CUtensorMap* tm, void* buf, uint64_t row_bytes, uint64_t rows, uint32_t box_rows) {
  cuuint64_t dims[2] = {row_bytes, rows}; cuuint64_t strides[1] = {row_bytes}; cuuint32_t box[2] = {128u, box_rows}; cuuint32_t es[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, buf, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int S>
static void run_ring(EncodeTiledFn enc, uint8_t* buf, size_t mb, unsigned long long* out, int box_rows, int boxes, int sms) {
  const uint64_t row_bytes = 4096, rows = mb * 1024 * 1024 / row_bytes;
  const size_t smem = 1024 + (size_t)S * box_rows * 128 * boxes + 8 * S + 64;
  if (smem > 227 * 1024) return;
  CUtensorMap tm;
  if (!make_map(enc, &tm, buf, row_bytes, rows, box_rows)) { printf("tensor map failed\n"); return; }
  cudaFuncSetAttribute(ring_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  for (int grid : {1, sms}) {
    const int iters = 2000;
    for (int rep = 0; rep < 2; ++rep) { ring_kernel<S><<<grid, 128, smem>>>(tm, out, iters, box_rows, boxes, (int)(rows / box_rows), (int)(row_bytes / 128)); cudaDeviceSynchronize(); }
    std::vector<unsigned long long> h(grid * 2);
    cudaMemcpy(h.data(), out, grid * 16, cudaMemcpyDeviceToHost);
    unsigned long long t0 = ~0ull, t1 = 0; bool ok = true; double per = 0;
    for (int i = 0; i < grid; ++i) { if (!h[2 * i + 1]) ok = false; if (h[2 * i] < t0) t0 = h[2 * i]; if (h[2 * i + 1] > t1) t1 = h[2 * i + 1]; per += (double)(h[2 * i + 1] - h[2 * i]); }
    const double bytes = (double)grid * iters * box_rows * 128.0 * boxes;
    printf("ring: buffer %4zu MB, box %3d rows x %d per stage, %d stages, %3d CTAs: %s %8.1f GB/s aggregate, %6.1f B/ns per SM, %.3f us per stage  (%s)\n", mb, box_rows, boxes, S, grid,
           ok ? "ok" : "WAIT EXPIRED", bytes / (double)(t1 - t0), bytes / grid / (per / grid), per / grid / 1e3 / iters, cudaGetErrorString(cudaGetLastError()));
  }
}

static bool make_map_rows(EncodeTiledFn enc, CUtensorMap* tm, void* buf, uint64_t row_bytes, uint64_t rows, uint32_t box_rows) {
  return make_map(enc, tm, buf, row_bytes, rows, box_rows);
}
template <int S>
static void run_gemm_ring(EncodeTiledFn enc, uint8_t* W, uint8_t* X, unsigned long long* out, int T, int O, int K, int tile_t, int extra, int grid, int cextra = 0) {
  CUtensorMap tmA, tmB;
  if (!make_map_rows(enc, &tmA, W, K, O, 128) || !make_map_rows(enc, &tmB, X, K, T, tile_t)) { printf("tensor map failed\n"); return; }
  const size_t smem = 1024 + (size_t)S * (tile_t * 128 + 16384) + 16 * S + 64;
  if (smem > 227 * 1024) return;
  cudaFuncSetAttribute(gemm_ring_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const int tiles_o = O / 128, tiles_t = (T + tile_t - 1) / tile_t, items = tiles_o * tiles_t, ksteps = K / 128;
  for (int rep = 0; rep < 3; ++rep) { gemm_ring_kernel<S><<<grid, 128, smem>>>(tmA, tmB, out, items, tiles_o, ksteps, tile_t, extra, cextra); cudaDeviceSynchronize(); }
  std::vector<unsigned long long> h(grid * 3);
  cudaMemcpy(h.data(), out, grid * 24, cudaMemcpyDeviceToHost);
  unsigned long long t0 = ~0ull, t1 = 0, maxsteps = 0, tot = 0; bool ok = true;
  for (int i = 0; i < grid; ++i) { if (!h[3 * i + 1]) ok = false; if (h[3 * i] < t0) t0 = h[3 * i]; if (h[3 * i + 1] > t1) t1 = h[3 * i + 1]; if (h[3 * i + 2] > maxsteps) maxsteps = h[3 * i + 2]; tot += h[3 * i + 2]; }
  const double bytes = (double)tot * (tile_t * 128.0 + 16384.0);
  printf("gemm ring: T %d O %d K %d, token tile %3d, %d stages, %3d / %3d extra producer / consumer instructions per stage: %s span %.2f us, %.3f us per stage of the busiest CTA, %.1f TB/s into shared memory  (%s)\n",
         T, O, K, tile_t, S, extra, cextra, ok ? "ok" : "WAIT EXPIRED", (t1 - t0) / 1e3, (t1 - t0) / 1e3 / (double)maxsteps, bytes / (double)(t1 - t0) / 1e3, cudaGetErrorString(cudaGetLastError()));
}

int main() {
  void* sym = nullptr; cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym) { printf("no cuTensorMapEncodeTiled\n"); return 1; }
  EncodeTiledFn enc = (EncodeTiledFn)sym;
  int sms = 0; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
  // ---- part 1
  {
    long long* out; cudaMalloc(&out, 128 * 148);
    uint8_t* buf; cudaMalloc(&buf, 64 << 20); cudaMemset(buf, 1, 64 << 20);
    CUtensorMap tm; make_map(enc, &tm, buf, 4096, 16384, 64);
    cudaFuncSetAttribute(issue_cost_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    for (int grid : {1, sms}) {
      for (int rep = 0; rep < 2; ++rep) { issue_cost_kernel<<<grid, 128, 227 * 1024>>>(tm, out); cudaDeviceSynchronize(); }
      std::vector<long long> h(16 * grid); cudaMemcpy(h.data(), out, 128 * grid, cudaMemcpyDeviceToHost);
      double m[16] = {0}; for (int b = 0; b < grid; ++b) for (int j = 0; j < 16; ++j) m[j] += (double)h[b * 16 + j] / grid;
      printf("issue cost, %3d CTAs (SM cycles, mean): arrive %.0f | try_wait on a completed phase %.0f | expect_tx %.0f | expect_tx + TMA issue %.0f each | "
             "6 boxes of 8 KB from L2: first landed after %.0f, all after %.0f  (%s)\n", grid, m[0], m[1], m[8], m[5], m[6], m[7], cudaGetErrorString(cudaGetLastError()));
    }
    cudaFree(buf); cudaFree(out);
  }
  // ---- part 2
  unsigned long long* out; cudaMalloc(&out, 16 * 148);
  for (size_t mb : {32, 64, 96, 1024}) {
    uint8_t* buf; cudaMalloc(&buf, mb << 20); cudaMemset(buf, 1, mb << 20);
    for (int box_rows : {64, 128, 256}) for (int boxes : {1, 2}) { run_ring<2>(enc, buf, mb, out, box_rows, boxes, sms); run_ring<4>(enc, buf, mb, out, box_rows, boxes, sms); }
    cudaFree(buf);
  }
  // ---- part 3: DeiT-B fc2 (25216 tokens, K = 3072 -> 768 out-features), one CTA per SM
  {
    const int T = 25216, O = 768, K = 3072;
    uint8_t *W, *X; unsigned long long* out3;
    cudaMalloc(&W, (size_t)O * K); cudaMalloc(&X, (size_t)T * K); cudaMalloc(&out3, 24 * 148);
    cudaMemset(W, 1, (size_t)O * K); cudaMemset(X, 1, (size_t)T * K);
    for (int extra : {0, 16, 32, 64, 128}) {
      run_gemm_ring<4>(enc, W, X, out3, T, O, K, 256, extra, sms);
      run_gemm_ring<4>(enc, W, X, out3, T, O, K, 128, extra, sms);
    }
    for (int cextra : {32, 64, 128}) run_gemm_ring<4>(enc, W, X, out3, T, O, K, 256, 0, sms, cextra);
    run_gemm_ring<4>(enc, W, X, out3, T, O, K, 256, 32, sms, 64);
    run_gemm_ring<2>(enc, W, X, out3, T, O, K, 128, 0, sms);
    run_gemm_ring<6>(enc, W, X, out3, T, O, K, 128, 0, sms);
    cudaFree(W); cudaFree(X); cudaFree(out3);
  }
  return 0;
}
