// Main-loop probe for sm_100a (harness only): the smallest complete dense INT8 GEMM main loop that the
// tcgen05 kernels of this repository are built around -- one producer thread (tiled TMA loads into a
// ring), one issuing warp (tcgen05.mma into tensor memory, tcgen05.commit releases the stage), eight
// epilogue warps (tcgen05.ld -> shared-memory patch -> global memory) -- with the parts of the epilogue
// switchable, to see what each part costs the main loop.  DeiT-B fc2 operands (25216 x 3072 activations,
// 768 x 3072 weights, INT32 out); single CTAs with 128 out-features x `tile_t` tokens per tile.
// Every wait is a bounded poll.  With all-ones operands every output equals K, which the host checks.
//   epi 0: no epilogue (accumulators are overwritten)      1: tcgen05.ld only
//       2: + transposed st.shared into the patch           3: + TMA store of the patch (the kernels' epilogue)
//       4: patch written out by plain 16-byte global stores 5: as 4, into a 4096-row window (stays in L2)
//   loads 0: the issuing warp issues no MMAs (stages are recycled at once);  loads 2: nothing is loaded
//   or multiplied, only the epilogue's stores run.
#include "nm_umma_common.cuh"

#include <cstdio>
#include <cstdlib>
#include <vector>

using namespace nm;

namespace mlprobe {

__device__ __forceinline__ bool poll(uint32_t bar, uint32_t par) {
  for (uint32_t i = 0; i < (1u << 16); ++i) if (mbar_try_wait(bar, par)) return true;      // a failed try_wait has already waited a while inside the instruction
  return false;
}

template <int S>
__global__ void __launch_bounds__(320, 1)
mainloop_kernel(int32_t* __restrict__ Y, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmY, int T, int O, unsigned long long* outg, int items, int tiles_o,
                int ksteps, int tile_t, int loads, int epi) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_slot;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bbytes = (uint32_t)tile_t * 128u, abytes = 16384u, sb = bbytes + abytes;
  const uint32_t patches = base + S * sb;
  const uint32_t full = patches + 8 * 4096, empty = full + 8 * S, tfull = empty + 8 * S, tempty = tfull + 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ksteps_run = (loads == 2) ? 0 : ksteps;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2 * S; ++s) mbar_init(full + 8 * s, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(tfull + 8 * b, 1); mbar_init(tempty + 8 * b, 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  if (threadIdx.x == 0) {
    // ---------------- producer
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool ok = true, wrapped = false;
    uint32_t s = 0, ph = 0; long steps = 0;
    for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
      const int o0 = (item % tiles_o) * 128, t0r = (item / tiles_o) * tile_t;
      for (int ks = 0; ks < ksteps_run; ++ks) {
        if (wrapped) { ok = poll(empty + 8 * s, ph ^ 1u); if (!ok) break; }
        const uint32_t st = base + s * sb;
        mbar_expect_tx(full + 8 * s, sb);
        tma_load_2d(st, &tmB, full + 8 * s, ks * 128, t0r);
        tma_load_2d(st + bbytes, &tmA, full + 8 * s, ks * 128, o0);
        ++steps;
        if (++s == S) { s = 0; ph ^= 1u; wrapped = true; }
      }
    }
    // the last loads must have landed and the MMAs that read them retired before the CTA leaves
    for (int d = 0; d < S && ok; ++d)
      if (steps > d) { const long g = steps - 1 - d; ok = poll(full + 8 * (uint32_t)(g % S), (uint32_t)((g / S) & 1)); }
    for (int d = 0; d < S && ok; ++d)
      if (steps > d) { const long g = steps - 1 - d; ok = poll(empty + 8 * (uint32_t)(g % S), (uint32_t)((g / S) & 1)); }
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    outg[blockIdx.x * 3] = t0; outg[blockIdx.x * 3 + 1] = ok ? t1 : 0; outg[blockIdx.x * 3 + 2] = (unsigned long long)steps;
  } else if (warp == 1) {
    // ---------------- MMA issuer (whole warp, the wrappers elect the issuing lane)
    const uint32_t idesc = ((uint32_t)(tile_t >> 3) << 17) | ((uint32_t)(128 >> 4) << 24) | (2u << 4) | (1u << 7) | (1u << 10);
    uint32_t s = 0, ph = 0; bool ok = true; int n = 0;
    for (int item = blockIdx.x; item < items && ok; item += gridDim.x, ++n) {
      const uint32_t buf = (uint32_t)(n & 1), use = (uint32_t)(n >> 1);
      const uint32_t d_tmem = tmem_base + buf * (uint32_t)tile_t;
      if (epi && use >= 1u) { ok = poll(tempty + 8 * buf, (use - 1u) & 1u); ok = __all_sync(0xffffffffu, ok); if (!ok) break; tc_fence_after(); }
      for (int ks = 0; ks < ksteps_run; ++ks) {
        ok = poll(full + 8 * s, ph);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (loads == 1) {
          const uint32_t st = base + s * sb;
          const uint64_t db0 = desc_sw128(st), da0 = desc_sw128(st + bbytes);
#pragma unroll
          for (int j = 0; j < 4; ++j) tc_mma_dense<NM_I8>(d_tmem, da0 + (uint64_t)(2 * j), db0 + (uint64_t)(2 * j), idesc, (ks > 0 || j > 0) ? 1u : 0u);
        }
        tc_commit(empty + 8 * s);
        if (++s == S) { s = 0; ph ^= 1u; }
      }
      if (!ok) break;
      if (epi) tc_commit(tfull + 8 * buf);
    }
  } else if (epi && warp >= 2) {
    // ---------------- epilogue warps 2..9 (the idle lanes of warp 0 must not come here): lane = out feature, register j = token
    const int e = warp - 2, q = warp & 3, h = e >> 2;
    const uint32_t patch = patches + (uint32_t)e * 4096u;
    int n = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, ++n) {
      const int o0 = (item % tiles_o) * 128, t0 = (item / tiles_o) * tile_t;
      const uint32_t buf = (uint32_t)(n & 1), use = (uint32_t)(n >> 1);
      uint32_t ok = 1;
      if (lane == 0) ok = poll(tfull + 8 * buf, use & 1u) ? 1u : 0u;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      const int o_base = o0 + q * 32;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)tile_t;
      for (int cc = (h ^ (n & 1)) * 32; cc < tile_t; cc += 64) {
        const int t = t0 + cc;
        if (t >= T) break;
        uint32_t r[32];
        if (lane == 0 && epi == 3) tma_store_wait_read();
        __syncwarp();
        tc_ld_32x32(lane_addr + (uint32_t)cc, r);
        if (epi == 1) {
          uint32_t x = 0;
#pragma unroll
          for (int j = 0; j < 32; ++j) x ^= r[j];
          if (x == 0x12345678u) outg[0] = x;      // keeps the loads alive
          continue;
        }
#pragma unroll
        for (int j = 0; j < 32; ++j)
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(patch + (uint32_t)j * 128u + (uint32_t)lane * 4u), "r"(r[j]) : "memory");
        if (epi == 2) continue;
        if (epi >= 4) {
          // 8 lanes write one 128-byte row segment with 16-byte stores, 4 rows per instruction
          __syncwarp();
          const int row0 = lane >> 3, c16 = lane & 7;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int row = row0 + 4 * i;
            uint32_t a0, a1, a2, a3;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                         : "r"(patch + (uint32_t)row * 128u + (uint32_t)c16 * 16u) : "memory");
            if (t + row < T && o_base + c16 * 4 < O) {
              int32_t* dst = Y + (size_t)((epi == 5) ? ((t + row) & 4095) : (t + row)) * O + o_base + c16 * 4;
              asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(a0), "r"(a1), "r"(a2), "r"(a3) : "memory");
            }
          }
          __syncwarp();
          continue;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && o_base < O) tma_store_2d(&tmY, patch, o_base * 4, t);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty + 8 * buf);
    }
    if (lane == 0) tma_store_wait_read();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

}  // namespace mlprobe
using namespace mlprobe;

static int32_t* g_Y = nullptr;

template <int S>
static void run(uint8_t* W, uint8_t* X, unsigned long long* out, int T, int O, int K, int tile_t, int loads, int epi, int grid) {
  CUtensorMap tmA, tmB, tmY;
  if (!make_map(&tmA, W, K, O, K, 128u, 128u, true) || !make_map(&tmB, X, K, T, K, 128u, (uint32_t)tile_t, true) ||
      !make_map(&tmY, g_Y, (uint64_t)O * 4, T, (uint64_t)O * 4, 128u, 32u, false)) { printf("tensor map failed\n"); return; }
  const size_t smem = 1024 + (size_t)S * (tile_t * 128 + 16384) + 8 * 4096 + 16 * S + 32 + 64;
  if (smem > 226 * 1024) { printf("does not fit\n"); return; }
  if (cudaFuncSetAttribute(mainloop_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) { printf("attribute failed\n"); return; }
  const int tiles_o = O / 128, tiles_t = (T + tile_t - 1) / tile_t, items = tiles_o * tiles_t, ksteps = K / 128;
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  float ms = 0;
  for (int rep = 0; rep < 3; ++rep) {
    cudaEventRecord(e0);
    mainloop_kernel<S><<<grid, 320, smem>>>(g_Y, tmA, tmB, tmY, T, O, out, items, tiles_o, ksteps, tile_t, loads, epi);
    cudaEventRecord(e1);
    if (cudaDeviceSynchronize() != cudaSuccess) { printf("launch failed: %s\n", cudaGetErrorString(cudaGetLastError())); exit(2); }
  }
  cudaEventElapsedTime(&ms, e0, e1);
  std::vector<unsigned long long> h(grid * 3);
  cudaMemcpy(h.data(), out, grid * 24, cudaMemcpyDeviceToHost);
  unsigned long long t0 = ~0ull, t1 = 0, maxsteps = 0; bool ok = true;
  for (int i = 0; i < grid; ++i) { if (!h[3 * i + 1]) ok = false; if (h[3 * i] < t0) t0 = h[3 * i]; if (h[3 * i + 1] > t1) t1 = h[3 * i + 1]; if (h[3 * i + 2] > maxsteps) maxsteps = h[3 * i + 2]; }
  long bad = -1;
  if (loads == 1 && (epi == 3 || epi == 4)) {
    std::vector<int32_t> y((size_t)T * O);
    cudaMemcpy(y.data(), g_Y, y.size() * 4, cudaMemcpyDeviceToHost);
    bad = 0;
    for (size_t i = 0; i < y.size(); ++i) if (y[i] != K) ++bad;
    cudaMemset(g_Y, 0, y.size() * 4);
  }
  static const char* lname[] = {"loads only", "loads + MMAs", "stores only"};
  static const char* ename[] = {"no epilogue", "tcgen05.ld", "tcgen05.ld + st.shared", "+ TMA stores", "+ plain 16-byte stores", "+ plain stores into an L2-resident window"};
  printf("tile %3d, %d stages, %-12s, %-42s: %s kernel %.1f us (isolated launch, events), producer's span %.2f us", tile_t, S, lname[loads], ename[epi],
         ok ? "ok" : "WAIT EXPIRED", ms * 1e3, (t1 - t0) / 1e3);
  if (maxsteps) printf(", %.3f us per K step", (t1 - t0) / 1e3 / (double)maxsteps);
  if (bad >= 0) printf(", wrong outputs %ld", bad);
  printf("\n");
}

int main() {
  setvbuf(stdout, NULL, _IONBF, 0);
  cudaFree(0);
  const int T = 25216, O = 768, K = 3072;
  int sms = 0; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
  uint8_t *W, *X; unsigned long long* out;
  cudaMalloc(&W, (size_t)O * K); cudaMalloc(&X, (size_t)T * K); cudaMalloc(&out, 24 * 160);
  cudaMemset(W, 1, (size_t)O * K); cudaMemset(X, 1, (size_t)T * K);
  cudaMalloc(&g_Y, (size_t)T * O * 4); cudaMemset(g_Y, 0, (size_t)T * O * 4);
  if (sms > 160) sms = 160;
  run<3>(W, X, out, T, O, K, 256, 0, 0, sms);
  for (int epi = 0; epi <= 5; ++epi) run<3>(W, X, out, T, O, K, 256, 1, epi, sms);
  run<4>(W, X, out, T, O, K, 128, 0, 0, sms);
  for (int epi : {0, 3, 4}) run<4>(W, X, out, T, O, K, 128, 1, epi, sms);
  run<3>(W, X, out, T, O, K, 256, 2, 3, sms);
  run<3>(W, X, out, T, O, K, 256, 2, 4, sms);
  return 0;
}
