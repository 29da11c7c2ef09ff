// C-ABI entry points (see include/nm.h): argument checks, host packing, dispatch.
#include <cuda_runtime.h>

#include <atomic>
#include <cstring>
#include <vector>

#include "nm_internal.h"

namespace nm {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static std::atomic<unsigned long long*> g_trace{nullptr};
unsigned long long* trace_buffer() { return g_trace.load(std::memory_order_relaxed); }

static uint32_t resolve_auto_images(int n, int m, bool clean24, int K, int eb) {
  uint32_t img = NM_IMG_CANONICAL;
  if (n == m) return img;                 // dense rows are already in the canonical values
  // A row that fits in one dense K step (128 bytes) gains nothing from the sparse tensor core,
  // whose K step spans 256 bytes of X that would be mostly padding (measured 21-33 % slower at K = 96).
  if (clean24 && K * eb > 128) img |= NM_IMG_HW24;
  else img |= NM_IMG_DENSE;
  return img;
}

static nm_status check_arch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return NM_ERR_CUDA;
  thread_local int cached_dev = -1, cached_ok = 0;      // per thread: no torn (device, answer) pair
  if (dev != cached_dev) {
    int major = 0, minor = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
      return NM_ERR_CUDA;
    cached_ok = (major == 10 && minor == 0);
    cached_dev = dev;
  }
  return cached_ok ? NM_OK : NM_ERR_ARCH;
}

static bool weight_ok(const nm_weight* w) {
  return w && w->magic == kWeightMagic && w->version == 1 && w->dev_base != nullptr;
}

}  // namespace nm

using namespace nm;

extern "C" {

const char* nm_status_string(nm_status s) {
  switch (s) {
    case NM_OK: return "NM_OK";
    case NM_ERR_INVALID_ARG: return "NM_ERR_INVALID_ARG";
    case NM_ERR_SHAPE: return "NM_ERR_SHAPE";
    case NM_ERR_ALIGN: return "NM_ERR_ALIGN";
    case NM_ERR_NOT_NM: return "NM_ERR_NOT_NM";
    case NM_ERR_UNSUPPORTED: return "NM_ERR_UNSUPPORTED";
    case NM_ERR_WORKSPACE: return "NM_ERR_WORKSPACE";
    case NM_ERR_ARCH: return "NM_ERR_ARCH";
    case NM_ERR_CUDA: return "NM_ERR_CUDA";
    case NM_ERR_TIMEOUT: return "NM_ERR_TIMEOUT";
  }
  return "NM_ERR_UNKNOWN";
}

uint64_t nm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

#ifdef NM_TRACE
// Trace builds only (not declared in nm.h): device buffer of 16 x uint64 per CTA that the following
// launches of the tcgen05 kernels stamp their phases into; nullptr switches the stamps off.
__attribute__((visibility("default"))) void nm_trace_set_buffer(void* dev_buf) {
  g_trace.store(static_cast<unsigned long long*>(dev_buf), std::memory_order_relaxed);
}
#endif

size_t nm_packed_size(int O, int K, int n, int m, nm_dtype dt, uint32_t images) {
  PackLayout L;
  uint32_t img = (images & NM_IMG_AUTO) ? (NM_IMG_CANONICAL | NM_IMG_HW24 | NM_IMG_DENSE | (images & NM_IMG_REMAP48)) : images;
  if (pack_layout(O, K, n, m, dt, img, &L) != NM_OK) return 0;
  return (size_t)L.bytes;
}

// Shared by nm_compress_host / nm_compress: validate, choose images, pack into `host`
// (resized to the layout's size when `host_cap` is null, else checked against *host_cap).
static nm_status pack_to_host(const void* W, int64_t ldw, int O, int K, int n, int m, nm_dtype dt,
                              uint32_t images, uint8_t* host_buf, size_t host_cap, std::vector<uint8_t>* host_vec,
                              nm_weight* out, int64_t* bad_row, int64_t* bad_group) {
  if (!W || !out || ldw < K) return NM_ERR_INVALID_ARG;
  CanonGeom g;
  nm_status st = canon_geom(O, K, n, m, dt, &g);
  if (st != NM_OK) return st;

  // canonical first: it is also the n:m validity check
  std::vector<uint8_t> canon(g.bytes);
  st = build_canonical(W, ldw, g, dt, canon.data(), bad_row, bad_group);
  if (st != NM_OK) return st;

  const bool always_clean = (n <= 2 && m % 4 == 0) || (m == 2 && n == 1);
  const bool is_auto = (images & NM_IMG_AUTO) != 0;
  const bool may_hw24 = (images & NM_IMG_HW24) || (is_auto && n != m);
  bool clean = always_clean && n != m;
  if (!clean && may_hw24) clean = is_24_clean(W, ldw, O, K, dt);
  uint32_t img;
  if (is_auto) {
    img = resolve_auto_images(n, m, clean, K, dt == NM_I8 ? 1 : 2) | (images & NM_IMG_DENSE);
    if ((images & NM_IMG_HW24) && clean) img |= NM_IMG_HW24;
  } else {
    img = images | NM_IMG_CANONICAL;
    if ((img & NM_IMG_HW24) && !clean) return NM_ERR_UNSUPPORTED;
  }
  // the K remap is only built on request, for weights it applies to (not dense, at most 4 nonzeros per 8 k)
  if (images & NM_IMG_REMAP48) {
    if (n == m || !is_48_remappable(W, ldw, O, K, dt)) return NM_ERR_UNSUPPORTED;
    img |= NM_IMG_REMAP48;
  }
  PackLayout L;
  st = pack_layout(O, K, n, m, dt, img, &L);
  if (st != NM_OK) return st;
  uint8_t* host = host_buf;
  if (host_vec) { host_vec->assign(L.bytes, 0); host = host_vec->data(); }
  else {
    if (!host_buf || host_cap < L.bytes) return NM_ERR_WORKSPACE;
    std::memset(host, 0, L.bytes);
  }
  std::memcpy(host + L.off_canonical, canon.data(), g.bytes);
  if (img & NM_IMG_HW24)
    build_hw24(W, ldw, O, K, dt, L, host + L.off_hw24_values, host + L.off_hw24_meta);
  if (L.off_dense) build_dense(W, ldw, O, K, dt, L, host + L.off_dense);
  if (L.off_remap_values) build_remap48(W, ldw, O, K, dt, L, host + L.off_remap_values, host + L.off_remap_meta);

  std::memset(out, 0, sizeof(*out));
  out->magic = kWeightMagic; out->version = 1;
  out->O = O; out->K = K; out->n = n; out->m = m; out->dtype = dt;
  out->images = L.images & ~(uint32_t)NM_IMG_AUTO;
  if (!L.off_dense) out->images &= ~(uint32_t)NM_IMG_DENSE;
  out->dev_base = nullptr; out->bytes = L.bytes;
  out->off_canonical = L.off_canonical;
  out->off_hw24_values = L.off_hw24_values; out->off_hw24_meta = L.off_hw24_meta;
  out->off_dense = L.off_dense;
  out->hw24_row_bytes = L.hw24_row_bytes; out->dense_row_bytes = L.dense_row_bytes;
  out->hw24_meta_kblocks = L.hw24_meta_kblocks;
  if (!L.off_remap_values) out->images &= ~(uint32_t)NM_IMG_REMAP48;
  out->off_remap_values = L.off_remap_values; out->off_remap_meta = L.off_remap_meta;
  out->remap_row_bytes = L.remap_row_bytes; out->remap_meta_kblocks = L.remap_meta_kblocks;
  out->remap_k = L.remap_k; out->remap_k_main = L.remap_k_main;
  return NM_OK;
}

nm_status nm_compress_host(const void* W, int64_t ldw, int O, int K, int n, int m, nm_dtype dt,
                           uint32_t images, void* host_buf, size_t host_bytes, nm_weight* out,
                           int64_t* bad_row, int64_t* bad_group) {
  return pack_to_host(W, ldw, O, K, n, m, dt, images, static_cast<uint8_t*>(host_buf), host_bytes, nullptr,
                      out, bad_row, bad_group);
}

nm_status nm_compress(const void* W, int64_t ldw, int O, int K, int n, int m, nm_dtype dt,
                      uint32_t images, void* dev_buf, size_t dev_bytes, void* stream,
                      nm_weight* out, int64_t* bad_row, int64_t* bad_group) {
  if (!dev_buf) return NM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev_buf) & 255) return NM_ERR_ALIGN;
  std::vector<uint8_t> host;
  nm_weight w;
  nm_status st = pack_to_host(W, ldw, O, K, n, m, dt, images, nullptr, 0, &host, &w, bad_row, bad_group);
  if (st != NM_OK) return st;
  if (dev_bytes < w.bytes) return NM_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(dev_buf, host.data(), w.bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return NM_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return NM_ERR_CUDA;
  w.dev_base = dev_buf;
  *out = w;
  return NM_OK;
}

nm_status nm_prune_magnitude(void* W, int64_t ldw, int O, int K, int n, int m, nm_dtype dt) {
  CanonGeom g;
  if (!W || ldw < K) return NM_ERR_INVALID_ARG;
  nm_status st = canon_geom(O, K, n, m, dt, &g);
  if (st != NM_OK) return st;
  for (int o = 0; o < O; ++o)
    for (int gi = 0; gi < g.G; ++gi) {
      const int64_t base = (int64_t)o * ldw + (int64_t)gi * m;
      int mag[16];
      for (int p = 0; p < m; ++p) {
        if (dt == NM_I8) { int v = static_cast<int8_t*>(W)[base + p]; mag[p] = v < 0 ? -v : v; }
        else mag[p] = static_cast<uint16_t*>(W)[base + p] & 0x7fff;   // fp16 magnitude order == bit order
      }
      uint32_t keep = 0;
      for (int r = 0; r < n; ++r) {
        int best = -1;
        for (int p = 0; p < m; ++p)
          if (!(keep & (1u << p)) && (best < 0 || mag[p] > mag[best])) best = p;
        keep |= 1u << best;
      }
      for (int p = 0; p < m; ++p)
        if (!(keep & (1u << p))) {
          if (dt == NM_I8) static_cast<int8_t*>(W)[base + p] = 0;
          else static_cast<uint16_t*>(W)[base + p] = 0;
        }
    }
  return NM_OK;
}

nm_status nm_export_canonical(const nm_weight* w, void* host_buf, size_t* bytes, void* stream) {
  if (!weight_ok(w) || !bytes) return NM_ERR_INVALID_ARG;
  CanonGeom g;
  nm_status st = canon_geom(w->O, w->K, w->n, w->m, w->dtype, &g);
  if (st != NM_OK) return st;
  if (!host_buf) { *bytes = g.bytes; return NM_OK; }
  if (*bytes < g.bytes) return NM_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_buf, static_cast<const uint8_t*>(w->dev_base) + w->off_canonical, g.bytes,
                      cudaMemcpyDeviceToHost, s) != cudaSuccess) return NM_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return NM_ERR_CUDA;
  *bytes = g.bytes;
  return NM_OK;
}

nm_status nm_decompress(const nm_weight* w, void* W_host, int64_t ldw, void* stream) {
  if (!weight_ok(w) || !W_host || ldw < w->K) return NM_ERR_INVALID_ARG;
  size_t bytes = 0;
  nm_status st = nm_export_canonical(w, nullptr, &bytes, stream);
  if (st != NM_OK) return st;
  std::vector<uint8_t> canon(bytes);
  st = nm_export_canonical(w, canon.data(), &bytes, stream);
  if (st != NM_OK) return st;
  return decode_canonical(canon.data(), bytes, W_host, ldw);
}

nm_status nm_spmm(const void* X, int64_t ldx, int T, const nm_weight* w, const nm_plan* plan,
                  void* Y, int64_t ldy, nm_out_dtype od, void* workspace, size_t workspace_bytes,
                  uint32_t* status, void* stream) {
  return nm_spmm_ex(X, ldx, T, w, plan, Y, ldy, od, nullptr, workspace, workspace_bytes, status, stream);
}

nm_status nm_spmm_ex(const void* X, int64_t ldx, int T, const nm_weight* w, const nm_plan* plan,
                     void* Y, int64_t ldy, nm_out_dtype od, const nm_epilogue* epi, void* workspace,
                     size_t workspace_bytes, uint32_t* status, void* stream) {
  if (!X || !Y || !weight_ok(w) || T < 1) return NM_ERR_INVALID_ARG;
  if (ldx < w->K || ldy < w->O) return NM_ERR_INVALID_ARG;
  if (epi) {
    if (w->dtype != NM_I8 || od != NM_OUT_I8 || !epi->scale_dev) return NM_ERR_INVALID_ARG;
  } else if (w->dtype == NM_I8 ? od != NM_OUT_I32 : (od != NM_OUT_F32 && od != NM_OUT_F16)) {
    return NM_ERR_INVALID_ARG;
  }
  nm_status st = check_arch();
  if (st != NM_OK) return st;

  const int eb = elem_bytes(w->dtype);
  const bool aligned = !(reinterpret_cast<uintptr_t>(X) & 15) && ((uint64_t)ldx * eb) % 16 == 0 &&
                       !(reinterpret_cast<uintptr_t>(Y) & 15);
  SpmmArgs a{X, ldx, T, w, {}, Y, ldy, od, workspace, workspace_bytes, status, stream, {}};
  if (epi) a.epi = *epi;
  if (plan) {
    a.plan = *plan;
    if (a.plan.path != NM_PATH_SIMT && !aligned) return NM_ERR_ALIGN;
  } else {
    int dev = 0, sms = kDefaultSMs;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return NM_ERR_CUDA;
    st = nm_plan_shape(T, w->O, w->K, w->n, w->m, (nm_dtype)w->dtype, od, w->images, sms, &a.plan);
    if (st != NM_OK) return st;
    // the automatic plan never fails on alignment or scratch: it degrades instead
    if (a.plan.path != NM_PATH_SIMT && !aligned) { a.plan.path = NM_PATH_SIMT; a.plan.split_k = 1; a.plan.workspace_bytes = 0; }
    if (a.plan.workspace_bytes > workspace_bytes || (a.plan.workspace_bytes && !workspace)) {
      if (a.plan.path == NM_PATH_UMMA_EXPAND) {      // no room for the dense copy: decode on chip instead
        a.plan.path = NM_PATH_UMMA_DECODE; a.plan.resident = NM_RES_W; a.plan.cta_group = 1; a.plan.issuers = 1;
      }
      a.plan.split_k = 1; a.plan.workspace_bytes = 0;
    }
  }
  // NM_PATH_UMMA_EXPAND: write the dense rows into the head of the workspace, then run the dense path on them
  nm_weight expanded;
  if (a.plan.path == NM_PATH_UMMA_EXPAND) {
    if (w->n == w->m) {
      a.plan.path = NM_PATH_UMMA_DENSE;              // dense rows are the canonical values already
    } else {
      const uint64_t head = expand_workspace_bytes(w->O, w->K, eb);
      if (!workspace || workspace_bytes < head) return NM_ERR_WORKSPACE;
      if (reinterpret_cast<uintptr_t>(workspace) & 15) return NM_ERR_ALIGN;
      st = launch_expand(w, workspace, stream);
      if (st != NM_OK) return st;
      expanded = *w;
      expanded.dev_base = workspace;
      expanded.images = NM_IMG_DENSE;
      expanded.off_dense = 0;
      expanded.dense_row_bytes = round_up((uint64_t)w->K * eb, 16);
      a.w = &expanded;
      a.w_fresh = true;
      a.plan.path = NM_PATH_UMMA_DENSE;
      a.workspace = static_cast<uint8_t*>(workspace) + head;
      a.workspace_bytes = workspace_bytes - head;
    }
  }
  // NM_PATH_UMMA_REMAP48: gather the third-chunk activations into the head of the workspace, then run the
  // sparse kernel over the remapped weight; its K steps beyond the main range read the gathered copy
  nm_weight remapped;
  if (a.plan.path == NM_PATH_UMMA_REMAP48) {
    if (!(w->images & NM_IMG_REMAP48) || !w->off_remap_values) return NM_ERR_UNSUPPORTED;
    if (a.plan.split_k > 1 || a.plan.resident != NM_RES_NONE || epi) return NM_ERR_INVALID_ARG;
    const uint64_t head = remap_workspace_bytes(T, w->K, eb);
    if (!workspace || workspace_bytes < head) return NM_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15) return NM_ERR_ALIGN;
    st = launch_remap_gather(X, ldx, T, w->K, w->dtype, workspace, stream);
    if (st != NM_OK) return st;
    remapped = *w;
    remapped.K = w->remap_k; remapped.n = 2; remapped.m = 4;
    remapped.images = NM_IMG_HW24;
    remapped.off_hw24_values = w->off_remap_values; remapped.off_hw24_meta = w->off_remap_meta;
    remapped.hw24_row_bytes = w->remap_row_bytes; remapped.hw24_meta_kblocks = w->remap_meta_kblocks;
    a.w = &remapped;
    a.X_ovf = workspace;
    a.ld_ovf = (int64_t)(round_up((uint64_t)(w->K / 2) * eb, 16) / eb);
    a.k_x = w->K; a.k_ovf = w->K / 2;
    a.ksteps_main = w->remap_k_main * eb / 256;
    a.plan.path = NM_PATH_UMMA_SP24;
    a.plan.cta_group = 1;
    a.workspace = static_cast<uint8_t*>(workspace) + head;
    a.workspace_bytes = workspace_bytes - head;
  }
  switch (a.plan.path) {
    case NM_PATH_SIMT: return launch_simt(a);
    case NM_PATH_UMMA_DENSE:
    case NM_PATH_UMMA_SP24:
    case NM_PATH_UMMA_DECODE: {
      if (a.plan.cta_group == 2) {           // CTA pairs are a request: the pair launcher declines what it cannot run
        bool handled = false;
        st = launch_umma_pair(a, &handled);
        if (handled || st != NM_OK) return st;
      }
      return launch_umma(a);
    }
    default: return NM_ERR_INVALID_ARG;
  }
}

nm_status nm_latency_table(const int32_t* shapes, int n_shapes, const int32_t* nm_pairs, int n_pairs,
                           nm_dtype dt, nm_out_dtype od, int reps, void* X, void* Wpack, size_t wpack_bytes,
                           void* Y, void* workspace, size_t workspace_bytes, nm_latency_row* rows, void* stream) {
  if (!shapes || !nm_pairs || !rows || !X || !Wpack || !Y || n_shapes < 1 || n_pairs < 1 || reps < 1)
    return NM_ERR_INVALID_ARG;
  nm_status st = check_arch();
  if (st != NM_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The measurements run on a private stream (the caller's may be the legacy default stream,
  // which cannot be captured into a graph) once the caller's stream has drained.
  if (cudaStreamSynchronize(s) != cudaSuccess) return NM_ERR_CUDA;
  cudaStream_t cs = nullptr;
  if (cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) != cudaSuccess) return NM_ERR_CUDA;
  void* const cs_arg = static_cast<void*>(cs);
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { cudaStreamDestroy(cs); return NM_ERR_CUDA; }
  const int eb = elem_bytes(dt);
  for (int si = 0; si < n_shapes; ++si) {
    const int T = shapes[3 * si], O = shapes[3 * si + 1], K = shapes[3 * si + 2];
    for (int pi = 0; pi < n_pairs; ++pi) {
      const int n = nm_pairs[2 * pi], m = nm_pairs[2 * pi + 1];
      nm_latency_row& r = rows[(size_t)si * n_pairs + pi];
      std::memset(&r, 0, sizeof r);
      r.T = T; r.O = O; r.K = K; r.n = n; r.m = m; r.dtype = dt; r.out_dtype = od; r.reps = reps;
      CanonGeom g;
      st = (T >= 1) ? canon_geom(O, K, n, m, dt, &g) : NM_ERR_INVALID_ARG;
      if (st != NM_OK) { r.status = st; continue; }
      // synthetic weight: every group keeps its first n positions, value 1
      std::vector<uint8_t> Wd((size_t)O * K * eb, 0);
      for (int o = 0; o < O; ++o)
        for (int k = 0; k < K; ++k)
          if (k % m < n) {
            if (dt == NM_I8) reinterpret_cast<int8_t*>(Wd.data())[(size_t)o * K + k] = 1;
            else reinterpret_cast<uint16_t*>(Wd.data())[(size_t)o * K + k] = 0x3c00;   // 1.0
          }
      nm_weight w;
      st = nm_compress(Wd.data(), K, O, K, n, m, dt, NM_IMG_AUTO, Wpack, wpack_bytes, cs_arg, &w, nullptr, nullptr);
      if (st != NM_OK) { r.status = st; continue; }
      nm_plan plan;
      st = nm_plan_create(T, &w, od, -1, &plan);
      if (st == NM_OK && plan.workspace_bytes > workspace_bytes) { plan.split_k = 1; plan.workspace_bytes = 0; }
      // rows of X that TMA cannot address (pitch not a 16-byte multiple) run on the CUDA-core path,
      // exactly as nm_spmm's automatic plan would
      if (st == NM_OK && ((uint64_t)K * eb) % 16 != 0) { plan.path = NM_PATH_SIMT; plan.split_k = 1; plan.workspace_bytes = 0; }
      if (st != NM_OK) { r.status = st; continue; }
      r.path = plan.path; r.tile_t = plan.tile_t; r.split_k = plan.split_k;
      float sum = 0.f, best = 1e30f;
      // Preferred timing: `reps` back-to-back calls captured in one CUDA graph on the private
      // stream and replayed, so that the figure is the steady-state cost of the operator inside a
      // model (launch latency hidden, prologue overlapped with the previous call) rather than
      // the cost of one isolated launch.  mean = best-of-three replays / reps.
      bool timed = false;
      for (int warm = 0; warm < 2 && st == NM_OK; ++warm)
        st = nm_spmm(X, K, T, &w, &plan, Y, O, od, workspace, workspace_bytes, nullptr, cs_arg);
      if (st == NM_OK && cudaStreamSynchronize(cs) != cudaSuccess) st = NM_ERR_CUDA;
      if (st == NM_OK && cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        nm_status cst = NM_OK;
        for (int it = 0; it < reps && cst == NM_OK; ++it)
          cst = nm_spmm(X, K, T, &w, &plan, Y, O, od, workspace, workspace_bytes, nullptr, cs_arg);
        cudaGraph_t graph = nullptr;
        cudaGraphExec_t exec = nullptr;
        const bool ended = cudaStreamEndCapture(cs, &graph) == cudaSuccess && graph != nullptr;
        if (ended && cst == NM_OK && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
          bool ok = cudaGraphLaunch(exec, cs) == cudaSuccess && cudaStreamSynchronize(cs) == cudaSuccess;
          for (int rep = 0; rep < 3 && ok; ++rep) {
            cudaEventRecord(e0, cs);
            ok = cudaGraphLaunch(exec, cs) == cudaSuccess;
            cudaEventRecord(e1, cs);
            ok = ok && cudaEventSynchronize(e1) == cudaSuccess;
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            ms /= (float)reps;
            sum += ms;
            best = ms < best ? ms : best;
          }
          if (ok) { sum = sum / 3.0f * (float)reps; timed = true; }
        }
        if (exec) cudaGraphExecDestroy(exec);
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
      }
      if (!timed) {            // capture unavailable: one event pair per call
        sum = 0.f; best = 1e30f;
        for (int it = 0; it < reps && st == NM_OK; ++it) {
          cudaEventRecord(e0, cs);
          st = nm_spmm(X, K, T, &w, &plan, Y, O, od, workspace, workspace_bytes, nullptr, cs_arg);
          cudaEventRecord(e1, cs);
          if (cudaEventSynchronize(e1) != cudaSuccess) st = NM_ERR_CUDA;
          float ms = 0.f;
          cudaEventElapsedTime(&ms, e0, e1);
          sum += ms; best = ms < best ? ms : best;
        }
      }
      r.status = st;
      if (st == NM_OK) { r.us_mean = 1e3f * sum / reps; r.us_min = 1e3f * best; }
    }
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaStreamSynchronize(cs);
  cudaStreamDestroy(cs);
  return NM_OK;
}

}  // extern "C"
