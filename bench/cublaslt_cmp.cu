// Dense library comparator for the benchmark harness: cuBLASLt matmul with an algorithm sweep.
//
// Y[T x O] (row-major) = X[T x K] * W[O x K]^T, INT8 -> INT32 (CUBLAS_COMPUTE_32I) or FP16 -> FP16
// with FP32 accumulation (CUBLAS_COMPUTE_32F), expressed for cuBLASLt as the column-major "TN"
// product C[O x T] = op(A)[O x K] * B[K x T] with A = W (lda = K, transposed) and B = X (ldb = K).
// cublasLtMatmulAlgoGetHeuristic returns up to `max_algos` candidate algorithms; every one that
// runs is timed with CUDA events over `reps` back-to-back calls and the fastest is reported next to
// the heuristic's first choice.  Harness only: nothing in the product library calls this.
#include <cublasLt.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

namespace {
cublasLtHandle_t handle() {
  static cublasLtHandle_t h = nullptr;
  if (!h) cublasLtCreate(&h);
  return h;
}
}  // namespace

extern "C" __attribute__((visibility("default")))
int lt_gemm_sweep(int dtype, int T, int O, int K, const void* X, const void* W, void* Y, void* workspace,
                  size_t workspace_bytes, int max_algos, int reps, void* stream_v, float* best_us,
                  float* heuristic_us, int* n_ok) {
  cublasLtHandle_t lt = handle();
  if (!lt || max_algos < 1 || reps < 1) return -1;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const bool i8 = dtype == 0;
  const cudaDataType_t in_t = i8 ? CUDA_R_8I : CUDA_R_16F, out_t = i8 ? CUDA_R_32I : CUDA_R_16F;
  cublasLtMatmulDesc_t op = nullptr;
  cublasLtMatrixLayout_t la = nullptr, lb = nullptr, lc = nullptr;
  cublasLtMatmulPreference_t pref = nullptr;
  int rc = 0;
  const cublasOperation_t ta = CUBLAS_OP_T, tb = CUBLAS_OP_N;
  if (cublasLtMatmulDescCreate(&op, i8 ? CUBLAS_COMPUTE_32I : CUBLAS_COMPUTE_32F, i8 ? CUDA_R_32I : CUDA_R_32F) != CUBLAS_STATUS_SUCCESS) return -2;
  cublasLtMatmulDescSetAttribute(op, CUBLASLT_MATMUL_DESC_TRANSA, &ta, sizeof ta);
  cublasLtMatmulDescSetAttribute(op, CUBLASLT_MATMUL_DESC_TRANSB, &tb, sizeof tb);
  if (cublasLtMatrixLayoutCreate(&la, in_t, K, O, K) != CUBLAS_STATUS_SUCCESS ||      // A: K x O column-major, used transposed
      cublasLtMatrixLayoutCreate(&lb, in_t, K, T, K) != CUBLAS_STATUS_SUCCESS ||      // B: K x T column-major
      cublasLtMatrixLayoutCreate(&lc, out_t, O, T, O) != CUBLAS_STATUS_SUCCESS ||     // C: O x T column-major = Y row-major
      cublasLtMatmulPreferenceCreate(&pref) != CUBLAS_STATUS_SUCCESS) rc = -3;
  std::vector<cublasLtMatmulHeuristicResult_t> res(max_algos);
  int found = 0;
  if (!rc) {
    cublasLtMatmulPreferenceSetAttribute(pref, CUBLASLT_MATMUL_PREF_MAX_WORKSPACE_BYTES, &workspace_bytes, sizeof workspace_bytes);
    if (cublasLtMatmulAlgoGetHeuristic(lt, op, la, lb, lc, lc, pref, max_algos, res.data(), &found) != CUBLAS_STATUS_SUCCESS || found < 1) rc = -4;
  }
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (!rc && (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess)) rc = -5;
  float best = 1e30f, first = -1.f;
  int ok_count = 0;
  const int32_t alpha_i = 1, beta_i = 0;
  const float alpha_f = 1.f, beta_f = 0.f;
  const void* alpha = i8 ? static_cast<const void*>(&alpha_i) : static_cast<const void*>(&alpha_f);
  const void* beta = i8 ? static_cast<const void*>(&beta_i) : static_cast<const void*>(&beta_f);
  for (int a = 0; !rc && a < found; ++a) {
    if (res[a].state != CUBLAS_STATUS_SUCCESS || res[a].workspaceSize > workspace_bytes) continue;
    auto run = [&]() {
      return cublasLtMatmul(lt, op, alpha, W, la, X, lb, beta, Y, lc, Y, lc, &res[a].algo, workspace, workspace_bytes, stream);
    };
    if (run() != CUBLAS_STATUS_SUCCESS || cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); continue; }
    float t_best = 1e30f;
    for (int round = 0; round < 2; ++round) {            // best of two timed rounds
      cudaEventRecord(e0, stream);
      bool ok = true;
      for (int r = 0; r < reps && ok; ++r) ok = run() == CUBLAS_STATUS_SUCCESS;
      cudaEventRecord(e1, stream);
      if (!ok || cudaEventSynchronize(e1) != cudaSuccess) { cudaGetLastError(); t_best = 1e30f; break; }
      float ms = 0.f;
      cudaEventElapsedTime(&ms, e0, e1);
      const float us = ms * 1e3f / reps;
      if (us < t_best) t_best = us;
    }
    if (t_best >= 1e29f) continue;
    ++ok_count;
    if (first < 0.f) first = t_best;                     // the heuristic's first usable choice
    if (t_best < best) best = t_best;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (pref) cublasLtMatmulPreferenceDestroy(pref);
  if (la) cublasLtMatrixLayoutDestroy(la);
  if (lb) cublasLtMatrixLayoutDestroy(lb);
  if (lc) cublasLtMatrixLayoutDestroy(lc);
  if (op) cublasLtMatmulDescDestroy(op);
  if (rc) return rc;
  if (ok_count == 0) return -6;
  *best_us = best; *heuristic_us = first; *n_ok = ok_count;
  return 0;
}
