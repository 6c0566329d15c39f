// C-ABI entry points that only validate and dispatch, plus the library's
// small amount of per-device state (architecture check, status word).
#include "common.cuh"

namespace peqa {

thread_local int g_last_cuda_error = 0;

// Written by kernels whose bounded waits expire: [0] = status code, [1..3] = where.
__device__ int g_status_word[4];

int status_word(int** dev_ptr) {
  void* p = nullptr;
  PEQA_CUDA(cudaGetSymbolAddress(&p, g_status_word));
  *dev_ptr = static_cast<int*>(p);
  return PEQA_OK;
}

int check_arch() {
  static thread_local int cached_dev = -1;
  static thread_local int cached_ok = 0;
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev != cached_dev) {
    int major = 0;
    PEQA_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    cached_dev = dev;
    cached_ok = (major == 10);
  }
  return cached_ok ? PEQA_OK : PEQA_ERR_ARCH;
}

int check_qweight(const peqa_qweight_t* w, int* g, int* G) {
  if (!w) return PEQA_ERR_NULL;
  if (!w->qweight || !w->zeros || !w->scales) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(w->out_features, w->in_features, w->bits, w->group_size));
  if (!aligned16(w->qweight) || !aligned16(w->scales)) return PEQA_ERR_ALIGNMENT;
  *g = effective_group(w->in_features, w->group_size);
  *G = w->in_features / *g;
  return PEQA_OK;
}

}  // namespace peqa

using namespace peqa;

extern "C" int peqa_version(void) { return 100; }

extern "C" int peqa_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" size_t peqa_workspace_bytes(int op, int T, const peqa_qweight_t* w) {
  if (!w || T <= 0) return 0;
  if (check_bits_shape(w->out_features, w->in_features, w->bits, w->group_size) != PEQA_OK)
    return 0;
  const int g = effective_group(w->in_features, w->group_size);
  switch (op) {
    case PEQA_OP_BWD: return ds_workspace_bytes(w, g, T);
    case PEQA_OP_DECODE: return decode_workspace_bytes(w, g, T);
    case PEQA_OP_BWD_DSDZ: return dsdz_workspace_bytes(w, g, T);
    case PEQA_OP_BWD_DS_FROM_Y: return g == w->in_features ? ds_from_y_workspace_bytes(w, T) : 0;
    default: return 0;
  }
}

static int check_gemm_shape(const peqa_qweight_t* w, int T) {
  if (T <= 0) return PEQA_ERR_BAD_SHAPE;
  if (w->in_features % 64 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  return PEQA_OK;
}

extern "C" int peqa_qlinear_fwd(const peqa_qweight_t* w, const void* X, int T, void* Y,
                                void* workspace, size_t workspace_bytes, void* stream) {
  (void)workspace; (void)workspace_bytes;
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!X || !Y) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(X) || !aligned16(Y)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  return launch_fwd(w, g, X, T, Y, as_stream(stream));
}

extern "C" int peqa_qlinear_bwd(const peqa_qweight_t* w, const void* X, const void* dY, int T,
                                void* dX, float* dS, void* workspace, size_t workspace_bytes,
                                void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!dY) return PEQA_ERR_NULL;
  if (dS && !X) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(dY) || (X && !aligned16(X)) || (dX && !aligned16(dX)) || (dS && !aligned16(dS)))
    return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  if (dS) {
    const size_t need = ds_workspace_bytes(w, g, T);
    if (need > 0) {
      if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
      if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
    }
  }
  if (dX) PEQA_TRY(launch_dx(w, g, dY, T, dX, as_stream(stream)));
  if (dS) PEQA_TRY(launch_ds(w, g, X, dY, T, dS, nullptr, nullptr, workspace, workspace_bytes, as_stream(stream)));
  return PEQA_OK;
}

extern "C" int peqa_qlinear_bwd_ds_adamw(const peqa_qweight_t* w, const void* X, const void* dY,
                                         int T, float* dS, float* m, float* v, float lr,
                                         float beta1, float beta2, float eps, float weight_decay,
                                         int64_t step, void* workspace, size_t workspace_bytes,
                                         void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!X || !dY || !dS || !m || !v) return PEQA_ERR_NULL;
  if (step < 1) return PEQA_ERR_BAD_SHAPE;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(X) || !aligned16(dY) || !aligned16(dS)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const size_t need = ds_workspace_bytes(w, g, T);
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  }
  DsAdam adam;
  adam.c = adamw_consts(lr, beta1, beta2, eps, weight_decay, (long long)step);
  adam.scales = const_cast<float*>(w->scales);
  adam.m = m;
  adam.v = v;
  return launch_ds(w, g, X, dY, T, dS, nullptr, &adam, workspace, workspace_bytes, as_stream(stream));
}

extern "C" int peqa_qlinear_bwd_dsdz(const peqa_qweight_t* w, const void* X, const void* dY, int T,
                                     float* dS, float* dZ, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!X || !dY || !dS || !dZ) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(X) || !aligned16(dY) || !aligned16(dS) || !aligned16(dZ)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const size_t need = dsdz_workspace_bytes(w, g, T);
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  }
  return launch_ds(w, g, X, dY, T, dS, dZ, nullptr, workspace, workspace_bytes, as_stream(stream));
}

extern "C" int peqa_qlinear_bwd_ds_from_y(const peqa_qweight_t* w, const void* dY, const void* Y,
                                          int T, float* dS, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!dY || !Y || !dS) return PEQA_ERR_NULL;
  if (G != 1) return PEQA_ERR_BAD_SHAPE;          // the identity holds for one scale per channel only
  if (T <= 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(dY) || !aligned16(Y) || !aligned16(dS)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const size_t need = ds_from_y_workspace_bytes(w, T);
  if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  return launch_ds_from_y(w, dY, Y, T, dS, workspace, as_stream(stream));
}

extern "C" int peqa_qlinear_decode(const peqa_qweight_t* w, const void* X, int M, void* Y,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!X || !Y) return PEQA_ERR_NULL;
  if (M < 1 || M > 16) return PEQA_ERR_BAD_SHAPE;
  if (w->in_features % 128 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(X) || !aligned16(Y)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const size_t need = decode_workspace_bytes(w, g, M);
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  }
  return launch_decode(w, g, X, M, Y, workspace, workspace_bytes, as_stream(stream));
}

extern "C" int peqa_qlinear_decode_multitask(const peqa_qweight_t* w, const float* scale_table,
                                             int n_tasks, const int32_t* task_ids, const void* X,
                                             int M, void* Y, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!scale_table || !task_ids || !X || !Y) return PEQA_ERR_NULL;
  if (M < 1 || M > 16 || n_tasks < 1) return PEQA_ERR_BAD_SHAPE;
  if (G != 1) return PEQA_ERR_BAD_SHAPE;          // task-specific scales are per channel here
  if (w->in_features % 128 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(X) || !aligned16(Y) || !aligned16(scale_table)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  if (!decode_stream_supported(w, g, M)) return PEQA_ERR_BAD_SHAPE;
  return launch_decode_stream(w, g, X, M, Y, scale_table, n_tasks, task_ids, as_stream(stream));
}

namespace {

// Two auxiliary streams and a pool of events per device for peqa_train_step_host, made on
// the first call on that device and kept until the process ends.
constexpr int kHostChunksMax = 8;
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, out_done = nullptr;
  cudaEvent_t x_landed[kHostChunksMax] = {};
  cudaEvent_t dy_landed[kHostChunksMax] = {};
  cudaEvent_t fwd_done[kHostChunksMax] = {};
  cudaEvent_t dx_done[kHostChunksMax] = {};
  bool ready = false;
};

int host_pipe(HostPipe** out) {
  static HostPipe pipes[64];
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return PEQA_ERR_BAD_SHAPE;
  HostPipe& hp = pipes[dev];
  if (!hp.ready) {
    PEQA_CUDA(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
    PEQA_CUDA(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
    PEQA_CUDA(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
    PEQA_CUDA(cudaEventCreateWithFlags(&hp.out_done, cudaEventDisableTiming));
    for (int c = 0; c < kHostChunksMax; ++c) {
      PEQA_CUDA(cudaEventCreateWithFlags(&hp.x_landed[c], cudaEventDisableTiming));
      PEQA_CUDA(cudaEventCreateWithFlags(&hp.dy_landed[c], cudaEventDisableTiming));
      PEQA_CUDA(cudaEventCreateWithFlags(&hp.fwd_done[c], cudaEventDisableTiming));
      PEQA_CUDA(cudaEventCreateWithFlags(&hp.dx_done[c], cudaEventDisableTiming));
    }
    hp.ready = true;
  }
  *out = &hp;
  return PEQA_OK;
}

}  // namespace

// The tokens go through in chunks so that the three engines overlap: chunk c+1 is on its
// way to the device (auxiliary stream `in`) while chunk c runs forward and dX on the
// caller's stream and chunk c-1 returns Y and dX (auxiliary stream `out`); PCIe carries both
// directions at once.  dS sums over all tokens, so it runs once after the last chunk, then
// AdamW.  Forward and dX treat tokens independently, so chunking does not change a bit of
// their results.
extern "C" int peqa_train_step_host(const peqa_qweight_t* w, int T,
                                    const void* h_X, const void* h_dY,
                                    void* h_Y, void* h_dX, float* h_dS,
                                    void* d_X, void* d_dY, void* d_Y, void* d_dX, float* d_dS,
                                    float* d_m, float* d_v,
                                    float lr, float beta1, float beta2, float eps,
                                    float weight_decay, int64_t step,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!h_X || !h_dY || !h_Y || !h_dX || !h_dS || !d_X || !d_dY || !d_Y || !d_dX || !d_dS ||
      !d_m || !d_v)
    return PEQA_ERR_NULL;
  if (T <= 0) return PEQA_ERR_BAD_SHAPE;
  PEQA_TRY(check_gemm_shape(w, T));
  cudaStream_t st = as_stream(stream);
  const size_t N = w->out_features, K = w->in_features;
  // chunks of whole 512-token tiles, at most kHostChunksMax of them
  int chunks = (T + 511) / 512;
  if (chunks > kHostChunksMax) chunks = kHostChunksMax;
  const int per = ((T + chunks - 1) / chunks + 7) & ~7;   // rows per chunk, 16-byte aligned slices
  chunks = (T + per - 1) / per;
  HostPipe* hp = nullptr;
  PEQA_TRY(host_pipe(&hp));
  const char* hX = static_cast<const char*>(h_X);
  const char* hdY = static_cast<const char*>(h_dY);
  char* hY = static_cast<char*>(h_Y);
  char* hdX = static_cast<char*>(h_dX);
  char* dX_in = static_cast<char*>(d_X);
  char* ddY = static_cast<char*>(d_dY);
  char* dY_out = static_cast<char*>(d_Y);
  char* ddX = static_cast<char*>(d_dX);
  // the auxiliary streams start after whatever the caller's stream already holds
  PEQA_CUDA(cudaEventRecord(hp->start, st));
  PEQA_CUDA(cudaStreamWaitEvent(hp->in, hp->start, 0));
  PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->start, 0));
  for (int c = 0; c < chunks; ++c) {
    const size_t t0 = (size_t)c * per;
    const size_t tc = (size_t)T - t0 < (size_t)per ? (size_t)T - t0 : (size_t)per;
    PEQA_CUDA(cudaMemcpyAsync(dX_in + t0 * K * 2, hX + t0 * K * 2, tc * K * 2, cudaMemcpyHostToDevice, hp->in));
    PEQA_CUDA(cudaEventRecord(hp->x_landed[c], hp->in));
    PEQA_CUDA(cudaMemcpyAsync(ddY + t0 * N * 2, hdY + t0 * N * 2, tc * N * 2, cudaMemcpyHostToDevice, hp->in));
    PEQA_CUDA(cudaEventRecord(hp->dy_landed[c], hp->in));
    // the forward needs only X: it runs while dY is still on its way
    PEQA_CUDA(cudaStreamWaitEvent(st, hp->x_landed[c], 0));
    PEQA_TRY(peqa_qlinear_fwd(w, dX_in + t0 * K * 2, (int)tc, dY_out + t0 * N * 2, workspace,
                              workspace_bytes, stream));
    PEQA_CUDA(cudaEventRecord(hp->fwd_done[c], st));
    PEQA_CUDA(cudaStreamWaitEvent(st, hp->dy_landed[c], 0));
    PEQA_TRY(peqa_qlinear_bwd(w, nullptr, ddY + t0 * N * 2, (int)tc, ddX + t0 * K * 2, nullptr,
                              workspace, workspace_bytes, stream));
    PEQA_CUDA(cudaEventRecord(hp->dx_done[c], st));
    // Y goes back while dX is still being computed
    PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->fwd_done[c], 0));
    PEQA_CUDA(cudaMemcpyAsync(hY + t0 * N * 2, dY_out + t0 * N * 2, tc * N * 2, cudaMemcpyDeviceToHost, hp->out));
    PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->dx_done[c], 0));
    PEQA_CUDA(cudaMemcpyAsync(hdX + t0 * K * 2, ddX + t0 * K * 2, tc * K * 2, cudaMemcpyDeviceToHost, hp->out));
  }
  PEQA_CUDA(cudaEventRecord(hp->out_done, hp->out));
  PEQA_TRY(peqa_qlinear_bwd_ds_adamw(w, d_X, d_dY, T, d_dS, d_m, d_v, lr, beta1, beta2, eps,
                                     weight_decay, step, workspace, workspace_bytes, stream));
  PEQA_CUDA(cudaMemcpyAsync(h_dS, d_dS, N * (size_t)G * 4, cudaMemcpyDeviceToHost, st));
  PEQA_CUDA(cudaStreamWaitEvent(st, hp->out_done, 0));
  PEQA_CUDA(cudaStreamSynchronize(st));
  return PEQA_OK;
}

extern "C" int peqa_check_status(void* stream) {
  int* dev = nullptr;
  PEQA_TRY(status_word(&dev));
  int host[4] = {0, 0, 0, 0};
  cudaStream_t st = as_stream(stream);
  PEQA_CUDA(cudaMemcpyAsync(host, dev, sizeof(host), cudaMemcpyDeviceToHost, st));
  PEQA_CUDA(cudaStreamSynchronize(st));
  if (host[0] != 0) {
    PEQA_CUDA(cudaMemsetAsync(dev, 0, sizeof(host), st));
    PEQA_CUDA(cudaStreamSynchronize(st));
    return PEQA_ERR_DEVICE_TIMEOUT;
  }
  return PEQA_OK;
}
