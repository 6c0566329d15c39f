// C-ABI entry points that only validate and dispatch, plus the library's
// small amount of per-device state (architecture check, status word).
#include <mutex>

#include "common.cuh"
#include "tensor_map.cuh"

namespace peqa {

thread_local int g_last_cuda_error = 0;

// Written by kernels whose bounded waits expire; one slot per stream (see common.cuh).
__device__ int g_status_slots[kStatusSlots][kStatusInts];

namespace {

constexpr int kMaxDevices = 64;
constexpr int kDefaultWaitLimitUs = 2000000;   // 2 s
struct DeviceStatus {
  int* base = nullptr;                 // device address of g_status_slots
  cudaStream_t keys[kStatusSlots] = {};
  int used = 0;
  int wait_limit_us = kDefaultWaitLimitUs;
  int selftest_knob = 0;
};
std::mutex g_status_mutex;
DeviceStatus g_device_status[kMaxDevices];

int write_all_slots(const DeviceStatus& ds) {
  int host[kStatusSlots][kStatusInts] = {};
  for (int q = 0; q < kStatusSlots; ++q) {
    host[q][4] = ds.wait_limit_us;
    host[q][5] = ds.selftest_knob;
  }
  PEQA_CUDA(cudaMemcpy(ds.base, host, sizeof(host), cudaMemcpyHostToDevice));
  return PEQA_OK;
}

// Caller holds g_status_mutex.
int device_status(DeviceStatus** out) {
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PEQA_ERR_TOO_LARGE;
  DeviceStatus& ds = g_device_status[dev];
  if (!ds.base) {
    void* p = nullptr;
    PEQA_CUDA(cudaGetSymbolAddress(&p, g_status_slots));
    ds.base = static_cast<int*>(p);
    const int rc = write_all_slots(ds);
    if (rc != PEQA_OK) {
      ds.base = nullptr;
      return rc;
    }
  }
  *out = &ds;
  return PEQA_OK;
}

}  // namespace

int status_word(cudaStream_t st, int** dev_ptr) {
  std::lock_guard<std::mutex> lock(g_status_mutex);
  DeviceStatus* ds = nullptr;
  PEQA_TRY(device_status(&ds));
  int slot = -1;
  for (int q = 0; q < ds->used; ++q)
    if (ds->keys[q] == st) slot = q;
  if (slot < 0) {
    if (ds->used < kStatusSlots - 1) {
      slot = ds->used++;
      ds->keys[slot] = st;
    } else {
      slot = kStatusSlots - 1;       // shared by every further stream
    }
  }
  *dev_ptr = ds->base + slot * kStatusInts;
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

int tensor_map_encoder(EncodeTiledFn* out) {
  static std::mutex mu;
  static EncodeTiledFn cached = nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cached) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    PEQA_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorUnknown);
    cached = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = cached;
  return PEQA_OK;
}

int sm_count_or(int fallback) {
  static thread_local int cached_dev = -1;
  static thread_local int cached_sms = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return fallback;
  if (dev != cached_dev) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      return fallback;
    cached_dev = dev;
    cached_sms = sms;
  }
  return cached_sms;
}

int check_qweight(const peqa_qweight_t* w, int* g, int* G, bool zeros_optional) {
  if (!w) return PEQA_ERR_NULL;
  if (!w->qweight || (!w->zeros && !zeros_optional) || !w->scales) return PEQA_ERR_NULL;
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
  return launch_fwd(w, nullptr, g, X, T, Y, as_stream(stream));
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
  if (dX) PEQA_TRY(launch_dx(w, nullptr, g, dY, T, dX, as_stream(stream)));
  if (dS) PEQA_TRY(launch_ds(w, nullptr, g, X, dY, T, dS, nullptr, nullptr, workspace, workspace_bytes, as_stream(stream)));
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
  return launch_ds(w, nullptr, g, X, dY, T, dS, nullptr, &adam, workspace, workspace_bytes, as_stream(stream));
}

// Checks of one linear of a layer step; fills the workspace need of its dS pass.
static int check_layer_linear(const peqa_layer_linear_t* L, int T, int apply_adamw, int* g_out) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(&L->w, &g, &G));
  if (!L->X_bf16 || !L->dY_bf16 || !L->Y_bf16 || !L->dX_bf16 || !L->dS) return PEQA_ERR_NULL;
  if (apply_adamw && (!L->m || !L->v)) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(&L->w, T));
  if (!aligned16(L->X_bf16) || !aligned16(L->dY_bf16) || !aligned16(L->Y_bf16) || !aligned16(L->dX_bf16) || !aligned16(L->dS))
    return PEQA_ERR_ALIGNMENT;
  const size_t need = ds_workspace_bytes(&L->w, g, T);
  if (need > 0) {
    if (!L->workspace || L->workspace_bytes < need) return PEQA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(L->workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  }
  *g_out = g;
  return PEQA_OK;
}

extern "C" int peqa_layer_train_step(const peqa_layer_linear_t* linears, int n_linears, int T,
                                     int apply_adamw, float lr, float beta1, float beta2, float eps,
                                     float weight_decay, int64_t step, void* stream) {
  if (!linears) return PEQA_ERR_NULL;
  if (n_linears < 1 || n_linears > PEQA_LAYER_MAX_LINEARS) return PEQA_ERR_BAD_SHAPE;
  if (apply_adamw && step < 1) return PEQA_ERR_BAD_SHAPE;
  int g[PEQA_LAYER_MAX_LINEARS];
  for (int i = 0; i < n_linears; ++i) PEQA_TRY(check_layer_linear(&linears[i], T, apply_adamw, &g[i]));
  PEQA_TRY(check_arch());
  cudaStream_t st = as_stream(stream);
  DsAdam adam;
  adam.c = adamw_consts(lr, beta1, beta2, eps, weight_decay, (long long)(apply_adamw ? step : 1));
  for (int i = 0; i < n_linears; ++i) {
    const peqa_layer_linear_t* L = &linears[i];
    PEQA_TRY(launch_fwd(&L->w, nullptr, g[i], L->X_bf16, T, L->Y_bf16, st));
    PEQA_TRY(launch_dx(&L->w, nullptr, g[i], L->dY_bf16, T, L->dX_bf16, st));
    adam.scales = const_cast<float*>(L->w.scales);
    adam.m = L->m;
    adam.v = L->v;
    PEQA_TRY(launch_ds(&L->w, nullptr, g[i], L->X_bf16, L->dY_bf16, T, L->dS, nullptr, apply_adamw ? &adam : nullptr,
                       L->workspace, L->workspace_bytes, st));
  }
  return PEQA_OK;
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
  return launch_ds(w, nullptr, g, X, dY, T, dS, dZ, nullptr, workspace, workspace_bytes, as_stream(stream));
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

extern "C" int peqa_qlinear_fwd_zf(const peqa_qweight_t* w, const float* zeros_f, const void* X,
                                   int T, void* Y, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G, true));
  if (!zeros_f || !X || !Y) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(X) || !aligned16(Y)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  return launch_fwd(w, zeros_f, g, X, T, Y, as_stream(stream));
}

extern "C" int peqa_qlinear_bwd_zf(const peqa_qweight_t* w, const float* zeros_f, const void* X,
                                   const void* dY, int T, void* dX, float* dS, float* dZ,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G, true));
  if (!zeros_f || !dY) return PEQA_ERR_NULL;
  if ((dS == nullptr) != (dZ == nullptr)) return PEQA_ERR_NULL;   // both gradients or neither
  if (dS && !X) return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(w, T));
  if (!aligned16(dY) || (X && !aligned16(X)) || (dX && !aligned16(dX)) || (dS && !aligned16(dS)) ||
      (dZ && !aligned16(dZ)))
    return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  if (dS) {
    const size_t need = dsdz_workspace_bytes(w, g, T);
    if (need > 0) {
      if (!workspace || workspace_bytes < need) return PEQA_ERR_WORKSPACE;
      if (reinterpret_cast<uintptr_t>(workspace) & 255u) return PEQA_ERR_ALIGNMENT;
    }
  }
  if (dX) PEQA_TRY(launch_dx(w, zeros_f, g, dY, T, dX, as_stream(stream)));
  if (dS) PEQA_TRY(launch_ds(w, zeros_f, g, X, dY, T, dS, dZ, nullptr, workspace, workspace_bytes, as_stream(stream)));
  return PEQA_OK;
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
  cudaEvent_t start = nullptr, out_done = nullptr, ds_done = nullptr;
  cudaEvent_t x_landed[kHostChunksMax] = {};
  cudaEvent_t dy_landed[kHostChunksMax] = {};
  cudaEvent_t fwd_done[kHostChunksMax] = {};
  cudaEvent_t dx_done[kHostChunksMax] = {};
  bool ready = false;
};

std::mutex g_pipe_mutex[64];

// Caller holds the device's g_pipe_mutex.  A partly created pipe is torn down again, so a
// later call starts from scratch instead of leaking.
int host_pipe(int dev, HostPipe** out) {
  static HostPipe pipes[64];
  HostPipe& hp = pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.out_done, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.ds_done, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; ok && c < kHostChunksMax; ++c)
      ok = cudaEventCreateWithFlags(&hp.x_landed[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.dy_landed[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.fwd_done[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.dx_done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      const cudaError_t e = cudaGetLastError();
      if (hp.in) cudaStreamDestroy(hp.in);
      if (hp.out) cudaStreamDestroy(hp.out);
      if (hp.start) cudaEventDestroy(hp.start);
      if (hp.out_done) cudaEventDestroy(hp.out_done);
      if (hp.ds_done) cudaEventDestroy(hp.ds_done);
      for (int c = 0; c < kHostChunksMax; ++c) {
        if (hp.x_landed[c]) cudaEventDestroy(hp.x_landed[c]);
        if (hp.dy_landed[c]) cudaEventDestroy(hp.dy_landed[c]);
        if (hp.fwd_done[c]) cudaEventDestroy(hp.fwd_done[c]);
        if (hp.dx_done[c]) cudaEventDestroy(hp.dx_done[c]);
      }
      hp = HostPipe();
      return cuda_fail(e == cudaSuccess ? cudaErrorUnknown : e);
    }
    hp.ready = true;
  }
  *out = &hp;
  return PEQA_OK;
}

// Everything that can still fail once work is enqueued has been checked before; if a CUDA
// call fails all the same, the three streams are drained before the error is returned, so no
// copy into the caller's host buffers is left in flight.
int drain_and_fail(HostPipe* hp, cudaStream_t st, int rc) {
  cudaStreamSynchronize(hp->in);
  cudaStreamSynchronize(hp->out);
  cudaStreamSynchronize(st);
  return rc;
}

// The tokens go through in chunks so that the three engines overlap: chunk c+1 is on its
// way to the device (auxiliary stream `in`) while chunk c runs forward and dX on the
// caller's stream and chunk c-1 returns Y and dX (auxiliary stream `out`); PCIe carries both
// directions at once.  dS sums over all tokens, so it runs once after the last chunk, then
// AdamW.  Forward and dX treat tokens independently, so chunking does not change a bit of
// their results.  With several linears the copies in of the next linear run while the
// kernels of the current one are still busy.

// Host-side checks of one linear of a host-buffer step; nothing is enqueued.
int check_host_linear(const peqa_layer_host_linear_t& L, int T) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(&L.w, &g, &G));
  if (!L.h_X || !L.h_dY || !L.h_Y || !L.h_dX || !L.h_dS || !L.d_X || !L.d_dY || !L.d_Y || !L.d_dX ||
      !L.d_dS || !L.d_m || !L.d_v)
    return PEQA_ERR_NULL;
  PEQA_TRY(check_gemm_shape(&L.w, T));
  if (!aligned16(L.d_X) || !aligned16(L.d_dY) || !aligned16(L.d_Y) || !aligned16(L.d_dX) || !aligned16(L.d_dS))
    return PEQA_ERR_ALIGNMENT;
  const size_t need = ds_workspace_bytes(&L.w, g, T);
  if (need > 0) {
    if (!L.workspace || L.workspace_bytes < need) return PEQA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(L.workspace) & 255u) return PEQA_ERR_ALIGNMENT;
  }
  return PEQA_OK;
}

// Enqueues one linear of a host-buffer step: its tokens travel in chunks, copies in on hp->in,
// kernels on st, copies out on hp->out.  The caller has checked
// every argument, holds the device's pipe mutex and has made hp->in and hp->out wait for
// whatever must precede the first copy.
int enqueue_host_linear(HostPipe* hp, cudaStream_t st, const peqa_layer_host_linear_t& L, int T,
                        float lr, float beta1, float beta2, float eps, float weight_decay,
                        int64_t step) {
  const peqa_qweight_t* w = &L.w;
  const size_t N = w->out_features, K = w->in_features;
  const size_t G = w->group_size == 0 ? 1 : K / (size_t)w->group_size;
  // chunks of 256 tokens or more, at most kHostChunksMax: short chunks shorten the time before
  // the first kernel can start and after the last one has ended, which is all copy time
  int chunks = (T + 255) / 256;
  if (chunks > kHostChunksMax) chunks = kHostChunksMax;
  const int per = ((T + chunks - 1) / chunks + 7) & ~7;   // rows per chunk, 16-byte aligned slices
  chunks = (T + per - 1) / per;
  const char* hX = static_cast<const char*>(L.h_X);
  const char* hdY = static_cast<const char*>(L.h_dY);
  char* hY = static_cast<char*>(L.h_Y);
  char* hdX = static_cast<char*>(L.h_dX);
  char* dX_in = static_cast<char*>(L.d_X);
  char* ddY = static_cast<char*>(L.d_dY);
  char* dY_out = static_cast<char*>(L.d_Y);
  char* ddX = static_cast<char*>(L.d_dX);
  void* stream = static_cast<void*>(st);
  for (int c = 0; c < chunks; ++c) {
    const size_t t0 = (size_t)c * per;
    const size_t tc = (size_t)T - t0 < (size_t)per ? (size_t)T - t0 : (size_t)per;
    PEQA_CUDA(cudaMemcpyAsync(dX_in + t0 * K * 2, hX + t0 * K * 2, tc * K * 2, cudaMemcpyHostToDevice, hp->in));
    PEQA_CUDA(cudaEventRecord(hp->x_landed[c], hp->in));
    PEQA_CUDA(cudaMemcpyAsync(ddY + t0 * N * 2, hdY + t0 * N * 2, tc * N * 2, cudaMemcpyHostToDevice, hp->in));
    PEQA_CUDA(cudaEventRecord(hp->dy_landed[c], hp->in));
    // the forward needs only X: it runs while dY is still on its way
    PEQA_CUDA(cudaStreamWaitEvent(st, hp->x_landed[c], 0));
    PEQA_TRY(peqa_qlinear_fwd(w, dX_in + t0 * K * 2, (int)tc, dY_out + t0 * N * 2, L.workspace,
                              L.workspace_bytes, stream));
    PEQA_CUDA(cudaEventRecord(hp->fwd_done[c], st));
    PEQA_CUDA(cudaStreamWaitEvent(st, hp->dy_landed[c], 0));
    PEQA_TRY(peqa_qlinear_bwd(w, nullptr, ddY + t0 * N * 2, (int)tc, ddX + t0 * K * 2, nullptr,
                              L.workspace, L.workspace_bytes, stream));
    PEQA_CUDA(cudaEventRecord(hp->dx_done[c], st));
    // Y goes back while dX is still being computed
    PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->fwd_done[c], 0));
    PEQA_CUDA(cudaMemcpyAsync(hY + t0 * N * 2, dY_out + t0 * N * 2, tc * N * 2, cudaMemcpyDeviceToHost, hp->out));
    PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->dx_done[c], 0));
    PEQA_CUDA(cudaMemcpyAsync(hdX + t0 * K * 2, ddX + t0 * K * 2, tc * K * 2, cudaMemcpyDeviceToHost, hp->out));
  }
  PEQA_TRY(peqa_qlinear_bwd_ds_adamw(w, L.d_X, L.d_dY, T, L.d_dS, L.d_m, L.d_v, lr, beta1, beta2, eps,
                                     weight_decay, step, L.workspace, L.workspace_bytes, stream));
  // dS follows on the copy-out stream, so that the next linear's kernels do not wait for it
  PEQA_CUDA(cudaEventRecord(hp->ds_done, st));
  PEQA_CUDA(cudaStreamWaitEvent(hp->out, hp->ds_done, 0));
  PEQA_CUDA(cudaMemcpyAsync(L.h_dS, L.d_dS, N * G * 4, cudaMemcpyDeviceToHost, hp->out));
  return PEQA_OK;
}

bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + nb && y < x + na;
}

}  // namespace

extern "C" int peqa_layer_train_step_host(const peqa_layer_host_linear_t* linears, int n_linears, int T,
                                          float lr, float beta1, float beta2, float eps,
                                          float weight_decay, int64_t step, void* stream) {
  if (!linears) return PEQA_ERR_NULL;
  if (n_linears < 1 || n_linears > PEQA_LAYER_MAX_LINEARS || T <= 0 || step < 1) return PEQA_ERR_BAD_SHAPE;
  // every check of every linear before anything is enqueued
  for (int i = 0; i < n_linears; ++i) PEQA_TRY(check_host_linear(linears[i], T));
  // the copies of a linear run ahead of the kernels of the linears before it: the device
  // staging buffers they write must not be buffers an earlier linear still reads
  for (int i = 0; i < n_linears; ++i) {
    const size_t xi = (size_t)T * linears[i].w.in_features * 2, yi = (size_t)T * linears[i].w.out_features * 2;
    for (int j = 0; j < i; ++j) {
      const size_t xj = (size_t)T * linears[j].w.in_features * 2, yj = (size_t)T * linears[j].w.out_features * 2;
      const void* bi[4] = {linears[i].d_X, linears[i].d_dY, linears[i].d_Y, linears[i].d_dX};
      const size_t ni[4] = {xi, yi, yi, xi};
      const void* bj[4] = {linears[j].d_X, linears[j].d_dY, linears[j].d_Y, linears[j].d_dX};
      const size_t nj[4] = {xj, yj, yj, xj};
      for (int a = 0; a < 4; ++a)
        for (int b = 0; b < 4; ++b)
          if (ranges_overlap(bi[a], ni[a], bj[b], nj[b])) return PEQA_ERR_BAD_SHAPE;
    }
  }
  PEQA_TRY(check_arch());
  cudaStream_t st = as_stream(stream);
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return PEQA_ERR_TOO_LARGE;
  // the auxiliary streams and events are shared by all calls on the device: one call at a time
  std::lock_guard<std::mutex> lock(g_pipe_mutex[dev]);
  HostPipe* hp = nullptr;
  PEQA_TRY(host_pipe(dev, &hp));
  // the auxiliary streams start after whatever the caller's stream already holds
  cudaError_t e = cudaEventRecord(hp->start, st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hp->in, hp->start, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hp->out, hp->start, 0);
  if (e != cudaSuccess) return drain_and_fail(hp, st, cuda_fail(e));
  for (int i = 0; i < n_linears; ++i) {
    const int rc = enqueue_host_linear(hp, st, linears[i], T, lr, beta1, beta2, eps, weight_decay, step);
    if (rc != PEQA_OK) return drain_and_fail(hp, st, rc);
  }
  e = cudaEventRecord(hp->out_done, hp->out);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, hp->out_done, 0);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return drain_and_fail(hp, st, cuda_fail(e));
  return PEQA_OK;
}

extern "C" int peqa_train_step_host(const peqa_qweight_t* w, int T,
                                    const void* h_X, const void* h_dY,
                                    void* h_Y, void* h_dX, float* h_dS,
                                    void* d_X, void* d_dY, void* d_Y, void* d_dX, float* d_dS,
                                    float* d_m, float* d_v,
                                    float lr, float beta1, float beta2, float eps,
                                    float weight_decay, int64_t step,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  if (!w) return PEQA_ERR_NULL;
  peqa_layer_host_linear_t L = {};
  L.w = *w;
  L.h_X = h_X; L.h_dY = h_dY; L.h_Y = h_Y; L.h_dX = h_dX; L.h_dS = h_dS;
  L.d_X = d_X; L.d_dY = d_dY; L.d_Y = d_Y; L.d_dX = d_dX; L.d_dS = d_dS;
  L.d_m = d_m; L.d_v = d_v;
  L.workspace = workspace; L.workspace_bytes = workspace_bytes;
  return peqa_layer_train_step_host(&L, 1, T, lr, beta1, beta2, eps, weight_decay, step, stream);
}

extern "C" int peqa_check_status(void* stream) {
  cudaStream_t st = as_stream(stream);
  int* dev = nullptr;
  PEQA_TRY(status_word(st, &dev));
  int host[4] = {0, 0, 0, 0};
  PEQA_CUDA(cudaMemcpyAsync(host, dev, sizeof(host), cudaMemcpyDeviceToHost, st));
  PEQA_CUDA(cudaStreamSynchronize(st));
  if (host[0] != 0) {
    PEQA_CUDA(cudaMemsetAsync(dev, 0, sizeof(host), st));
    PEQA_CUDA(cudaStreamSynchronize(st));
    return PEQA_ERR_DEVICE_TIMEOUT;
  }
  return PEQA_OK;
}

extern "C" int peqa_selftest_configure(int wait_limit_us, int starve_forward) {
  if (wait_limit_us < 0) return PEQA_ERR_BAD_SHAPE;
  std::lock_guard<std::mutex> lock(g_status_mutex);
  DeviceStatus* ds = nullptr;
  PEQA_TRY(device_status(&ds));
  PEQA_CUDA(cudaDeviceSynchronize());
  ds->wait_limit_us = wait_limit_us == 0 ? kDefaultWaitLimitUs : wait_limit_us;
  ds->selftest_knob = starve_forward ? 1 : 0;
  // the status codes of all slots are cleared along with the knobs
  return write_all_slots(*ds);
}
