// Shared host-side helpers of the PEQA sm_100a library: argument checks,
// CUDA error capture and the device status word.
#pragma once

#include <math.h>

#include <cuda_runtime.h>
#include <stdint.h>

#include "peqa.h"

namespace peqa {

extern thread_local int g_last_cuda_error;

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return PEQA_ERR_CUDA;
}

#define PEQA_CUDA(expr)                                   \
  do {                                                    \
    cudaError_t _e = (expr);                              \
    if (_e != cudaSuccess) return ::peqa::cuda_fail(_e);  \
  } while (0)

#define PEQA_TRY(expr)              \
  do {                              \
    int _s = (expr);                \
    if (_s != PEQA_OK) return _s;   \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Effective group size (per-channel when 0 or K) or 0 when invalid.
inline int effective_group(int K, int group_size) {
  if (group_size == 0 || group_size == K) return K;
  if (group_size < 0 || group_size % 32 != 0 || K % group_size != 0) return 0;
  return group_size;
}

inline int check_bits_shape(int N, int K, int bits, int group_size) {
  if (bits != 3 && bits != 4) return PEQA_ERR_BAD_BITS;
  if (N <= 0 || K <= 0 || K % 32 != 0) return PEQA_ERR_BAD_SHAPE;
  if (effective_group(K, group_size) == 0) return PEQA_ERR_BAD_SHAPE;
  return PEQA_OK;
}

// Validates a layer descriptor; fills g (effective group) and G.  With zeros_optional the
// integer zero-points may be absent (entry points that take real-valued ones).
int check_qweight(const peqa_qweight_t* w, int* g, int* G, bool zeros_optional = false);

// The current device must be compute capability 10.x (cached per device).
int check_arch();

// Device address of the status slot kernels launched on `st` report to, on the current
// device.  A slot is int[8]: [0] status code, [1..3] where, [4] bound of a single device-side
// wait in microseconds, [5] self-test knob (see peqa_selftest_configure), [6..7] unused.
// Streams get slots of their own (first come, first served; the last slot is shared by any
// further streams).  The first call on a device initialises the table with a blocking copy.
constexpr int kStatusSlots = 32;
constexpr int kStatusInts = 8;
int status_word(cudaStream_t st, int** dev_ptr);

// Multiprocessor count of the current device (cached per device); `fallback` when the query
// fails.
int sm_count_or(int fallback);

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// One AdamW step on a scale (App. A; decoupled decay, bias-corrected moments).  The bias
// corrections 1 - b^t are formed on the host in double and passed as reciprocals, as are
// 1 - b1 and 1 - b2.  Every operation is a single rounded binary32 operation, so the
// stand-alone kernel and the kernels that apply the step where dS is produced agree bit
// for bit.
struct AdamWConsts {
  float lr, b1, b2, omb1, omb2, eps, decay, inv_c1, inv_c2;
};

inline AdamWConsts adamw_consts(float lr, float beta1, float beta2, float eps, float weight_decay,
                                long long step) {
  AdamWConsts c;
  const double c1 = pow((double)beta1, (double)step), c2 = pow((double)beta2, (double)step);
  c.lr = lr;
  c.b1 = beta1;
  c.b2 = beta2;
  c.omb1 = (float)(1.0 - (double)beta1);
  c.omb2 = (float)(1.0 - (double)beta2);
  c.eps = eps;
  c.decay = (float)(1.0 - (double)lr * (double)weight_decay);
  c.inv_c1 = (float)(1.0 / (1.0 - c1));
  c.inv_c2 = (float)(1.0 / (1.0 - c2));
  return c;
}

#ifdef __CUDACC__
__device__ __forceinline__ void adamw_update(float& s, float gr, float& m, float& v,
                                             const AdamWConsts& c) {
  const float mn = __fmaf_rn(c.b1, m, __fmul_rn(c.omb1, gr));
  const float vn = __fmaf_rn(c.b2, v, __fmul_rn(__fmul_rn(c.omb2, gr), gr));
  const float denom = __fadd_rn(sqrtf(__fmul_rn(vn, c.inv_c2)), c.eps);
  s = __fsub_rn(__fmul_rn(s, c.decay), __fdiv_rn(__fmul_rn(c.lr, __fmul_rn(mn, c.inv_c1)), denom));
  m = mn;
  v = vn;
}
#endif

// Work items of the CTA-pair kernels (forward, dX).  A tile is 512 tokens x 256 outputs held as
// two accumulators of 256 tokens.  Tiles are dealt round-robin to the pairs; when the last round
// would keep at most half of the pairs busy, its tiles are cut into two items of 256 tokens each,
// so that round takes about half as long.  Items [0, full_items) are whole tiles, the rest are
// halves: item full_items + 2*i + h is half h of tile full_items + i.
struct PairItems {
  int o_tiles;       // 256-wide tiles along the output dimension
  int full_items;    // items that are whole tiles
  int total_items;
};
inline PairItems make_pair_items(int o_tiles, int t_tiles, int T, int pairs) {
  PairItems it;
  const int tiles = o_tiles * t_tiles;
  it.o_tiles = o_tiles;
  it.full_items = tiles;
  it.total_items = tiles;
  const int rem = pairs > 0 ? tiles % pairs : 0;
  if (T % 512 == 0 && tiles > pairs && rem > 0 && 2 * rem <= pairs) {
    it.full_items = tiles - rem;
    it.total_items = tiles + rem;
  }
  return it;
}
#ifdef __CUDACC__
// Output tile, first token and token blocks (1 or 2) of an item.
__device__ __forceinline__ void pair_item(const PairItems& it, int item, int T, int& o_tile, int& tt0,
                                          int& blocks) {
  int tile = item, half = -1;
  if (item >= it.full_items) {
    const int h = item - it.full_items;
    tile = it.full_items + (h >> 1);
    half = h & 1;
  }
  const int t_tile = tile / it.o_tiles;
  o_tile = tile - t_tile * it.o_tiles;
  tt0 = t_tile * 512;
  if (half >= 0) {
    tt0 += half * 256;
    blocks = 1;
  } else {
    blocks = tt0 + 256 < T ? 2 : 1;
  }
}
#endif

// Entry points implemented in the individual translation units.
// zeros_f != nullptr: real-valued zero-points [N, G] (App. K) replace w->zeros
int launch_fwd(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, int T, void* Y,
               cudaStream_t st);
bool fwd_pair_supported(const peqa_qweight_t* w);
int launch_fwd_pair(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, int T,
                    void* Y, cudaStream_t st);
bool dx_pair_supported(const peqa_qweight_t* w);
int launch_dx_pair(const peqa_qweight_t* w, const float* zeros_f, int g, const void* dY, int T,
                   void* dX, cudaStream_t st);
int launch_dx(const peqa_qweight_t* w, const float* zeros_f, int g, const void* dY, int T, void* dX,
              cudaStream_t st);
// adam != nullptr: the AdamW step on (w->scales, m, v) is applied where dS is produced
struct DsAdam {
  AdamWConsts c;
  float* scales;
  float* m;
  float* v;
};
// zeros_f != nullptr needs dZ: dS is then taken with the real-valued zero-point
int launch_ds(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, const void* dY,
              int T, float* dS, float* dZ, const DsAdam* adam, void* workspace,
              size_t workspace_bytes, cudaStream_t st);
size_t dsdz_workspace_bytes(const peqa_qweight_t* w, int g, int T);
size_t ds_workspace_bytes(const peqa_qweight_t* w, int g, int T);
size_t ds_from_y_workspace_bytes(const peqa_qweight_t* w, int T);
int launch_ds_from_y(const peqa_qweight_t* w, const void* dY, const void* Y, int T, float* dS,
                     void* workspace, cudaStream_t st);
bool decode_stream_supported(const peqa_qweight_t* w, int g, int M);
int launch_decode_stream(const peqa_qweight_t* w, int g, const void* X, int M, void* Y,
                         const float* scale_table, int n_tasks, const int32_t* task_ids,
                         cudaStream_t st);
int launch_decode(const peqa_qweight_t* w, int g, const void* X, int M, void* Y,
                  void* workspace, size_t workspace_bytes, cudaStream_t st);
size_t decode_workspace_bytes(const peqa_qweight_t* w, int g, int M);

}  // namespace peqa
