// Forward of the PEQA layer, Y = X * W_hat^T (Eq. 2), on CTA pairs with the
// dequantised weight operand in tensor memory.
//
// A pair of CTAs (cta_group::2) owns a tile of 256 output channels x 256 tokens.
// CTA `rank` owns channels [r0 + 128*rank, +128): it rebuilds their (Q - z)
// [* bf16(s)] as bf16 and writes them with tcgen05.st into tensor memory, where
// tcgen05.mma reads them as its A operand (lane = channel, one 32-bit column =
// two consecutive contraction elements).  The activation tile is the B operand:
// each CTA TMA-loads 128 of the 256 tokens into its own shared memory and the
// pair's MMAs read both halves.  Only the activations go through shared memory
// at MMA rate: 16 KiB in and 32 KiB out per 64-deep stage, against the 96 KiB a
// single-CTA kernel with both operands in shared memory moves -- and it is that
// shared-memory traffic which bounds the single-CTA kernel.
//
// Packed codes reach the dequant warps through their own TMA ring (one box =
// 128 channels x 64 columns of codes), so the global reads are bulk copies.
// Four groups of four dequant warps take the stages round-robin, so that one
// group's wait -> read -> convert -> store -> signal chain overlaps the others'.
//
// Tensor memory (512 columns): [0,256) fp32 accumulator (256 tokens),
// [256,512) eight weight stages of 32 columns (64 contraction elements).
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"

namespace peqa {

namespace {

using namespace ptx;

constexpr int PM = 128;            // output channels per CTA (TMEM lanes)
constexpr int PN = 256;            // tokens per pair tile (MMA N)
constexpr int PK = 64;             // contraction elements per stage
constexpr int PSTAGES = 8;
constexpr int PB_BYTES = (PN / 2) * PK * 2;          // activation half tile: 16 KiB
constexpr int PQ_BYTES = PM * 32;                    // packed codes of one stage: 128 rows x 8 words
constexpr int P_TMEM_COLS = 512;
constexpr int P_ACC_COL = 0;
constexpr int P_A_COL = 256;
constexpr int P_SMEM_BYTES = PSTAGES * (PB_BYTES + PQ_BYTES) + 1024 + 512;
constexpr int P_GROUPS = 4;        // dequant groups (four warps each)
constexpr int kPairThreads = 896;  // warps: 0 act TMA, 1 MMA, 2 TMEM alloc, 3 code TMA, 4-7 and 24-27 epilogue, 8-23 dequant

struct PairBarriers {
  uint64_t full_a[PSTAGES];     // leader: weight stage written to tensor memory by both CTAs
  uint64_t full_b[PSTAGES];     // leader: activation bytes of both CTAs landed
  uint64_t empty[PSTAGES];      // each CTA: MMAs that read the stage completed
  uint64_t pk_full[PSTAGES];    // each CTA: packed codes landed
  uint64_t pk_empty[PSTAGES];   // each CTA: the group that owns the slot has read it
  uint64_t acc_full;            // each CTA: accumulator ready
  uint64_t acc_empty;           // leader: both CTAs' epilogues drained the accumulator
  uint32_t tmem_base;
  int abort_flag;
};

struct PairParams {
  const uint8_t* zeros;
  const float* scales;
  __nv_bfloat16* out;   // Y [T, N]
  int N, K, G, g, g_shift, T;
  int r_tiles, t_tiles, k_blocks;   // 256-channel tiles, 256-token tiles, 64-deep stages
  int* status;
};

__device__ __forceinline__ int pair_group_of(const PairParams& p, int col) {
  if (p.G == 1) return 0;
  return p.g_shift >= 0 ? (col >> p.g_shift) : (col / p.g);
}

template <int BITS, bool FOLD>
__global__ void __launch_bounds__(kPairThreads, 1)
qfwd_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_q,
                 const PairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* sm_b = base;                                   // PSTAGES x 16 KiB, 128B-swizzled
  uint8_t* sm_q = base + PSTAGES * PB_BYTES;              // PSTAGES x 4 KiB, plain 32-byte rows
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(sm_q + PSTAGES * PQ_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(smem_u32(&bars->full_a[s]), 8);           // 4 warps of one group in each CTA
      mbar_init(smem_u32(&bars->full_b[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
      mbar_init(smem_u32(&bars->pk_full[s]), 1);
      mbar_init(smem_u32(&bars->pk_empty[s]), 4);         // 4 warps of the owning group
    }
    mbar_init(smem_u32(&bars->acc_full), 1);
    mbar_init(smem_u32(&bars->acc_empty), 16);            // 8 epilogue warps in each CTA
    bars->abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_x);
    prefetch_tmap(&tmap_q);
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(&bars->tmem_base), P_TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = p.r_tiles * p.t_tiles;
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;
  const int my_tiles = (total_tiles - pair + n_pairs - 1) / n_pairs;

  if (warp == 0) {
    // ------------------------------------------ activation TMA (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        const int t0 = (tile / p.r_tiles) * PN + (int)rank * (PN / 2);
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_arrive_expect_tx(smem_u32(&bars->full_b[s]), 2 * PB_BYTES);
          tma_load_2d_pair(smem_u32(sm_b + s * PB_BYTES), &tmap_x,
                           mapa_shared(smem_u32(&bars->full_b[s]), 0), kb * PK, t0);
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------ packed-code TMA (one lane)
    // A box is 128 rows x 8 words holding the stage's 64 columns; for 3-bit codes the 6
    // words start 2 words into the box on odd k-blocks, which keeps the box start
    // 16-byte aligned.
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        const int r0 = (tile % p.r_tiles) * (2 * PM) + (int)rank * PM;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int q = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!mbar_wait(smem_u32(&bars->pk_empty[q]), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t bar = smem_u32(&bars->pk_full[q]);
          mbar_arrive_expect_tx(bar, PQ_BYTES);
          tma_load_2d(smem_u32(sm_q + q * PQ_BYTES), &tmap_q, bar,
                      BITS == 3 ? 6 * kb - 2 * (kb & 1) : 8 * kb, r0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------ MMA issuer (leader CTA, one lane)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(2 * PM, PN, 0, 0);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
        if (!mbar_wait_cluster(smem_u32(&bars->acc_empty), (uint32_t)(local & 1) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + P_ACC_COL;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->full_a[s]), ph, abort_flag) ||
              !mbar_wait_cluster(smem_u32(&bars->full_b[s]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t b_addr = smem_u32(sm_b + s * PB_BYTES);
          const uint32_t a_tmem = tmem_base + P_A_COL + s * (PK / 2);
#pragma unroll
          for (int k = 0; k < PK / 16; ++k) {
            const uint64_t bdesc = smem_desc_sw128(b_addr + k * 32, 16, 1024);
            mma_bf16_ts_pair(d_tmem, a_tmem + k * 8, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit_pair(smem_u32(&bars->empty[s]), 3);
        }
        if (ok) mma_commit_pair(smem_u32(&bars->acc_full), 3);
      }
    }
  } else if ((warp >= 4 && warp < 8) || warp >= 24) {
    // ------------------------------------------ epilogue (lane = output channel)
    // Two warps per TMEM lane quarter: warps 4-7 take tokens [0,128) of the tile,
    // warps 24-27 tokens [128,256).
    const int ew = warp & 3;
    const int thalf = warp >= 24 ? 1 : 0;
    const uint32_t acc_empty_leader = mapa_shared(smem_u32(&bars->acc_empty), 0);
    int local = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
      const int r0 = (tile % p.r_tiles) * (2 * PM) + (int)rank * PM;
      const int t0 = (tile / p.r_tiles) * PN;
      if (!mbar_wait_cluster(smem_u32(&bars->acc_full), (uint32_t)(local & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int r = r0 + ew * 32 + lane;
      float scale = 1.0f;
      if (!FOLD && r < p.N) scale = __ldg(p.scales + r);
#pragma unroll 1
      for (int cc = thalf * (PN / 64); cc < (thalf + 1) * (PN / 64); ++cc) {
        const int tc0 = t0 + cc * 32;
        if (tc0 >= p.T) break;
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(ew * 32) << 16) + P_ACC_COL + cc * 32, v);
        tmem_ld_wait();
        if (r < p.N) {
          __nv_bfloat16* dst = p.out + (size_t)tc0 * p.N + r;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (tc0 + j < p.T) dst[(size_t)j * p.N] = __float2bfloat16_rn(__uint_as_float(v[j]) * scale);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
    }
  } else if (warp >= 8 && warp < 24) {
    // ------------------------------------------ weight dequant -> tensor memory
    // Group g (four warps) serves the stages with it % 4 == g.  Warp (w % 4) owns TMEM
    // lanes 32*(w % 4)..+31, so a thread is one output channel; it converts the 64
    // contraction elements of the stage (two units of 32 columns) and stores them as
    // 32 tensor-memory columns.
    const int grp = (warp - 8) >> 2;
    const int q4 = warp & 3;
    const int row = q4 * 32 + lane;
    const uint32_t full_a_leader0 = mapa_shared(smem_u32(&bars->full_a[0]), 0);
    const uint32_t total_it = (uint32_t)my_tiles * (uint32_t)p.k_blocks;
    // cursor of the stage whose (s, z) is being prefetched, walked without divisions
    int pf_tile = pair, pf_kb = grp;
    while (pf_kb >= p.k_blocks) { pf_kb -= p.k_blocks; pf_tile += n_pairs; }
    int pf_r = (pf_tile % p.r_tiles) * (2 * PM) + (int)rank * PM + row;
    auto load_zs = [&](uint32_t (&z)[2], float (&sc)[2]) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        z[u] = 0u;
        sc[u] = 0.0f;
        if (pf_r < p.N) {
          const size_t gi = (size_t)pf_r * p.G + pair_group_of(p, pf_kb * PK + 32 * u);
          z[u] = __ldg(p.zeros + gi);
          if (FOLD) sc[u] = __ldg(p.scales + gi);
        }
      }
      pf_kb += P_GROUPS;
      while (pf_kb >= p.k_blocks) {
        pf_kb -= p.k_blocks;
        pf_tile += n_pairs;
        pf_r = (pf_tile % p.r_tiles) * (2 * PM) + (int)rank * PM + row;
      }
    };
    uint32_t z[2], zn[2];
    float sc[2], scn[2];
    int cur_kb = pf_kb;
    if ((uint32_t)grp < total_it) load_zs(z, sc);
    for (uint32_t it = grp; it < total_it; it += P_GROUPS) {
      const int next_kb = pf_kb;
      if (it + P_GROUPS < total_it) load_zs(zn, scn);
      const int s = it % PSTAGES;
      const uint32_t ph = (it / PSTAGES) & 1u;
      if (!mbar_wait(smem_u32(&bars->pk_full[s]), ph, abort_flag)) break;
      uint32_t w[2][BITS];
      {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(sm_q + s * PQ_BYTES) + row * 8;
        const uint4 lo = *reinterpret_cast<const uint4*>(src);
        const uint4 hi = *reinterpret_cast<const uint4*>(src + 4);
        const uint32_t w8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        if constexpr (BITS == 4) {
#pragma unroll
          for (int e = 0; e < 4; ++e) { w[0][e] = w8[e]; w[1][e] = w8[4 + e]; }
        } else {
          const bool odd = (cur_kb & 1) != 0;
#pragma unroll
          for (int e = 0; e < 3; ++e) {
            w[0][e] = odd ? w8[2 + e] : w8[e];
            w[1][e] = odd ? w8[5 + e] : w8[3 + e];
          }
        }
      }
      uint32_t o[32];
      {
        uint32_t o0[16], o1[16];
        dq::unit32_natural<BITS, FOLD>(w[0], z[0], sc[0], o0);
        dq::unit32_natural<BITS, FOLD>(w[1], z[1], sc[1], o1);
#pragma unroll
        for (int e = 0; e < 16; ++e) { o[e] = o0[e]; o[16 + e] = o1[e]; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->pk_empty[s]));   // codes consumed: slot free
      if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) break;
      tc_fence_after();
      tmem_st_32x32(tmem_base + ((uint32_t)(q4 * 32) << 16) + P_A_COL + s * (PK / 2), o);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(full_a_leader0 + s * 8);
      z[0] = zn[0]; z[1] = zn[1];
      sc[0] = scn[0]; sc[1] = scn[1];
      cur_kb = next_kb;
    }
  }

  if (*abort_flag) {
    // let copies and MMAs already in flight finish before memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, P_TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) {
    atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
    p.status[1] = (int)blockIdx.x;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int encode_fn(EncodeTiledFn* out) {
  static EncodeTiledFn cached = nullptr;
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

template <int BITS, bool FOLD>
int launch_pair_t(const CUtensorMap& tx, const CUtensorMap& tq, const PairParams& p, int pairs,
                  cudaStream_t st) {
  auto kern = qfwd_pair_kernel<BITS, FOLD>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = P_SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, tx, tq, p));
  return PEQA_OK;
}

}  // namespace

// The pair kernel needs a 16-byte row pitch of the packed matrix for its code
// boxes (always true for 4-bit, K % 128 == 0 for 3-bit); other shapes take the
// single-CTA kernel.
bool fwd_pair_supported(const peqa_qweight_t* w) {
  return ((size_t)w->in_features * w->bits / 8) % 16 == 0;
}

int launch_fwd_pair(const peqa_qweight_t* w, int g, const void* X, int T, void* Y, cudaStream_t st) {
  PairParams p;
  p.zeros = w->zeros;
  p.scales = w->scales;
  p.out = static_cast<__nv_bfloat16*>(Y);
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  p.g_shift = -1;
  for (int b = 5; b < 31; ++b)
    if ((1 << b) == g) p.g_shift = b;
  p.T = T;
  p.r_tiles = (p.N + 2 * PM - 1) / (2 * PM);
  p.t_tiles = (T + PN - 1) / PN;
  p.k_blocks = p.K / PK;
  PEQA_TRY(status_word(&p.status));
  EncodeTiledFn enc = nullptr;
  PEQA_TRY(encode_fn(&enc));
  CUtensorMap tx, tq;
  {
    cuuint64_t dims[2] = {(cuuint64_t)p.K, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)p.K * 2};
    cuuint32_t box[2] = {64, PN / 2};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  {
    const int wpr = p.K * w->bits / 32;
    cuuint64_t dims[2] = {(cuuint64_t)wpr, (cuuint64_t)p.N};
    cuuint64_t strides[1] = {(cuuint64_t)wpr * 4};
    cuuint32_t box[2] = {8, PM};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(w->qweight), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int tiles = p.r_tiles * p.t_tiles;
  const int max_pairs = sms / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  const bool fold = p.G > 1;
  if (w->bits == 4)
    return fold ? launch_pair_t<4, true>(tx, tq, p, pairs, st) : launch_pair_t<4, false>(tx, tq, p, pairs, st);
  return fold ? launch_pair_t<3, true>(tx, tq, p, pairs, st) : launch_pair_t<3, false>(tx, tq, p, pairs, st);
}

}  // namespace peqa
