// Backward with respect to the input, dX = dY * W_hat (chain rule on Eq. 2), on
// CTA pairs.
//
// A pair of CTAs (cta_group::2) owns a tile of 512 tokens x 256 input columns j,
// held as two 256 x 256 accumulators that fill tensor memory.  The tokens are
// the MMA "M" side: CTA `rank` TMA-loads two blocks of 128 tokens of dY per
// stage (A operands, K-major: the contraction index i is contiguous in dY) and
// keeps their accumulator rows.  The weights are the "N" side, split between the
// two CTAs: each dequantises the 128 columns [j0 + 128*rank, +128) of the
// stage's 64 weight rows into its own shared memory, MN-major (a row of packed
// codes is unpacked along j, exactly as it is stored), and both token blocks
// multiply the same weight stage.  A weight element is therefore rebuilt once
// per 512 tokens, which brings the conversion work per stage (8192 elements per
// CTA) under the time the tensor cores need for it (two 256x256x64 products);
// and the accumulator is token-major, so an epilogue thread writes contiguous
// runs of dX.
//
// Packed codes come through their own TMA ring (one box = 64 weight rows x the
// CTA's 128 columns); four groups of four dequant warps take the stages
// round-robin.  A tile whose second token block lies wholly beyond T runs with
// one block.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace peqa {

namespace {

using namespace ptx;

constexpr int XK = 64;                       // contraction elements (weight rows i) per stage
constexpr int XSTAGES = 4;
constexpr int XBLK_BYTES = 128 * XK * 2;     // one block of 128 tokens of dY: 16 KiB
constexpr int XA_BYTES = 2 * XBLK_BYTES;     // this CTA's two token blocks
constexpr int XB_BYTES = XK * 128 * 2;       // this CTA's 128 weight columns: 16 KiB
constexpr int XSTAGE_BYTES = XA_BYTES + XB_BYTES;
constexpr int XQ_SLOTS = 4;
constexpr int XE_BYTES = 32 * 64;            // one epilogue warp's staging tile: 32 tokens x 32 columns
constexpr int XQ_BYTES = 4096;               // 64 rows x up to 64 B of codes
constexpr int X_TMEM_COLS = 512;
constexpr int X_SMEM_BYTES = XSTAGES * XSTAGE_BYTES + XQ_SLOTS * XQ_BYTES + 8 * XE_BYTES + 1024 + 512;
constexpr int X_GROUPS = 4;
constexpr int kDxThreads = 896;  // warps: 0 act TMA, 1 MMA, 2 TMEM alloc, 3 code TMA, 4-11 epilogue, 12-27 dequant

struct DxBarriers {
  uint64_t full_act[XSTAGES];   // leader: dY bytes of both CTAs landed
  uint64_t full_w[XSTAGES];     // leader: weight halves of both CTAs written
  uint64_t empty[XSTAGES];      // each CTA: MMAs that read the stage completed
  uint64_t pk_full[XQ_SLOTS];   // each CTA: packed codes landed
  uint64_t pk_empty[XQ_SLOTS];  // each CTA: the owning group has read the slot
  uint64_t acc_full;            // each CTA: both accumulators ready
  uint64_t acc_empty;           // leader: both CTAs' epilogues drained them
  uint32_t tmem_base;
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

struct DxParams {
  const uint8_t* zeros;
  const float* zeros_f;   // real-valued zero-points (App. K) or nullptr; replaces `zeros`
  const float* scales;
  __nv_bfloat16* out;   // dX [T, K]
  int N, K, G, g, g_shift, T;
  int j_tiles, t_tiles, k_blocks;   // 256-column tiles, 512-token tiles, 64-row stages over N
  PairItems items;
  int* status;
};

__device__ __forceinline__ int dx_group_of(const DxParams& p, int col) {
  if (p.G == 1) return 0;
  return p.g_shift >= 0 ? (col >> p.g_shift) : (col / p.g);
}

template <int BITS, bool ZF>
__global__ void __launch_bounds__(kDxThreads, 1)
qdx_pair_kernel(const __grid_constant__ CUtensorMap tmap_dy, const __grid_constant__ CUtensorMap tmap_q,
                const __grid_constant__ CUtensorMap tmap_out,
                const DxParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* sm_q = base + XSTAGES * XSTAGE_BYTES;
  uint8_t* sm_e = sm_q + XQ_SLOTS * XQ_BYTES;             // 8 epilogue warps x 2 KiB, 64-byte swizzle
  DxBarriers* bars = reinterpret_cast<DxBarriers*>(sm_e + 8 * XE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < XSTAGES; ++s) {
      mbar_init(smem_u32(&bars->full_act[s]), 1);
      mbar_init(smem_u32(&bars->full_w[s]), 8);           // 4 warps of one group in each CTA
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int q = 0; q < XQ_SLOTS; ++q) {
      mbar_init(smem_u32(&bars->pk_full[q]), 1);
      mbar_init(smem_u32(&bars->pk_empty[q]), 4);
    }
    mbar_init(smem_u32(&bars->acc_full), 1);
    mbar_init(smem_u32(&bars->acc_empty), 16);            // 8 epilogue warps in each CTA
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    fence_mbar_init();
    prefetch_tmap(&tmap_dy);
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_out);
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(&bars->tmem_base), X_TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  // Set-up is done.  The next kernel of the stream may begin its own (programmatic launch);
  // everything below touches memory that the preceding kernel may still be writing.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = p.items.total_items;      // work items: whole tiles, then halves
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;
  const int my_tiles = (total_tiles - pair + n_pairs - 1) / n_pairs;

  if (warp == 0) {
    // ------------------------------------------ dY TMA (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        int j_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, j_tile, tt0, blocks);
        const int t0 = tt0 + (int)rank * 128;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % XSTAGES;
          const uint32_t ph = (it / XSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_arrive_expect_tx(smem_u32(&bars->full_act[s]), 2 * blocks * XBLK_BYTES);
          const uint32_t bar = mapa_shared(smem_u32(&bars->full_act[s]), 0);
          tma_load_2d_pair(smem_u32(base + s * XSTAGE_BYTES), &tmap_dy, bar, kb * XK, t0);
          if (blocks == 2)
            tma_load_2d_pair(smem_u32(base + s * XSTAGE_BYTES + XBLK_BYTES), &tmap_dy, bar, kb * XK, t0 + 256);
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------ packed-code TMA (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        int j_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, j_tile, tt0, blocks);
        const int w0 = j_tile * 256 + (int)rank * 128;   // first column of this CTA
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int q = it % XQ_SLOTS;
          const uint32_t ph = (it / XQ_SLOTS) & 1u;
          if (!mbar_wait(smem_u32(&bars->pk_empty[q]), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t bar = smem_u32(&bars->pk_full[q]);
          mbar_arrive_expect_tx(bar, 64 * 16 * BITS);
          tma_load_2d(smem_u32(sm_q + q * XQ_BYTES), &tmap_q, bar, (w0 >> 5) * BITS, kb * XK);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------ MMA issuer (leader CTA, one lane)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(256, 256, 0, 1);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
        int j_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, j_tile, tt0, blocks);
        if (!mbar_wait_cluster(smem_u32(&bars->acc_empty), (uint32_t)(local & 1) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % XSTAGES;
          const uint32_t ph = (it / XSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->full_w[s]), ph, abort_flag) ||
              !mbar_wait_cluster(smem_u32(&bars->full_act[s]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(base + s * XSTAGE_BYTES);
          const uint32_t b_addr = a_addr + XA_BYTES;
          for (int m = 0; m < blocks; ++m) {
#pragma unroll
            for (int k = 0; k < XK / 16; ++k) {
              const uint64_t adesc = smem_desc_sw128(a_addr + m * XBLK_BYTES + k * 32, 16, 1024);
              const uint64_t bdesc = smem_desc_sw128(b_addr + k * (16 * 128), 64 * 128, 1024);
              mma_bf16_ss_pair(tmem_base + m * 256, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
            }
          }
          mma_commit_pair(smem_u32(&bars->empty[s]), 3);
        }
        if (ok) mma_commit_pair(smem_u32(&bars->acc_full), 3);
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------------ epilogue: thread = token, 256 columns
    // A warp drains 32 tokens x 32 columns at a time through its 2 KiB staging tile (64-byte
    // swizzle of the output tensor map: 16-byte chunk c of row r at c ^ ((r >> 1) & 3)) and one
    // tiled bulk store, so the copy engine writes whole sectors of dX; the accumulators are
    // released as soon as the last chunk has left tensor memory.
    const int quarter = warp & 3;
    const int m = (warp - 4) >> 2;                 // token block = accumulator
    const uint32_t acc_empty_leader = mapa_shared(smem_u32(&bars->acc_empty), 0);
    uint8_t* stage = sm_e + (warp - 4) * XE_BYTES;
    uint8_t* srow = stage + lane * 64;
    const int sw = (lane >> 1) & 3;
    int local = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
      int j_tile, tt0, blocks;
      pair_item(p.items, tile, p.T, j_tile, tt0, blocks);
      const int j0 = j_tile * 256;
      const int row0 = tt0 + m * 256 + (int)rank * 128 + quarter * 32;   // first token of this warp
      if (!mbar_wait_cluster(smem_u32(&bars->acc_full), (uint32_t)(local & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      int chunks = m < blocks ? (p.K - j0 + 31) / 32 : 0;                // K is a multiple of 32
      chunks = chunks > 8 ? 8 : chunks;
#pragma unroll 1
      for (int cc = 0; cc < chunks; ++cc) {
        const int c0 = j0 + cc * 32;
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + m * 256 + cc * 32, v);
        tmem_ld_wait();
        if (cc + 1 == chunks) {
          // nothing of this tile is left in tensor memory for this warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
        }
        // the previous store must have finished reading the staging tile
        if (lane == 0) bulk_wait_group_read0();
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 o;
          __nv_bfloat162 h;
          h = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])); o.x = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])); o.y = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])); o.z = *reinterpret_cast<uint32_t*>(&h);
          h = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])); o.w = *reinterpret_cast<uint32_t*>(&h);
          *reinterpret_cast<uint4*>(srow + ((q ^ sw) << 4)) = o;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < p.T) {
          tma_store_2d(&tmap_out, smem_u32(stage), c0, row0);
          bulk_commit_group();
        }
      }
      if (chunks == 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
      }
    }
    if (lane == 0) bulk_wait_group0();             // every store has left shared memory and landed
  } else if (warp >= 12) {
    // ------------------------------------------ weight dequant (this CTA's 128 columns)
    // Group g (four warps) serves the stages with it % 4 == g.  A stage is 64 weight rows x
    // 4 units of 32 columns; lanes = 8 rows x 4 units, a thread converts (row, u) and
    // (row + 32, u) and writes them MN-major: chunk (u / 2) of 64 columns, 128 bytes per row.
    const int grp = (warp - 12) >> 2;
    const int gw = (warp - 12) & 3;
    const int row8 = lane & 7, u4 = lane >> 3;
    const int row_a = gw * 8 + row8, row_b = row_a + 32;
    const int chunk0 = (u4 & 1) * 4;
    const int swz = row_a & 7;
    const uint32_t off_a = (uint32_t)((u4 >> 1) * (64 * 128) + row_a * 128);
    const uint32_t off_b = (uint32_t)((u4 >> 1) * (64 * 128) + row_b * 128);
    const uint32_t full_w_leader0 = mapa_shared(smem_u32(&bars->full_w[0]), 0);
    const uint32_t total_it = (uint32_t)my_tiles * (uint32_t)p.k_blocks;
    int pf_tile = pair, pf_kb = grp;
    while (pf_kb >= p.k_blocks) { pf_kb -= p.k_blocks; pf_tile += n_pairs; }
    auto item_col = [&](int item) {
      int j_tile, tt0, blocks;
      pair_item(p.items, item, p.T, j_tile, tt0, blocks);
      return j_tile * 256 + (int)rank * 128 + 32 * u4;
    };
    int pf_col = item_col(pf_tile);
    // cz: the constant term -delta * s of a real-valued zero-point (ZF), else unused
    auto load_zs = [&](uint32_t (&z)[2], float (&sc)[2], float (&cz)[2]) {
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int i = pf_kb * XK + (k ? row_b : row_a);
        z[k] = 0u;
        sc[k] = 0.0f;
        cz[k] = 0.0f;
        if (i < p.N && pf_col < p.K) {
          const size_t gi = (size_t)i * p.G + dx_group_of(p, pf_col);
          sc[k] = __ldg(p.scales + gi);
          if (ZF) {
            float delta;
            dq::split_zero_point<BITS>(__ldg(p.zeros_f + gi), z[k], delta);
            cz[k] = -delta * sc[k];
          } else {
            z[k] = __ldg(p.zeros + gi);
          }
        }
      }
      pf_kb += X_GROUPS;
      while (pf_kb >= p.k_blocks) {
        pf_kb -= p.k_blocks;
        pf_tile += n_pairs;
        pf_col = item_col(pf_tile);
      }
    };
    uint32_t z[2], zn[2];
    float sc[2], scn[2], cz[2], czn[2];
    if ((uint32_t)grp < total_it) load_zs(z, sc, cz);
    for (uint32_t it = grp; it < total_it; it += X_GROUPS) {
      if (it + X_GROUPS < total_it) load_zs(zn, scn, czn);
      const int s = it % XSTAGES;
      const int q = it % XQ_SLOTS;
      if (!mbar_wait(smem_u32(&bars->pk_full[q]), (it / XQ_SLOTS) & 1u, abort_flag)) break;
      uint32_t wa[BITS], wb[BITS];
      {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(sm_q + q * XQ_BYTES) + u4 * BITS;
        if constexpr (BITS == 4) {
          // a unit is 16 aligned bytes: one vector load per row
          const uint4 va = *reinterpret_cast<const uint4*>(src + row_a * 16);
          const uint4 vb = *reinterpret_cast<const uint4*>(src + row_b * 16);
          wa[0] = va.x; wa[1] = va.y; wa[2] = va.z; wa[3] = va.w;
          wb[0] = vb.x; wb[1] = vb.y; wb[2] = vb.z; wb[3] = vb.w;
        } else {
#pragma unroll
          for (int e = 0; e < BITS; ++e) {
            wa[e] = src[row_a * (4 * BITS) + e];
            wb[e] = src[row_b * (4 * BITS) + e];
          }
        }
      }
      uint32_t oa[16], ob[16];
      if constexpr (ZF) {
        dq::unit32_affine<BITS>(wa, z[0], sc[0], cz[0], oa);
        dq::unit32_affine<BITS>(wb, z[1], sc[1], cz[1], ob);
      } else {
        dq::unit32_natural<BITS, true>(wa, z[0], sc[0], oa);
        dq::unit32_natural<BITS, true>(wb, z[1], sc[1], ob);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->pk_empty[q]));   // codes consumed: slot free
      if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ((it / XSTAGES) & 1u) ^ 1u, abort_flag)) break;
      uint8_t* wbuf = base + s * XSTAGE_BYTES + XA_BYTES;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        *reinterpret_cast<uint4*>(wbuf + off_a + (((chunk0 + c) ^ swz) << 4)) =
            make_uint4(oa[4 * c], oa[4 * c + 1], oa[4 * c + 2], oa[4 * c + 3]);
        *reinterpret_cast<uint4*>(wbuf + off_b + (((chunk0 + c) ^ swz) << 4)) =
            make_uint4(ob[4 * c], ob[4 * c + 1], ob[4 * c + 2], ob[4 * c + 3]);
      }
      // make the tile visible to the tensor cores of both CTAs, then tell the leader
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_release(full_w_leader0 + s * 8);
      z[0] = zn[0]; z[1] = zn[1];
      sc[0] = scn[0]; sc[1] = scn[1];
      cz[0] = czn[0]; cz[1] = czn[1];
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
    tmem_dealloc_pair(tmem_base, X_TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) {
    atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
    p.status[1] = (int)blockIdx.x;
  }
}

template <int BITS, bool ZF>
int launch_dx_pair_t(const CUtensorMap& ta, const CUtensorMap& tq, const CUtensorMap& to, const DxParams& p, int pairs,
                     cudaStream_t st) {
  auto kern = qdx_pair_kernel<BITS, ZF>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, X_SMEM_BYTES));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kDxThreads, 1, 1);
  cfg.dynamicSmemBytes = X_SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // barrier set-up and the tensor-memory allocation may overlap the tail of the kernel before
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, ta, tq, to, p));
  return PEQA_OK;
}

}  // namespace

// Same shape rule as the forward pair kernel: the code boxes need a 16-byte row pitch.
bool dx_pair_supported(const peqa_qweight_t* w) {
  return ((size_t)w->in_features * w->bits / 8) % 16 == 0;
}

int launch_dx_pair(const peqa_qweight_t* w, const float* zeros_f, int g, const void* dY, int T,
                   void* dX, cudaStream_t st) {
  DxParams p;
  p.zeros = w->zeros;
  p.zeros_f = zeros_f;
  p.scales = w->scales;
  p.out = static_cast<__nv_bfloat16*>(dX);
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  p.g_shift = -1;
  for (int b = 5; b < 31; ++b)
    if ((1 << b) == g) p.g_shift = b;
  p.T = T;
  p.j_tiles = (p.K + 255) / 256;
  p.t_tiles = (T + 511) / 512;
  p.k_blocks = (p.N + XK - 1) / XK;
  PEQA_TRY(status_word(st, &p.status));
  EncodeTiledFn enc = nullptr;
  PEQA_TRY(tensor_map_encoder(&enc));
  CUtensorMap ta, tq, to;
  {
    // output dX [T, K]: boxes of 32 columns x 32 tokens, 64-byte swizzle (the epilogue's staging tile)
    cuuint64_t dims[2] = {(cuuint64_t)p.K, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)p.K * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&to, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, dX, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  {
    cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)p.N * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(dY), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  {
    const int wpr = p.K * w->bits / 32;
    cuuint64_t dims[2] = {(cuuint64_t)wpr, (cuuint64_t)p.N};
    cuuint64_t strides[1] = {(cuuint64_t)wpr * 4};
    cuuint32_t box[2] = {(cuuint32_t)(4 * w->bits), 64};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(w->qweight), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int tiles = p.j_tiles * p.t_tiles;
  const int max_pairs = sms / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  p.items = make_pair_items(p.j_tiles, p.t_tiles, T, pairs);
  if (zeros_f)
    return w->bits == 4 ? launch_dx_pair_t<4, true>(ta, tq, to, p, pairs, st)
                        : launch_dx_pair_t<3, true>(ta, tq, to, p, pairs, st);
  return w->bits == 4 ? launch_dx_pair_t<4, false>(ta, tq, to, p, pairs, st)
                      : launch_dx_pair_t<3, false>(ta, tq, to, p, pairs, st);
}

}  // namespace peqa
