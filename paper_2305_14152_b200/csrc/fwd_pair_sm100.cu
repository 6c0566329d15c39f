// Forward of the PEQA layer, Y = X * W_hat^T (Eq. 2), on CTA pairs.
//
// A pair of CTAs (cta_group::2) owns a tile of 512 tokens x 256 output channels,
// held as two 256 x 256 accumulators that fill tensor memory.  The tokens are
// the MMA "M" side: CTA `rank` TMA-loads two blocks of 128 tokens of X per
// 64-deep stage (A operands, K-major).  The weights are the "N" side, split
// between the two CTAs: each rebuilds (Q - z) [* bf16(s)] of its 128 channels
// [n0 + 128*rank, +128) as bf16 in its own shared memory, K-major with the
// 128-byte swizzle the tensor core expects, and both token blocks multiply the
// same weight stage.  A weight element is therefore rebuilt once per 512
// tokens, which brings the conversion work per stage (8192 elements per CTA)
// under the time the tensor cores need for it (two 256x256x64 products), and
// the accumulator is token-major, so an epilogue thread writes contiguous runs
// of Y.
//
// Packed codes reach the dequant warps through their own TMA ring (one box =
// 128 channels x 64 columns of codes).  Four groups of four dequant warps take
// the stages round-robin, so that one group's wait -> read -> convert -> store
// -> signal chain overlaps the others'.  A tile whose second token block lies
// wholly beyond T runs with one block.
//
// With one scale per channel (G == 1) the weights stay the exact integers
// Q - z and the fp32 scale multiplies the accumulator columns in the epilogue;
// with grouped scales the product (Q - z) * bf16(s) is formed before the MMA.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace peqa {

namespace {

using namespace ptx;

constexpr int PK = 64;                       // contraction elements per stage
constexpr int PSTAGES = 4;
constexpr int PBLK_BYTES = 128 * PK * 2;     // one block of 128 tokens of X: 16 KiB
constexpr int PA_BYTES = 2 * PBLK_BYTES;     // this CTA's two token blocks
constexpr int PB_BYTES = 128 * PK * 2;       // this CTA's 128 channels: 16 KiB
constexpr int PSTAGE_BYTES = PA_BYTES + PB_BYTES;
constexpr int PQ_SLOTS = 4;
constexpr int PE_BYTES = 32 * 64;            // one epilogue warp's staging tile: 32 tokens x 32 channels
constexpr int PQ_BYTES = 128 * 32;           // packed codes of one stage: 128 rows x 8 words
constexpr int P_TMEM_COLS = 512;
constexpr int P_SMEM_BYTES = PSTAGES * PSTAGE_BYTES + PQ_SLOTS * PQ_BYTES + 8 * PE_BYTES + 1024 + 512;
constexpr int P_GROUPS = 4;        // dequant groups (four warps each)
constexpr int kPairThreads = 896;  // warps: 0 act TMA, 1 MMA, 2 TMEM alloc, 3 code TMA, 4-11 epilogue, 12-27 dequant

struct PairBarriers {
  uint64_t full_act[PSTAGES];   // leader: X bytes of both CTAs landed
  uint64_t full_w[PSTAGES];     // leader: weight halves of both CTAs written
  uint64_t empty[PSTAGES];      // each CTA: MMAs that read the stage completed
  uint64_t pk_full[PQ_SLOTS];   // each CTA: packed codes landed
  uint64_t pk_empty[PQ_SLOTS];  // each CTA: the group that owns the slot has read it
  uint64_t acc_full;            // each CTA: both accumulators ready
  uint64_t acc_empty;           // leader: both CTAs' epilogues drained them
  uint32_t tmem_base;
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

struct PairParams {
  const uint8_t* zeros;
  const float* zeros_f;   // real-valued zero-points (App. K) or nullptr; replaces `zeros`
  const float* scales;
  __nv_bfloat16* out;   // Y [T, N]
  int N, K, G, g, g_shift, T;
  int n_tiles, t_tiles, k_blocks;   // 256-channel tiles, 512-token tiles, 64-deep stages
  PairItems items;
  int* status;
};

__device__ __forceinline__ int pair_group_of(const PairParams& p, int col) {
  if (p.G == 1) return 0;
  return p.g_shift >= 0 ? (col >> p.g_shift) : (col / p.g);
}

template <int BITS, bool FOLD, bool ZF>
__global__ void __launch_bounds__(kPairThreads, 1)
qfwd_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_q,
                 const __grid_constant__ CUtensorMap tmap_y, const PairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* sm_q = base + PSTAGES * PSTAGE_BYTES;          // PQ_SLOTS x 4 KiB, plain 32-byte rows
  uint8_t* sm_e = sm_q + PQ_SLOTS * PQ_BYTES;             // 8 epilogue warps x 2 KiB, 64-byte swizzle
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(sm_e + 8 * PE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(smem_u32(&bars->full_act[s]), 1);
      mbar_init(smem_u32(&bars->full_w[s]), 8);           // 4 warps of one group in each CTA
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int q = 0; q < PQ_SLOTS; ++q) {
      mbar_init(smem_u32(&bars->pk_full[q]), 1);
      mbar_init(smem_u32(&bars->pk_empty[q]), 4);         // 4 warps of the owning group
    }
    mbar_init(smem_u32(&bars->acc_full), 1);
    mbar_init(smem_u32(&bars->acc_empty), 16);            // 8 epilogue warps in each CTA
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    fence_mbar_init();
    prefetch_tmap(&tmap_x);
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_y);
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(&bars->tmem_base), P_TMEM_COLS);
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
    // ------------------------------------------ activation TMA (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      // self-test knob (peqa_selftest_configure): announce one byte more than will arrive, so
      // that the stage never fills and the bounded waits have to end the kernel
      const uint32_t starve = p.status[5] != 0 ? 1u : 0u;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        int n_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, n_tile, tt0, blocks);
        const int t0 = tt0 + (int)rank * 128;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_arrive_expect_tx(smem_u32(&bars->full_act[s]), 2 * blocks * PBLK_BYTES + starve);
          const uint32_t bar = mapa_shared(smem_u32(&bars->full_act[s]), 0);
          tma_load_2d_pair(smem_u32(base + s * PSTAGE_BYTES), &tmap_x, bar, kb * PK, t0);
          if (blocks == 2)
            tma_load_2d_pair(smem_u32(base + s * PSTAGE_BYTES + PBLK_BYTES), &tmap_x, bar, kb * PK, t0 + 256);
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
        int n_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, n_tile, tt0, blocks);
        const int r0 = n_tile * 256 + (int)rank * 128;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int q = it % PQ_SLOTS;
          const uint32_t ph = (it / PQ_SLOTS) & 1u;
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
      constexpr uint32_t idesc = idesc_bf16_f32(256, 256, 0, 0);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
        int n_tile, tt0, blocks;
        pair_item(p.items, tile, p.T, n_tile, tt0, blocks);
        if (!mbar_wait_cluster(smem_u32(&bars->acc_empty), (uint32_t)(local & 1) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->full_w[s]), ph, abort_flag) ||
              !mbar_wait_cluster(smem_u32(&bars->full_act[s]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(base + s * PSTAGE_BYTES);
          const uint32_t b_addr = a_addr + PA_BYTES;
          for (int m = 0; m < blocks; ++m) {
#pragma unroll
            for (int k = 0; k < PK / 16; ++k) {
              const uint64_t adesc = smem_desc_sw128(a_addr + m * PBLK_BYTES + k * 32, 16, 1024);
              const uint64_t bdesc = smem_desc_sw128(b_addr + k * 32, 16, 1024);
              mma_bf16_ss_pair(tmem_base + m * 256, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
            }
          }
          mma_commit_pair(smem_u32(&bars->empty[s]), 3);
        }
        if (ok) mma_commit_pair(smem_u32(&bars->acc_full), 3);
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------------ epilogue: thread = token, 256 channels
    // A warp drains 32 tokens x 32 channels at a time: tensor memory -> registers -> bf16 ->
    // its 2 KiB staging tile (rows of 64 bytes, 16-byte chunk c of row r at c ^ ((r >> 1) & 3):
    // the 64-byte swizzle of the output tensor map, which also keeps the stores free of bank
    // conflicts) -> one tiled bulk store.  The copy engine writes whole sectors of Y; a
    // thread-per-row store by the warp itself cost 32 half-filled sectors per instruction and
    // made the drain take ~11,000 cycles a tile.  The accumulators are released as soon as the
    // last chunk has left tensor memory.
    const int quarter = warp & 3;
    const int m = (warp - 4) >> 2;                 // token block = accumulator
    const uint32_t acc_empty_leader = mapa_shared(smem_u32(&bars->acc_empty), 0);
    uint8_t* stage = sm_e + (warp - 4) * PE_BYTES;
    uint8_t* srow = stage + lane * 64;
    const int sw = (lane >> 1) & 3;
    int local = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
      int n_tile, tt0, blocks;
      pair_item(p.items, tile, p.T, n_tile, tt0, blocks);
      const int n0 = n_tile * 256;
      const int row0 = tt0 + m * 256 + (int)rank * 128 + quarter * 32;   // first token of this warp
      if (!mbar_wait_cluster(smem_u32(&bars->acc_full), (uint32_t)(local & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      int chunks = m < blocks ? (p.N - n0 + 31) / 32 : 0;
      chunks = chunks > 8 ? 8 : chunks;
#pragma unroll 1
      for (int cc = 0; cc < chunks; ++cc) {
        const int c0 = n0 + cc * 32;
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + m * 256 + cc * 32, v);
        tmem_ld_wait();
        if (cc + 1 == chunks) {
          // nothing of this tile is left in tensor memory for this warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
        }
        if (!FOLD) {
          // one scale per channel: every lane reads the same 32 scales (broadcast loads)
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float sc = c0 + j < p.N ? __ldg(p.scales + c0 + j) : 0.0f;
            v[j] = __float_as_uint(__uint_as_float(v[j]) * sc);
          }
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
          tma_store_2d(&tmap_y, smem_u32(stage), c0, row0);
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
    // ------------------------------------------ weight dequant (this CTA's 128 channels)
    // Group g (four warps) serves the stages with it % 4 == g.  A thread is one channel:
    // it converts the 64 contraction elements of the stage (two units of 32 columns)
    // and writes them as the channel's 128-byte row, 16-byte chunk c at position
    // c ^ (row % 8) (the 128-byte swizzle).
    const int grp = (warp - 12) >> 2;
    const int row = ((warp - 12) & 3) * 32 + lane;
    const int swz = row & 7;
    const uint32_t full_w_leader0 = mapa_shared(smem_u32(&bars->full_w[0]), 0);
    const uint32_t total_it = (uint32_t)my_tiles * (uint32_t)p.k_blocks;
    // cursor of the stage whose (s, z) is being prefetched, walked without divisions
    int pf_tile = pair, pf_kb = grp;
    while (pf_kb >= p.k_blocks) { pf_kb -= p.k_blocks; pf_tile += n_pairs; }
    auto item_row = [&](int item) {
      int n_tile, tt0, blocks;
      pair_item(p.items, item, p.T, n_tile, tt0, blocks);
      return n_tile * 256 + (int)rank * 128 + row;
    };
    int pf_r = item_row(pf_tile);
    // every lane reads another row, so each load of a warp touches 32 sectors: the two
    // units of a stage share one load when they share a group (g >= 64, or one scale per
    // channel), and one 2-byte / 8-byte load when the groups are 32 columns wide
    const bool one_group = p.G == 1 || (p.g & 63) == 0;
    const bool pair_load = !one_group && p.g == 32 && (p.G & 1) == 0;
    // cz: the constant term -delta * s of a real-valued zero-point (ZF), else unused
    auto load_zs = [&](uint32_t (&z)[2], float (&sc)[2], float (&cz)[2]) {
      z[0] = z[1] = 0u;
      sc[0] = sc[1] = 0.0f;
      cz[0] = cz[1] = 0.0f;
      const int col = pf_kb * PK;
      if (pf_r < p.N && col < p.K) {
        const size_t gi = (size_t)pf_r * p.G + pair_group_of(p, col);
        if (ZF) {
          float delta;
          sc[0] = __ldg(p.scales + gi);
          dq::split_zero_point<BITS>(__ldg(p.zeros_f + gi), z[0], delta);
          cz[0] = -delta * sc[0];
          z[1] = z[0]; sc[1] = sc[0]; cz[1] = cz[0];
          if (!one_group && col + 32 < p.K) {
            const size_t g1 = (size_t)pf_r * p.G + pair_group_of(p, col + 32);
            sc[1] = __ldg(p.scales + g1);
            dq::split_zero_point<BITS>(__ldg(p.zeros_f + g1), z[1], delta);
            cz[1] = -delta * sc[1];
          }
        } else if (one_group) {
          z[0] = z[1] = __ldg(p.zeros + gi);
          if (FOLD) sc[0] = sc[1] = __ldg(p.scales + gi);
        } else if (pair_load) {
          const uint32_t z2 = __ldg(reinterpret_cast<const unsigned short*>(p.zeros + gi));
          z[0] = z2 & 0xFFu;
          z[1] = z2 >> 8;
          if (FOLD) {
            const float2 s2 = __ldg(reinterpret_cast<const float2*>(p.scales + gi));
            sc[0] = s2.x;
            sc[1] = s2.y;
          }
        } else {
          z[0] = __ldg(p.zeros + gi);
          if (FOLD) sc[0] = __ldg(p.scales + gi);
          if (col + 32 < p.K) {
            const size_t g1 = (size_t)pf_r * p.G + pair_group_of(p, col + 32);
            z[1] = __ldg(p.zeros + g1);
            if (FOLD) sc[1] = __ldg(p.scales + g1);
          }
        }
      }
      pf_kb += P_GROUPS;
      while (pf_kb >= p.k_blocks) {
        pf_kb -= p.k_blocks;
        pf_tile += n_pairs;
        pf_r = item_row(pf_tile);
      }
    };
    uint32_t z[2], zn[2];
    float sc[2], scn[2], cz[2], czn[2];
    int cur_kb = pf_kb;
    if ((uint32_t)grp < total_it) load_zs(z, sc, cz);
    for (uint32_t it = grp; it < total_it; it += P_GROUPS) {
      const int next_kb = pf_kb;
      if (it + P_GROUPS < total_it) load_zs(zn, scn, czn);
      const int s = it % PSTAGES;
      const int q = it % PQ_SLOTS;
      if (!mbar_wait(smem_u32(&bars->pk_full[q]), (it / PQ_SLOTS) & 1u, abort_flag)) break;
      uint32_t w[2][BITS];
      {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(sm_q + q * PQ_BYTES) + row * 8;
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
      uint32_t o0[16], o1[16];
      if constexpr (ZF) {
        dq::unit32_affine<BITS>(w[0], z[0], sc[0], cz[0], o0);
        dq::unit32_affine<BITS>(w[1], z[1], sc[1], cz[1], o1);
      } else {
        dq::unit32_natural<BITS, FOLD>(w[0], z[0], sc[0], o0);
        dq::unit32_natural<BITS, FOLD>(w[1], z[1], sc[1], o1);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->pk_empty[q]));   // codes consumed: slot free
      if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ((it / PSTAGES) & 1u) ^ 1u, abort_flag)) break;
      uint8_t* wrow = base + s * PSTAGE_BYTES + PA_BYTES + row * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        *reinterpret_cast<uint4*>(wrow + ((c ^ swz) << 4)) =
            make_uint4(o0[4 * c], o0[4 * c + 1], o0[4 * c + 2], o0[4 * c + 3]);
        *reinterpret_cast<uint4*>(wrow + (((4 + c) ^ swz) << 4)) =
            make_uint4(o1[4 * c], o1[4 * c + 1], o1[4 * c + 2], o1[4 * c + 3]);
      }
      // make the rows visible to the tensor cores of both CTAs, then tell the leader
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_release(full_w_leader0 + s * 8);
      z[0] = zn[0]; z[1] = zn[1];
      sc[0] = scn[0]; sc[1] = scn[1];
      cz[0] = czn[0]; cz[1] = czn[1];
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

template <int BITS, bool FOLD, bool ZF>
int launch_pair_t(const CUtensorMap& tx, const CUtensorMap& tq, const CUtensorMap& ty, const PairParams& p,
                  int pairs, cudaStream_t st) {
  auto kern = qfwd_pair_kernel<BITS, FOLD, ZF>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = P_SMEM_BYTES;
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
  PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, tx, tq, ty, p));
  return PEQA_OK;
}

}  // namespace

// The pair kernel needs a 16-byte row pitch of the packed matrix for its code
// boxes (always true for 4-bit, K % 128 == 0 for 3-bit); other shapes take the
// single-CTA kernel.
bool fwd_pair_supported(const peqa_qweight_t* w) {
  return ((size_t)w->in_features * w->bits / 8) % 16 == 0;
}

int launch_fwd_pair(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, int T,
                    void* Y, cudaStream_t st) {
  PairParams p;
  p.zeros = w->zeros;
  p.zeros_f = zeros_f;
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
  p.n_tiles = (p.N + 255) / 256;
  p.t_tiles = (T + 511) / 512;
  p.k_blocks = (p.K + PK - 1) / PK;
  PEQA_TRY(status_word(st, &p.status));
  EncodeTiledFn enc = nullptr;
  PEQA_TRY(tensor_map_encoder(&enc));
  CUtensorMap tx, tq, ty;
  {
    // output Y [T, N]: boxes of 32 channels x 32 tokens, 64-byte swizzle (the epilogue's staging tile)
    cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)p.N * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  {
    cuuint64_t dims[2] = {(cuuint64_t)p.K, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)p.K * 2};
    cuuint32_t box[2] = {64, 128};
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
    cuuint32_t box[2] = {8, 128};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tq, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(w->qweight), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int tiles = p.n_tiles * p.t_tiles;
  const int max_pairs = sms / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  p.items = make_pair_items(p.n_tiles, p.t_tiles, T, pairs);
  const bool fold = p.G > 1;
  if (zeros_f)   // a real-valued zero-point is folded into the operand whatever the group size
    return w->bits == 4 ? launch_pair_t<4, true, true>(tx, tq, ty, p, pairs, st)
                        : launch_pair_t<3, true, true>(tx, tq, ty, p, pairs, st);
  if (w->bits == 4)
    return fold ? launch_pair_t<4, true, false>(tx, tq, ty, p, pairs, st)
                : launch_pair_t<4, false, false>(tx, tq, ty, p, pairs, st);
  return fold ? launch_pair_t<3, true, false>(tx, tq, ty, p, pairs, st)
              : launch_pair_t<3, false, false>(tx, tq, ty, p, pairs, st);
}

}  // namespace peqa
