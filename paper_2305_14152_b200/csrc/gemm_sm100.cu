// Tensor-core kernels of the PEQA layer for sm_100a.
//
//   qgemm_kernel<TRANS=false>  Y[t,i]  = sum_j X[t,j]  * W_hat[i,j]     (forward, Eq. 2)
//   qgemm_kernel<TRANS=true>   dX[t,j] = sum_i dY[t,i] * W_hat[i,j]     (backward wrt input)
//   ds_kernel                  dS[i,g] = sum_{j in g} (Q-z)[i,j] * (dY^T X)[i,j]
//
// All three are persistent, warp-specialised kernels: one CTA per SM walks a
// static list of 128x256 output tiles.  Activations arrive by TMA into
// 128-byte-swizzled shared memory, tcgen05.mma accumulates fp32 in tensor
// memory (two 256-column accumulators, so the epilogue of one tile overlaps
// the main loop of the next), and every mbarrier wait is bounded.
//
// In qgemm the weight operand never exists in HBM as bf16: dedicated warps
// read the packed codes, rebuild (Q - z) [times bf16(s) when the scale varies
// along the contraction] in registers and write the bf16 tile straight into
// the swizzled layout the tensor core reads.  The weight tile is the MMA "A"
// operand (M = 128 weight rows/columns), the activation tile the "B" operand
// (N = 256 tokens), so each weight is dequantised once per 256 tokens.
//   forward : A is K-major   (row = out channel i, 64 contraction columns j)
//   dX      : A is MN-major  (row = contraction index i, 128 columns j) --
//             the same row-wise unpack, only the descriptor differs, so Q is
//             "read transposed" without any transposed copy.
//
// In ds_kernel both operands are activations (dY^T and X, MN-major straight
// from their row-major storage); the 128x256 dW tile stays in tensor memory,
// and the epilogue multiplies it by (Q - z) and sums over column pieces that
// lie inside one group.  dW never reaches HBM.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace peqa {

namespace {

using namespace ptx;

constexpr int BM = 128;      // weight rows per tile (MMA M, TMEM lanes)
constexpr int BN = 256;      // tokens (qgemm) / weight columns (ds) per tile (MMA N)
constexpr int BK = 64;       // contraction elements per pipeline stage
constexpr int UMMA_K = 16;   // contraction elements per tcgen05.mma
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;   // 16 KiB
constexpr int B_BYTES = BN * BK * 2;   // 32 KiB
constexpr int PK_BYTES = 4096;         // packed codes of one stage (qgemm)
constexpr int PK_SLOTS = 8;            // their own, deeper ring: the codes run ahead of the operands
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 512;         // two fp32 accumulators of 256 columns
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + PK_SLOTS * PK_BYTES + 1024 /*align*/ + 512 /*barriers*/;

constexpr int kQgemmThreads = 512;     // warps: 0 TMA, 1 MMA, 2 TMEM alloc, 4-7 epilogue, 8-15 dequant
constexpr int kDequantThreads = 256;
constexpr int DQ_GROUPS = 4;           // dequant warp groups that take the stages round-robin
constexpr int kDsThreads = 384;        // warps: 0 TMA, 1 MMA, 2 TMEM alloc, 4-11 epilogue

struct Barriers {
  uint64_t full_a[STAGES];   // dequantised weight tile written (qgemm only)
  uint64_t full_b[STAGES];   // TMA bytes landed
  uint64_t full_pk[PK_SLOTS];   // packed codes landed (qgemm with TMA-staged codes)
  uint64_t empty_pk[PK_SLOTS];  // all dequant warps have read the slot
  uint64_t empty[STAGES];    // MMAs that read the stage have completed
  uint64_t acc_full[2];      // accumulator ready for the epilogue
  uint64_t acc_empty[2];     // accumulator drained by the epilogue
  uint32_t tmem_base;
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

struct SmemView {
  uint8_t* a[STAGES];
  uint8_t* b[STAGES];
  uint8_t* pk[PK_SLOTS];
  Barriers* bars;
};

__device__ __forceinline__ SmemView carve_smem(uint8_t* raw) {
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  SmemView v;
#pragma unroll
  for (int s = 0; s < STAGES; ++s) {
    v.a[s] = base + s * STAGE_BYTES;
    v.b[s] = base + s * STAGE_BYTES + A_BYTES;
  }
#pragma unroll
  for (int q = 0; q < PK_SLOTS; ++q) v.pk[q] = base + STAGES * STAGE_BYTES + q * PK_BYTES;
  v.bars = reinterpret_cast<Barriers*>(base + STAGES * STAGE_BYTES + PK_SLOTS * PK_BYTES);
  return v;
}

// After a bounded wait gave up: let copies and MMAs already in flight finish
// before shared and tensor memory are released.
__device__ __forceinline__ void drain_after_abort() {
  for (int i = 0; i < 64; ++i) __nanosleep(1000);
}

struct QGemmParams {
  const uint32_t* qw;
  const uint8_t* zeros;
  const float* zeros_f;   // real-valued zero-points (App. K) or nullptr; replaces `zeros`
  const float* scales;
  __nv_bfloat16* out;   // [T, R]
  int N, K, G, g, T;
  int g_shift;          // log2(g) when g is a power of two, else -1
  int wpr;              // packed words per weight row
  int R, C;             // output features, contraction length
  int r_tiles, t_tiles, k_blocks;
  int* status;
};

// Packed words, zero-point and scale of one 32-column unit of one weight row.
template <int BITS>
struct Unit {
  uint32_t w[BITS];
  uint32_t z;
  float s;
  float c;   // -delta * s of a real-valued zero-point z + delta (App. K), else 0
};

__device__ __forceinline__ int group_of(const QGemmParams& p, int col) {
  if (p.G == 1) return 0;
  return p.g_shift >= 0 ? (col >> p.g_shift) : (col / p.g);
}

// Weight row i, columns [col0, col0 + 32): zero-point and scale, plus the packed
// words when WORDS is set (otherwise the caller takes them from shared memory).
template <int BITS, bool WORDS = true>
__device__ __forceinline__ Unit<BITS> load_unit(const QGemmParams& p, int i, int col0) {
  Unit<BITS> u;
#pragma unroll
  for (int q = 0; q < BITS; ++q) u.w[q] = 0u;
  if (i < p.N && col0 < p.K) {
    if (WORDS) {
      const uint32_t* src = p.qw + (size_t)i * p.wpr + (col0 >> 5) * BITS;
      if constexpr (BITS == 4) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
        u.w[0] = v.x; u.w[1] = v.y; u.w[2] = v.z; u.w[3] = v.w;
      } else {
        u.w[0] = __ldg(src); u.w[1] = __ldg(src + 1); u.w[2] = __ldg(src + 2);
      }
    }
    const size_t gidx = (size_t)i * p.G + group_of(p, col0);
    u.s = __ldg(p.scales + gidx);
    u.c = 0.0f;
    if (p.zeros_f) {
      float delta;
      dq::split_zero_point<BITS>(__ldg(p.zeros_f + gidx), u.z, delta);
      u.c = -delta * u.s;
    } else {
      u.z = __ldg(p.zeros + gidx);
    }
  } else {
    // Outside the matrix: codes equal to the zero-point dequantise to exactly 0.
    u.z = 0u;
    u.s = 0.0f;
    u.c = 0.0f;
  }
  return u;
}

// (q - z) [* bf16(s)] of one unit; with a real-valued zero-point (zf, uniform over the
// launch, only with FOLD) the affine form (q - zi) * s + c.
template <int BITS, bool FOLD>
__device__ __forceinline__ void dequant_unit(const Unit<BITS>& u, bool zf, uint32_t (&o)[16]) {
  if (FOLD && zf) dq::unit32_affine<BITS>(u.w, u.z, u.s, u.c, o);
  else dq::unit32_natural<BITS, FOLD>(u.w, u.z, u.s, o);
}

// PKTMA: the packed codes of a stage arrive by TMA in shared memory (needs a
// 16-byte row pitch of the packed matrix); otherwise the dequant threads read
// them from global memory themselves.
template <int BITS, bool TRANS, bool FOLD, bool PKTMA>
__global__ void __launch_bounds__(kQgemmThreads, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmap_act,
             const __grid_constant__ CUtensorMap tmap_pk, const QGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  SmemView sm = carve_smem(smem_raw);
  Barriers* bars = sm.bars;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars->full_a[s]), kDequantThreads / DQ_GROUPS);   // the threads of one dequant group
      mbar_init(smem_u32(&bars->full_b[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int q = 0; q < PK_SLOTS; ++q) {
      mbar_init(smem_u32(&bars->full_pk[q]), 1);
      mbar_init(smem_u32(&bars->empty_pk[q]), (kDequantThreads / 32) / DQ_GROUPS);   // the warps of one group
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);
      mbar_init(smem_u32(&bars->acc_empty[b]), 128);
    }
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    fence_mbar_init();
    prefetch_tmap(&tmap_act);
    if (PKTMA) prefetch_tmap(&tmap_pk);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(&bars->tmem_base), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  const int total_tiles = p.r_tiles * p.t_tiles;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const int t0 = (tile / p.r_tiles) * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t bar = smem_u32(&bars->full_b[s]);
          mbar_arrive_expect_tx(bar, B_BYTES);
          tma_load_2d(smem_u32(sm.b[s]), &tmap_act, bar, kb * BK, t0);
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------ packed-code TMA producer (one lane)
    // forward: a box is 128 rows x 8 words holding the stage's 64 columns (3-bit: on odd
    // k-blocks the 6 words start 2 words into the box, which keeps the box start
    // 16-byte aligned); dX: 64 rows x the tile's 128 columns.
    if (PKTMA && lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const int w0 = (tile % p.r_tiles) * BM;   // first weight row (forward) / column (dX)
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int q = it % PK_SLOTS;
          const uint32_t ph = (it / PK_SLOTS) & 1u;
          if (!mbar_wait(smem_u32(&bars->empty_pk[q]), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t pbar = smem_u32(&bars->full_pk[q]);
          if (!TRANS) {
            mbar_arrive_expect_tx(pbar, 128 * 32);
            tma_load_2d(smem_u32(sm.pk[q]), &tmap_pk, pbar,
                        BITS == 3 ? 6 * kb - 2 * (kb & 1) : 8 * kb, w0);
          } else {
            mbar_arrive_expect_tx(pbar, 64 * 16 * BITS);
            tma_load_2d(smem_u32(sm.pk[q]), &tmap_pk, pbar, (w0 >> 5) * BITS, kb * BK);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------- MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(BM, BN, TRANS ? 1 : 0, 0);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bars->acc_empty[buf]), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(smem_u32(&bars->full_a[s]), ph, abort_flag) ||
              !mbar_wait(smem_u32(&bars->full_b[s]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(sm.a[s]);
          const uint32_t b_addr = smem_u32(sm.b[s]);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = TRANS
                ? smem_desc_sw128(a_addr + k * (UMMA_K * 128), 64 * 128, 1024)
                : smem_desc_sw128(a_addr + k * (UMMA_K * 2), 16, 1024);
            const uint64_t bdesc = smem_desc_sw128(b_addr + k * (UMMA_K * 2), 16, 1024);
            mma_bf16_ss(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit(smem_u32(&bars->empty[s]));
        }
        if (ok) mma_commit(smem_u32(&bars->acc_full[buf]));
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ------------------------------------------------------------- epilogue
    const int ew = warp - 4;  // == warp % 4: the TMEM lane quarter this warp may read
    int local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++local) {
      const int r0 = (tile % p.r_tiles) * BM;
      const int t0 = (tile / p.r_tiles) * BN;
      const int buf = local & 1;
      const uint32_t acc_ph = (local >> 1) & 1u;
      if (!mbar_wait(smem_u32(&bars->acc_full[buf]), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int r = r0 + ew * 32 + lane;
      float scale = 1.0f;
      if (!FOLD && r < p.R) scale = __ldg(p.scales + r);  // per-channel forward: s[i] applied here
#pragma unroll 1
      for (int cc = 0; cc < BN / 32; ++cc) {
        const int tc0 = t0 + cc * 32;
        if (tc0 >= p.T) break;
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(ew * 32) << 16) + buf * BN + cc * 32, v);
        tmem_ld_wait();
        if (r < p.R) {
          __nv_bfloat16* dst = p.out + (size_t)tc0 * p.R + r;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (tc0 + j < p.T) dst[(size_t)j * p.R] = __float2bfloat16_rn(__uint_as_float(v[j]) * scale);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&bars->acc_empty[buf]));
    }
  } else if (warp >= 8) {
    // ------------------------------------------------------- weight dequant
    // DQ_GROUPS groups of warps take the stages round-robin, so that one group's
    // wait -> read -> convert -> store -> signal chain overlaps the other groups';
    // a thread converts UPT units (32 columns each) of its group's stage, all of
    // them into registers before it waits for the stage buffer to be released.
    constexpr int UPT = DQ_GROUPS;                      // 256 units per stage / threads per group
    constexpr int GW = (kDequantThreads / 32) / DQ_GROUPS;   // warps per group
    const int dw = warp - 8;
    const int grp = dw / GW;
    const int gw = dw % GW;
    const int my_tiles = (total_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const uint32_t total_it = (uint32_t)my_tiles * (uint32_t)p.k_blocks;
    // forward: stage = 128 weight rows x 2 units; lanes = 32 consecutive rows; the
    //          thread's units are (row, 0), (row, 1), (row + 32*GW, 0), ...
    // dX:      stage = 64 weight rows x 4 units; lanes = 8 rows x 4 units; further
    //          units of the thread are the same columns 8*GW rows further down.
    const int u4 = lane >> 3;
    int rowl[UPT], col_off[UPT], chunk0[UPT], row_off[UPT];
#pragma unroll
    for (int k = 0; k < UPT; ++k) {
      if constexpr (!TRANS) {
        rowl[k] = gw * 32 + lane + (k >> 1) * (32 * GW);
        col_off[k] = 32 * (k & 1);
        chunk0[k] = 4 * (k & 1);
        row_off[k] = rowl[k] * 128;
      } else {
        rowl[k] = gw * 8 + (lane & 7) + k * (8 * GW);
        col_off[k] = 32 * u4;
        chunk0[k] = (u4 & 1) * 4;
        row_off[k] = (u4 >> 1) * (64 * 128) + rowl[k] * 128;
      }
    }
    const int swz = rowl[0] & 7;            // all rows of a thread agree modulo 8
    // cursor of the stage being prefetched (this group's next stage), no divisions
    int pf_tile = blockIdx.x, pf_kb = grp;
    while (pf_kb >= p.k_blocks) { pf_kb -= p.k_blocks; pf_tile += gridDim.x; }
    int pf_w0 = (pf_tile % p.r_tiles) * BM;
    auto load_next = [&](Unit<BITS> (&u)[UPT]) {
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
        if constexpr (!TRANS) u[k] = load_unit<BITS, !PKTMA>(p, pf_w0 + rowl[k], pf_kb * BK + col_off[k]);
        else u[k] = load_unit<BITS, !PKTMA>(p, pf_kb * BK + rowl[k], pf_w0 + col_off[k]);
      }
      pf_kb += DQ_GROUPS;
      while (pf_kb >= p.k_blocks) {
        pf_kb -= p.k_blocks;
        pf_tile += gridDim.x;
        pf_w0 = (pf_tile % p.r_tiles) * BM;
      }
    };
    Unit<BITS> cur[UPT], nxt[UPT];
    int cur_kb = pf_kb;                      // k-block of the stage about to be processed
    if ((uint32_t)grp < total_it) load_next(cur);
    for (uint32_t it = grp; it < total_it; it += DQ_GROUPS) {
      const int next_kb = pf_kb;
      if (it + DQ_GROUPS < total_it) load_next(nxt);
      const int s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1u;
      if (PKTMA) {
        const int pq = it % PK_SLOTS;
        if (!mbar_wait(smem_u32(&bars->full_pk[pq]), (it / PK_SLOTS) & 1u, abort_flag)) break;
        const uint32_t* src = reinterpret_cast<const uint32_t*>(sm.pk[pq]);
        if constexpr (!TRANS) {
          // a row of the slot is 32 bytes: read it whole with two 16-byte loads (consecutive
          // lanes are consecutive rows, so narrower loads would pile onto four banks) and
          // pick this stage's words: 4-bit uses all eight, 3-bit six starting at word 0 or 2
#pragma unroll
          for (int k = 0; k < UPT; k += 2) {
            const uint4 lo = *reinterpret_cast<const uint4*>(src + rowl[k] * 8);
            const uint4 hi = *reinterpret_cast<const uint4*>(src + rowl[k] * 8 + 4);
            const uint32_t w8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            if constexpr (BITS == 4) {
#pragma unroll
              for (int e = 0; e < 4; ++e) { cur[k].w[e] = w8[e]; cur[k + 1].w[e] = w8[4 + e]; }
            } else {
              const bool odd = (cur_kb & 1) != 0;
#pragma unroll
              for (int e = 0; e < 3; ++e) {
                cur[k].w[e] = odd ? w8[2 + e] : w8[e];
                cur[k + 1].w[e] = odd ? w8[5 + e] : w8[3 + e];
              }
            }
          }
        } else {
#pragma unroll
          for (int k = 0; k < UPT; ++k) {
            const uint32_t* r = src + rowl[k] * (4 * BITS) + u4 * BITS;
#pragma unroll
            for (int e = 0; e < BITS; ++e) cur[k].w[e] = r[e];
          }
        }
      }
      uint32_t o[UPT][16];
#pragma unroll
      for (int k = 0; k < UPT; ++k) dequant_unit<BITS, FOLD>(cur[k], p.zeros_f != nullptr, o[k]);
      if (PKTMA) {
        // every lane has consumed its codes by now: hand the slot back
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->empty_pk[it % PK_SLOTS]));
      }
      if (!mbar_wait(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) break;
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
        uint8_t* row_ptr = sm.a[s] + row_off[k];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(row_ptr + (((chunk0[k] + q) ^ swz) << 4)) =
              make_uint4(o[k][4 * q], o[k][4 * q + 1], o[k][4 * q + 2], o[k][4 * q + 3]);
      }
      fence_proxy_async_smem();
      mbar_arrive(smem_u32(&bars->full_a[s]));
#pragma unroll
      for (int k = 0; k < UPT; ++k) cur[k] = nxt[k];
      cur_kb = next_kb;
    }
  }

  // ---------------------------------------------------------------- teardown
  if (*abort_flag) drain_after_abort();
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) {
    atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
    p.status[1] = (int)blockIdx.x;
  }
}

// ------------------------------------------------------------------- dS ---
struct DsParams {
  const uint32_t* qw;
  const uint8_t* zeros;
  const float* zeros_f;   // real-valued zero-points (App. K) or nullptr; only with DZ
  float* out;        // [N, K / piece]: dS itself when piece == g, else partial sums
  float* out_z;      // same shape: dZ (or its partial sums of dW); only read by ds_kernel<.., true>
  const float* scales;
  // ds_kernel<.., ADAM = true> and the reduction kernel: AdamW applied where dS is final
  AdamWConsts adam;
  float* adam_s;
  float* adam_m;
  float* adam_v;
  int N, K, G, g, T;
  int wpr;
  int piece;         // columns per output piece: 32, 64 or 128; divides g
  int i_tiles, j_tiles, k_blocks;
  int band, band_rows;   // tile order: tiles per band and which dimension is banded (see ds_tile)
  int* status;
};

// Tile order of the dS kernel.  One of the two tile dimensions is taken in bands of `band`
// tiles (row tiles of dY^T when band_rows, else column tiles of X); within a band the other
// dimension moves slowest.  The pairs that run at the same time then share a band of operand
// rows (band x 2 MiB at T = 4096) that stays in L2 while the other operand is swept once per
// band; with the plain order (all row tiles for one column tile) dY was re-read from HBM for
// every few column tiles: 4x the algorithmic bytes on the 8192 x 8192 layer.
__device__ __forceinline__ void ds_tile(const DsParams& p, int tile, int& it, int& jt) {
  const int banded = p.band_rows ? p.i_tiles : p.j_tiles;   // tiles along the banded dimension
  const int other = p.band_rows ? p.j_tiles : p.i_tiles;
  const int per_band = p.band * other;
  const int b = tile / per_band;
  const int r = tile - b * per_band;
  const int width = min(p.band, banded - b * p.band);
  const int o = r / width;
  const int w = b * p.band + (r - o * width);
  it = p.band_rows ? w : o;
  jt = p.band_rows ? o : w;
}

// A CTA pair (cta_group::2) owns a 256 x 256 tile of dW: CTA `rank` holds rows
// [i0 + 128*rank, +128) of dY^T as its A operand and accumulator, and loads the
// 128 columns [j0 + 128*rank, +128) of X as its half of the shared B operand.
// The leader CTA (rank 0) issues every MMA; both CTAs' TMA loads credit the
// leader's "full" barrier and tcgen05.commit releases the stage in both CTAs.
constexpr int DS_STAGES = 6;
constexpr int DS_STAGE_BYTES = 2 * (BM * BK * 2);                      // A 16 KiB + B half 16 KiB
constexpr int DS_SMEM_BYTES = DS_STAGES * DS_STAGE_BYTES + 1024 + 512;

struct DsBarriers {
  uint64_t full[DS_STAGES];     // leader: bytes of both CTAs landed
  uint64_t empty[DS_STAGES];    // each CTA: MMAs that read the stage completed
  uint64_t acc_full[2];         // each CTA: accumulator ready
  uint64_t acc_empty[2];        // leader: both CTAs' epilogues drained the accumulator
  uint32_t tmem_base;
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

template <int BITS, bool DZ, bool ADAM>
__global__ void __launch_bounds__(kDsThreads, 1)
ds_kernel(const __grid_constant__ CUtensorMap tmap_dy, const __grid_constant__ CUtensorMap tmap_x,
          const DsParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  DsBarriers* bars = reinterpret_cast<DsBarriers*>(base + DS_STAGES * DS_STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < DS_STAGES; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);
      mbar_init(smem_u32(&bars->acc_empty[b]), 16);   // 8 epilogue warps in each of the 2 CTAs
    }
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    fence_mbar_init();
    prefetch_tmap(&tmap_dy);
    prefetch_tmap(&tmap_x);
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(&bars->tmem_base), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // barriers of both CTAs initialised before any remote arrive
  tc_fence_after();
  // Set-up is done.  The next kernel of the stream may begin its own (programmatic launch);
  // everything below touches memory that the preceding kernel may still be writing.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t tmem_base = bars->tmem_base;
  const int total_tiles = p.i_tiles * p.j_tiles;   // pair tiles (256 x 256)
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        int ti, tj;
        ds_tile(p, tile, ti, tj);
        const int i0 = ti * (2 * BM) + (int)rank * BM;
        const int j0 = tj * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % DS_STAGES;
          const uint32_t ph = (it / DS_STAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t bar = mapa_shared(smem_u32(&bars->full[s]), 0);
          if (leader) mbar_arrive_expect_tx(smem_u32(&bars->full[s]), 2 * DS_STAGE_BYTES);
          uint8_t* st = base + s * DS_STAGE_BYTES;
          // Each box is 64 contiguous features x 64 tokens = one 8 KiB MN-major chunk.
#pragma unroll
          for (int m = 0; m < 2; ++m)
            tma_load_2d_pair(smem_u32(st) + m * 8192, &tmap_dy, bar, i0 + 64 * m, kb * BK);
#pragma unroll
          for (int m = 0; m < 2; ++m)
            tma_load_2d_pair(smem_u32(st) + 16384 + m * 8192, &tmap_x, bar, j0 + 64 * m, kb * BK);
        }
      }
    }
  } else if (warp == 1) {
    if (leader && lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(2 * BM, BN, 1, 1);
      uint32_t it = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
        const int buf = local & 1;
        const uint32_t acc_ph = (local >> 1) & 1u;
        if (!mbar_wait_cluster(smem_u32(&bars->acc_empty[buf]), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % DS_STAGES;
          const uint32_t ph = (it / DS_STAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&bars->full[s]), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(base + s * DS_STAGE_BYTES);
          const uint32_t b_addr = a_addr + 16384;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = smem_desc_sw128(a_addr + k * (UMMA_K * 128), 8192, 1024);
            const uint64_t bdesc = smem_desc_sw128(b_addr + k * (UMMA_K * 128), 8192, 1024);
            mma_bf16_ss_pair(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit_pair(smem_u32(&bars->empty[s]), 3);
        }
        if (ok) mma_commit_pair(smem_u32(&bars->acc_full[buf]), 3);
      }
    }
  } else if (warp >= 4) {
    // Epilogue: thread = one weight row i (TMEM lane) and one 128-column half.
    const int quarter = warp & 3;
    const int half = (warp - 4) >> 2;
    const int npieces = p.K / p.piece;
    const int chunks_per_piece = p.piece >> 5;
    const uint32_t acc_empty_leader0 = mapa_shared(smem_u32(&bars->acc_empty[0]), 0);
    const uint32_t acc_empty_leader1 = mapa_shared(smem_u32(&bars->acc_empty[1]), 0);
    int local = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < total_tiles; tile += n_pairs, ++local) {
      int ti, tj;
      ds_tile(p, tile, ti, tj);
      const int i0 = ti * (2 * BM) + (int)rank * BM;
      const int j0 = tj * BN;
      const int buf = local & 1;
      const uint32_t acc_ph = (local >> 1) & 1u;
      if (!mbar_wait_cluster(smem_u32(&bars->acc_full[buf]), acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int i = i0 + quarter * 32 + lane;
      float acc = 0.0f, accz = 0.0f;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        const int col0 = j0 + half * 128 + cc * 32;
        if (col0 >= p.K) break;
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN + half * 128 + cc * 32, v);
        const bool row_ok = i < p.N;
        uint32_t w[BITS];
        uint32_t z = 0u;
        float delta = 0.0f;   // real-valued zero-point = z + delta
#pragma unroll
        for (int q = 0; q < BITS; ++q) w[q] = 0u;
        if (row_ok) {
          const uint32_t* src = p.qw + (size_t)i * p.wpr + (col0 >> 5) * BITS;
          if constexpr (BITS == 4) {
            const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(src));
            w[0] = q4.x; w[1] = q4.y; w[2] = q4.z; w[3] = q4.w;
          } else {
            w[0] = __ldg(src); w[1] = __ldg(src + 1); w[2] = __ldg(src + 2);
          }
          if (DZ && p.zeros_f) dq::split_zero_point<BITS>(__ldg(p.zeros_f + (size_t)i * p.G + col0 / p.g), z, delta);
          else z = __ldg(p.zeros + (size_t)i * p.G + col0 / p.g);
        }
        uint32_t o[16];
        dq::unit32_natural<BITS, false>(w, z, 0.0f, o);
        tmem_ld_wait();   // warp-wide: every lane executes it, ragged rows included
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          acc = fmaf(__uint_as_float(v[2 * q]), __uint_as_float(o[q] << 16), acc);
          acc = fmaf(__uint_as_float(v[2 * q + 1]), __uint_as_float(o[q] & 0xFFFF0000u), acc);
          if (DZ) accz += __uint_as_float(v[2 * q]) + __uint_as_float(v[2 * q + 1]);
        }
        if (((cc + 1) % chunks_per_piece) == 0) {
          if (row_ok) {
            // with a real-valued zero-point, sum (q - z) dW = sum (q - zi) dW - delta * sum dW;
            // partial pieces are stored raw and corrected after they have been added
            if (DZ && p.zeros_f && p.piece == p.g) acc = fmaf(-delta, accz, acc);
            p.out[(size_t)i * npieces + col0 / p.piece] = acc;
            if (ADAM) {
              // pieces are whole groups here (the launcher only asks for this then): acc is
              // the final dS of scale (i, group), owned by this thread alone
              const size_t e = (size_t)i * npieces + col0 / p.piece;
              float sv = p.adam_s[e], mv = p.adam_m[e], vv = p.adam_v[e];
              adamw_update(sv, acc, mv, vv, p.adam);
              p.adam_s[e] = sv;
              p.adam_m[e] = mv;
              p.adam_v[e] = vv;
            }
            if (DZ) {
              // a piece that is a whole group is dZ itself: -s * sum of dW; otherwise the
              // reduction kernel applies -s after adding the pieces
              const float f = p.piece == p.g ? -__ldg(p.scales + (size_t)i * p.G + col0 / p.g) : 1.0f;
              p.out_z[(size_t)i * npieces + col0 / p.piece] = f * accz;
            }
          }
          acc = 0.0f;
          accz = 0.0f;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(buf ? acc_empty_leader1 : acc_empty_leader0);
    }
  }

  if (*abort_flag) drain_after_abort();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // no CTA leaves while its peer may still signal its barriers
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) {
    atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
    p.status[1] = (int)blockIdx.x;
  }
}

// Real-valued zero-point, groups wider than a piece: dS = sum(pieces) - delta * sum(dW pieces)
// and dZ = -s * sum(dW pieces), pieces added in index order.
__global__ void ds_reduce_zf_kernel(const float* __restrict__ partial_s, const float* __restrict__ partial_w,
                                    float* __restrict__ dS, float* __restrict__ dZ, long long n_out,
                                    int pieces_per_group, const float* __restrict__ zeros_f,
                                    const float* __restrict__ scales, int bits) {
  long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_out) return;
  float acc_s = 0.0f, acc_w = 0.0f;
  for (int q = 0; q < pieces_per_group; ++q) {
    acc_s += partial_s[e * pieces_per_group + q];
    acc_w += partial_w[e * pieces_per_group + q];
  }
  uint32_t zi;
  float delta;
  if (bits == 3) dq::split_zero_point<3>(zeros_f[e], zi, delta);
  else dq::split_zero_point<4>(zeros_f[e], zi, delta);
  dS[e] = fmaf(-delta, acc_w, acc_s);
  dZ[e] = -scales[e] * acc_w;
}

// dS[i, gi] = sum of the group's partial pieces, in index order (deterministic); with
// neg_scales the sum is multiplied by -s[i, gi] (the zero-point gradient); with adam_s the
// AdamW step on scale e follows at once.
__global__ void ds_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dS,
                                 long long n_out, int pieces_per_group,
                                 const float* __restrict__ neg_scales, AdamWConsts adam,
                                 float* __restrict__ adam_s, float* __restrict__ adam_m,
                                 float* __restrict__ adam_v) {
  long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_out) return;
  const float* src = partial + e * pieces_per_group;
  float acc = 0.0f;
  for (int q = 0; q < pieces_per_group; ++q) acc += src[q];
  dS[e] = neg_scales ? -neg_scales[e] * acc : acc;
  if (adam_s) {
    float sv = adam_s[e], mv = adam_m[e], vv = adam_v[e];
    adamw_update(sv, acc, mv, vv, adam);
    adam_s[e] = sv;
    adam_m[e] = mv;
    adam_v[e] = vv;
  }
}

// --------------------------------------------------------------- host side

// bf16 row-major [outer, inner] tensor, box = [box_outer rows, 64 elements], 128B swizzle,
// out-of-bounds elements read as zero.
int make_tmap_bf16(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer,
                   uint32_t box_outer) {
  EncodeTiledFn enc = nullptr;
  PEQA_TRY(tensor_map_encoder(&enc));
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {64, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);
  return PEQA_OK;
}

int sm_count(int* n) {
  static thread_local int cached_dev = -1, cached_n = 0;
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev != cached_dev) {
    PEQA_CUDA(cudaDeviceGetAttribute(&cached_n, cudaDevAttrMultiProcessorCount, dev));
    cached_dev = dev;
  }
  *n = cached_n;
  return PEQA_OK;
}

template <typename Kern>
int set_smem(Kern k) {
  PEQA_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
  return PEQA_OK;
}

template <int BITS, bool TRANS, bool FOLD, bool PKTMA>
int launch_qgemm_k(const CUtensorMap& tmap, const CUtensorMap& tmap_pk, const QGemmParams& p,
                   int grid, cudaStream_t st) {
  auto kern = qgemm_kernel<BITS, TRANS, FOLD, PKTMA>;
  PEQA_TRY(set_smem(kern));
  kern<<<grid, kQgemmThreads, SMEM_BYTES, st>>>(tmap, tmap_pk, p);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

template <int BITS, bool TRANS, bool FOLD>
int launch_qgemm_t(const CUtensorMap& tmap, const CUtensorMap& tmap_pk, bool pktma,
                   const QGemmParams& p, int grid, cudaStream_t st) {
  return pktma ? launch_qgemm_k<BITS, TRANS, FOLD, true>(tmap, tmap_pk, p, grid, st)
               : launch_qgemm_k<BITS, TRANS, FOLD, false>(tmap, tmap_pk, p, grid, st);
}

int launch_qgemm(const peqa_qweight_t* w, const float* zeros_f, int g, const void* act, int T,
                 void* out, bool trans, cudaStream_t st) {
  QGemmParams p;
  p.qw = w->qweight;
  p.zeros = w->zeros;
  p.zeros_f = zeros_f;
  p.scales = w->scales;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  p.g_shift = -1;
  for (int b = 5; b < 31; ++b)
    if ((1 << b) == g) p.g_shift = b;
  p.T = T;
  p.wpr = p.K * w->bits / 32;
  p.R = trans ? p.K : p.N;
  p.C = trans ? p.N : p.K;
  p.r_tiles = (p.R + BM - 1) / BM;
  p.t_tiles = (T + BN - 1) / BN;
  p.k_blocks = (p.C + BK - 1) / BK;
  PEQA_TRY(status_word(st, &p.status));
  CUtensorMap tmap;
  PEQA_TRY(make_tmap_bf16(&tmap, act, (uint64_t)p.C, (uint64_t)T, BN));
  int sms = 0;
  PEQA_TRY(sm_count(&sms));
  const int tiles = p.r_tiles * p.t_tiles;
  const int grid = tiles < sms ? tiles : sms;
  const bool fold = trans || p.G > 1 || zeros_f != nullptr;
  // Packed codes by TMA need a 16-byte row pitch: always true for 4-bit, K % 128 == 0 for 3-bit.
  const bool pktma = ((size_t)p.wpr * 4) % 16 == 0;
  CUtensorMap tmap_pk = tmap;
  if (pktma) {
    EncodeTiledFn enc = nullptr;
    PEQA_TRY(tensor_map_encoder(&enc));
    cuuint64_t dims[2] = {(cuuint64_t)p.wpr, (cuuint64_t)p.N};
    cuuint64_t strides[1] = {(cuuint64_t)p.wpr * 4};
    cuuint32_t box[2] = {trans ? (cuuint32_t)(4 * w->bits) : 8u, trans ? 64u : 128u};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap_pk, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(w->qweight), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  if (w->bits == 4) {
    if (trans) return launch_qgemm_t<4, true, true>(tmap, tmap_pk, pktma, p, grid, st);
    return fold ? launch_qgemm_t<4, false, true>(tmap, tmap_pk, pktma, p, grid, st)
                : launch_qgemm_t<4, false, false>(tmap, tmap_pk, pktma, p, grid, st);
  }
  if (trans) return launch_qgemm_t<3, true, true>(tmap, tmap_pk, pktma, p, grid, st);
  return fold ? launch_qgemm_t<3, false, true>(tmap, tmap_pk, pktma, p, grid, st)
              : launch_qgemm_t<3, false, false>(tmap, tmap_pk, pktma, p, grid, st);
}

int gcd_int(int a, int b) { return b == 0 ? a : gcd_int(b, a % b); }

// Columns per dS output piece: the largest of {32, 64, 128} that divides g, so
// that a piece never crosses a group or a 128-column epilogue half.
int ds_piece(int g) { return gcd_int(g, 128); }

}  // namespace

int launch_fwd(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, int T, void* Y,
               cudaStream_t st) {
  if (fwd_pair_supported(w)) return launch_fwd_pair(w, zeros_f, g, X, T, Y, st);
  return launch_qgemm(w, zeros_f, g, X, T, Y, false, st);
}

int launch_dx(const peqa_qweight_t* w, const float* zeros_f, int g, const void* dY, int T, void* dX,
              cudaStream_t st) {
  if (dx_pair_supported(w)) return launch_dx_pair(w, zeros_f, g, dY, T, dX, st);
  return launch_qgemm(w, zeros_f, g, dY, T, dX, true, st);
}

size_t ds_workspace_bytes(const peqa_qweight_t* w, int g, int T) {
  (void)T;
  const int piece = ds_piece(g);
  if (piece == g) return 0;
  return (size_t)w->out_features * (size_t)(w->in_features / piece) * sizeof(float);
}

// with dZ: a second array of partial sums behind the first
size_t dsdz_workspace_bytes(const peqa_qweight_t* w, int g, int T) {
  return 2 * ds_workspace_bytes(w, g, T);
}

int launch_ds(const peqa_qweight_t* w, const float* zeros_f, int g, const void* X, const void* dY,
              int T, float* dS, float* dZ, const DsAdam* adam, void* workspace,
              size_t workspace_bytes, cudaStream_t st) {
  if (adam && dZ) return PEQA_ERR_BAD_SHAPE;   // dZ reads the scales the step would be rewriting
  if (zeros_f && !dZ) return PEQA_ERR_NULL;    // the correction needs the sums dZ is made of
  (void)workspace_bytes;
  DsParams p;
  p.qw = w->qweight;
  p.zeros = w->zeros;
  p.zeros_f = zeros_f;
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  p.T = T;
  p.wpr = p.K * w->bits / 32;
  p.piece = ds_piece(g);
  const bool direct = (p.piece == g);
  p.out = direct ? dS : static_cast<float*>(workspace);
  p.scales = w->scales;
  const size_t n_pieces = (size_t)p.N * (size_t)(p.K / p.piece);
  p.out_z = dZ ? (direct ? dZ : static_cast<float*>(workspace) + n_pieces) : nullptr;
  p.adam = adam ? adam->c : AdamWConsts{};
  p.adam_s = adam ? adam->scales : nullptr;
  p.adam_m = adam ? adam->m : nullptr;
  p.adam_v = adam ? adam->v : nullptr;
  const bool adam_in_kernel = adam && direct;
  p.i_tiles = (p.N + 2 * BM - 1) / (2 * BM);   // 256-row pair tiles
  p.j_tiles = (p.K + BN - 1) / BN;
  p.k_blocks = (T + BK - 1) / BK;
  {
    // a band of about 32 MiB of one operand; band the dimension that gives less HBM traffic:
    // rows: dY once + X once per band of rows; columns: X once + dY once per band of columns
    int band = (int)((32u << 20) / ((size_t)512 * (size_t)T));
    band = band < 1 ? 1 : band;
    const double by_rows = (double)p.N + (double)p.K * ((p.i_tiles + band - 1) / band);
    const double by_cols = (double)p.K + (double)p.N * ((p.j_tiles + band - 1) / band);
    p.band_rows = by_rows <= by_cols ? 1 : 0;
    const int dim = p.band_rows ? p.i_tiles : p.j_tiles;
    p.band = band < dim ? band : dim;
  }
  PEQA_TRY(status_word(st, &p.status));
  CUtensorMap tmap_dy, tmap_x;
  PEQA_TRY(make_tmap_bf16(&tmap_dy, dY, (uint64_t)p.N, (uint64_t)T, BK));
  PEQA_TRY(make_tmap_bf16(&tmap_x, X, (uint64_t)p.K, (uint64_t)T, BK));
  int sms = 0;
  PEQA_TRY(sm_count(&sms));
  const int tiles = p.i_tiles * p.j_tiles;
  const int max_pairs = sms / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kDsThreads, 1, 1);
  cfg.dynamicSmemBytes = DS_SMEM_BYTES;
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
#define PEQA_DS_LAUNCH(B, Z, A)                                                                       \
  do {                                                                                               \
    auto kern = ds_kernel<B, Z, A>;                                                                  \
    PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,                \
                                   DS_SMEM_BYTES));                                                  \
    PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, tmap_dy, tmap_x, p));                                   \
  } while (0)
  if (w->bits == 4) {
    if (dZ) PEQA_DS_LAUNCH(4, true, false);
    else if (adam_in_kernel) PEQA_DS_LAUNCH(4, false, true);
    else PEQA_DS_LAUNCH(4, false, false);
  } else {
    if (dZ) PEQA_DS_LAUNCH(3, true, false);
    else if (adam_in_kernel) PEQA_DS_LAUNCH(3, false, true);
    else PEQA_DS_LAUNCH(3, false, false);
  }
#undef PEQA_DS_LAUNCH
  if (!direct) {
    const long long n_out = (long long)p.N * p.G;
    const int ppg = g / p.piece;
    const int blocks = (int)((n_out + 255) / 256);
    if (zeros_f) {
      ds_reduce_zf_kernel<<<blocks, 256, 0, st>>>(p.out, p.out_z, dS, dZ, n_out, ppg, zeros_f, w->scales,
                                                  w->bits);
      PEQA_CUDA(cudaGetLastError());
      return PEQA_OK;
    }
    ds_reduce_kernel<<<blocks, 256, 0, st>>>(p.out, dS, n_out, ppg, nullptr, p.adam, p.adam_s,
                                             p.adam_m, p.adam_v);
    PEQA_CUDA(cudaGetLastError());
    if (dZ) {
      ds_reduce_kernel<<<blocks, 256, 0, st>>>(p.out_z, dZ, n_out, ppg, w->scales, AdamWConsts{},
                                               nullptr, nullptr, nullptr);
      PEQA_CUDA(cudaGetLastError());
    }
  }
  return PEQA_OK;
}

}  // namespace peqa
