// Small-batch forward (token generation): Y[m,i] = sum_j X[m,j] * s[i,g(j)] * (Q[i,j] - z[i,g(j)])
// for M <= 16 tokens: the cluster kernel, used for groups narrower than 128
// columns and for batches whose activations do not fit the streaming kernel's
// staging (decode_stream.cu serves the rest).  The packed weights are read from
// HBM exactly once, by TMA into a two-slot ring per CTA.
//
// Work split: a CTA owns 128 weight rows and one slice of the K range; the
// CTAs that share the same rows form a thread-block cluster along K and add
// their partial sums through distributed shared memory in rank order, so the
// result is deterministic and needs neither atomics nor a workspace.
//
// Inside a CTA each warp owns 32 rows.  The multiply-accumulate runs on the
// warp-level tensor-core instruction mma.m16n8k16 with the *weights* as the
// 16-row operand and the tokens as the 8-wide operand (M <= 8: one MMA per 16
// rows; M <= 16: two).  Lane (g, c) = (lane/4, lane%4) streams 128 consecutive
// codes of rows g and g+8 per step (48 B for 3-bit, 64 B for 4-bit), so the
// four lanes of a row read one contiguous 192/256-byte run.  Codes become bf16
// pairs (column k, column k+4) with one shift/funnel-shift, one logic op and
// one bf16x2 subtract (see dequant.cuh); the contraction order inside an MMA is
// free, so the activations are simply stored in shared memory in that same
// pair order and no register permutation is needed.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include <cuda.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace cg = cooperative_groups;

namespace peqa {

namespace {

constexpr int kDecWarps = 4;                            // compute warps
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecBlock = kDecThreads + 32;             // + one warp that issues the TMA copies
constexpr int kDecSlots = 2;                            // weight steps in flight per CTA
constexpr int kDecBoxBytes = 128 * 64;                  // one TMA box: 128 rows x 16 words
constexpr int kRowsPerWarp = 32;
constexpr int kRowsPerCta = kDecWarps * kRowsPerWarp;   // 128
constexpr int kStepCols = 512;                          // columns per warp step (4 lanes x 128)
constexpr int kBlockBytes = 288;                        // 128 activations (256 B) + 32 B bank skew
constexpr int kMaxSplit = 8;                            // portable cluster size

struct DecodeParams {
  const uint32_t* qw;
  const uint8_t* zeros;
  const float* scales;
  const __nv_bfloat16* X;   // [M, K]
  __nv_bfloat16* Y;         // [M, N]
  int N, K, G, g, M;
  int wpr;                  // packed words per row
  int total_steps;          // ceil(K / 512)
  int split;                // CTAs per cluster along K
  int x_pitch;              // bytes between token rows of the staged activations
  int* status;
};

struct DecBarriers {
  uint64_t full[kDecSlots];    // weight step landed in its slot
  uint64_t empty[kDecSlots];   // all compute warps have read the slot
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
      "{%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// 128 consecutive codes of one row: WORDS = 4 * BITS packed words.
template <int BITS>
struct RowChunk {
  uint4 v[BITS];
};

template <int BITS>
__device__ __forceinline__ void unit_words(const RowChunk<BITS>& r, int u, uint32_t (&w)[BITS]) {
  const uint32_t* flat = reinterpret_cast<const uint32_t*>(r.v);
#pragma unroll
  for (int q = 0; q < BITS; ++q) w[q] = flat[u * BITS + q];
}

// The two bf16x2 registers one lane contributes to one MMA for one weight row:
// pairs (8*BLK + E, +4) and (8*BLK + E + 1, +4).
template <int BITS, int BLK, int E, bool FOLD>
__device__ __forceinline__ void two_pairs(const uint32_t (&w)[BITS], uint32_t zc, uint32_t s2,
                                          uint32_t& p0, uint32_t& p1) {
  // Per-channel layers (!FOLD) feed the biased values (bias + q) straight to the MMA and
  // take the (bias + z) * sum(x) term out of the result at the end: one operation less
  // per pair in the loop that decides whether the weight stream can be kept up with.
  p0 = dq::pair_raw<BITS, 8 * BLK + E>(w);
  p1 = dq::pair_raw<BITS, 8 * BLK + E + 1>(w);
  if (FOLD) {
    p0 = dq::bf162_mul(dq::bf162_sub(p0, zc), s2);
    p1 = dq::bf162_mul(dq::bf162_sub(p1, zc), s2);
  }
}

template <int BITS, int NT, bool FOLD>
__global__ void __launch_bounds__(kDecBlock, BITS == 3 ? 4 : 3)
decode_kernel(const __grid_constant__ CUtensorMap tmap_q, const DecodeParams p) {
  extern __shared__ uint8_t dec_smem_raw[];
  // layout: [weight slots: kDecSlots x BITS boxes of 8 KiB, 64-byte-swizzled]
  //         [staged activations: M rows of x_pitch bytes][partials: 128 rows x (8*NT) fp32]
  //         [activation sums 2 x 16 fp32][barriers]
  constexpr int kStepBytes = BITS * kDecBoxBytes;     // 512 columns of 128 rows
  uint8_t* slots = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dec_smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  uint8_t* dec_smem = slots + kDecSlots * kStepBytes;
  const int rank = blockIdx.y;   // position along K inside the cluster
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, c4 = lane & 3;
  const bool is_producer = warp == kDecWarps;

  const int steps_lo = (int)(((long long)p.total_steps * rank) / p.split);
  const int steps_hi = (int)(((long long)p.total_steps * (rank + 1)) / p.split);
  const int kbeg = steps_lo * kStepCols;
  const int nsteps = steps_hi - steps_lo;

  uint8_t* xs = dec_smem;
  float* partial = reinterpret_cast<float*>(dec_smem + (((size_t)p.M * p.x_pitch + 15) & ~(size_t)15));
  DecBarriers* bars = reinterpret_cast<DecBarriers*>(partial + kRowsPerCta * 8 * NT + 32);
  volatile int* abort_flag = &bars->abort_flag;

  // One weight step (128 rows x 512 columns) = BITS boxes of 16 words x 128 rows.
  auto issue_step = [&](int st) {
    const int slot = st % kDecSlots;
    const uint32_t bar = ptx::smem_u32(&bars->full[slot]);
    ptx::mbar_arrive_expect_tx(bar, kStepBytes);
#pragma unroll
    for (int b = 0; b < BITS; ++b)
      ptx::tma_load_2d(ptx::smem_u32(slots + slot * kStepBytes + b * kDecBoxBytes), &tmap_q, bar,
                       (steps_lo + st) * (16 * BITS) + 16 * b, blockIdx.x * kRowsPerCta);
  };
  if (is_producer && lane == 0) {
    // The weight copies are requested before anything else: they do not depend on the
    // activations, so their latency overlaps the staging below.
    ptx::prefetch_tmap(&tmap_q);
    for (int q = 0; q < kDecSlots; ++q) {
      ptx::mbar_init(ptx::smem_u32(&bars->full[q]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->empty[q]), kDecWarps);
    }
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    ptx::fence_mbar_init();
    for (int st = 0; st < nsteps && st < kDecSlots; ++st) issue_step(st);
  }

  // The first weight chunks are requested before anything else: they do not depend on
  // the activations, so their latency overlaps the staging below.
  const int row_base = blockIdx.x * kRowsPerCta + warp * kRowsPerWarp;
  // rows of this lane: fragment rows g and g+8 of the two 16-row blocks
  int rows[4] = {row_base + g8, row_base + g8 + 8, row_base + 16 + g8, row_base + 24 + g8};

  float acc[2][NT][4];
#pragma unroll
  for (int rb = 0; rb < 2; ++rb)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[rb][nt][e] = 0.0f;

  float z_row[4] = {0.f, 0.f, 0.f, 0.f};   // per-channel zero-points of this lane's rows
  if (!FOLD) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
      if (rows[r] < p.N) z_row[r] = (float)__ldg(p.zeros + rows[r]);
  }

  // token rows this lane reads as the MMA "B" operand (token index = lane / 4);
  // lanes beyond M read row 0: their accumulator columns are never stored.
  const uint8_t* xrow0 = xs + (size_t)(g8 < p.M ? g8 : 0) * p.x_pitch;
  const uint8_t* xrow1 = xs + (size_t)(g8 + 8 < p.M ? g8 + 8 : 0) * p.x_pitch;

  RowChunk<BITS> cur[4];
  // Where this lane's 16-byte pieces of a step sit in a slot: word w of the step's row is
  // in box w/16, 16-byte chunk (w%16)/4, and the 64-byte swizzle XORs the chunk index with
  // bits 1-2 of the row (equal for the lane's four rows, which differ by multiples of 8).
  uint32_t piece_off[BITS];
#pragma unroll
  for (int q = 0; q < BITS; ++q) {
    const int w = 4 * BITS * c4 + 4 * q;
    piece_off[q] = (uint32_t)((w >> 4) * kDecBoxBytes + ((((w & 15) >> 2) ^ ((g8 >> 1) & 3)) << 4));
  }
  const uint32_t row_off0 = (uint32_t)(warp * kRowsPerWarp + g8) * 64u;   // local rows g8, +8, +16, +24

  // ---- stage the activation slice: blocks of 8 columns stored as (0,4,1,5,2,6,3,7)
  {
    const int blocks8 = nsteps * (kStepCols / 8);
    for (int idx = threadIdx.x; idx < p.M * blocks8; idx += kDecBlock) {
      const int m = idx / blocks8;
      const int b8 = idx - m * blocks8;
      const int col = kbeg + b8 * 8;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (col < p.K) v = __ldg(reinterpret_cast<const uint4*>(p.X + (size_t)m * p.K + col));
      const int lcol = b8 * 8;
      uint8_t* dst = xs + (size_t)m * p.x_pitch + (lcol >> 7) * kBlockBytes + (lcol & 127) * 2;
      *reinterpret_cast<uint2*>(dst) =
          make_uint2(dq::prmt(v.x, v.z, 0x5410u), dq::prmt(v.x, v.z, 0x7632u));
      *reinterpret_cast<uint2*>(dst + 8) =
          make_uint2(dq::prmt(v.y, v.w, 0x5410u), dq::prmt(v.y, v.w, 0x7632u));
    }
  }
  __syncthreads();

  // Per-channel path: sums of the staged activations over the columns that land in the
  // low and in the high half of the bf16 pairs (they carry different biases).  In the
  // staged order every 32-bit word is one (low, high) pair.  Fixed summation order.
  float* xsum = partial + kRowsPerCta * 8 * NT;   // [2][16]
  if (!FOLD && !is_producer) {
    for (int m = warp; m < p.M; m += kDecWarps) {
      const uint8_t* xr = xs + (size_t)m * p.x_pitch;
      float lo = 0.f, hi = 0.f;
      for (int blk = 0; blk < nsteps * 4; ++blk) {
        const uint32_t* wds = reinterpret_cast<const uint32_t*>(xr + blk * kBlockBytes);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t v = wds[lane + 32 * h];
          lo += __uint_as_float(v << 16);
          hi += __uint_as_float(v & 0xFFFF0000u);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        lo += __shfl_xor_sync(0xffffffffu, lo, o);
        hi += __shfl_xor_sync(0xffffffffu, hi, o);
      }
      if (lane == 0) { xsum[m] = lo; xsum[16 + m] = hi; }
    }
  }

  if (is_producer) {
    // keep the slots full: step st goes into slot st % kDecSlots once every compute warp
    // has finished with the step that was there
    if (lane == 0) {
      for (int st = kDecSlots; st < nsteps; ++st) {
        const int slot = st % kDecSlots;
        if (!ptx::mbar_wait(ptx::smem_u32(&bars->empty[slot]), ((st / kDecSlots) & 1u) ^ 1u, abort_flag)) break;
        issue_step(st);
      }
    }
  } else
  for (int st = 0; st < nsteps; ++st) {
    const int col0 = kbeg + st * kStepCols + c4 * 128;   // first column of this lane's chunk
    const int slot = st % kDecSlots;
    if (!ptx::mbar_wait(ptx::smem_u32(&bars->full[slot]), (st / kDecSlots) & 1u, abort_flag)) break;
    {
      const uint8_t* sb = slots + slot * kStepBytes + row_off0;
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int q = 0; q < BITS; ++q)
          cur[r].v[q] = *reinterpret_cast<const uint4*>(sb + r * (8 * 64) + piece_off[q]);
    }
    const int xoff = (st * 4 + c4) * kBlockBytes;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      uint32_t w[4][BITS];
      uint32_t zc[4], s2[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        unit_words<BITS>(cur[r], u, w[r]);
        if (FOLD) {
          const int col = col0 + u * 32;
          uint32_t z = 0u;
          float s = 0.0f;
          if (rows[r] < p.N && col < p.K) {
            const size_t gi = (size_t)rows[r] * p.G + col / p.g;
            z = __ldg(p.zeros + gi);
            s = __ldg(p.scales + gi);
          }
          zc[r] = dq::zero_const<BITS>(z);
          s2[r] = dq::bf162_broadcast(s);
        } else {
          zc[r] = 0u;
          s2[r] = 0u;
        }
      }
#pragma unroll
      for (int blk = 0; blk < 4; ++blk) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          // activations of pairs (2*hh, 2*hh+1) of this 8-column block
          const int xo = xoff + u * 64 + blk * 16 + hh * 8;
          const uint2 b0 = *reinterpret_cast<const uint2*>(xrow0 + xo);
          uint2 b1 = make_uint2(0u, 0u);
          if (NT == 2) b1 = *reinterpret_cast<const uint2*>(xrow1 + xo);
#pragma unroll
          for (int rb = 0; rb < 2; ++rb) {
            uint32_t a[4];
            if (hh == 0) {
              if (blk == 0) { two_pairs<BITS, 0, 0, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 0, 0, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 1) { two_pairs<BITS, 1, 0, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 1, 0, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 2) { two_pairs<BITS, 2, 0, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 2, 0, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 3) { two_pairs<BITS, 3, 0, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 3, 0, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
            } else {
              if (blk == 0) { two_pairs<BITS, 0, 2, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 0, 2, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 1) { two_pairs<BITS, 1, 2, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 1, 2, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 2) { two_pairs<BITS, 2, 2, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 2, 2, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
              if (blk == 3) { two_pairs<BITS, 3, 2, FOLD>(w[2 * rb], zc[2 * rb], s2[2 * rb], a[0], a[2]);
                              two_pairs<BITS, 3, 2, FOLD>(w[2 * rb + 1], zc[2 * rb + 1], s2[2 * rb + 1], a[1], a[3]); }
            }
            mma_16816(acc[rb][0], a, b0.x, b0.y);
            if (NT == 2) mma_16816(acc[rb][1], a, b1.x, b1.y);
          }
        }
      }
    }
    // the codes of this step are in registers and consumed: hand the slot back
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->empty[slot]));
  }

  // ---- partial sums of this CTA: [128 rows][8*NT tokens]
  constexpr int TOK = 8 * NT;
  if (!FOLD) __syncthreads();   // xsum of every token is written
  constexpr float kBiasLo = BITS == 4 ? 128.0f : 8.0f;
  if (!is_producer)
#pragma unroll
  for (int rb = 0; rb < 2; ++rb)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int lr = warp * kRowsPerWarp + rb * 16 + g8;
      const int tk = nt * 8 + c4 * 2;
      float c00 = 0.f, c01 = 0.f, c10 = 0.f, c11 = 0.f;
      if (!FOLD) {
        // (bias + z) * sum(x) over this CTA's K slice, per row and token
        const float lo0 = tk < p.M ? xsum[tk] : 0.f, hi0 = tk < p.M ? xsum[16 + tk] : 0.f;
        const float lo1 = tk + 1 < p.M ? xsum[tk + 1] : 0.f, hi1 = tk + 1 < p.M ? xsum[16 + tk + 1] : 0.f;
        const float za = z_row[2 * rb], zb = z_row[2 * rb + 1];
        c00 = (kBiasLo + za) * lo0 + (128.0f + za) * hi0;
        c01 = (kBiasLo + za) * lo1 + (128.0f + za) * hi1;
        c10 = (kBiasLo + zb) * lo0 + (128.0f + zb) * hi0;
        c11 = (kBiasLo + zb) * lo1 + (128.0f + zb) * hi1;
      }
      partial[lr * TOK + tk] = acc[rb][nt][0] - c00;
      partial[lr * TOK + tk + 1] = acc[rb][nt][1] - c01;
      partial[(lr + 8) * TOK + tk] = acc[rb][nt][2] - c10;
      partial[(lr + 8) * TOK + tk + 1] = acc[rb][nt][3] - c11;
    }

  // ---- add the K-slices of the cluster in rank order and write Y
  const int rows_per_rank = kRowsPerCta / p.split;
  if (p.split > 1) {
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    for (int idx = threadIdx.x; idx < rows_per_rank * p.M; idx += kDecBlock) {
      const int m = idx / rows_per_rank;
      const int lr = rank * rows_per_rank + (idx - m * rows_per_rank);
      const int row = blockIdx.x * kRowsPerCta + lr;
      float sum = 0.0f;
      for (int r = 0; r < p.split; ++r) {
        const float* remote = cluster.map_shared_rank(partial, r);
        sum += remote[lr * TOK + m];
      }
      if (row < p.N) {
        if (!FOLD) sum *= __ldg(p.scales + row);
        p.Y[(size_t)m * p.N + row] = __float2bfloat16_rn(sum);
      }
    }
    cluster.sync();   // keep every CTA's shared memory alive until all ranks have read it
  } else {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kRowsPerCta * p.M; idx += kDecBlock) {
      const int m = idx / kRowsPerCta;
      const int lr = idx - m * kRowsPerCta;
      const int row = blockIdx.x * kRowsPerCta + lr;
      if (row < p.N) {
        float sum = partial[lr * TOK + m];
        if (!FOLD) sum *= __ldg(p.scales + row);
        p.Y[(size_t)m * p.N + row] = __float2bfloat16_rn(sum);
      }
    }
  }
  if (threadIdx.x == 0 && bars->abort_flag) atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
}

int sm_count_cached(int* n) {
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

template <int BITS, int NT, bool FOLD>
int launch_decode_t(const CUtensorMap& tmap_q, const DecodeParams& p, int row_blocks, size_t smem,
                    cudaStream_t st) {
  auto kern = decode_kernel<BITS, NT, FOLD>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(row_blocks, p.split, 1);
  cfg.blockDim = dim3(kDecBlock, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = p.split;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, tmap_q, p));
  return PEQA_OK;
}

}  // namespace

size_t decode_workspace_bytes(const peqa_qweight_t*, int, int) { return 0; }

int launch_decode(const peqa_qweight_t* w, int g, const void* X, int M, void* Y,
                  void* workspace, size_t workspace_bytes, cudaStream_t st) {
  (void)workspace; (void)workspace_bytes;
  if (decode_stream_supported(w, g, M)) return launch_decode_stream(w, g, X, M, Y, nullptr, 1, nullptr, st);
  DecodeParams p;
  p.qw = w->qweight;
  p.zeros = w->zeros;
  p.scales = w->scales;
  p.X = static_cast<const __nv_bfloat16*>(X);
  p.Y = static_cast<__nv_bfloat16*>(Y);
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  p.M = M;
  p.wpr = p.K * w->bits / 32;
  p.total_steps = (p.K + kStepCols - 1) / kStepCols;

  int sms = 0;
  PEQA_TRY(sm_count_cached(&sms));
  const int row_blocks = (p.N + kRowsPerCta - 1) / kRowsPerCta;
  // Enough CTAs for about three waves of the machine, split a power of two <= 8.
  int split = 1;
  while (split < kMaxSplit && row_blocks * split < 3 * sms && split * 2 <= p.total_steps) split *= 2;
  const int NT = M <= 8 ? 1 : 2;
  size_t smem = 0;
  for (;;) {
    p.split = split;
    const int max_steps = (p.total_steps + split - 1) / split;
    const int nblk = max_steps * (kStepCols / 128);
    // pitch = nblk*288 + pad with pitch % 128 == 8: consecutive tokens land 2 banks apart
    const int pad = ((8 - (nblk * kBlockBytes) % 128) % 128 + 128) % 128;
    p.x_pitch = nblk * kBlockBytes + pad;
    smem = 1024 /*alignment*/ + (size_t)kDecSlots * w->bits * kDecBoxBytes /*weight slots*/ +
           (((size_t)M * p.x_pitch + 15) & ~(size_t)15) + (size_t)kRowsPerCta * 8 * NT * sizeof(float) +
           32 * sizeof(float) /*activation sums*/ + sizeof(DecBarriers) + 16;
    if (smem <= 200 * 1024 || split == kMaxSplit) break;
    split *= 2;
  }
  if (smem > 227 * 1024) return PEQA_ERR_TOO_LARGE;
  PEQA_TRY(status_word(st, &p.status));
  // packed matrix as uint32 [N, wpr]; box = 16 words x 128 rows, 64-byte swizzle
  CUtensorMap tmap_q;
  {
    EncodeTiledFn enc = nullptr;
    PEQA_TRY(tensor_map_encoder(&enc));
    cuuint64_t dims[2] = {(cuuint64_t)p.wpr, (cuuint64_t)p.N};
    cuuint64_t strides[1] = {(cuuint64_t)p.wpr * 4};
    cuuint32_t box[2] = {16, (cuuint32_t)kRowsPerCta};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap_q, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(w->qweight), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  const bool fold = p.G > 1;
  if (w->bits == 4) {
    if (NT == 1) return fold ? launch_decode_t<4, 1, true>(tmap_q, p, row_blocks, smem, st)
                             : launch_decode_t<4, 1, false>(tmap_q, p, row_blocks, smem, st);
    return fold ? launch_decode_t<4, 2, true>(tmap_q, p, row_blocks, smem, st)
                : launch_decode_t<4, 2, false>(tmap_q, p, row_blocks, smem, st);
  }
  if (NT == 1) return fold ? launch_decode_t<3, 1, true>(tmap_q, p, row_blocks, smem, st)
                           : launch_decode_t<3, 1, false>(tmap_q, p, row_blocks, smem, st);
  return fold ? launch_decode_t<3, 2, true>(tmap_q, p, row_blocks, smem, st)
              : launch_decode_t<3, 2, false>(tmap_q, p, row_blocks, smem, st);
}

}  // namespace peqa
