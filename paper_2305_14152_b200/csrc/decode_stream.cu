// Small-batch forward (token generation), streaming variant:
//   Y[m,i] = sum_j X[m,j] * s[i,g(j)] * (Q[i,j] - z[i,g(j)])      (Eq. 2, M <= 16 tokens)
// for layers with one scale per channel or with groups that are multiples of
// 128 columns, when the staged activations fit in shared memory.
//
// The packed weights are read exactly once, and the design goal is that every
// byte a CTA will need is requested from HBM within the first microsecond:
//   * one CTA per SM owns a contiguous range of rows (a multiple of 8) and all
//     of K for them, so no sum crosses a CTA and there is no workspace;
//   * four producer warps copy the range into a ring in shared memory with
//     16-byte asynchronous copies through the load/store unit, a step of 32
//     rows x 512 columns of codes (192 B per row for 3-bit, 256 B for 4-bit)
//     at a time.  TMA is not used here on purpose: fed by TMA boxes the same
//     ring filled at about 2 TB/s over the whole GPU, whatever the box shape,
//     while the load/store path keeps the whole ring in flight.  A thread can
//     track only a few batches of such copies at a time, so a producer warp
//     issues a whole step (12 or 16 copies per lane) per tracked arrival.  The
//     ring has up to 32 steps (about 190 KiB), which for the shapes of a
//     7B-65B model is nearly the CTA's whole range, so the copies hardly ever
//     wait for compute;
//   * rows sit in the ring at a padded pitch (208 / 320 bytes) chosen so that
//     the eight rows a warp reads together fall in different banks.
//
// Sixteen compute warps split K: warp w takes the 512-column steps w, w+16, ...
// of every 32-row block.  The multiply-accumulate is the warp-level
// mma.m16n8k16 with the weights as the 16-row operand, as in the cluster
// kernel; here the four lanes of a row share one 128-column block (32 columns
// each), so all contraction slots of an MMA lie in one quantization group.
// That lets the codes go to the tensor core as the biased integers (bias + q)
// they already are after one logic operation, and the group's zero-point and
// scale are applied to the accumulator once per 128 columns:
//   y += s * (acc - z * sum(x) - sum(bias * x)),
// with both sums per 128-column block tabulated once per CTA.  Because the
// order of the contraction is free here (the activations are staged to match),
// 3-bit codes are taken two pairs per shifted window (stream_lo / stream_hi in
// dequant.cuh), a fifth fewer integer operations than pairing (k, k+4) only.
// The products are exact integers times bf16 in fp32, which is also closer to
// the reference than multiplying by a bf16-rounded scale first.
//
// The warps' partial sums of a 32-row block meet in shared memory and are added
// in warp order, so the result does not depend on timing.
//
// What bounds it: one shift and one logic operation per pair of codes, on the
// integer pipe, which issues at half the rate of the floating-point pipe; for
// 8192 x 8192 3-bit that is about as long as HBM needs for the weights.
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"

namespace peqa {

namespace {

constexpr int kSWarps = 16;                        // compute warps
constexpr int kSThreads = kSWarps * 32;
constexpr int kSProducers = 4;                     // producer warps
constexpr int kSProdThreads = kSProducers * 32;
constexpr int kSBlock = kSThreads + kSProdThreads;
constexpr int kSMaxSlots = 32;
constexpr int kSMaxXLoads = 8;                     // 16-byte activation loads per thread
constexpr int kSStepCols = 512;
constexpr int kSBlockBytes = 288;                  // 128 activations (256 B) + 32 B bank skew
constexpr int kSSmemLimit = 227 * 1024;

template <int BITS>
struct StreamGeom {
  static constexpr int piece = 64 * BITS;                  // bytes of 512 codes of one row
  static constexpr int pitch = BITS == 3 ? 208 : 320;      // row pitch in a ring slot
  static constexpr int cpr = piece / 16;                   // 16-byte chunks per row piece
  static constexpr int slot = 32 * pitch;                  // one step: 32 rows
};

struct StreamParams {
  const uint32_t* qw;
  const uint8_t* zeros;
  const float* scales;
  const __nv_bfloat16* X;   // [M, K]
  __nv_bfloat16* Y;         // [M, N]
  int N, K, G, g, M;
  int wpr;                  // packed words per row
  int nchunks;              // ceil(K / 512)
  int rows_per_cta;         // multiple of 8
  int x_blocks;             // 128-column blocks staged per token (4 * nchunks)
  int x_pitch;              // bytes between staged token rows
  int slots;                // ring depth
  // multi-task decode (one scale per channel only): token m uses the scales at
  // scales + clamp(task_ids[m], 0, n_tasks - 1) * N; task_ids == nullptr: one task
  const int32_t* task_ids;
  int n_tasks;
  int* status;
};

struct StreamBarriers {
  uint64_t full[kSMaxSlots];    // the step's row pieces have landed
  uint64_t empty[kSMaxSlots];   // the warp that owns the step has read it
  int abort_flag;
  int wait_limit_us;    // must follow abort_flag (read by the bounded waits)
};

__device__ __forceinline__ void smma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                           uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
      "{%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// MMA 2*BLK + HH of the lane's 32-column unit (pairs 4*BLK + 2*HH and the next one, see
// stream_lo in dequant.cuh) for both 16-row halves of the 32-row block.
template <int BITS, int NT, int BLK, int HH>
__device__ __forceinline__ void unit_mma(const uint32_t (&w)[4][BITS], const uint8_t* x0,
                                         const uint8_t* x1, float (&acc)[2][NT][4]) {
  const uint2 b0 = *reinterpret_cast<const uint2*>(x0 + BLK * 16 + HH * 8);
  uint2 b1 = make_uint2(0u, 0u);
  if (NT == 2) b1 = *reinterpret_cast<const uint2*>(x1 + BLK * 16 + HH * 8);
#pragma unroll
  for (int rb = 0; rb < 2; ++rb) {
    uint32_t a[4];
    dq::mma_pairs_stream<BITS, 2 * BLK + HH>(w[2 * rb], a[0], a[2]);
    dq::mma_pairs_stream<BITS, 2 * BLK + HH>(w[2 * rb + 1], a[1], a[3]);
    smma_16816(acc[rb][0], a, b0.x, b0.y);
    if (NT == 2) smma_16816(acc[rb][1], a, b1.x, b1.y);
  }
}

template <int BITS, int NT, bool GROUPED>
__global__ void __launch_bounds__(kSBlock, 1)
decode_stream_kernel(const StreamParams p) {
  using Geo = StreamGeom<BITS>;
  constexpr int TOKP = 8 * NT;                       // token columns of the MMAs
  extern __shared__ uint8_t stream_smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(stream_smem_raw) + 127) &
                                             ~static_cast<uintptr_t>(127));
  uint8_t* xs = ring + (size_t)p.slots * Geo::slot;
  float* xtab = reinterpret_cast<float*>(xs + (((size_t)p.M * p.x_pitch + 15) & ~(size_t)15));
  float* xtot = xtab + (size_t)p.x_blocks * TOKP * 2;      // [TOKP][lo, hi] over all of K
  float* partial = xtot + TOKP * 2;                         // [2][kSWarps][32][TOKP]
  StreamBarriers* bars = reinterpret_cast<StreamBarriers*>(partial + 2 * kSWarps * 32 * TOKP);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, c4 = lane & 3;
  const bool is_producer = warp >= kSWarps;
  const int row0 = blockIdx.x * p.rows_per_cta;
  const int row_end = min(p.N, row0 + p.rows_per_cta);
  const int nrb = (row_end - row0 + 31) >> 5;          // 32-row blocks of this CTA
  const int total_steps = nrb * p.nchunks;

  // The activation loads are issued before the weight copies start: behind a CTA's worth
  // of weight traffic they would wait for microseconds, and everything waits for them.
  const int units = p.x_blocks * 4;                    // 32-column units per token, zero past K
  uint4 xv[kSMaxXLoads];
  if (threadIdx.x == kSThreads) {
    for (int q = 0; q < p.slots; ++q) {
      ptx::mbar_init(ptx::smem_u32(&bars->full[q]), 32);   // one arrival per lane of the issuing warp
      ptx::mbar_init(ptx::smem_u32(&bars->empty[q]), 1);
    }
    bars->abort_flag = 0;
    bars->wait_limit_us = p.status[4];
    ptx::fence_mbar_init();
  } else if (!is_producer) {
#pragma unroll
    for (int q = 0; q < kSMaxXLoads / 4; ++q) {
      const int idx = q * kSThreads + threadIdx.x;       // one 32-column unit of one token
      const int m = idx / units;
      const int col = (idx - m * units) * 32;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        xv[4 * q + e] = make_uint4(0u, 0u, 0u, 0u);
        if (m < p.M && col + 8 * e < p.K)
          xv[4 * q + e] = __ldg(reinterpret_cast<const uint4*>(p.X + (size_t)m * p.K + col + 8 * e));
      }
    }
  }
  __syncthreads();

  if (is_producer) {
    // ------------------------------------------------ weight copies
    // Producer warp q issues the steps q, q + 4, ... whole: 12 (16) copies per lane and
    // one tracked arrival.  A thread can keep only a few such tracked batches in flight,
    // so the batches are made as large as a step allows.
    const uint32_t row_bytes = (uint32_t)p.wpr * 4u;
    const uint8_t* qbytes = reinterpret_cast<const uint8_t*>(p.qw);
    for (int s = warp - kSWarps; s < total_steps; s += kSProducers) {
      const int rb = s / p.nchunks, ch = s - rb * p.nchunks;
      const int slot = s % p.slots;
      if (s >= p.slots) {
        int good = 1;
        if (lane == 0)
          good = ptx::mbar_wait(ptx::smem_u32(&bars->empty[slot]), (((uint32_t)(s / p.slots)) & 1u) ^ 1u,
                                abort_flag) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) break;
      }
      const int rbase = row0 + rb * 32;
      const uint32_t off = (uint32_t)ch * Geo::piece;
      uint8_t* sdst = ring + (size_t)slot * Geo::slot;
      // rows beyond the CTA's range and chunks beyond the end of a row are not copied:
      // whatever the slot holds there meets accumulator rows that are never stored, or
      // activations that were staged as zero
#pragma unroll
      for (int c = lane; c < 32 * Geo::cpr; c += 32) {
        const int row = c / Geo::cpr, k = c - row * Geo::cpr;
        if (rbase + row < row_end && off + 16u * k < row_bytes)
          ptx::cp_async_16(ptx::smem_u32(sdst + row * Geo::pitch + 16 * k),
                           qbytes + (size_t)(rbase + row) * row_bytes + off + 16u * k);
      }
      ptx::cp_async_mbar_arrive_noinc(ptx::smem_u32(&bars->full[slot]));
    }
  } else {
    // ------------------------------------------------ stage the activations
    // A unit of 32 columns is stored as its 16 pairs (low column, high column) in the order
    // in which the weights' pairs come out of the packed codes (stream_lo, stream_hi), so that MMA
    // m of a unit reads its four activations as one 8-byte word; columns beyond K are zero.
#pragma unroll
    for (int q = 0; q < kSMaxXLoads / 4; ++q) {
      const int idx = q * kSThreads + threadIdx.x;
      const int m = idx / units;
      const int col = (idx - m * units) * 32;
      if (m < p.M) {
        const uint32_t src[16] = {xv[4 * q].x, xv[4 * q].y, xv[4 * q].z, xv[4 * q].w,
                                  xv[4 * q + 1].x, xv[4 * q + 1].y, xv[4 * q + 1].z, xv[4 * q + 1].w,
                                  xv[4 * q + 2].x, xv[4 * q + 2].y, xv[4 * q + 2].z, xv[4 * q + 2].w,
                                  xv[4 * q + 3].x, xv[4 * q + 3].y, xv[4 * q + 3].z, xv[4 * q + 3].w};
        uint32_t outw[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int lo = dq::stream_lo(BITS, k), hi = dq::stream_hi(BITS, k);
          // bytes 0-1: column lo (half lo % 2 of its word), bytes 2-3: column hi
          const uint32_t sel = (uint32_t)(2 * (lo & 1)) | ((uint32_t)(2 * (lo & 1) + 1) << 4) |
                               ((uint32_t)(4 + 2 * (hi & 1)) << 8) | ((uint32_t)(5 + 2 * (hi & 1)) << 12);
          outw[k] = dq::prmt(src[lo >> 1], src[hi >> 1], sel);
        }
        // token rows are 8-byte aligned only (their pitch is skewed by 8 bytes)
        uint2* dst = reinterpret_cast<uint2*>(xs + (size_t)m * p.x_pitch + (col >> 7) * kSBlockBytes +
                                              (col & 127) * 2);
#pragma unroll
        for (int e = 0; e < 8; ++e) dst[e] = make_uint2(outw[2 * e], outw[2 * e + 1]);
      }
    }
    // entries of tokens beyond M are read by the lanes that hold those (unused) columns
    for (int idx = threadIdx.x; idx < p.x_blocks * TOKP * 2; idx += kSThreads) xtab[idx] = 0.0f;
    ptx::named_barrier_sync(1, kSThreads);
    // Per 128-column block and token: S = sum of the staged activations and B = sum of
    // (bias of the code that meets it) * activation.  The MMAs see (bias + q), so what has
    // to come off the accumulator is sum (bias + z) x = z * S + B.  In the staged order every
    // 32-bit word is one (low, high) pair and word k of a unit is pair k: lane l reads words
    // l and l + 32 of the block, both pair l % 16.
    float bias_lo = 128.0f, bias_hi = 128.0f;
    if (BITS == 3) {
      const bool alt = (dq::stream_alt_mask3() >> (lane & 15)) & 1u;
      bias_lo = alt ? 64.0f : 8.0f;
      bias_hi = alt ? 16.0f : 128.0f;
    }
    for (int idx = warp; idx < p.x_blocks * p.M; idx += kSWarps) {
      const int blk = idx / p.M, m = idx - blk * p.M;
      const uint32_t* wds =
          reinterpret_cast<const uint32_t*>(xs + (size_t)m * p.x_pitch + blk * kSBlockBytes);
      const uint32_t v0 = wds[lane], v1 = wds[lane + 32];
      const float lo = __uint_as_float(v0 << 16) + __uint_as_float(v1 << 16);
      const float hi = __uint_as_float(v0 & 0xFFFF0000u) + __uint_as_float(v1 & 0xFFFF0000u);
      float sm = lo + hi;
      float bs = fmaf(bias_hi, hi, bias_lo * lo);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sm += __shfl_xor_sync(0xffffffffu, sm, o);
        bs += __shfl_xor_sync(0xffffffffu, bs, o);
      }
      if (lane == 0) { xtab[(blk * TOKP + m) * 2] = sm; xtab[(blk * TOKP + m) * 2 + 1] = bs; }
    }
    ptx::named_barrier_sync(1, kSThreads);
    if (!GROUPED && warp < p.M) {
      // whole-row sums for token `warp`: lanes stride over the blocks, then a fixed tree
      float lo = 0.f, hi = 0.f;
      for (int blk = lane; blk < p.x_blocks; blk += 32) {
        lo += xtab[(blk * TOKP + warp) * 2];
        hi += xtab[(blk * TOKP + warp) * 2 + 1];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        lo += __shfl_xor_sync(0xffffffffu, lo, o);
        hi += __shfl_xor_sync(0xffffffffu, hi, o);
      }
      if (lane == 0) { xtot[warp * 2] = lo; xtot[warp * 2 + 1] = hi; }
    }

    // token rows this lane reads as the MMA "B" operand (token index = lane / 4); lanes
    // beyond M read row 0: their accumulator columns are never stored
    const uint8_t* xrow0 = xs + (size_t)(g8 < p.M ? g8 : 0) * p.x_pitch;
    const uint8_t* xrow1 = xs + (size_t)(g8 + 8 < p.M ? g8 + 8 : 0) * p.x_pitch;
    const bool vec_zs = GROUPED && p.g == 128 && (p.G & 3) == 0;
    bool ok = true;

    for (int rb = 0; rb < nrb; ++rb) {
      int rows[4];
      bool valid[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        rows[r] = row0 + rb * 32 + r * 8 + g8;
        valid[r] = rows[r] < row_end;
      }
      float acc[2][NT][4], tot[2][NT][4];
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) { acc[h][nt][e] = 0.0f; tot[h][nt][e] = 0.0f; }

      for (int ch = warp; ch < p.nchunks; ch += kSWarps) {
        const int s = rb * p.nchunks + ch;
        const int slot = s % p.slots;
        // zero-points and scales of the step's four 128-column blocks, requested before
        // the wait so that their latency is hidden behind it
        float zq[4][4], sq[4][4];
        if (GROUPED) {
          if (vec_zs) {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              uint32_t z4 = 0u;
              float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
              if (valid[r]) {
                const size_t gi = (size_t)rows[r] * p.G + ch * 4;
                z4 = __ldg(reinterpret_cast<const uint32_t*>(p.zeros + gi));
                s4 = __ldg(reinterpret_cast<const float4*>(p.scales + gi));
              }
              zq[r][0] = (float)(z4 & 0xFFu); zq[r][1] = (float)((z4 >> 8) & 0xFFu);
              zq[r][2] = (float)((z4 >> 16) & 0xFFu); zq[r][3] = (float)(z4 >> 24);
              sq[r][0] = s4.x; sq[r][1] = s4.y; sq[r][2] = s4.z; sq[r][3] = s4.w;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int col = ch * kSStepCols + j * 128;
              const int gidx = col < p.K ? col / p.g : 0;
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                zq[r][j] = 0.f;
                sq[r][j] = 0.f;
                if (valid[r] && col < p.K) {
                  const size_t gi = (size_t)rows[r] * p.G + gidx;
                  zq[r][j] = (float)__ldg(p.zeros + gi);
                  sq[r][j] = __ldg(p.scales + gi);
                }
              }
            }
          }
        }
        if (ok && !ptx::mbar_wait(ptx::smem_u32(&bars->full[slot]), ((uint32_t)(s / p.slots)) & 1u, abort_flag))
          ok = false;
        if (ok) {
          const uint8_t* sb = ring + (size_t)slot * Geo::slot + g8 * Geo::pitch;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4][BITS];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const uint8_t* src = sb + r * (8 * Geo::pitch) + (4 * j + c4) * (BITS * 4);
              if constexpr (BITS == 4) {
                const uint4 v = *reinterpret_cast<const uint4*>(src);
                w[r][0] = v.x; w[r][1] = v.y; w[r][2] = v.z; w[r][3] = v.w;
              } else {
                const uint32_t* s32 = reinterpret_cast<const uint32_t*>(src);
                w[r][0] = s32[0]; w[r][1] = s32[1]; w[r][2] = s32[2];
              }
            }
            const int xo = (ch * 4 + j) * kSBlockBytes + c4 * 64;
            const uint8_t* x0 = xrow0 + xo;
            const uint8_t* x1 = xrow1 + xo;
            unit_mma<BITS, NT, 0, 0>(w, x0, x1, acc);
            unit_mma<BITS, NT, 0, 1>(w, x0, x1, acc);
            unit_mma<BITS, NT, 1, 0>(w, x0, x1, acc);
            unit_mma<BITS, NT, 1, 1>(w, x0, x1, acc);
            unit_mma<BITS, NT, 2, 0>(w, x0, x1, acc);
            unit_mma<BITS, NT, 2, 1>(w, x0, x1, acc);
            unit_mma<BITS, NT, 3, 0>(w, x0, x1, acc);
            unit_mma<BITS, NT, 3, 1>(w, x0, x1, acc);
            if (GROUPED) {
              // close the 128-column block: zero-point term out, scale in
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) {
                const float4 xt = *reinterpret_cast<const float4*>(
                    xtab + ((size_t)(ch * 4 + j) * TOKP + nt * 8 + 2 * c4) * 2);   // S0 B0 S1 B1
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                  for (int q = 0; q < 2; ++q) {      // q = 0: row g8 of the half, q = 1: row g8 + 8
                    const float z = zq[2 * h + q][j], sc = sq[2 * h + q][j];
                    const float c0 = fmaf(z, xt.x, xt.y);      // z * S + B, token tk
                    const float c1 = fmaf(z, xt.z, xt.w);      // token tk + 1
                    tot[h][nt][2 * q] = fmaf(sc, acc[h][nt][2 * q] - c0, tot[h][nt][2 * q]);
                    tot[h][nt][2 * q + 1] = fmaf(sc, acc[h][nt][2 * q + 1] - c1, tot[h][nt][2 * q + 1]);
                    acc[h][nt][2 * q] = 0.0f;
                    acc[h][nt][2 * q + 1] = 0.0f;
                  }
                }
              }
            }
          }
        }
        // the codes of this step are consumed: hand the slot back
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->empty[slot]));
      }

      // ---- this warp's partial sums of the block: [32 rows][TOKP]
      float* mine = partial + (size_t)(((rb & 1) * kSWarps + warp) * 32) * TOKP;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int lr = h * 16 + g8;
          const int tk = nt * 8 + c4 * 2;
          const float* v = GROUPED ? tot[h][nt] : acc[h][nt];
          *reinterpret_cast<float2*>(mine + lr * TOKP + tk) = make_float2(v[0], v[1]);
          *reinterpret_cast<float2*>(mine + (lr + 8) * TOKP + tk) = make_float2(v[2], v[3]);
        }
      ptx::named_barrier_sync(1, kSThreads);
      // ---- add the warps' sums in warp order and write Y
      const float* buf = partial + (size_t)((rb & 1) * kSWarps * 32) * TOKP;
      for (int idx = threadIdx.x; idx < 32 * p.M; idx += kSThreads) {
        const int m = idx >> 5, lr = idx & 31;
        const int row = row0 + rb * 32 + lr;
        if (row < row_end) {
          float sum = 0.0f;
#pragma unroll
          for (int wv = 0; wv < kSWarps; ++wv) sum += buf[(wv * 32 + lr) * TOKP + m];
          if (!GROUPED) {
            const float z = (float)__ldg(p.zeros + row);
            const float* sc = p.scales;
            if (p.task_ids) {
              const int task = min(max(__ldg(p.task_ids + m), 0), p.n_tasks - 1);
              sc += (size_t)task * p.N;
            }
            sum = (sum - fmaf(z, xtot[m * 2], xtot[m * 2 + 1])) * __ldg(sc + row);
          }
          p.Y[(size_t)m * p.N + row] = __float2bfloat16_rn(sum);
        }
      }
    }
  }

  __syncthreads();
  if (*abort_flag) {
    // copies still in flight must land before the shared memory is given back
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    if (threadIdx.x == 0) {
      atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
      p.status[1] = (int)blockIdx.x;
    }
  }
}

struct StreamPlan {
  int rows_per_cta, grid, nchunks, x_blocks, x_pitch, slots;
  size_t smem;
};

// Shared-memory plan; slots == 0 when the streaming kernel does not apply.
int plan_stream(const peqa_qweight_t* w, int g, int M, StreamPlan* plan) {
  plan->slots = 0;
  const int N = w->out_features, K = w->in_features;
  const int G = K / g;
  if (K % 128 != 0 || N % 8 != 0) return PEQA_OK;
  if (G > 1 && g % 128 != 0) return PEQA_OK;
  const int NT = M <= 8 ? 1 : 2;
  const int TOKP = 8 * NT;
  if ((long long)M * (((K + kSStepCols - 1) / kSStepCols) * 64) > (long long)kSMaxXLoads * kSThreads)
    return PEQA_OK;   // the activations do not fit the registers they are fetched through
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int groups8 = N / 8;
  const int per_cta = (groups8 + sms - 1) / sms;
  plan->rows_per_cta = 8 * per_cta;
  plan->grid = (N + plan->rows_per_cta - 1) / plan->rows_per_cta;
  plan->nchunks = (K + kSStepCols - 1) / kSStepCols;
  plan->x_blocks = 4 * plan->nchunks;
  // pitch = blocks*288 + pad with pitch % 128 == 8: consecutive tokens land 2 banks apart
  const int raw = plan->x_blocks * kSBlockBytes;
  plan->x_pitch = raw + ((8 - raw % 128) % 128 + 128) % 128;
  const size_t fixed = 128 /*alignment*/ + (((size_t)M * plan->x_pitch + 15) & ~(size_t)15) +
                       (size_t)plan->x_blocks * TOKP * 2 * sizeof(float) + (size_t)TOKP * 2 * sizeof(float) +
                       (size_t)2 * kSWarps * 32 * TOKP * sizeof(float) + sizeof(StreamBarriers) + 16;
  const size_t slot = w->bits == 3 ? StreamGeom<3>::slot : StreamGeom<4>::slot;
  if (fixed + 8 * slot > (size_t)kSSmemLimit) return PEQA_OK;   // activations too large to stage
  size_t slots = ((size_t)kSSmemLimit - fixed) / slot;
  if (slots > (size_t)kSMaxSlots) slots = kSMaxSlots;
  const size_t steps = (size_t)((plan->rows_per_cta + 31) / 32) * plan->nchunks;
  if (slots > steps) slots = steps;
  plan->slots = (int)slots;
  plan->smem = fixed + slots * slot;
  return PEQA_OK;
}

template <int BITS, int NT, bool GROUPED>
int launch_stream_t(const StreamParams& p, int grid, size_t smem, cudaStream_t st) {
  auto kern = decode_stream_kernel<BITS, NT, GROUPED>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<grid, kSBlock, smem, st>>>(p);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

}  // namespace

// One scale per channel or groups that are multiples of 128 columns, and staged
// activations small enough to leave the ring at least one step per compute warp.
bool decode_stream_supported(const peqa_qweight_t* w, int g, int M) {
  StreamPlan plan;
  if (plan_stream(w, g, M, &plan) != PEQA_OK) return false;
  return plan.slots > 0;
}

int launch_decode_stream(const peqa_qweight_t* w, int g, const void* X, int M, void* Y,
                         const float* scale_table, int n_tasks, const int32_t* task_ids,
                         cudaStream_t st) {
  StreamPlan plan;
  PEQA_TRY(plan_stream(w, g, M, &plan));
  if (plan.slots == 0) return PEQA_ERR_BAD_SHAPE;
  StreamParams p;
  p.qw = w->qweight;
  p.zeros = w->zeros;
  p.scales = task_ids ? scale_table : w->scales;
  p.task_ids = task_ids;
  p.n_tasks = n_tasks;
  p.X = static_cast<const __nv_bfloat16*>(X);
  p.Y = static_cast<__nv_bfloat16*>(Y);
  p.N = w->out_features;
  p.K = w->in_features;
  p.g = g;
  p.G = p.K / g;
  if (task_ids && p.G != 1) return PEQA_ERR_BAD_SHAPE;
  p.M = M;
  p.wpr = p.K * w->bits / 32;
  p.nchunks = plan.nchunks;
  p.rows_per_cta = plan.rows_per_cta;
  p.x_blocks = plan.x_blocks;
  p.x_pitch = plan.x_pitch;
  p.slots = plan.slots;
  PEQA_TRY(status_word(st, &p.status));
  const bool grouped = p.G > 1;
  const int NT = M <= 8 ? 1 : 2;
  if (w->bits == 4) {
    if (NT == 1) return grouped ? launch_stream_t<4, 1, true>(p, plan.grid, plan.smem, st)
                                : launch_stream_t<4, 1, false>(p, plan.grid, plan.smem, st);
    return grouped ? launch_stream_t<4, 2, true>(p, plan.grid, plan.smem, st)
                   : launch_stream_t<4, 2, false>(p, plan.grid, plan.smem, st);
  }
  if (NT == 1) return grouped ? launch_stream_t<3, 1, true>(p, plan.grid, plan.smem, st)
                              : launch_stream_t<3, 1, false>(p, plan.grid, plan.smem, st);
  return grouped ? launch_stream_t<3, 2, true>(p, plan.grid, plan.smem, st)
                 : launch_stream_t<3, 2, false>(p, plan.grid, plan.smem, st);
}

}  // namespace peqa
