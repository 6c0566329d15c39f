// Small-batch forward (token generation) from a prepared copy of the frozen
// weights:  Y[m,i] = sum_g s[i,g] * sum_{j in g} X[m,j] * (Q[i,j] - z[i,g])   (Eq. 2 with
// M <= 16 tokens; Sec. 3.1 / 3.3: the memory-bound matrix-vector regime).
//
// The frozen matrix never changes after quantization (Sec. 3.3), so a server
// can keep it in whatever order suits the kernel.  The prepared layout stores the
// same bits as the canonical packed matrix, rearranged so that
//   * everything one warp needs for one step (8 rows x 512 columns) is one
//     contiguous block that a single bulk copy moves into shared memory, in the
//     order the lanes read it (16 bytes per lane and read, no bank conflicts);
//   * the sixteen contraction slots of one warp-level MMA are sixteen columns of
//     one 32-column run, so they share a quantization group and the scale and
//     zero-point can be applied per group to the accumulator;
//   * the two codes one logic operation extracts as a bf16 pair are the codes of
//     two ADJACENT columns, so the activations are used in their natural order.
//
// Layout.  rg = row / 8, r = row % 8, step t = column / 512 (T = ceil(K / 512)
// steps; columns beyond K hold zero codes), C = bits.  Block (rg, t) is C*512
// bytes at byte offset (((rg/2)*T + t)*2 + rg%2)*C*512, so the two row groups of a
// pair alternate step by step and a pair's consecutive steps are contiguous
// (an odd count of row groups is padded with a group of zero codes): chunk c
// (0..C-1), lane l (0..31), 16 bytes each, chunk-major.  Lane l = 4*r + c4 owns, of row 8*rg + r, columns
// 8*c4 .. 8*c4+7 of each of the step's sixteen 32-column runs.  Its 4*C words are
// four strings of C words; string s holds runs 4s .. 4s+3, its string column
// cs = 8*(run % 4) + (column % 8); string column 2k sits at code position
// stream_lo(k) and 2k+1 at stream_hi(k) (dequant.cuh), code position p being bits
// [bits*p, bits*p + bits) of the string read as a little-endian bit string.
//
// Work split.  One CTA per SM owns a contiguous range of 8-row groups and all
// of K for them, so no sum crosses a CTA: no workspace, no atomics.  Row
// groups 2P and 2P+1 form a "pair", the 16 rows of a warp-level mma.m16n8k16
// whose 8-wide side are the tokens (a range that starts or ends inside a pair
// runs that group as a half pair).  The CTA's (pair, step) list, pair-major, is cut into sixteen
// contiguous ranges of equal cost, one per warp.  A warp streams its range
// through a private ring in shared memory: lane 0 issues one bulk copy per slot
// (one or two steps of a pair: 3 to 8 KiB of contiguous memory; streaming reads
// on this part want few, large copies and well over 100 KiB in flight per SM)
// and all lanes wait on the slot's mbarrier.  Codes reach the tensor core as the biased integers
// (bias + q) they are after one logic operation; the zero-point and bias terms
// come off the sum when a group (or the row) is complete:
//   y += s * (acc - z * sum_j x_j - sum_j bias_j x_j).
// When a warp's range crosses into the next pair it parks its sums in shared
// memory; at the end the parked sums of each pair are added in warp order, so
// results do not depend on timing.
//
// Activations are staged in shared memory, all of K when they fit, otherwise in
// chunks of steps with the per-output sums carried in shared memory.
//
// Launch overlap.  The kernel is launched with programmatic stream
// serialization: it lets the next kernel in the stream start as soon as SMs
// free up, requests its own first weights at once, and only then waits for the
// preceding kernel before it touches X or Y.  The prepared weights are
// therefore read before earlier work in the stream is known to be complete:
// they must be final when the call is made.
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"

namespace peqa {

namespace {

using namespace ptx;

#ifndef PEQA_PREP_WARPS
#define PEQA_PREP_WARPS 16
#endif
constexpr int kPWarps = PEQA_PREP_WARPS;
constexpr int kPThreads = kPWarps * 32;
constexpr int kPSmemLimit = 227 * 1024;
constexpr int kPMaxSlots = 4;
constexpr int kStepCols = 512;
constexpr int kPBarBytes = kPWarps * kPMaxSlots * 8;              // the warps' mbarriers
// + abort flag, wait limit and, per warp, the bounds of its steps and its first and last pair
constexpr int kPHeadBytes = (kPBarBytes + 32 + 3 * (kPWarps + 1) * 4 + 127) / 128 * 128;

// Pitch (floats) of a row's tokens in the per-output tables of shared memory.
__host__ __device__ inline int tok_pitch(int toks) { return toks + ((6 - (toks & 3)) & 3); }

struct PrepParams {
  const uint8_t* P;         // prepared weights
  const uint8_t* zeros;     // [N, G]
  const float* scales;      // [N, G] or table [n_tasks, N, G]
  const __nv_bfloat16* X;   // [M, K]
  __nv_bfloat16* Y;         // [M, N]
  const int32_t* task_ids;  // nullptr: one task
  int n_tasks;
  int N, K, G, M;
  int rgs;                  // row groups in the matrix (N / 8)
  int rg_per_cta;
  int T;                    // steps of 512 columns per row group
  int spc;                  // steps per staged chunk of activations
  int nchunks;
  int slots;                // ring slots per warp
  int sps;                  // steps per slot (1 or 2)
  int maxseg;               // parked partial sums per warp and chunk
  int x_pitch;              // bytes between staged token rows
  int pairs_per_cta;
  int* status;
};

__device__ __forceinline__ void pmma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                           uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
      "{%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Contiguous bulk copy global -> shared memory; its bytes are credited to `bar`.  Both
// addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}

// 16 bytes of a ring slot.  Volatile at both compiler levels: the read must be issued before
// the bulk copy that refills the slot, and neither the compiler nor the assembler can see
// that the copy writes this memory, so an ordinary load could be moved behind it.
__device__ __forceinline__ uint4 ring_load(uint32_t addr) {
  uint4 v;
  asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(addr)
               : "memory");
  return v;
}

// One lane's weights of one step: row r of the pair's two groups.
template <int BITS>
struct StepRegs {
  uint4 a[BITS];
  uint4 b[BITS];
};

// MMAs 2*MM and 2*MM + 1 of string S: run 4*S + MM of the step, whose eight columns of this
// lane are one 16-byte word of activations per token.
template <int BITS, int NT, bool HAS_B, int MM>
__device__ __forceinline__ void run_mma2(const uint32_t (&wa)[BITS], const uint32_t (&wb)[BITS],
                                         const uint8_t* x0, const uint8_t* x1,
                                         float (&acc)[NT][4], float (&acc2)[NT][4]) {
  const uint4 xa = *reinterpret_cast<const uint4*>(x0 + MM * 64);
  uint4 xb = make_uint4(0u, 0u, 0u, 0u);
  if (NT == 2) xb = *reinterpret_cast<const uint4*>(x1 + MM * 64);
  uint32_t f0[4], f1[4];
  dq::mma_pairs_stream<BITS, 2 * MM>(wa, f0[0], f0[2]);
  dq::mma_pairs_stream<BITS, 2 * MM + 1>(wa, f1[0], f1[2]);
  f0[1] = f0[3] = f1[1] = f1[3] = 0u;
  if (HAS_B) {
    dq::mma_pairs_stream<BITS, 2 * MM>(wb, f0[1], f0[3]);
    dq::mma_pairs_stream<BITS, 2 * MM + 1>(wb, f1[1], f1[3]);
  }
  // the two MMAs of a run go to different accumulators, so that consecutive MMAs of a warp do
  // not wait for one another (a single chain of 32 dependent MMAs per step cost 5 % of the
  // kernel); the halves are added when the sums are taken off
  pmma_16816(acc[0], f0, xa.x, xa.y);
  pmma_16816(acc2[0], f1, xa.z, xa.w);
  if (NT == 2) {
    pmma_16816(acc[1], f0, xb.x, xb.y);
    pmma_16816(acc2[1], f1, xb.z, xb.w);
  }
}

// Bias the code of string column cs (0..31) carries when it reaches the tensor core.
template <int BITS>
__host__ __device__ constexpr float column_bias(int cs) {
  if (BITS == 4) return 128.0f;
  return dq::stream_alt(3, cs >> 1) ? ((cs & 1) ? 16.0f : 64.0f) : ((cs & 1) ? 128.0f : 8.0f);
}

// GSH: quantization groups of 32 << GSH columns (1: 64, 2: 128, 3: 256), or 0: one group
// per row or groups that are multiples of 512 columns (the sums of a whole staged chunk of
// steps are taken off at once, which needs the chunk to lie inside one group).
template <int BITS, int NT, int GSH>
__global__ void __launch_bounds__(kPThreads, 1)
decode_prep_kernel(const PrepParams p) {
  constexpr int C = BITS;                            // 16-byte chunks per lane, step and group
  constexpr int BLK = C * 512;                       // bytes of one block (rg, t)
  constexpr int TOKP = 8 * NT;
  constexpr bool GROUPED = GSH != 0;
  constexpr int RUNS_PER_GROUP = GROUPED ? (1 << GSH) : 16;
  constexpr int GPS = 16 / RUNS_PER_GROUP;           // groups per step (GROUPED)
  extern __shared__ uint8_t prep_smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(prep_smem_raw) + 127) &
                                             ~static_cast<uintptr_t>(127));
  uint64_t* bars = reinterpret_cast<uint64_t*>(base);                        // [warps][kPMaxSlots]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base + kPBarBytes);   // [0] flag, [1] limit
  int* wbound = const_cast<int*>(abort_flag) + 8;                            // [warps + 1] bounds of the chunk
  int* wfirst = wbound + kPWarps + 1;                                        // [warps] first pair of the range
  int* wlast = wfirst + kPWarps + 1;                                         // [warps] last pair, -1: no steps
  const int toks = (p.M + 1) & ~1;                                           // tokens kept of a tile
  // pitch of a row's tokens in the per-output tables: toks rounded up to 2 mod 4, so that the
  // sixteen rows a warp reads for one token fall into sixteen different banks
  const int tp = tok_pitch(toks);
  float* part = reinterpret_cast<float*>(base + kPHeadBytes);                // [warps][maxseg][16][tp]
  float* yacc = part + (size_t)kPWarps * p.maxseg * 16 * tp;                 // [pairs][16][tp]
  float* sums = yacc + (p.nchunks > 1 ? (size_t)p.pairs_per_cta * 16 * tp : 0);
  // sums, GROUPED: [groups of the chunk][TOKP][2] = (sum x, sum bias*x) per group and token;
  // else [16 warps][TOKP][2]: every warp's share of the chunk's sums, added in warp order
  const int sum_rows = GROUPED ? p.spc * GPS : kPWarps;
  // cterm (GROUPED): [pairs][16][tp], the part of every output that does not depend on the weights
  float* cterm = sums + (size_t)sum_rows * TOKP * 2;
  uint8_t* xs = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(cterm + (GROUPED ? (size_t)p.pairs_per_cta * 16 * tp : 0)) + 127) &
      ~static_cast<uintptr_t>(127));
  uint8_t* ring = xs + (((size_t)p.M * p.x_pitch + 127) & ~static_cast<size_t>(127));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r8 = lane >> 2, c4 = lane & 3;
  const int rg0 = blockIdx.x * p.rg_per_cta;
  const int rg_end = min(p.rgs, rg0 + p.rg_per_cta);
  // pairs are (2P, 2P+1) for the whole matrix; a range that starts (ends) at an odd row group
  // has a half pair in front (at the end)
  const int P0 = rg0 >> 1;
  const int lead = rg0 & 1;
  const int rest = rg_end - rg0 - lead;
  const int trail = rest & 1;
  const int F = rest >> 1;                           // full pairs
  const int npairs = lead + F + trail;
  const int slot_bytes = 2 * BLK * p.sps;

  // the next kernel of the stream may be scheduled as SMs free up
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (threadIdx.x == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = p.status[4];
  }
  if (lane == 0) {
    for (int s = 0; s < p.slots; ++s) mbar_init(smem_u32(&bars[warp * kPMaxSlots + s]), 1);
    fence_mbar_init();
  }
  __syncwarp();

  // ---- this warp's steps of a chunk: [bound(w), bound(w+1)) of the pair-major list, cut so
  // that the warps' costs are equal (a step of a full pair costs 4, of a half pair 3)
  auto spc_of = [&](int ch) { return min(p.spc, p.T - ch * p.spc); };
  auto bound = [&](int w, int spc_c) {
    // measured: a step of a half pair takes about three quarters of a full pair's step (half
    // the code extraction, the same MMAs and activation reads)
    constexpr int CF = 4, CH = 3;
    const int tot = (CH * (lead + trail) + CF * F) * spc_c;
    int b = (int)(((long long)w * tot) / kPWarps);
    int at = 0;
    if (lead) {
      if (b <= CH * spc_c) return (b + CH / 2) / CH;
      b -= CH * spc_c;
      at = spc_c;
    }
    if (b <= CF * F * spc_c) return at + (b + CF / 2) / CF;
    return at + F * spc_c + (b - CF * F * spc_c + CH / 2) / CH;
  };
  auto pair_full = [&](int lp) { return lp >= lead && lp < lead + F; };
  // first row group of local pair lp (the only one of a half pair)
  auto pair_rg = [&](int lp) { return lp == 0 ? rg0 : 2 * (P0 + lp); };
  // ---- ring: issue cursor (only lane 0 uses it)
  const uint32_t ring_w = smem_u32(ring) + (uint32_t)warp * (uint32_t)(p.slots * slot_bytes);
  const uint32_t bar_w = smem_u32(&bars[warp * kPMaxSlots]);
  int i_ch = 0, i_lin = 0, i_hi = 0, i_spc = 1;
  int i_lp = 0, i_tl = 0, i_slot = 0;               // pair and step of i_lin; slot of the next copy
  auto issue_seek = [&]() {       // moves to the first chunk (from i_ch on) where this warp has steps
    while (i_ch < p.nchunks) {
      i_spc = spc_of(i_ch);
      i_lin = bound(warp, i_spc);
      i_hi = bound(warp + 1, i_spc);
      i_lp = i_lin / i_spc;
      i_tl = i_lin - i_lp * i_spc;
      if (i_lin < i_hi) return;
      ++i_ch;
    }
  };
  auto issue_next = [&]() {
    if (i_ch >= p.nchunks) return;
    const int lp = i_lp, tl = i_tl;
    const int t = i_ch * p.spc + tl;
    const int n = (p.sps == 2 && i_lin + 1 < i_hi && tl + 1 < i_spc) ? 2 : 1;
    const int rg = pair_rg(lp);
    const int slot = i_slot;
    const uint32_t bar = bar_w + slot * 8;
    const uint32_t dst = ring_w + slot * slot_bytes;
    // block (rg, t) lies at (((rg >> 1) * T + t) * 2 + (rg & 1)) * BLK
    const uint8_t* src = p.P + ((((size_t)(rg >> 1) * p.T + t) * 2 + (rg & 1)) * BLK);
    if (pair_full(lp)) {
      mbar_arrive_expect_tx(bar, n * 2 * BLK);
      bulk_load(dst, src, n * 2 * BLK, bar);                       // steps t .. t+n-1 are contiguous
    } else {
      mbar_arrive_expect_tx(bar, n * BLK);
      bulk_load(dst, src, BLK, bar);
      if (n == 2) bulk_load(dst + 2 * BLK, src + 2 * BLK, BLK, bar);
    }
    i_slot = i_slot + 1 == p.slots ? 0 : i_slot + 1;
    i_lin += n;
    i_tl += n;
    if (i_tl >= i_spc) {
      i_tl = 0;
      ++i_lp;
    }
    if (i_lin >= i_hi) {
      ++i_ch;
      issue_seek();
    }
  };
  // One slot per warp is requested while the preceding kernel drains; the others follow the
  // activation requests of the first chunk, which would otherwise queue behind a full ring of
  // weights on their way into this SM (the CTAs that start last wait longest for them).
  if (lane == 0) {
    issue_seek();
    issue_next();
  }

  // everything below reads X or writes Y: the preceding kernel must have completed
  asm volatile("griddepcontrol.wait;" ::: "memory");

  int c_slot = 0;
  uint32_t c_phase = 0;                              // parity of the ring's current round
  bool ok = true;

  for (int ch = 0; ch < p.nchunks; ++ch) {
    const int spc_c = spc_of(ch);
    const int col0 = ch * p.spc * kStepCols;                       // first column of the chunk
    const int ccols = min(p.K - col0, spc_c * kStepCols);          // real columns in it
    if (ch > 0) __syncthreads();                                   // the previous chunk is no longer read
    // ---- stage X[:, chunk] (columns beyond K read as zero) and take, per token, the sum of x
    // and the sum of bias * x: per group (a thread stages and sums whole groups), or over the
    // pieces this thread staged itself, added up per warp (the warps' shares are added in
    // warp order when the rows are finished)
    const int pieces = spc_c * (kStepCols / 8);                    // 16-byte pieces per token
    if (threadIdx.x <= kPWarps) {
      const int wl = bound(threadIdx.x, spc_c);
      wbound[threadIdx.x] = wl;
      if (threadIdx.x < kPWarps) {
        const int wh = bound(threadIdx.x + 1, spc_c);
        wfirst[threadIdx.x] = wl / spc_c;
        wlast[threadIdx.x] = wh > wl ? (wh - 1) / spc_c : -1;
      }
    }
    // bias of the two columns in word e of a piece whose run in the step is run % 4 == rq
    auto piece_sums = [&](const uint8_t* ptr, int rq, float& sx, float& sb) {
      const uint4 v = *reinterpret_cast<const uint4*>(ptr);
      const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = __uint_as_float(wv[e] << 16), hi = __uint_as_float(wv[e] & 0xFFFF0000u);
        sx += lo + hi;
        float b0 = 128.0f, b1 = 128.0f;
        if (BITS == 3) {
          const bool alt = (dq::stream_alt_mask3() >> (4 * rq + e)) & 1u;
          b0 = alt ? 64.0f : 8.0f;
          b1 = alt ? 16.0f : 128.0f;
        }
        sb = fmaf(b0, lo, sb);
        sb = fmaf(b1, hi, sb);
      }
    };
    auto stage_piece = [&](int m, int pc) {
      uint8_t* dst = xs + (size_t)m * p.x_pitch + pc * 16;
      if (pc * 8 < ccols) cp_async_16(smem_u32(dst), p.X + (size_t)m * p.K + col0 + pc * 8);
      else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
    };
    if (GROUPED) {
      const int ngr = spc_c * GPS;
      constexpr int gpieces = RUNS_PER_GROUP * 4;                  // 16-byte pieces per group
      for (int idx = threadIdx.x; idx < ngr * p.M; idx += kPThreads) {
        const int gi = idx / p.M, m = idx - gi * p.M;
        for (int pc = 0; pc < gpieces; ++pc) stage_piece(m, gi * gpieces + pc);
      }
      if (ch == 0 && lane == 0)
        for (int s = 1; s < p.slots; ++s) issue_next();
      asm volatile("cp.async.wait_all;" ::: "memory");
      for (int idx = threadIdx.x; idx < ngr * p.M; idx += kPThreads) {
        const int gi = idx / p.M, m = idx - gi * p.M;
        const uint8_t* row = xs + (size_t)m * p.x_pitch + (size_t)gi * gpieces * 16;
        float sx = 0.0f, sb = 0.0f;
        for (int pc = 0; pc < gpieces; ++pc)
          piece_sums(row + pc * 16, (gi * RUNS_PER_GROUP + (pc >> 2)) & 3, sx, sb);
        sums[((size_t)gi * TOKP + m) * 2] = sx;
        sums[((size_t)gi * TOKP + m) * 2 + 1] = sb;
      }
    } else {
      // A token belongs to 16 / Mp warps (Mp: M rounded up to a power of two); a warp copies
      // every (16 / Mp)-th block of 32 pieces of its token and sums what it copied itself, so
      // it needs no other warp's copies and reduces once.  run % 4 of a lane's pieces is fixed.
      int mp = 1;
      while (mp < p.M) mp <<= 1;
      const int wpt = kPWarps / mp;                                // warps per token
      const int tok = warp / wpt, sub = warp - tok * wpt;
      if (tok < p.M)
        for (int pc = sub * 32 + lane; pc < pieces; pc += wpt * 32) stage_piece(tok, pc);
      if (ch == 0 && lane == 0)
        for (int s = 1; s < p.slots; ++s) issue_next();
      // this warp's row of the table: zero but for its own token
      for (int i = lane; i < TOKP * 2; i += 32) sums[warp * TOKP * 2 + i] = 0.0f;
      asm volatile("cp.async.wait_all;" ::: "memory");
      __syncwarp();
      if (tok < p.M) {
        float sx = 0.0f, sb = 0.0f;
        const uint8_t* row = xs + (size_t)tok * p.x_pitch;
        for (int pc = sub * 32 + lane; pc < pieces; pc += wpt * 32)
          piece_sums(row + pc * 16, (lane >> 2) & 3, sx, sb);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          sx += __shfl_xor_sync(0xffffffffu, sx, o);
          sb += __shfl_xor_sync(0xffffffffu, sb, o);
        }
        if (lane == 0) {
          sums[(warp * TOKP + tok) * 2] = sx;
          sums[(warp * TOKP + tok) * 2 + 1] = sb;
        }
      }
    }
    __syncthreads();

    // ---- per-row terms: when every output of the CTA has a thread of its own, that thread fetches
    // the row's zero-point and scale now, so that the final reduce does not wait for them
    const bool own_output = !GROUPED && npairs * 16 * p.M <= kPThreads;
    float z_own = 0.0f, s_own = 0.0f;
    if (own_output && threadIdx.x < npairs * 16 * p.M) {
      const int lp = threadIdx.x / (16 * p.M);
      const int rem = threadIdx.x - lp * 16 * p.M;
      const int m = rem >> 4, lr = rem & 15;
      if (pair_full(lp) || lr < 8) {
        const int row = pair_rg(lp) * 8 + lr;
        const int gg = p.G == 1 ? 0 : col0 / (p.K / p.G);
        z_own = (float)__ldg(p.zeros + (size_t)row * p.G + gg);
        const float* tab = p.scales;
        if (p.task_ids) tab += (size_t)min(max(__ldg(p.task_ids + m), 0), p.n_tasks - 1) * p.N * p.G;
        s_own = __ldg(tab + (size_t)row * p.G + gg);
      }
    }

    // ---- this warp's steps of the chunk
    const int lo = wbound[warp], hi = wbound[warp + 1];
    int seg = 0, cur_pair = -1;
    float acc[NT][4], acc2[NT][4], yv[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[nt][e] = acc2[nt][e] = yv[nt][e] = 0.0f;
    auto fold = [&]() {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          acc[nt][e] += acc2[nt][e];
          acc2[nt][e] = 0.0f;
        }
    };
    auto park = [&]() {
      fold();
      float* mine = part + ((size_t)(warp * p.maxseg + seg) * 16) * tp;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int tk = nt * 8 + c4 * 2;
        const float* v = GROUPED ? yv[nt] : acc[nt];
        if (seg < p.maxseg && tk < toks) {
          *reinterpret_cast<float2*>(mine + r8 * tp + tk) = make_float2(v[0], v[1]);
          *reinterpret_cast<float2*>(mine + (r8 + 8) * tp + tk) = make_float2(v[2], v[3]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = yv[nt][e] = 0.0f;
      }
      ++seg;
    };
    const uint8_t* xl = xs + (size_t)(r8 < p.M ? r8 : 0) * p.x_pitch + c4 * 16;
    const uint8_t* xh = xs + (size_t)(r8 + 8 < p.M ? r8 + 8 : 0) * p.x_pitch + c4 * 16;

    int lin = lo;
    int lp = lo / spc_c, tl = lo - lp * spc_c;
    while (ok && lin < hi) {
      const int nsteps = (p.sps == 2 && lin + 1 < hi && tl + 1 < spc_c) ? 2 : 1;
      const int slot = c_slot;
      if (!mbar_wait(bar_w + slot * 8, c_phase, abort_flag)) { ok = false; break; }
      if (++c_slot == p.slots) {
        c_slot = 0;
        c_phase ^= 1u;
      }
      for (int j = 0; j < nsteps; ++j) {
        if (lp != cur_pair) {
          if (cur_pair >= 0) park();
          cur_pair = lp;
        }
        const bool has_b = pair_full(lp);
        StepRegs<BITS> w;
        {
          const uint32_t sp = ring_w + (uint32_t)(slot * slot_bytes + j * 2 * BLK + lane * 16);
#pragma unroll
          for (int c = 0; c < C; ++c) w.a[c] = ring_load(sp + c * 512);
          if (has_b) {
#pragma unroll
            for (int c = 0; c < C; ++c) w.b[c] = ring_load(sp + (C + c) * 512);
          } else {
#pragma unroll
            for (int c = 0; c < C; ++c) w.b[c] = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        if (j + 1 == nsteps) {
          // every lane has issued its reads of the slot: it can be refilled
          __syncwarp();
          if (lane == 0) issue_next();
        }

        // scales of this lane's two rows for the groups of the step (GROUPED, one task): the
        // sum of a group is only scaled here; its zero-point and bias terms, which do not depend
        // on the weights, come off where the rows are finished
        const int rowa = pair_rg(lp) * 8 + r8, rowb = rowa + 8;
        const int gstep0 = ((ch * p.spc + tl) * GPS);              // first group of the step
        float gsa[GPS], gsb[GPS];
        if (GROUPED && !p.task_ids) {
          const float* pa = p.scales + (size_t)rowa * p.G + gstep0;
          const float* pb = p.scales + (size_t)rowb * p.G + gstep0;
          if ((p.G % GPS) == 0 && gstep0 < p.G) {
            // G is a multiple of the groups per step: whole, aligned vectors
            if (GPS >= 4) {
#pragma unroll
              for (int q = 0; q < GPS / 4; ++q) {
                const float4 va = __ldg(reinterpret_cast<const float4*>(pa) + q);
                const float4 vb = has_b ? __ldg(reinterpret_cast<const float4*>(pb) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                gsa[4 * q + 0] = va.x; gsa[4 * q + 1] = va.y; gsa[4 * q + 2] = va.z; gsa[4 * q + 3] = va.w;
                gsb[4 * q + 0] = vb.x; gsb[4 * q + 1] = vb.y; gsb[4 * q + 2] = vb.z; gsb[4 * q + 3] = vb.w;
              }
            } else {
              const float2 va = __ldg(reinterpret_cast<const float2*>(pa));
              const float2 vb = has_b ? __ldg(reinterpret_cast<const float2*>(pb)) : make_float2(0.f, 0.f);
              gsa[0] = va.x; gsa[GPS - 1] = va.y;
              gsb[0] = vb.x; gsb[GPS - 1] = vb.y;
            }
          } else {
#pragma unroll
            for (int q = 0; q < GPS; ++q) {
              const bool in = gstep0 + q < p.G;
              gsa[q] = in ? __ldg(pa + q) : 0.0f;
              gsb[q] = in && has_b ? __ldg(pb + q) : 0.0f;
            }
          }
        }
        // group gi of the step is complete: take z * sum x + sum bias * x off and scale
        auto flush = [&](int gi) {
          fold();
          const int gg = gstep0 + gi;                              // group index in the row
          const float* sm = sums + ((size_t)(tl * GPS + gi) * TOKP) * 2;
          if (!p.task_ids) {
            const float sa = gsa[gi], sb = gsb[gi];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              yv[nt][0] = fmaf(sa, acc[nt][0], yv[nt][0]);
              yv[nt][1] = fmaf(sa, acc[nt][1], yv[nt][1]);
              yv[nt][2] = fmaf(sb, acc[nt][2], yv[nt][2]);
              yv[nt][3] = fmaf(sb, acc[nt][3], yv[nt][3]);
            }
          } else if (gg < p.G) {
            // every token has the scales of its own task (Sec. 3.3)
            const float za = (float)__ldg(p.zeros + (size_t)rowa * p.G + gg);
            const float zb = has_b ? (float)__ldg(p.zeros + (size_t)rowb * p.G + gg) : 0.0f;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const float4 sv = *reinterpret_cast<const float4*>(sm + (nt * 8 + c4 * 2) * 2);
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int tok = nt * 8 + c4 * 2 + e;
                const int task = tok < p.M ? min(max(__ldg(p.task_ids + tok), 0), p.n_tasks - 1) : 0;
                const float* tab = p.scales + (size_t)task * p.N * p.G;
                const float sa = __ldg(tab + (size_t)rowa * p.G + gg);
                const float sb = has_b ? __ldg(tab + (size_t)rowb * p.G + gg) : 0.0f;
                const float sx = e ? sv.z : sv.x, sbx = e ? sv.w : sv.y;
                yv[nt][e] = fmaf(sa, acc[nt][e] - fmaf(za, sx, sbx), yv[nt][e]);
                yv[nt][2 + e] = fmaf(sb, acc[nt][2 + e] - fmaf(zb, sx, sbx), yv[nt][2 + e]);
              }
            }
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nt][e] = 0.0f;
        };

        const uint32_t* fa = reinterpret_cast<const uint32_t*>(w.a);
        const uint32_t* fb = reinterpret_cast<const uint32_t*>(w.b);
        const uint8_t* x0 = xl + (size_t)tl * (kStepCols * 2);
        const uint8_t* x1 = xh + (size_t)tl * (kStepCols * 2);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          uint32_t wa[BITS], wb[BITS];
#pragma unroll
          for (int e = 0; e < BITS; ++e) {
            wa[e] = fa[s * BITS + e];
            wb[e] = fb[s * BITS + e];
          }
          const uint8_t* xs0 = x0 + s * 256;
          const uint8_t* xs1 = x1 + s * 256;
          if (has_b) {
            run_mma2<BITS, NT, true, 0>(wa, wb, xs0, xs1, acc, acc2);
            run_mma2<BITS, NT, true, 1>(wa, wb, xs0, xs1, acc, acc2);
            if (GROUPED && RUNS_PER_GROUP == 2) flush(2 * s);
            run_mma2<BITS, NT, true, 2>(wa, wb, xs0, xs1, acc, acc2);
            run_mma2<BITS, NT, true, 3>(wa, wb, xs0, xs1, acc, acc2);
          } else {
            run_mma2<BITS, NT, false, 0>(wa, wb, xs0, xs1, acc, acc2);
            run_mma2<BITS, NT, false, 1>(wa, wb, xs0, xs1, acc, acc2);
            if (GROUPED && RUNS_PER_GROUP == 2) flush(2 * s);
            run_mma2<BITS, NT, false, 2>(wa, wb, xs0, xs1, acc, acc2);
            run_mma2<BITS, NT, false, 3>(wa, wb, xs0, xs1, acc, acc2);
          }
          if (GROUPED && RUNS_PER_GROUP == 2) flush(2 * s + 1);
          if (GROUPED && RUNS_PER_GROUP == 4) flush(s);
          if (GROUPED && RUNS_PER_GROUP == 8 && (s & 1)) flush(s >> 1);
        }
        ++lin;
        if (++tl == spc_c) {
          tl = 0;
          ++lp;
        }
      }
    }
    if (cur_pair >= 0) park();
    __syncthreads();

    // ---- grouped scales of one task: the terms of the chunk's groups that do not depend on the
    // weights, per row and token:  sum_g s[row, g] * (z[row, g] * sum x_g + sum bias * x_g).
    // A warp takes rows warp, warp + 16, ...; the loads of all its rows are issued before the
    // first is used (this pass is pure latency otherwise), a lane owns four adjacent groups.
    const bool last = ch + 1 == p.nchunks;
    const bool group_terms = GROUPED && !p.task_ids;
    if (group_terms) {
      constexpr int RB = 8;                                        // rows of a warp in flight
      const int nrows = npairs * 16;
      const int g0 = ch * p.spc * GPS;
      const int ng = min(p.G - g0, spc_c * GPS);
      const bool vec = ((p.G | g0) & 3) == 0;                      // a lane's four scales are 16-byte aligned
      for (int rbase = warp; rbase < nrows; rbase += kPWarps * RB) {
        for (int gb = 0; gb < ng; gb += 128) {
          const int gl = gb + 4 * lane;                            // this lane's first group of the block
          float4 sv[RB];
          uint32_t zv[RB];
#pragma unroll
          for (int i = 0; i < RB; ++i) {
            const int r = rbase + i * kPWarps;
            const int lp = r >> 4, lr = r & 15;
            sv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            zv[i] = 0u;
            if (r < nrows && (pair_full(lp) || lr < 8) && gl < ng) {
              const size_t off = (size_t)(pair_rg(lp) * 8 + lr) * p.G + g0 + gl;
              if (vec && gl + 4 <= ng) {
                sv[i] = __ldg(reinterpret_cast<const float4*>(p.scales + off));
                zv[i] = __ldg(reinterpret_cast<const uint32_t*>(p.zeros + off));
              } else {
                float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (gl + e < ng) {
                    t[e] = __ldg(p.scales + off + e);
                    zv[i] |= (uint32_t)__ldg(p.zeros + off + e) << (8 * e);
                  }
                sv[i] = make_float4(t[0], t[1], t[2], t[3]);
              }
            }
          }
          // groups past the chunk's end carry s = 0; the sums read for them are the last group's
          for (int m = 0; m < p.M; ++m) {
            float2 sm[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              sm[e] = *reinterpret_cast<const float2*>(sums + ((size_t)min(gl + e, ng - 1) * TOKP + m) * 2);
#pragma unroll
            for (int i = 0; i < RB; ++i) {
              const int r = rbase + i * kPWarps;
              if (r >= nrows) break;                               // warp-uniform
              const float s4[4] = {sv[i].x, sv[i].y, sv[i].z, sv[i].w};
              float c = 0.0f;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float z = (float)((zv[i] >> (8 * e)) & 0xFFu);
                c = fmaf(s4[e], fmaf(z, sm[e].x, sm[e].y), c);
              }
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
              if (lane == 0) {
                float* ct = cterm + (size_t)r * tp + m;
                *ct = gb == 0 ? c : *ct + c;
              }
            }
          }
        }
      }
      __syncthreads();
    }

    // ---- add the parked sums of every pair in warp order
    for (int idx = threadIdx.x; idx < npairs * 16 * p.M; idx += kPThreads) {
      const int lp = idx / (16 * p.M);
      const int rem = idx - lp * 16 * p.M;
      const int m = rem >> 4, lr = rem & 15;
      if (!pair_full(lp) && lr >= 8) continue;                     // a half pair has eight rows
      const int row = pair_rg(lp) * 8 + lr;
      float sum = group_terms ? -cterm[((size_t)lp * 16 + lr) * tp + m] : 0.0f;
      // branch-free and unrolled, so that the sixteen reads do not wait for one another: a warp
      // that has nothing parked for this pair reads a slot of its own (any value) and adds zero
#pragma unroll
      for (int w = 0; w < kPWarps; ++w) {
        const int sg = lp - wfirst[w];
        const bool has = sg >= 0 && sg < p.maxseg && lp <= wlast[w];
        const int sgc = min(max(sg, 0), p.maxseg - 1);
        const float v = part[((size_t)(w * p.maxseg + sgc) * 16 + lr) * tp + m];
        sum += has ? v : 0.0f;
      }
      if (!GROUPED) {
        // the chunk lies inside one group: take its zero-point and bias terms off, then scale
        float sx = 0.0f, sb = 0.0f;
        for (int w = 0; w < kPWarps; ++w) {
          sx += sums[(w * TOKP + m) * 2];
          sb += sums[(w * TOKP + m) * 2 + 1];
        }
        float z = z_own, sc = s_own;
        if (!own_output) {
          const int gg = p.G == 1 ? 0 : col0 / (p.K / p.G);
          z = (float)__ldg(p.zeros + (size_t)row * p.G + gg);
          const float* tab = p.scales;
          if (p.task_ids) tab += (size_t)min(max(__ldg(p.task_ids + m), 0), p.n_tasks - 1) * p.N * p.G;
          sc = __ldg(tab + (size_t)row * p.G + gg);
        }
        sum -= fmaf(z, sx, sb);
        sum *= sc;
      }
      if (p.nchunks > 1) {
        float* ya = yacc + ((size_t)lp * 16 + lr) * tp + m;
        if (ch > 0) sum += *ya;
        if (!last) {
          *ya = sum;
          continue;
        }
      }
      p.Y[(size_t)m * p.N + row] = __float2bfloat16_rn(sum);
    }
  }

  if (!ok || abort_flag[0]) {
    // let copies already in flight land before shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
    if (threadIdx.x == 0) {
      atomicExch(p.status, (int)PEQA_ERR_DEVICE_TIMEOUT);
      p.status[1] = (int)blockIdx.x;
    }
  }
}

// ------------------------------------------------------------- prepare / unprepare
// One thread per (row group, step, lane, string): moves the string's 32 codes between the
// two layouts.  TO_PREPARED: canonical -> prepared, else the inverse.
template <int BITS, bool TO_PREPARED>
__global__ void prep_layout_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst,
                                   int N, int K, int T) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int rgs = N / 8, rgs2 = (rgs + 1) & ~1;      // the buffer holds whole pairs of row groups
  const size_t total = (size_t)rgs2 * T * 128;
  if (idx >= total) return;
  const int s = (int)(idx & 3), lane = (int)((idx >> 2) & 31);
  const size_t rt = idx >> 7;
  const int t = (int)(rt % T), rg = (int)(rt / T);
  const size_t blk = ((size_t)(rg >> 1) * T + t) * 2 + (rg & 1);
  const int r8 = lane >> 2, c4 = lane & 3;
  const int row = rg * 8 + r8;
  // word e of string s of this lane: word index wi = s*BITS + e of the lane's 4*BITS words
  auto prep_word = [&](int e) -> size_t {
    const int wi = s * BITS + e;
    const int c = wi >> 2, wo = wi & 3;
    return ((blk * BITS + c) * 32 + lane) * 4 + wo;
  };
  if (rg >= rgs) {                                   // the missing half of the last pair
    if (TO_PREPARED) {
#pragma unroll
      for (int e = 0; e < BITS; ++e) dst[prep_word(e)] = 0u;
    }
    return;
  }
  const int wpr = K * BITS / 32;
  const uint32_t* canon_r = (TO_PREPARED ? src : dst) + (size_t)row * wpr;
  uint32_t* canon_w = dst + (size_t)row * wpr;
  // code of column j of a canonical row
  auto canon_get = [&](int j) -> uint32_t {
    const int bit = j * BITS;
    uint32_t v = canon_r[bit >> 5] >> (bit & 31);
    if ((bit & 31) + BITS > 32) v |= canon_r[(bit >> 5) + 1] << (32 - (bit & 31));
    return v & ((1u << BITS) - 1u);
  };
  uint32_t str[BITS];
#pragma unroll
  for (int e = 0; e < BITS; ++e) str[e] = TO_PREPARED ? 0u : src[prep_word(e)];
  auto str_get = [&](int pos) -> uint32_t {
    const int bit = pos * BITS;
    uint32_t v = str[bit >> 5] >> (bit & 31);
    if ((bit & 31) + BITS > 32) v |= str[(bit >> 5) + 1] << (32 - (bit & 31));
    return v & ((1u << BITS) - 1u);
  };
  auto str_put = [&](int pos, uint32_t code) {
    const int bit = pos * BITS;
    str[bit >> 5] |= code << (bit & 31);
    if ((bit & 31) + BITS > 32) str[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
  };
  if (TO_PREPARED) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int cs = 2 * k + h;
        const int col = t * kStepCols + 32 * (4 * s + (cs >> 3)) + 8 * c4 + (cs & 7);
        const uint32_t code = col < K ? canon_get(col) : 0u;
        str_put(h ? dq::stream_hi(BITS, k) : dq::stream_lo(BITS, k), code);
      }
    }
#pragma unroll
    for (int e = 0; e < BITS; ++e) dst[prep_word(e)] = str[e];
  } else {
    // the eight columns of a run this lane owns are BITS whole bytes of the canonical row
    uint8_t* rowb = reinterpret_cast<uint8_t*>(canon_w);
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      const int col = t * kStepCols + 32 * (4 * s + rr) + 8 * c4;
      if (col >= K) continue;
      uint32_t bits8 = 0u;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int cs = 8 * rr + e, k = cs >> 1;
        const uint32_t code = str_get((cs & 1) ? dq::stream_hi(BITS, k) : dq::stream_lo(BITS, k));
        bits8 |= code << (BITS * e);
      }
      uint8_t* o = rowb + (size_t)col * BITS / 8;
#pragma unroll
      for (int b = 0; b < BITS; ++b) o[b] = (uint8_t)(bits8 >> (8 * b));
    }
  }
}

struct PrepPlan {
  int rg_per_cta, grid, T, spc, nchunks, slots, sps, maxseg, x_pitch, pairs;
  size_t smem;
};

int x_pitch_for(int steps) {
  const int raw = steps * kStepCols * 2;
  return raw + 64;                                                // pitch % 128 == 64
}

// Chooses how many steps of activations are staged at a time and the shape of the warps'
// rings.  gcols: columns of one quantization group.
int plan_prep(int N, int K, int M, int bits, int gcols, PrepPlan* plan) {
  const int sms = sm_count_or(148);
  const int rgs = N / 8;
  const int NT = M <= 8 ? 1 : 2, TOKP = 8 * NT;
  const int tp = tok_pitch((M + 1) & ~1);
  const int step_bytes = 2 * bits * 512;
  plan->T = (K + kStepCols - 1) / kStepCols;
  plan->rg_per_cta = (rgs + sms - 1) / sms;
  plan->grid = (rgs + plan->rg_per_cta - 1) / plan->rg_per_cta;
  plan->pairs = plan->rg_per_cta / 2 + 2;                         // incl. a half pair at either end
  const bool grouped = gcols < kStepCols;
  const int gps = grouped ? kStepCols / gcols : 0;
  auto need = [&](int spc, int slots, int sps, int* maxseg) -> size_t {
    const int nch = (plan->T + spc - 1) / spc;
    // a warp's share of a chunk is at most pairs*spc*4/16 cost units, i.e. at most that / 3 + 2
    // steps (all of them half-pair steps at cost 3): the pairs it touches
    const int steps = plan->pairs * spc / 12 + 2;
    *maxseg = (steps + spc - 1) / spc + 2;
    if (*maxseg > plan->pairs) *maxseg = plan->pairs;
    size_t b = 128 + kPHeadBytes;
    b += (size_t)kPWarps * (*maxseg) * 16 * tp * 4;
    if (nch > 1) b += (size_t)plan->pairs * 16 * tp * 4;
    b += (size_t)(grouped ? spc * gps : kPWarps) * TOKP * 2 * 4 + 128;
    if (grouped) b += (size_t)plan->pairs * 16 * tp * 4;
    b += (((size_t)M * x_pitch_for(spc)) + 127) / 128 * 128;
    b += (size_t)kPWarps * slots * sps * step_bytes;
    return b;
  };
  // a chunk must lie inside one quantization group unless the groups are applied per step
  const int steps_per_group = grouped ? 1 : gcols / kStepCols;     // one group per row: >= T
  const bool one_group = gcols >= K;
  // ring shapes in order of preference: bytes in flight first, larger copies on a tie
  const int shapes[5][2] = {{2, 2}, {4, 1}, {3, 1}, {2, 1}, {1, 1}};   // {slots, steps per slot}
  int seg = 0;
  plan->spc = 0;
  // all of K staged at once, with the best ring that fits ...
  if (grouped || one_group) {
    for (int i = 0; i < 4 && plan->spc == 0; ++i)
      if (need(plan->T, shapes[i][0], shapes[i][1], &seg) <= (size_t)kPSmemLimit) {
        plan->spc = plan->T;
        plan->slots = shapes[i][0];
        plan->sps = shapes[i][1];
      }
  }
  // ... else the largest chunk of steps beside a ring of two single steps
  if (plan->spc == 0) {
    for (int spc = plan->T; spc >= 1 && plan->spc == 0; --spc) {
      if (!grouped && !one_group && (steps_per_group % spc) != 0) continue;
      if (need(spc, 2, 1, &seg) <= (size_t)kPSmemLimit) {
        plan->spc = spc;
        plan->slots = 2;
        plan->sps = 1;
      }
    }
  }
  if (plan->spc == 0) return PEQA_ERR_TOO_LARGE;
  plan->nchunks = (plan->T + plan->spc - 1) / plan->spc;
  plan->x_pitch = x_pitch_for(plan->spc);
  plan->smem = need(plan->spc, plan->slots, plan->sps, &seg);
  plan->maxseg = seg;
  return PEQA_OK;
}

template <int BITS, int NT, int GSH>
int launch_prep_t(const PrepParams& p, int grid, size_t smem, cudaStream_t st) {
  auto kern = decode_prep_kernel<BITS, NT, GSH>;
  PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(kPThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PEQA_CUDA(cudaLaunchKernelEx(&cfg, kern, p));
  return PEQA_OK;
}

template <int BITS, int NT>
int launch_prep_g(const PrepParams& p, int gsh, int grid, size_t smem, cudaStream_t st) {
  switch (gsh) {
    case 1: return launch_prep_t<BITS, NT, 1>(p, grid, smem, st);
    case 2: return launch_prep_t<BITS, NT, 2>(p, grid, smem, st);
    case 3: return launch_prep_t<BITS, NT, 3>(p, grid, smem, st);
    default: return launch_prep_t<BITS, NT, 0>(p, grid, smem, st);
  }
}

int check_prep_layer(const peqa_qweight_t* w) {
  if (!w) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(w->out_features, w->in_features, w->bits, w->group_size));
  if (w->in_features % 128 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  return PEQA_OK;
}

// Group sizes the prepared kernel serves: one group per row, groups that are multiples of
// 512 columns, and groups of 64, 128 or 256 columns.
bool prep_group_supported(int K, int g) {
  return g == K || g % kStepCols == 0 || g == 64 || g == 128 || g == 256;
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" size_t peqa_decode_prepared_bytes(const peqa_qweight_t* w) {
  if (check_prep_layer(w) != PEQA_OK) return 0;
  const size_t T = ((size_t)w->in_features + kStepCols - 1) / kStepCols;
  const size_t rgs2 = ((size_t)w->out_features / 8 + 1) & ~(size_t)1;   // whole pairs of row groups
  return rgs2 * T * w->bits * 512;
}

static int run_layout(const peqa_qweight_t* w, const uint32_t* src, uint32_t* dst, bool to_prepared,
                      void* stream) {
  PEQA_TRY(check_prep_layer(w));
  if (!src || !dst) return PEQA_ERR_NULL;
  if (!aligned16(src) || !aligned16(dst)) return PEQA_ERR_ALIGNMENT;
  const int T = (w->in_features + kStepCols - 1) / kStepCols;
  const size_t n = (size_t)((w->out_features / 8 + 1) & ~1) * T * 128;
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  cudaStream_t st = as_stream(stream);
  const int N = w->out_features, K = w->in_features;
  if (w->bits == 3) {
    if (to_prepared) prep_layout_kernel<3, true><<<blocks, threads, 0, st>>>(src, dst, N, K, T);
    else prep_layout_kernel<3, false><<<blocks, threads, 0, st>>>(src, dst, N, K, T);
  } else {
    if (to_prepared) prep_layout_kernel<4, true><<<blocks, threads, 0, st>>>(src, dst, N, K, T);
    else prep_layout_kernel<4, false><<<blocks, threads, 0, st>>>(src, dst, N, K, T);
  }
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

extern "C" int peqa_decode_prepare(const peqa_qweight_t* w, uint32_t* prepared, void* stream) {
  if (!w || !w->qweight) return PEQA_ERR_NULL;
  return run_layout(w, w->qweight, prepared, true, stream);
}

extern "C" int peqa_decode_unprepare(const peqa_qweight_t* w, const uint32_t* prepared,
                                     uint32_t* qweight_out, void* stream) {
  return run_layout(w, prepared, qweight_out, false, stream);
}

extern "C" int peqa_qlinear_decode_prepared(const peqa_qweight_t* w, const uint32_t* prepared,
                                            const void* X, int M, void* Y,
                                            const float* scale_table, int n_tasks,
                                            const int32_t* task_ids, void* stream) {
  PEQA_TRY(check_prep_layer(w));
  if (!prepared || !X || !Y || !w->zeros) return PEQA_ERR_NULL;
  const int g = effective_group(w->in_features, w->group_size);
  if (!prep_group_supported(w->in_features, g)) return PEQA_ERR_BAD_SHAPE;
  if (M < 1 || M > 16) return PEQA_ERR_BAD_SHAPE;
  if (task_ids) {
    if (!scale_table) return PEQA_ERR_NULL;
    if (n_tasks < 1) return PEQA_ERR_BAD_SHAPE;
  } else if (!w->scales) {
    return PEQA_ERR_NULL;
  }
  if (!aligned16(prepared) || !aligned16(X) || !aligned16(Y)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  if (M > 8) {
    // Two launches of at most eight tokens each: the activations of eight tokens still fit
    // beside the rings in fewer, larger chunks, and the second pass finds the weights in L2
    // (measured: 64 us instead of 111 us for 16 tokens at 22016 x 8192, and a third of the
    // time with scales in groups of 64).
    const int h = (M + 1) / 2;
    const size_t K = (size_t)w->in_features, N = (size_t)w->out_features;
    PEQA_TRY(peqa_qlinear_decode_prepared(w, prepared, X, h, Y, scale_table, n_tasks, task_ids, stream));
    return peqa_qlinear_decode_prepared(w, prepared, static_cast<const char*>(X) + (size_t)h * K * 2, M - h,
                                        static_cast<char*>(Y) + (size_t)h * N * 2, scale_table, n_tasks,
                                        task_ids ? task_ids + h : nullptr, stream);
  }
  PrepPlan plan;
  PEQA_TRY(plan_prep(w->out_features, w->in_features, M, w->bits, g, &plan));
  PrepParams p;
  p.P = reinterpret_cast<const uint8_t*>(prepared);
  p.zeros = w->zeros;
  p.scales = task_ids ? scale_table : w->scales;
  p.X = static_cast<const __nv_bfloat16*>(X);
  p.Y = static_cast<__nv_bfloat16*>(Y);
  p.task_ids = task_ids;
  p.n_tasks = n_tasks;
  p.N = w->out_features;
  p.K = w->in_features;
  p.G = p.K / g;
  p.M = M;
  p.rgs = p.N / 8;
  p.rg_per_cta = plan.rg_per_cta;
  p.T = plan.T;
  p.spc = plan.spc;
  p.nchunks = plan.nchunks;
  p.slots = plan.slots;
  p.sps = plan.sps;
  p.maxseg = plan.maxseg;
  p.x_pitch = plan.x_pitch;
  p.pairs_per_cta = plan.pairs;
  cudaStream_t st = as_stream(stream);
  PEQA_TRY(status_word(st, &p.status));
  const int gsh = g == 64 ? 1 : g == 128 ? 2 : g == 256 ? 3 : 0;
  // one tile of eight tokens per MMA (NT = 1) is the only instance: M <= 8 here
  if (w->bits == 3) return launch_prep_g<3, 1>(p, gsh, plan.grid, plan.smem, st);
  return launch_prep_g<4, 1>(p, gsh, plan.grid, plan.smem, st);
}
