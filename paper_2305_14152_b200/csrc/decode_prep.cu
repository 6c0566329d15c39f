// Small-batch forward (token generation) from a prepared copy of the frozen
// weights:  Y[m,i] = s[i] * sum_j X[m,j] * (Q[i,j] - z[i])   (Eq. 2, M <= 16 tokens,
// one scale per channel; Sec. 3.1 / 3.3: the memory-bound matrix-vector regime).
//
// The frozen matrix never changes after quantization (Sec. 3.3), so a server
// can keep it in whatever order suits the kernel.  The prepared layout stores the
// same bits as the canonical packed matrix, rearranged so that
//   * the 16-byte piece every lane of a warp needs next lies in one contiguous
//     512-byte run (no shared-memory staging of the weights: they go from HBM
//     straight to registers, several 16-byte loads per lane in flight), and
//   * inside every 32-column run, the two codes one logic operation extracts as
//     a bf16 pair are the codes of two ADJACENT columns, so the activations are
//     used in their natural order.
//
// Layout.  rg = row / 8, r = row % 8, unit u = column / 128 (U = K / 128 units),
// C = bits (16-byte chunks per unit of one row: 48 or 64 bytes).  Chunk c of the
// unit (row, u) is stored at 16-byte index ((rg * C + c) * U + u) * 8 + r.  The
// 4*bits words of a unit are its four 32-column runs in order; within a run, the
// code of column 2k sits at bit position bits*stream_lo(k) and the code of column
// 2k+1 at bits*stream_hi(k) (k = 0..15; dequant.cuh).
//
// Work split.  One CTA per SM owns a contiguous range of 8-row groups and all
// of K for them, so no sum crosses a CTA: no workspace, no atomics.  Two row
// groups form a "pair", the 16 rows of a warp-level mma.m16n8k16 whose 8-wide
// side are the tokens.  Lane (r, c) = (lane / 4, lane % 4) holds, for rows r of
// both groups, one unit of 128 columns; a warp step is four units.  The sixteen
// warps are arranged as PG pairs x S splits of the unit range, chosen on the
// host so that all warps have the same number of steps.  Codes reach the tensor
// core as the biased integers (bias + q) they are after one logic operation;
// the zero-point and bias terms come off the sum at the end:
//   y = s * (acc - z * sum_j x_j - sum_j bias_j x_j).
// Warps' partial sums meet in shared memory after each round and are added in
// warp order, so results do not depend on timing.
//
// Activations are staged in shared memory, all of K when they fit, otherwise in
// chunks of units with the per-output sums carried in shared memory.
//
// Launch overlap.  The kernel is launched with programmatic stream
// serialization: it lets the next kernel in the stream start as soon as SMs
// free up, requests its own first weights at once, and only then waits for the
// preceding kernel before it touches X or Y.  The prepared weights, zero-points
// and scales are therefore read before earlier work in the stream is known to be
// complete: they must be final when the call is made.
#include <cuda_bf16.h>

#include "common.cuh"
#include "dequant.cuh"
#include "sm100_ptx.cuh"

namespace peqa {

namespace {

constexpr int kPWarps = 16;
constexpr int kPThreads = kPWarps * 32;
constexpr int kPUnitPitch = 272;                   // 128 activations (256 B) + 16 B bank skew
constexpr int kPSmemLimit = 227 * 1024;

struct PrepParams {
  const uint4* P;           // prepared weights
  const uint8_t* zeros;     // [N]
  const float* scales;      // [N] or table [n_tasks, N]
  const __nv_bfloat16* X;   // [M, K]
  __nv_bfloat16* Y;         // [M, N]
  const int32_t* task_ids;  // nullptr: one task
  int n_tasks;
  int N, K, U, M;
  int rgs;                  // row groups in the matrix (N / 8)
  int rg_per_cta;
  int S, PG;                // splits of a pair's unit range, pairs per round (S * PG = 16)
  int rounds;               // ceil(pairs per CTA / PG)
  int chunk_units;          // units of K staged at a time
  int nchunks;
  int ups;                  // units per split within a full chunk (multiple of 4)
  int spr;                  // steps per split and round (ups / 4)
  int x_pitch;              // bytes between staged token rows
  int pairs_per_cta;
};

__device__ __forceinline__ void pmma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                           uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
      "{%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// One lane's weights of one step: rows r of the pair's two groups, one unit each.
template <int BITS>
struct StepRegs {
  uint4 a[BITS];
  uint4 b[BITS];
};

// MMAs 2*MM and 2*MM + 1 of a 32-column run: the run's pairs 4*MM .. 4*MM + 3, i.e. its
// columns 8*MM .. 8*MM + 7, whose activations are one 16-byte word per token.
template <int BITS, int NT, int MM>
__device__ __forceinline__ void run_mma2(const uint32_t (&wa)[BITS], const uint32_t (&wb)[BITS],
                                         bool has_b, const uint8_t* x0, const uint8_t* x1,
                                         float (&acc)[NT][4]) {
  const uint4 xa = *reinterpret_cast<const uint4*>(x0 + MM * 16);
  uint4 xb = make_uint4(0u, 0u, 0u, 0u);
  if (NT == 2) xb = *reinterpret_cast<const uint4*>(x1 + MM * 16);
  uint32_t f0[4], f1[4];
  dq::mma_pairs_stream<BITS, 2 * MM>(wa, f0[0], f0[2]);
  dq::mma_pairs_stream<BITS, 2 * MM + 1>(wa, f1[0], f1[2]);
  f0[1] = f0[3] = f1[1] = f1[3] = 0u;
  if (has_b) {
    dq::mma_pairs_stream<BITS, 2 * MM>(wb, f0[1], f0[3]);
    dq::mma_pairs_stream<BITS, 2 * MM + 1>(wb, f1[1], f1[3]);
  }
  pmma_16816(acc[0], f0, xa.x, xa.y);
  pmma_16816(acc[0], f1, xa.z, xa.w);
  if (NT == 2) {
    pmma_16816(acc[1], f0, xb.x, xb.y);
    pmma_16816(acc[1], f1, xb.z, xb.w);
  }
}

template <int BITS, int NT>
__device__ __forceinline__ void step_compute(const StepRegs<BITS>& w, bool has_b, const uint8_t* x0,
                                             const uint8_t* x1, float (&acc)[NT][4]) {
  const uint32_t* fa = reinterpret_cast<const uint32_t*>(w.a);
  const uint32_t* fb = reinterpret_cast<const uint32_t*>(w.b);
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    uint32_t wa[BITS], wb[BITS];
#pragma unroll
    for (int e = 0; e < BITS; ++e) {
      wa[e] = fa[s * BITS + e];
      wb[e] = fb[s * BITS + e];
    }
    run_mma2<BITS, NT, 0>(wa, wb, has_b, x0 + s * 64, x1 + s * 64, acc);
    run_mma2<BITS, NT, 1>(wa, wb, has_b, x0 + s * 64, x1 + s * 64, acc);
    run_mma2<BITS, NT, 2>(wa, wb, has_b, x0 + s * 64, x1 + s * 64, acc);
    run_mma2<BITS, NT, 3>(wa, wb, has_b, x0 + s * 64, x1 + s * 64, acc);
  }
}

// Bias the code of column j (0..31) of a run carries when it reaches the tensor core.
template <int BITS>
__host__ __device__ constexpr float column_bias(int j) {
  if (BITS == 4) return 128.0f;
  return dq::stream_alt(3, j >> 1) ? ((j & 1) ? 16.0f : 64.0f) : ((j & 1) ? 128.0f : 8.0f);
}

template <int BITS, int NT>
__global__ void __launch_bounds__(kPThreads, 1)
decode_prep_kernel(const PrepParams p) {
  constexpr int C = BITS;                            // 16-byte chunks per unit of one row
  constexpr int TOKP = 8 * NT;
  extern __shared__ uint8_t prep_smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(prep_smem_raw) + 127) &
                                             ~static_cast<uintptr_t>(127));
  float* partial = reinterpret_cast<float*>(base);                 // [2][16 warps][16 rows][TOKP]
  float* yacc = partial + 2 * kPWarps * 16 * TOKP;                  // [pairs][16][TOKP]
  float* xtot = yacc + (size_t)p.pairs_per_cta * 16 * TOKP;         // [TOKP][2]: sum x, sum bias*x
  uint8_t* xzero = reinterpret_cast<uint8_t*>(xtot + TOKP * 2);     // 256 B of zeros
  uint8_t* xs = xzero + 256;                                        // [M][x_pitch]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r8 = lane >> 2, c4 = lane & 3;
  const int rg0 = blockIdx.x * p.rg_per_cta;
  const int rg_end = min(p.rgs, rg0 + p.rg_per_cta);
  const int split = warp % p.S, pr = warp / p.S;

  // the next kernel of the stream may be scheduled as SMs free up
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- weight stream of this warp: step i = (chunk, round, st)
  const int steps_per_chunk = p.rounds * p.spr;
  const int total = p.nchunks * steps_per_chunk;
  auto step_unit = [&](int i, int& chunk, int& round, bool& active) -> int {
    chunk = i / steps_per_chunk;
    const int rem = i - chunk * steps_per_chunk;
    round = rem / p.spr;
    const int st = rem - round * p.spr;
    const int cu0 = chunk * p.chunk_units;
    const int cend = min(p.U, cu0 + p.chunk_units);
    const int u = cu0 + split * p.ups + 4 * st + c4;
    active = u < min(cend, cu0 + (split + 1) * p.ups);
    return u;
  };
  auto load_step = [&](int i, StepRegs<BITS>& w) {
#pragma unroll
    for (int c = 0; c < C; ++c) {
      w.a[c] = make_uint4(0u, 0u, 0u, 0u);
      w.b[c] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (i >= total) return;
    int chunk, round;
    bool active;
    const int u = step_unit(i, chunk, round, active);
    const int rga = rg0 + 2 * (round * p.PG + pr);
    if (!active || rga >= rg_end) return;
    const size_t plane = (size_t)p.U * 8;                         // 16-byte pieces per (rg, c)
    const uint4* pa = p.P + (size_t)rga * C * plane + (size_t)u * 8 + r8;
#pragma unroll
    for (int c = 0; c < C; ++c) w.a[c] = ldg_stream(pa + c * plane);
    if (rga + 1 < rg_end) {
      const uint4* pb = pa + C * plane;
#pragma unroll
      for (int c = 0; c < C; ++c) w.b[c] = ldg_stream(pb + c * plane);
    }
  };

  StepRegs<BITS> w0, w1;
  load_step(0, w0);
  load_step(1, w1);

  for (int i = threadIdx.x; i < 64 + TOKP * 2; i += kPThreads) {
    if (i < 64) reinterpret_cast<uint32_t*>(xzero)[i] = 0u;
    else xtot[i - 64] = 0.0f;
  }

  // everything below reads X or writes Y: the preceding kernel must have completed
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // bias of the eight columns of a 16-byte piece of X: piece q = (piece index) % 4 of its run
  float bias8[8];
  {
    const int q = lane & 3;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float b = column_bias<BITS>(e);
      if (q == 1) b = column_bias<BITS>(8 + e);
      if (q == 2) b = column_bias<BITS>(16 + e);
      if (q == 3) b = column_bias<BITS>(24 + e);
      bias8[e] = b;
    }
  }

  int i = 0;
  for (int chunk = 0; chunk < p.nchunks; ++chunk) {
    const int cu0 = chunk * p.chunk_units;
    const int cun = min(p.U, cu0 + p.chunk_units) - cu0;           // units in this chunk
    if (chunk > 0) __syncthreads();                                // the previous chunk is no longer read
    // ---- stage X[:, chunk]: 16 pieces of 16 bytes per unit and token
    for (int idx = threadIdx.x; idx < p.M * cun * 16; idx += kPThreads) {
      const int m = idx / (cun * 16);
      const int rem = idx - m * cun * 16;
      const int uu = rem >> 4, piece = rem & 15;
      ptx::cp_async_16(ptx::smem_u32(xs + (size_t)m * p.x_pitch + uu * kPUnitPitch + piece * 16),
                       p.X + (size_t)m * p.K + (size_t)(cu0 + uu) * 128 + piece * 8);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    // ---- per token: sum of x and sum of bias * x over the chunk, added to the running totals
    if (warp < p.M) {
      float sx = 0.0f, sb = 0.0f;
      const uint8_t* row = xs + (size_t)warp * p.x_pitch;
      for (int pc = lane; pc < cun * 16; pc += 32) {               // pc % 4 == lane % 4
        const uint4 v = *reinterpret_cast<const uint4*>(row + (pc >> 4) * kPUnitPitch + (pc & 15) * 16);
        const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(wv[e] << 16), hi = __uint_as_float(wv[e] & 0xFFFF0000u);
          sx += lo + hi;
          sb = fmaf(bias8[2 * e], lo, sb);
          sb = fmaf(bias8[2 * e + 1], hi, sb);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sx += __shfl_xor_sync(0xffffffffu, sx, o);
        sb += __shfl_xor_sync(0xffffffffu, sb, o);
      }
      if (lane == 0) {
        xtot[warp * 2] += sx;
        xtot[warp * 2 + 1] += sb;
      }
    }

    for (int round = 0; round < p.rounds; ++round) {
      const int pair = round * p.PG + pr;
      const int rga = rg0 + 2 * pair;
      const bool has_b = rga + 1 < rg_end;
      float acc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = 0.0f;

      for (int st = 0; st < p.spr; ++st, ++i) {
        int ch2, rd2;
        bool active;
        const int u = step_unit(i, ch2, rd2, active);
        active = active && rga < rg_end;
        const uint8_t* x0 = xzero;
        const uint8_t* x1 = xzero;
        if (active) {
          const uint8_t* xu = xs + (u - cu0) * kPUnitPitch;
          x0 = xu + (size_t)(r8 < p.M ? r8 : 0) * p.x_pitch;
          x1 = xu + (size_t)(r8 + 8 < p.M ? r8 + 8 : 0) * p.x_pitch;
        }
        step_compute<BITS, NT>(w0, has_b, x0, x1, acc);
        w0 = w1;
        load_step(i + 2, w1);
      }

      // ---- this warp's partial sums: [16 rows][TOKP]
      const int buf = (chunk * p.rounds + round) & 1;
      float* mine = partial + (size_t)((buf * kPWarps + warp) * 16) * TOKP;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int tk = nt * 8 + c4 * 2;
        *reinterpret_cast<float2*>(mine + r8 * TOKP + tk) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2*>(mine + (r8 + 8) * TOKP + tk) = make_float2(acc[nt][2], acc[nt][3]);
      }
      __syncthreads();
      // ---- add the splits of every pair of this round in warp order
      const float* bufp = partial + (size_t)(buf * kPWarps * 16) * TOKP;
      for (int idx = threadIdx.x; idx < p.PG * 16 * p.M; idx += kPThreads) {
        const int q = idx / (16 * p.M);
        const int rem = idx - q * 16 * p.M;
        const int m = rem >> 4, lr = rem & 15;
        const int pr2 = round * p.PG + q;
        const int rg = rg0 + 2 * pr2 + (lr >> 3);
        if (rg >= rg_end) continue;
        float sum = 0.0f;
        for (int sp = 0; sp < p.S; ++sp) sum += bufp[((q * p.S + sp) * 16 + lr) * TOKP + m];
        if (p.nchunks > 1) {
          float* ya = yacc + ((size_t)pr2 * 16 + lr) * TOKP + m;
          if (chunk > 0) sum += *ya;
          if (chunk + 1 < p.nchunks) {
            *ya = sum;
            continue;
          }
        }
        const int row = rg * 8 + (lr & 7);
        const float z = (float)__ldg(p.zeros + row);
        const float* sc = p.scales;
        if (p.task_ids) {
          const int task = min(max(__ldg(p.task_ids + m), 0), p.n_tasks - 1);
          sc += (size_t)task * p.N;
        }
        sum = (sum - fmaf(z, xtot[m * 2], xtot[m * 2 + 1])) * __ldg(sc + row);
        p.Y[(size_t)m * p.N + row] = __float2bfloat16_rn(sum);
      }
    }
  }
}

// ------------------------------------------------------------- prepare / unprepare
// One thread per (row, 32-column run): moves the run's words between the two layouts and
// permutes the codes inside it.  TO_PREPARED: canonical -> prepared, else the inverse.
template <int BITS, bool TO_PREPARED>
__global__ void prep_layout_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst,
                                   int N, int K) {
  const int runs = K / 32, U = K / 128;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)N * runs) return;
  const int row = (int)(idx / runs), run = (int)(idx - (size_t)row * runs);
  const int u = run >> 2, s = run & 3;
  const int rg = row >> 3, r = row & 7;
  const uint32_t* canon = (TO_PREPARED ? src : dst) + (size_t)row * (K * BITS / 32) + (size_t)run * BITS;
  uint32_t* canon_w = const_cast<uint32_t*>(canon);
  auto prep_word = [&](int e) -> size_t {
    const int wi = s * BITS + e;
    const int c = wi >> 2, wo = wi & 3;
    return ((((size_t)rg * BITS + c) * U + u) * 8 + r) * 4 + wo;
  };
  uint32_t in[BITS], out[BITS];
#pragma unroll
  for (int e = 0; e < BITS; ++e) {
    in[e] = TO_PREPARED ? canon[e] : src[prep_word(e)];
    out[e] = 0u;
  }
  auto get = [&](int pos) -> uint32_t {
    const int bit = pos * BITS;
    uint32_t v = in[bit >> 5] >> (bit & 31);
    if ((bit & 31) + BITS > 32) v |= in[(bit >> 5) + 1] << (32 - (bit & 31));
    return v & ((1u << BITS) - 1u);
  };
  auto put = [&](int pos, uint32_t code) {
    const int bit = pos * BITS;
    out[bit >> 5] |= code << (bit & 31);
    if ((bit & 31) + BITS > 32) out[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
  };
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int lo = dq::stream_lo(BITS, k), hi = dq::stream_hi(BITS, k);
    if (TO_PREPARED) {
      put(lo, get(2 * k));
      put(hi, get(2 * k + 1));
    } else {
      put(2 * k, get(lo));
      put(2 * k + 1, get(hi));
    }
  }
#pragma unroll
  for (int e = 0; e < BITS; ++e) {
    if (TO_PREPARED) dst[prep_word(e)] = out[e];
    else canon_w[e] = out[e];
  }
}

struct PrepPlan {
  int rg_per_cta, grid, S, PG, rounds, chunk_units, nchunks, ups, spr, x_pitch, pairs;
  size_t smem;
};

int x_pitch_for(int units) {
  const int raw = units * kPUnitPitch;
  return raw + ((64 - raw % 128) % 128 + 128) % 128;              // pitch % 128 == 64
}

// Chooses the split of the sixteen warps (PG pairs x S splits) and the units of K staged at a
// time so that the warps' step counts are equal and as small as possible.
int plan_prep(int N, int K, int M, PrepPlan* plan) {
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int rgs = N / 8, U = K / 128;
  const int NT = M <= 8 ? 1 : 2, TOKP = 8 * NT;
  plan->rg_per_cta = (rgs + sms - 1) / sms;
  plan->grid = (rgs + plan->rg_per_cta - 1) / plan->rg_per_cta;
  plan->pairs = (plan->rg_per_cta + 1) / 2;
  const size_t fixed = 128 + (size_t)2 * kPWarps * 16 * TOKP * 4 + (size_t)plan->pairs * 16 * TOKP * 4 +
                       (size_t)TOKP * 2 * 4 + 256 + 64;
  long long best = -1;
  for (int S = 1; S <= kPWarps; S *= 2) {
    const int PG = kPWarps / S;
    const int rounds = (plan->pairs + PG - 1) / PG;
    // largest chunk that fits, a multiple of 4 * S units unless all of K fits
    int cu = U;
    while (cu > 0 && fixed + (size_t)M * x_pitch_for(cu) > (size_t)kPSmemLimit) --cu;
    if (cu <= 0) continue;
    if (cu < U) cu -= cu % (4 * S);
    if (cu <= 0) continue;
    long long cost = 0;
    const int nchunks = (U + cu - 1) / cu;
    for (int c = 0; c < nchunks; ++c) {
      const int ups = (((cu + S - 1) / S + 3) / 4) * 4;
      cost += (long long)rounds * (ups / 4) * 8 + rounds + 6;      // steps (x8), barriers, staging
    }
    if (best < 0 || cost < best) {
      best = cost;
      plan->S = S;
      plan->PG = PG;
      plan->rounds = rounds;
      plan->chunk_units = cu;
      plan->nchunks = nchunks;
      plan->ups = (((cu + S - 1) / S + 3) / 4) * 4;
      plan->spr = plan->ups / 4;
      plan->x_pitch = x_pitch_for(cu);
      plan->smem = fixed + (size_t)M * plan->x_pitch;
    }
  }
  return best < 0 ? PEQA_ERR_TOO_LARGE : PEQA_OK;
}

template <int BITS, int NT>
int launch_prep_t(const PrepParams& p, int grid, size_t smem, cudaStream_t st) {
  auto kern = decode_prep_kernel<BITS, NT>;
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

int check_prep_layer(const peqa_qweight_t* w) {
  if (!w) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(w->out_features, w->in_features, w->bits, w->group_size));
  if (w->in_features % 128 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  return PEQA_OK;
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" size_t peqa_decode_prepared_bytes(const peqa_qweight_t* w) {
  if (check_prep_layer(w) != PEQA_OK) return 0;
  return (size_t)w->out_features * w->in_features * w->bits / 8;
}

static int run_layout(const peqa_qweight_t* w, const uint32_t* src, uint32_t* dst, bool to_prepared,
                      void* stream) {
  PEQA_TRY(check_prep_layer(w));
  if (!src || !dst) return PEQA_ERR_NULL;
  if (!aligned16(src) || !aligned16(dst)) return PEQA_ERR_ALIGNMENT;
  const size_t n = (size_t)w->out_features * (w->in_features / 32);
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  cudaStream_t st = as_stream(stream);
  if (w->bits == 3) {
    if (to_prepared) prep_layout_kernel<3, true><<<blocks, threads, 0, st>>>(src, dst, w->out_features, w->in_features);
    else prep_layout_kernel<3, false><<<blocks, threads, 0, st>>>(src, dst, w->out_features, w->in_features);
  } else {
    if (to_prepared) prep_layout_kernel<4, true><<<blocks, threads, 0, st>>>(src, dst, w->out_features, w->in_features);
    else prep_layout_kernel<4, false><<<blocks, threads, 0, st>>>(src, dst, w->out_features, w->in_features);
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
  if (effective_group(w->in_features, w->group_size) != w->in_features) return PEQA_ERR_BAD_SHAPE;
  if (M < 1 || M > 16) return PEQA_ERR_BAD_SHAPE;
  if (task_ids) {
    if (!scale_table) return PEQA_ERR_NULL;
    if (n_tasks < 1) return PEQA_ERR_BAD_SHAPE;
  } else if (!w->scales) {
    return PEQA_ERR_NULL;
  }
  if (!aligned16(prepared) || !aligned16(X) || !aligned16(Y)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  PrepPlan plan;
  PEQA_TRY(plan_prep(w->out_features, w->in_features, M, &plan));
  PrepParams p;
  p.P = reinterpret_cast<const uint4*>(prepared);
  p.zeros = w->zeros;
  p.scales = task_ids ? scale_table : w->scales;
  p.X = static_cast<const __nv_bfloat16*>(X);
  p.Y = static_cast<__nv_bfloat16*>(Y);
  p.task_ids = task_ids;
  p.n_tasks = n_tasks;
  p.N = w->out_features;
  p.K = w->in_features;
  p.U = p.K / 128;
  p.M = M;
  p.rgs = p.N / 8;
  p.rg_per_cta = plan.rg_per_cta;
  p.S = plan.S;
  p.PG = plan.PG;
  p.rounds = plan.rounds;
  p.chunk_units = plan.chunk_units;
  p.nchunks = plan.nchunks;
  p.ups = plan.ups;
  p.spr = plan.spr;
  p.x_pitch = plan.x_pitch;
  p.pairs_per_cta = plan.pairs;
  cudaStream_t st = as_stream(stream);
  const int NT = M <= 8 ? 1 : 2;
  if (w->bits == 3)
    return NT == 1 ? launch_prep_t<3, 1>(p, plan.grid, plan.smem, st) : launch_prep_t<3, 2>(p, plan.grid, plan.smem, st);
  return NT == 1 ? launch_prep_t<4, 1>(p, plan.grid, plan.smem, st) : launch_prep_t<4, 2>(p, plan.grid, plan.smem, st);
}
