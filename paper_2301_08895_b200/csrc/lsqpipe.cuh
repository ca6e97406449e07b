// Least squares on bf16 data, HBM-bound form: Eq. 2 (U = 1) for all selected workers of a round as
// one stream of bulk row copies.
//
// Work item = (selected worker i, group g of 8 minibatch rows).  Items are dealt round-robin to one
// persistent CTA per SM.  A producer warp copies an item's rows X[idx_b][:] (8 KB each at d = 4096)
// and the model vector of the worker's version into a ring of shared-memory stages with
// cp.async.bulk + mbarrier; 512 consumer threads take a stage, each reading ITS columns of all
// rows once into registers (column slice = the 16-byte vector tid of every row), and from those
// registers form the partial dot products (block-reduced in a fixed order to the residuals
// r_b = x_b . w_v - y_b) and then the gradient contribution sum_b r_b x_b into accumulators that
// persist over all items of the CTA.  Every sample row is read from HBM exactly once and from
// shared memory exactly once.  The copies keep up easily (the producer waits for free stages a third
// of the time); what bounds a CTA is the consumers' instruction issue and the shared-memory /
// shuffle pipe, so their inner loops are packed FMAs on operands kept in 64-bit registers and the
// block reduction costs each warp one store, one 16-byte load and 19 shuffles per item.  Eq. 3 only
// needs the sum over workers: a CTA writes one partial sum, and one partial loss sum per item; the
// Eq. 3 kernel adds both up in a fixed order.
#pragma once
#include "common.cuh"
#include "ctl.cuh"
#include "tc.cuh"

namespace absb {
namespace lsqp {

constexpr int GROUP = 8;                 // rows per item / stage
constexpr int CONSUMERS = 512;           // one 16-byte column slice each: d <= 4096
constexpr int NWARPS = CONSUMERS / 32;
constexpr int THREADS = CONSUMERS + 32;  // + producer warp
constexpr int MAX_ITEMS = 64;            // items whose sample indices and targets are staged at once
constexpr int MAX_STAGES = 6;
constexpr int RS = 20;                   // floats between rows of the partial-dot table [GROUP][RS]: 16-byte reads of a row's
                                         // quarters by 8 lanes fall into different banks

struct Args {
  DevState* st;
  RoundInfo* ri;
  const int* sel; const int* job; const int* sel_tau;
  const __nv_bfloat16* X; const float* y;
  const __nv_bfloat16* ring; size_t slot_stride;
  float* loss_part;     // [K * groups] sum over the item's rows of 1/2 r_b^2
  float* G;             // [gridDim.x][slot_stride] per-CTA partial gradient sums
  int d;                // features, multiple of 8, at most 4096
  int stages;           // pipeline depth (2..MAX_STAGES)
  int groups;           // ceil(B / GROUP)
};

inline size_t stage_bytes(int d) { return (size_t)(GROUP + 1) * d * 2; }
inline size_t smem_bytes(int d, int stages) {
  return (size_t)stages * stage_bytes(d) + (size_t)MAX_ITEMS * GROUP * 8 + MAX_ITEMS * 8 + 2 * GROUP * RS * 4 +
         2 * MAX_STAGES * 8 + 64;
}

// Two binary32 values in one 64-bit register (first value in the low word).  The consumers are bound
// by instruction issue: a packed FMA (each half rounds like a scalar fma) halves their FMA count, and
// operands that are created, kept and consumed as 64-bit registers need no moves around it.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// the two bf16 values of a 32-bit word as binary32 values (exact): element 0 (low half) first; a byte
// permute and a mask, both on the integer pipe, so that the FMA pipe is left to the packed FMAs
__device__ __forceinline__ f32x2 bf16x2_to_f32x2(uint32_t u) {
  f32x2 r;
  asm("{\n\t.reg .b32 lo, hi;\n\tprmt.b32 lo, %1, 0, 0x1044;\n\tand.b32 hi, %1, 0xffff0000;\n\tmov.b64 %0, {lo, hi};\n\t}"
      : "=l"(r) : "r"(u));
  return r;
}
__device__ __forceinline__ void ffma2(f32x2& d, f32x2 a, f32x2 b) {      // d += a * b, per half
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

__device__ __forceinline__ void bulk_row(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(THREADS, 1) lsq_pipe_kernel(Args a) {
  grid_dependency_sync();
  extern __shared__ __align__(128) unsigned char lsm[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int K = ri->K, B = st->B, d = a.d, W = st->W, S = st->S, t = ri->t;
  const int groups = a.groups, n_items = K * groups;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = d >> 3;
  const uint32_t row_bytes = (uint32_t)d * 2u;
  const size_t stg = (size_t)(GROUP + 1) * row_bytes;
  const int STAGES = a.stages;
  unsigned char* stage0 = lsm;
  int* m_idx = reinterpret_cast<int*>(lsm + (size_t)STAGES * stg);         // [MAX_ITEMS][GROUP] sample index
  float* m_y = reinterpret_cast<float*>(m_idx + MAX_ITEMS * GROUP);        // [MAX_ITEMS][GROUP] target
  int* m_slot = reinterpret_cast<int*>(m_y + MAX_ITEMS * GROUP);           // [MAX_ITEMS] ring slot of the worker
  float* m_sa = reinterpret_cast<float*>(m_slot + MAX_ITEMS);              // [MAX_ITEMS] weight of the worker's gradient in Eq. 3
  float* red = m_sa + MAX_ITEMS;                                           // [2][GROUP][RS] partial dots, [row][warp]
  uint64_t* full = reinterpret_cast<uint64_t*>(red + 2 * GROUP * RS);      // [STAGES]
  uint64_t* empty = full + MAX_STAGES;                                     // [STAGES]
  volatile int* abort = reinterpret_cast<volatile int*>(empty + MAX_STAGES);
  volatile int* okflag = abort + 1;
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], CONSUMERS / 32); }
    *abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const i64 M = st->n_samples;
  const uint32_t key0 = st->key0, key1 = st->key1;
  // items of this CTA: it = blockIdx.x + q * gridDim.x, q = 0 .. my_items - 1
  const int my_items = n_items > (int)blockIdx.x ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  f32x2 acc[4];                     // gradient sums of this thread's 8 columns (all-zero bits = two zeros)
#pragma unroll
  for (int j = 0; j < 4; ++j) acc[j] = 0ull;
  int stage = 0, buf = 0;
  uint32_t phase = 0;
  bool ok = true;

  for (int q0 = 0; q0 < my_items && ok; q0 += MAX_ITEMS) {
    const int nq = min(MAX_ITEMS, my_items - q0);
    __syncthreads();                        // the staged indices of the previous chunk are no longer read
    // ---- sample indices (Philox block b / 4, word b % 4) and targets of the chunk's rows, all at once
    for (int e = tid; e < nq * GROUP; e += THREADS) {
      const int q = e / GROUP, r = e - q * GROUP;
      const int it = (int)blockIdx.x + (q0 + q) * (int)gridDim.x;
      const int i = it / groups, g = it - i * groups;
      const int b = g * GROUP + r;
      const int wn = a.sel[i];
      if (r == 0) {
        m_slot[q] = (t - a.sel_tau[i]) % (S + 1);
        m_sa[q] = st->sa_penalty ? sa_weight(a.sel_tau[i]) : 1.f;     // staleness-aware step size
      }
      int idx = -1;
      float yv = 0.f;
      if (b < B) {
        const i64 lo = ((i64)wn * M) / W, hi = ((i64)(wn + 1) * M) / W;
        uint32_t w4[4];
        philox4x32_10((uint32_t)wn, (uint32_t)a.job[wn], 1u, (uint32_t)(b >> 2), key0, key1, w4);
        const uint32_t wd = (b & 3) == 0 ? w4[0] : (b & 3) == 1 ? w4[1] : (b & 3) == 2 ? w4[2] : w4[3];
        idx = (int)lo + (int)(((u64)wd * (u64)(hi - lo)) >> 32);
        yv = a.y[idx];
      }
      m_idx[e] = idx;
      m_y[e] = yv;
    }
    __syncthreads();

    if (warp == CONSUMERS / 32) {
      // ------------------------------------------------------------------ producer warp
      for (int q = 0; q < nq; ++q) {
        if (lane == 0) ok = tc::mbar_wait(&empty[stage], phase ^ 1u, abort);
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok) break;
        unsigned char* sb = stage0 + (size_t)stage * stg;
        const int idx = lane < GROUP ? m_idx[q * GROUP + lane] : -1;
        const unsigned rows = __popc(__ballot_sync(0xffffffffu, idx >= 0));
        if (lane == 0) tc::mbar_expect_tx(&full[stage], (rows + 1u) * row_bytes);
        __syncwarp();
        if (idx >= 0) bulk_row(sb + (size_t)lane * row_bytes, a.X + (size_t)idx * d, row_bytes, &full[stage]);
        if (lane == GROUP)
          bulk_row(sb + (size_t)GROUP * row_bytes, a.ring + (size_t)m_slot[q] * a.slot_stride, row_bytes, &full[stage]);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    } else {
      // ------------------------------------------------------------------ consumers
      const int vec = tid;                           // the 16-byte column slice this thread owns
      const bool in = vec < nvec;
      for (int q = 0; q < nq; ++q) {
        // one thread waits (bounded) and tells the others, so all consumers take the same decision
        if (tid == 0) *okflag = tc::mbar_wait(&full[stage], phase, abort) ? 1 : 0;
        asm volatile("bar.sync 2, %0;" ::"n"(CONSUMERS) : "memory");
        if (*okflag == 0) { ok = false; break; }
        (void)tc::mbar_test(&full[stage], phase);     // every thread's own acquire of the copied bytes
        const unsigned char* sb = stage0 + (size_t)stage * stg;
        const int it = (int)blockIdx.x + (q0 + q) * (int)gridDim.x;
        const int g = it % groups;
        const int rows = min(GROUP, B - g * GROUP);
        uint4 xr[GROUP], wr;
        if (rows == GROUP && nvec == CONSUMERS) {      // the usual case (uniform in the CTA): no predicates
          wr = *reinterpret_cast<const uint4*>(sb + (size_t)GROUP * row_bytes + (size_t)vec * 16);
#pragma unroll
          for (int r = 0; r < GROUP; ++r) xr[r] = *reinterpret_cast<const uint4*>(sb + (size_t)r * row_bytes + (size_t)vec * 16);
        } else {
          wr = in ? *reinterpret_cast<const uint4*>(sb + (size_t)GROUP * row_bytes + (size_t)vec * 16) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
          for (int r = 0; r < GROUP; ++r)
            xr[r] = (in && r < rows) ? *reinterpret_cast<const uint4*>(sb + (size_t)r * row_bytes + (size_t)vec * 16)
                                     : make_uint4(0u, 0u, 0u, 0u);
        }
        // the stage is in registers now: hand it back to the producer
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&empty[stage]);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        // partial dot products of the 8 rows over this thread's 8 columns
        float pd[GROUP];
        {
          const f32x2 w2[4] = {bf16x2_to_f32x2(wr.x), bf16x2_to_f32x2(wr.y), bf16x2_to_f32x2(wr.z), bf16x2_to_f32x2(wr.w)};
#pragma unroll
          for (int r = 0; r < GROUP; ++r) {
            f32x2 s2 = 0ull;               // (sum over even columns, sum over odd columns)
            ffma2(s2, bf16x2_to_f32x2(xr[r].x), w2[0]);
            ffma2(s2, bf16x2_to_f32x2(xr[r].y), w2[1]);
            ffma2(s2, bf16x2_to_f32x2(xr[r].z), w2[2]);
            ffma2(s2, bf16x2_to_f32x2(xr[r].w), w2[3]);
            float s0, s1;
            unpack2(s2, s0, s1);
            pd[r] = s0 + s1;
          }
        }
        // warp sum of the 8 values with 9 shuffles: each exchange halves the rows a lane still carries;
        // afterwards lane l holds the warp's sum for row (l >> 2) & 7
        float k4[4], k2[2], k1;
        {
          const bool hi = (lane & 16) != 0;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float recv = __shfl_xor_sync(0xffffffffu, hi ? pd[i] : pd[i + 4], 16);
            k4[i] = (hi ? pd[i + 4] : pd[i]) + recv;
          }
          const bool h8 = (lane & 8) != 0;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float recv = __shfl_xor_sync(0xffffffffu, h8 ? k4[i] : k4[i + 2], 8);
            k2[i] = (h8 ? k4[i + 2] : k4[i]) + recv;
          }
          const bool h4 = (lane & 4) != 0;
          const float recv = __shfl_xor_sync(0xffffffffu, h4 ? k2[0] : k2[1], 4);
          k1 = (h4 ? k2[1] : k2[0]) + recv;
          k1 += __shfl_xor_sync(0xffffffffu, k1, 2);
          k1 += __shfl_xor_sync(0xffffffffu, k1, 1);
        }
        float* rb = red + buf * (GROUP * RS);
        if ((lane & 3) == 0) rb[(lane >> 2) * RS + warp] = k1;
        asm volatile("bar.sync 1, %0;" ::"n"(CONSUMERS) : "memory");
        // every warp adds the 16 warps' sums of a row up in the same order: lane l takes row l & 7 and
        // the four warps of quarter l >> 3 (one 16-byte load), then the quarters are added across lanes
        const int row = lane & 7;
        const float4 four = *reinterpret_cast<const float4*>(rb + row * RS + 4 * (lane >> 3));
        float mine = (four.x + four.y) + (four.z + four.w);
        mine += __shfl_xor_sync(0xffffffffu, mine, 8);
        mine += __shfl_xor_sync(0xffffffffu, mine, 16);
        mine = row < rows ? mine - m_y[q * GROUP + row] : 0.f;
        float res[GROUP], lsum = 0.f;
#pragma unroll
        for (int r = 0; r < GROUP; ++r) {
          res[r] = __shfl_sync(0xffffffffu, mine, r);
          lsum += 0.5f * res[r] * res[r];
        }
        if (tid == 0) a.loss_part[it] = lsum;
        const float sa = m_sa[q];
#pragma unroll
        for (int r = 0; r < GROUP; ++r) {
          const float rr = res[r] * sa;
          const f32x2 r2 = pack2(rr, rr);
          ffma2(acc[0], bf16x2_to_f32x2(xr[r].x), r2);
          ffma2(acc[1], bf16x2_to_f32x2(xr[r].y), r2);
          ffma2(acc[2], bf16x2_to_f32x2(xr[r].z), r2);
          ffma2(acc[3], bf16x2_to_f32x2(xr[r].w), r2);
        }
        buf ^= 1;
      }
    }
    ok = __syncthreads_and(ok ? 1 : 0) != 0;
  }
  // the producer's copies have all been consumed (every full barrier was waited on), unless a wait
  // gave up: then let copies in flight land before the shared memory goes away
  if (!ok && tid == 0) {
    const unsigned long long t0 = tc::global_ns();
    while (tc::global_ns() - t0 < 200000ull) {}
    st->timeout_where = 200;
    st->status = ST_TIMEOUT;
  }
  if (tid < CONSUMERS) {
    float* gout = a.G + (size_t)blockIdx.x * a.slot_stride;
    if (tid < nvec) {
      float g[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) unpack2(acc[j], g[2 * j], g[2 * j + 1]);
      reinterpret_cast<float4*>(gout + (size_t)tid * 8)[0] = make_float4(g[0], g[1], g[2], g[3]);
      reinterpret_cast<float4*>(gout + (size_t)tid * 8)[1] = make_float4(g[4], g[5], g[6], g[7]);
    }
  }
}

}  // namespace lsqp
}  // namespace absb
