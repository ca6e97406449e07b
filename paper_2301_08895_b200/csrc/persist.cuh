// Whole rounds of Algorithm 1 inside one kernel, for least-squares problems so small that a
// round is a few microseconds of work: launch gaps and dependent global-memory round trips
// between kernels would otherwise dominate.  One CTA keeps the version ring and the fp32 master
// copy in shared memory, and per round runs the control step (arrival selection, Eq. 4-6), the
// minibatch gradients of the K arrivals (Eq. 2) and the server step (Eq. 3).  Global memory holds
// the same state as on the multi-kernel path after every round, so the two can be mixed.
#pragma once
#include "common.cuh"
#include "ctl.cuh"
#include "narrow.cuh"

namespace absb {

struct LsqRoundsArgs {
  const void* X; const float* y;
  float* master; void* ring;
  size_t d_pad;
  int d;
  float lr;
};

constexpr int LSQ_ROUNDS_NTG = 256;               // threads that compute gradients (>= number of workers)
constexpr int LSQ_ROUNDS_NT = LSQ_ROUNDS_NTG + 32;  // plus one warp that prepares job durations ahead of time
constexpr int LSQ_ROUNDS_MAX_D = 256;               // a row is at most one warp of 8-element vectors
constexpr int LSQ_ROUNDS_MAX_ROWS = 4096;           // K * B gradient rows of a round

// dynamic shared memory: control-step scratch, ring [S+1][d], master [d], per-warp partial
// gradients [NTG/32][d], per-row losses and ring slots [MAX_ROWS] each, shard bounds [NTG] x 2
__host__ __device__ inline size_t lsq_rounds_smem(int S, int d) {
  return round_up((int)sizeof(CtlShared), 16) +
         4 * ((size_t)(S + 1) * d + d + (LSQ_ROUNDS_NTG / 32) * (size_t)d + 2 * LSQ_ROUNDS_MAX_ROWS + 2 * LSQ_ROUNDS_NTG);
}

// value a ring slot of this element type returns for m
__device__ __forceinline__ float as_stored(const float*, float m) { return m; }
__device__ __forceinline__ float as_stored(const __nv_bfloat16*, float m) { return __bfloat162float(__float2bfloat16_rn(m)); }

__device__ __forceinline__ void gradient_threads_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(LSQ_ROUNDS_NTG) : "memory");
}

template <typename T>
__global__ void __launch_bounds__(LSQ_ROUNDS_NT, 1)
abs_lsq_rounds_kernel(CtlArgs a, LsqRoundsArgs q, int t_first, int n_rounds) {
  constexpr int NT = LSQ_ROUNDS_NT, NTG = LSQ_ROUNDS_NTG, NW = NTG / 32, ITER = 8;
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char rounds_smem[];
  CtlShared& sh = *reinterpret_cast<CtlShared*>(rounds_smem);
  DevState* st = a.st;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool grad_thread = tid < NTG;
  const int W = st->W, S = st->S, B = st->B, d = q.d;
  const i64 M = st->n_samples;
  const uint32_t key0 = st->key0, key1 = st->key1;
  float* ring_s = reinterpret_cast<float*>(rounds_smem + round_up((int)sizeof(CtlShared), 16));   // [S+1][d], values as stored
  float* master_s = ring_s + (size_t)(S + 1) * d;                                                   // [d]
  float* red_s = master_s + d;                                                                      // [NW][d]
  float* rowloss_s = red_s + NW * d;                                                                // [K B]
  int* rslot_s = reinterpret_cast<int*>(rowloss_s + LSQ_ROUNDS_MAX_ROWS);                           // [K B] ring slot of every row
  int* wlo_s = rslot_s + LSQ_ROUNDS_MAX_ROWS;                                                       // [W] shard start of every worker
  unsigned* wlen_s = reinterpret_cast<unsigned*>(wlo_s + NTG);                                      // [W] shard length
  // the sort buffers of the control step are free between two control steps
  int* sidx_s = reinterpret_cast<int*>(sh.keysA);    // [K B] sample index of every row (keysA and keysB, 16 KB)
  const T* X = (const T*)q.X;
  T* ring = (T*)q.ring;
  for (int i = tid; i < (S + 1) * d; i += NT) {
    const int s = i / d, j = i - s * d;
    ring_s[i] = ldf(ring + (size_t)s * q.d_pad, j);
  }
  for (int j = tid; j < d; j += NT) master_s[j] = q.master[j];
  if (tid < W) {                             // shard n = [n M / N, (n+1) M / N)
    const i64 lo = ((i64)tid * M) / W, hi = ((i64)(tid + 1) * M) / W;
    wlo_s[tid] = (int)lo;
    wlen_s[tid] = (unsigned)(hi - lo);
  }
  const int nvec = d >> 3;
  int lpr = 1;                               // lanes that share a row
  while (lpr < nvec) lpr <<= 1;
  const int rpw = 32 / lpr;                  // rows a warp handles at a time
  const int sub = lane / lpr, v = lane - sub * lpr;
  __syncthreads();

  const bool sa_on = st->sa_penalty != 0;          // staleness-aware step size
  for (int r = 0; r < n_rounds; ++r) {
    const int t = t_first + r;
    if (ctl_round<NT>(a, sh, 1, 1, t)) return;
    __syncthreads();
    const int K = sh.scalar[4];
    const int R = K * B;
    if (!grad_thread) {
      // meanwhile the extra warp prepares the duration of the job each worker starts next (it
      // depends on (worker, job index) only), so that the control step finds it ready
      for (int n = lane; n < W; n += 32) {
        const int j = sh.job[n] + 1;
        if (a.dur_job[n] != j) {
          a.next_dur[n] = job_ticks(st->dist, key0, key1, n, j);
          a.dur_job[n] = j;
        }
      }
    } else {
      // sample indices of all K B rows: sample b of job (n, j) = word b%4 of Philox block
      // (n, j, 1, b/4), mapped into the worker's shard; ring slot of every row
      const int blocks_per = (B + 3) >> 2;
      for (int item = tid; item < K * blocks_per; item += NTG) {
        const int i = item / blocks_per, blk = item - i * blocks_per;
        const int wn = sh.sel_n[i];
        const int lo = wlo_s[wn];
        const u64 len = (u64)wlen_s[wn];
        const int slot = sh.version[wn] % (S + 1);            // the arrival computed on w^{t - tau}
        uint32_t w4[4];
        philox4x32_10((uint32_t)wn, (uint32_t)sh.job[wn], 1u, (uint32_t)blk, key0, key1, w4);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (blk * 4 + c < B) {
            sidx_s[i * B + blk * 4 + c] = lo + (int)(((u64)w4[c] * len) >> 32);
            rslot_s[i * B + blk * 4 + c] = slot;
          }
      }
      gradient_threads_sync();
      // Eq. 2 for all arrivals: a group of lpr lanes owns a row, keeps its 8-element piece in
      // registers for both the residual and the gradient, and adds into one running sum because
      // Eq. 3 only needs the sum over the arrivals.  The loads of ITER rows per lane group are
      // issued back to back so that one memory latency covers them all.
      float acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = 0.f;
      const int rows_it = NW * rpw;
      for (int r0 = 0; r0 < R; r0 += ITER * rows_it) {
        float xv[ITER][8], yv[ITER];
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
          const int row = r0 + k * rows_it + warp * rpw + sub;
#pragma unroll
          for (int j = 0; j < 8; ++j) xv[k][j] = 0.f;
          yv[k] = 0.f;
          if (row < R && v < nvec) {
            const int idx = sidx_s[row];
            load8(X + (size_t)idx * d + v * 8, xv[k]);
            if (v == 0) yv[k] = q.y[idx];
          }
        }
#pragma unroll
        for (int k = 0; k < ITER; ++k) {
          if (r0 + k * rows_it >= R) break;                   // same for the whole CTA
          const int row = r0 + k * rows_it + warp * rpw + sub;
          const bool valid = row < R;
          float dot = 0.f;
          if (valid && v < nvec) {
            const float4* w = reinterpret_cast<const float4*>(ring_s + (size_t)rslot_s[row] * d + v * 8);
            const float4 w0 = w[0], w1 = w[1];
            dot = fmaf(xv[k][0], w0.x, dot); dot = fmaf(xv[k][1], w0.y, dot);
            dot = fmaf(xv[k][2], w0.z, dot); dot = fmaf(xv[k][3], w0.w, dot);
            dot = fmaf(xv[k][4], w1.x, dot); dot = fmaf(xv[k][5], w1.y, dot);
            dot = fmaf(xv[k][6], w1.z, dot); dot = fmaf(xv[k][7], w1.w, dot);
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {                  // fixed trip count; steps >= lpr add nothing
            const float other = __shfl_xor_sync(0xffffffffu, dot, o);
            if (o < lpr) dot += other;
          }
          const float res = dot - __shfl_sync(0xffffffffu, yv[k], sub * lpr);
          if (valid && v == 0) rowloss_s[row] = 0.5f * res * res;
          // staleness-aware step size: the row's weight follows from the ring slot it was computed on
          const float rg = (sa_on && valid) ? res * sa_weight((t - rslot_s[row]) % (S + 1)) : res;
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] = fmaf(rg, xv[k][j], acc[j]);   // xv = 0 where there is no row
        }
      }
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float other = __shfl_xor_sync(0xffffffffu, acc[j], o);
          if (o >= lpr) acc[j] += other;
        }
      }
      if (sub == 0 && v < nvec) {
#pragma unroll
        for (int j = 0; j < 8; ++j) red_s[warp * d + v * 8 + j] = acc[j];
      }
    }
    __syncthreads();
    // minibatch loss of each arrival (fixed summation order)
    int bad = 0;
    if (grad_thread) {
      for (int i = warp; i < K; i += NW) {
        float part = 0.f;
        for (int b = lane; b < B; b += 32) part += rowloss_s[i * B + b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        const float loss = __fdiv_rn(part, (float)B);
        if (lane == 0) a.loss[i] = loss;
        bad |= !isfinite(loss);
      }
    }
    bad = __syncthreads_or(bad);
    // Eq. 3: w^{t+1} = w^t - eta / (K B) * sum, to the master copy and to ring slot (t+1) mod (S+1);
    // a non-finite loss leaves the model alone and the next control step reports divergence
    if (!bad) {
      const float step = __fdiv_rn(q.lr, (float)(K * B));
      const int slot = (t + 1) % (S + 1);
      for (int j = tid; j < d; j += NT) {
        float g = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) g += red_s[w * d + j];
        const float m = fmaf(-step, g, master_s[j]);
        master_s[j] = m;
        q.master[j] = m;
        stf(ring + (size_t)slot * q.d_pad, j, m);
        ring_s[(size_t)slot * d + j] = as_stored(ring, m);
      }
    }
    __syncthreads();
  }
  ctl_round<NT>(a, sh, 1, 0, t_first + n_rounds);
}

}  // namespace absb
