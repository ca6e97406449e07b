// Local SGD inside a job (Eq. 2 with U > 1): one CTA per selected worker runs the worker's U
// minibatch steps one after the other on its own copy of the model, which starts at the version the
// worker holds (its ring slot) and lives in shared memory as fp32 (bf16 configurations compute each
// step with the bf16 rounding of that copy, as their tensor-core paths must).  Step u draws its minibatch from
// Philox blocks (n, j, 1, u * ceil(B/4) + b/4).  The upload is the sum over the steps of the
// per-sample gradient sums, G = (B / eta) (w^{.,0} - w^{.,U}), and the average of the U mean
// minibatch losses (Algorithm 1, last worker line); Eq. 3 then reads the K uploads like the
// partial sums of the U = 1 path.  Single-layer models only (least squares, soft-max regression
// with at most 16 classes): their parameter vector fits in shared memory twice.
// The chains of different workers are independent but each is strictly sequential, so the kernel
// is latency-bound by design; a step is B short dot products and one rank-B update.
#pragma once
#include "common.cuh"
#include "ctl.cuh"
#include "narrow.cuh"

namespace absb {
namespace local {

constexpr int MAX_PARAMS = 12288;     // fp32 parameters of the local model (twice in shared memory)
constexpr int MAX_C = 16;
constexpr int MAX_BC = 8192;          // B * C deltas of one step
constexpr int NT_MAX = 1024;          // threads per CTA: only K CTAs run, so a large model gets wide CTAs
inline int threads_for(int n_par) { return n_par >= 2048 ? NT_MAX : 256; }

struct Args {
  DevState* st;
  RoundInfo* ri;
  const int* sel; const int* job; const int* sel_tau;
  const void* X; const void* y;       // y: float targets (least squares) or int labels
  const void* ring; size_t slot_stride;
  float* loss;                        // [W] uploaded loss of each selected worker
  float* G;                           // [W][slot_stride] uploaded gradient sums
  int lsq;                            // 1: least squares (C = 1, no bias)
  int in, C, U;
  float lr;
};

inline size_t smem_bytes(int n_par, int B, int C) {
  return sizeof(float) * ((size_t)2 * n_par + (size_t)B * C + B + 64) + sizeof(int) * (size_t)B;
}

// (d0, d1) += x * (w0, w1) as one packed binary32 FMA (each lane rounds like a scalar fma).
__device__ __forceinline__ void ffma2_bcast(float& d0, float& d1, float x, const float2 w) {
  asm("{\n\t.reg .b64 ra, rb, rc;\n\tmov.b64 ra, {%2, %2};\n\tmov.b64 rb, {%3, %4};\n\tmov.b64 rc, {%0, %1};\n\t"
      "fma.rn.f32x2 rc, ra, rb, rc;\n\tmov.b64 {%0, %1}, rc;\n\t}"
      : "+f"(d0), "+f"(d1) : "f"(x), "f"(w.x), "f"(w.y));
}

template <typename T>
__global__ void __launch_bounds__(NT_MAX) local_sgd_kernel(Args a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char loc_raw[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.x;
  if (i >= ri->K) return;
  const int B = st->B, in = a.in, C = a.C, U = a.U, W = st->W;
  const int n_w = in * C, n_par = a.lsq ? in : n_w + C;
  float* wl = reinterpret_cast<float*>(loc_raw);        // [n_par] local model
  float* gs = wl + n_par;                                // [n_par] sum of the steps' gradient sums
  float* dl = gs + n_par;                                // [B][C] deltas of the step (residuals for least squares)
  float* rl = dl + (size_t)B * C;                        // [B] sample losses of the step
  float* red = rl + B;                                   // [64]
  int* sidx = reinterpret_cast<int*>(red + 64);          // [B] sample indices of the step
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NT = (int)blockDim.x;
  const bool even_c = (C & 1) == 0;
  const int wn = a.sel[i], jb = a.job[wn];
  const int slot = (ri->t - a.sel_tau[i]) % (st->S + 1);
  const T* w0 = (const T*)a.ring + (size_t)slot * a.slot_stride;
  const T* X = (const T*)a.X;
  const i64 M = st->n_samples;
  const i64 lo = ((i64)wn * M) / W, hi = ((i64)(wn + 1) * M) / W;
  const u64 len = (u64)(hi - lo);
  const uint32_t key0 = st->key0, key1 = st->key1;
  const int nblk = (B + 3) >> 2;
  const float step = __fdiv_rn(a.lr, (float)B);
  for (int p = tid; p < n_par; p += NT) { wl[p] = ldf(w0, p); gs[p] = 0.f; }
  float loss_sum = 0.f;
  for (int u = 0; u < U; ++u) {
    for (int blk = tid; blk < nblk; blk += NT) {
      uint32_t w4[4];
      philox4x32_10((uint32_t)wn, (uint32_t)jb, 1u, (uint32_t)(u * nblk + blk), key0, key1, w4);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (blk * 4 + q < B) sidx[blk * 4 + q] = (int)lo + (int)(((u64)w4[q] * len) >> 32);
    }
    __syncthreads();
    // ---- forward at the local model: one warp per row
    for (int b = warp; b < B; b += NT / 32) {
      const T* x = X + (size_t)sidx[b] * in;
      float acc[MAX_C];
#pragma unroll
      for (int c = 0; c < MAX_C; ++c) acc[c] = 0.f;
#pragma unroll 8
      for (int m = lane; m < in; m += 32) {
        const float xv = ldf(x, m);
        if (even_c) {                 // class pairs: one 8-byte shared-memory read and one packed FMA per pair
          const float2* wp = reinterpret_cast<const float2*>(wl + m * C);
#pragma unroll
          for (int c = 0; c < MAX_C; c += 2)
            if (c < C) {
              float2 w = wp[c >> 1];
              w.x = round_store(w.x, (const T*)nullptr);
              w.y = round_store(w.y, (const T*)nullptr);
              ffma2_bcast(acc[c], acc[c + 1], xv, w);
            }
        } else {
#pragma unroll
          for (int c = 0; c < MAX_C; ++c)
            if (c < C) acc[c] = fmaf(xv, round_store(wl[m * C + c], (const T*)nullptr), acc[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < MAX_C; ++c)
        if (c < C) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        }
      if (a.lsq) {
        const float r = acc[0] - ((const float*)a.y)[sidx[b]];
        if (lane == 0) { dl[b] = r; rl[b] = 0.5f * r * r; }
      } else {
        const int y = ((const int*)a.y)[sidx[b]];
        float zmax = -3.0e38f, zy = 0.f;
#pragma unroll
        for (int c = 0; c < MAX_C; ++c)
          if (c < C) { acc[c] += round_store(wl[n_w + c], (const T*)nullptr); zmax = fmaxf(zmax, acc[c]); if (c == y) zy = acc[c]; }
        float se = 0.f;
#pragma unroll
        for (int c = 0; c < MAX_C; ++c)
          if (c < C) { acc[c] = expf(acc[c] - zmax); se += acc[c]; }
        const float inv = 1.f / se;
        float mine = 0.f;
#pragma unroll
        for (int c = 0; c < MAX_C; ++c)
          if (c == lane) mine = acc[c] * inv - (c == y ? 1.f : 0.f);
        // a delta is a stored quantity of the bf16 configurations: rounded like every other delta
        if (lane < C) dl[b * C + lane] = round_store(mine, (const T*)nullptr);
        if (lane == 0) rl[b] = logf(se) - (zy - zmax);
      }
    }
    __syncthreads();
    // ---- mean loss of the step (fixed order: strided partial sums, then a shuffle tree, then the warps in order)
    {
      float part = 0.f;
      for (int b = tid; b < B; b += NT) part += rl[b];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      if (lane == 0) red[warp] = part;
    }
    // ---- gradient sum of the step, one feature per thread (all classes), and the local step
    for (int m = tid; m < in; m += NT) {
      float acc[MAX_C];
#pragma unroll
      for (int c = 0; c < MAX_C; ++c) acc[c] = 0.f;
#pragma unroll 8
      for (int b = 0; b < B; ++b) {
        const float xv = ldf(X, (size_t)sidx[b] * in + m);
        if (even_c) {
          const float2* dp = reinterpret_cast<const float2*>(dl + b * C);
#pragma unroll
          for (int c = 0; c < MAX_C; c += 2)
            if (c < C) ffma2_bcast(acc[c], acc[c + 1], xv, dp[c >> 1]);
        } else {
#pragma unroll
          for (int c = 0; c < MAX_C; ++c)
            if (c < C) acc[c] = fmaf(xv, dl[b * C + c], acc[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < MAX_C; ++c)
        if (c < C) {
          gs[m * C + c] += acc[c];
          wl[m * C + c] = fmaf(-step, acc[c], wl[m * C + c]);
        }
    }
    if (!a.lsq && tid < C) {
      float acc = 0.f;
      for (int b = 0; b < B; ++b) acc += dl[b * C + tid];
      gs[n_w + tid] += acc;
      wl[n_w + tid] = fmaf(-step, acc, wl[n_w + tid]);
    }
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
      for (int q = 0; q < NT / 32; ++q) tot += red[q];
      loss_sum += __fdiv_rn(tot, (float)B);
    }
  }
  float* g = a.G + (size_t)i * a.slot_stride;
  const float sa = st->sa_penalty ? sa_weight(a.sel_tau[i]) : 1.f;   // staleness-aware step size: weight of the upload in Eq. 3
  for (int p = tid; p < n_par; p += NT) g[p] = gs[p] * sa;
  if (tid == 0) {
    const float loss = __fdiv_rn(loss_sum, (float)U);
    a.loss[i] = loss;
    if (!isfinite(loss)) ri->diverged = 1;
  }
}

}  // namespace local
}  // namespace absb
