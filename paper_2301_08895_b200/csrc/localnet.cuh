// Local SGD inside a job (Eq. 2 with U > 1) for multi-layer networks.
// After its first local step every selected worker computes with weights of its own, so the
// workers' copies live in HBM: an fp32 copy (the local model), for the bf16 configurations a bf16
// copy of it (the operand the gradient kernels read), and the fp32 sum of the steps' gradient sums
// (the upload), each [W][d_pad] and indexed by the worker's position in the round's selection.
// One local step of all selected workers is one pass of the grouped forward / backward kernels
// (tensor-core or FP32-FMA, as for U = 1) in which
//   - the rows of worker i are rows [i * RBp, i * RBp + B) (RBp = B rounded up to the row-tile
//     height; the rest is padding with sample index -1),
//   - the "model version" of a row tile is the worker's own copy (slot i of the private store), and
//   - the weight gradient is split per worker (split i = the rows of worker i) instead of summed,
// followed by the workers' local updates.  Eq. 3 then adds the K uploads like the partial sums of
// the U = 1 path.  Minibatch of step u: Philox blocks (n, j, 1, u * ceil(B/4) + b/4).
#pragma once
#include "common.cuh"
#include "ctl.cuh"

namespace absb {
namespace lnet {

struct Args {
  DevState* st;
  RoundInfo* ri;
  const int* sel; const int* job; const int* sel_tau;
  int* row_idx; int* tile_slot;        // the round's row layout, rewritten for every local step
  const void* ring;                    // [S+1][d_pad] model versions, storage type
  __nv_bfloat16* priv16;               // [W][d_pad] bf16 operand copies of the local models (bf16 configurations)
  float* priv32;                       // [W][d_pad] local models
  float* gsum;                         // [W][d_pad] uploads: sum over the steps of the gradient sums
  const float* G;                      // [W][d_pad] gradient sums of the current step, per worker
  const float* row_loss;               // sample losses of the current step, by row
  float* loss_acc;                     // [W] sum of the steps' mean losses
  float* loss;                         // [W] uploaded losses
  size_t d_pad;
  int RBp;                             // rows reserved per worker
  int U;
  float lr;
};

// Start of a job's local steps: the worker's copies are the model version it holds.
template <typename T>
__global__ void __launch_bounds__(256) local_begin_kernel(Args a) {
  grid_dependency_sync();
  const DevState* st = a.st;
  const RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  const int slot = (ri->t - a.sel_tau[i]) % (st->S + 1);
  const T* ring_slot = (const T*)a.ring + (size_t)slot * a.d_pad;
  uint2* d16 = reinterpret_cast<uint2*>(a.priv16 + (size_t)i * a.d_pad);
  float4* d32 = reinterpret_cast<float4*>(a.priv32 + (size_t)i * a.d_pad);
  float4* gs = reinterpret_cast<float4*>(a.gsum + (size_t)i * a.d_pad);
  const size_t n4 = a.d_pad / 4;
  for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (size_t)gridDim.x * blockDim.x) {
    if (sizeof(T) == 4) {
      d32[v] = reinterpret_cast<const float4*>(ring_slot)[v];
    } else {
      const uint2 pk = reinterpret_cast<const uint2*>(ring_slot)[v];
      d16[v] = pk;
      const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&pk.x);
      const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&pk.y);
      const float2 f0 = __bfloat1622float2(lo), f1 = __bfloat1622float2(hi);
      d32[v] = make_float4(f0.x, f0.y, f1.x, f1.y);
    }
    gs[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) a.loss_acc[i] = 0.f;
}

// Row layout of local step u: sample indices of every selected worker's minibatch, the owner of
// every row tile, and the row count of the pass.
__global__ void __launch_bounds__(128) local_layout_kernel(Args a, int u) {
  grid_dependency_sync();
  const DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int K = ri->K;
  if (blockIdx.x == 0 && threadIdx.x == 0) ri->n_rows = K * a.RBp;
  const int i = blockIdx.x;
  if (i >= K) return;
  const int B = st->B, W = st->W, RB = st->RB;
  const int wn = a.sel[i], jb = a.job[wn];
  const i64 M = st->n_samples;
  const i64 lo = ((i64)wn * M) / W, hi = ((i64)(wn + 1) * M) / W;
  const u64 len = (u64)(hi - lo);
  const int nblk = (B + 3) >> 2;
  for (int blk = threadIdx.x; blk < a.RBp / 4; blk += blockDim.x) {
    int idx[4] = {-1, -1, -1, -1};
    if (blk < nblk) {
      uint32_t w4[4];
      philox4x32_10((uint32_t)wn, (uint32_t)jb, 1u, (uint32_t)(u * nblk + blk), st->key0, st->key1, w4);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (blk * 4 + q < B) idx[q] = (int)lo + (int)(((u64)w4[q] * len) >> 32);
    }
    *reinterpret_cast<int4*>(a.row_idx + (size_t)i * a.RBp + blk * 4) = make_int4(idx[0], idx[1], idx[2], idx[3]);
  }
  const int tiles = a.RBp / RB;
  for (int q = threadIdx.x; q < tiles; q += blockDim.x) a.tile_slot[i * tiles + q] = i;
}

// Output-layer gradient of every worker: dst_i[j] = sum over the worker's row chunks of part[q][j].
// Block = 32 outputs x 8 chunk lanes (lane w adds chunks w, w+8, ... in order, then the lanes in order).
__global__ void __launch_bounds__(256) chunk_reduce_worker_kernel(const DevState* st, const RoundInfo* ri, const float* part, int len,
                                                                  float* dst, size_t d_pad, int chunk_rows, int RBp) {
  grid_dependency_sync();
  __shared__ float red[8][33];
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  const int per = RBp / chunk_rows, q0 = i * per;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + lane;
  float acc = 0.f;
  if (j < len)
    for (int q = w; q < per; q += 8) acc += part[(size_t)(q0 + q) * len + j];
  red[w][lane] = acc;
  __syncthreads();
  if (w == 0 && j < len) {
    float tot = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) tot += red[q][lane];
    dst[(size_t)i * d_pad + j] = tot;
  }
}

// The workers' local updates after step u (Eq. 2): w_i -= eta / B * G_i, upload += G_i, new
// operand copy (bf16 configurations); block (0, i) also adds the step's mean loss and, after the
// last step, writes the uploaded loss (the average of the U mean minibatch losses; Algorithm 1,
// last worker line).
template <typename T>
__global__ void __launch_bounds__(256) local_step_kernel(Args a, int last) {
  grid_dependency_sync();
  __shared__ float red[8];
  const DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  const int B = st->B;
  const float step = __fdiv_rn(a.lr, (float)B);
  const float4* g = reinterpret_cast<const float4*>(a.G + (size_t)i * a.d_pad);
  float4* gs = reinterpret_cast<float4*>(a.gsum + (size_t)i * a.d_pad);
  float4* w32 = reinterpret_cast<float4*>(a.priv32 + (size_t)i * a.d_pad);
  uint2* w16 = reinterpret_cast<uint2*>(a.priv16 + (size_t)i * a.d_pad);
  const size_t n4 = a.d_pad / 4;
  for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (size_t)gridDim.x * blockDim.x) {
    const float4 gv = g[v];
    float4 s = gs[v];
    s.x += gv.x; s.y += gv.y; s.z += gv.z; s.w += gv.w;
    gs[v] = s;
    float4 m = w32[v];
    m.x = fmaf(-step, gv.x, m.x); m.y = fmaf(-step, gv.y, m.y);
    m.z = fmaf(-step, gv.z, m.z); m.w = fmaf(-step, gv.w, m.w);
    w32[v] = m;
    if (sizeof(T) == 2) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(m.x, m.y), hi = __floats2bfloat162_rn(m.z, m.w);
      uint2 pk;
      pk.x = *reinterpret_cast<const unsigned*>(&lo);
      pk.y = *reinterpret_cast<const unsigned*>(&hi);
      w16[v] = pk;
    }
  }
  if (blockIdx.x == 0) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float part = 0.f;
    for (int b = threadIdx.x; b < B; b += blockDim.x) part += a.row_loss[(size_t)i * a.RBp + b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) red[warp] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int q = 0; q < 8; ++q) tot += red[q];
      const float acc = a.loss_acc[i] + __fdiv_rn(tot, (float)B);
      a.loss_acc[i] = acc;
      if (last) {
        const float loss = __fdiv_rn(acc, (float)a.U);
        a.loss[i] = loss;
        if (!isfinite(loss)) ri->diverged = 1;
      }
    }
  }
}

}  // namespace lnet
}  // namespace absb
