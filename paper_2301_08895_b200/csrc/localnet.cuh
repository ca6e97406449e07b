// Local SGD inside a job (Eq. 2 with U > 1) for multi-layer networks.
// After its first local step every selected worker computes with weights of its own, so the
// workers' copies live in HBM, each [W][d_pad] and indexed by the worker's position in the round's
// selection: the copy the gradient kernels read (storage type) and the fp32 upload, i.e. the sum of
// the steps' gradient sums so far.  The local model after u steps is the model version the worker
// started from minus eta / B times that sum (Eq. 2 unrolled), so no third copy is kept.
// One local step of all selected workers is one pass of the grouped forward / backward kernels
// (tensor-core or FP32-FMA, as for U = 1) in which
//   - the rows of worker i are rows [i * RBp, i * RBp + B) (RBp = B rounded up to the row-tile
//     height; the rest is padding with sample index -1),
//   - the "model version" of a row tile is the worker's own copy (slot i of the private store), and
//   - the weight gradient is split per worker (split i = the rows of worker i) and added to the
//     worker's upload instead of summed over the workers,
// followed by the refresh of the workers' copies.  Eq. 3 then adds the K uploads like the partial
// sums of the U = 1 path.  Minibatch of step u: Philox blocks (n, j, 1, u * ceil(B/4) + b/4).
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
  void* priv;                          // [W][d_pad] the workers' copies, storage type
  float* gsum;                         // [W][d_pad] uploads: sum over the steps of the gradient sums
  const float* row_loss;               // sample losses of the current step, by row
  float* loss_acc;                     // [W] sum of the steps' mean losses
  float* loss;                         // [W] uploaded losses
  size_t d_pad;
  int RBp;                             // rows reserved per worker
  int U;
  float lr;
};

// Row layout of local step u for selected worker i (one block): the sample indices of its minibatch
// and the owner of its row tiles.
__device__ __forceinline__ void write_layout(const Args& a, const DevState* st, int i, int u) {
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

// Start of a job's local steps: the worker's copy is the model version it holds, its upload zero;
// block (0, i) also writes the row layout of step 0 (and block (0, 0) the row count of the passes).
template <typename T>
__global__ void __launch_bounds__(256) local_begin_kernel(Args a) {
  grid_dependency_sync();
  const DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  if (blockIdx.x == 0) {
    if (i == 0 && threadIdx.x == 0) ri->n_rows = ri->K * a.RBp;
    write_layout(a, st, i, 0);
  }
  const int slot = (ri->t - a.sel_tau[i]) % (st->S + 1);
  const uint4* src = reinterpret_cast<const uint4*>((const T*)a.ring + (size_t)slot * a.d_pad);
  uint4* dst = reinterpret_cast<uint4*>((T*)a.priv + (size_t)i * a.d_pad);
  float4* gs = reinterpret_cast<float4*>(a.gsum + (size_t)i * a.d_pad);
  const size_t n16 = a.d_pad * sizeof(T) / 16, n4 = a.d_pad / 4;
  for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (size_t)gridDim.x * blockDim.x) {
    if (v < n16) dst[v] = src[v];
    gs[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) a.loss_acc[i] = 0.f;
}

// Output-layer gradient of every worker, added to its upload: dst_i[j] += sum over the worker's row
// chunks, in order, of part[q][j].  One thread per output (a worker has only RBp / chunk_rows chunks).
__global__ void __launch_bounds__(256) chunk_reduce_worker_kernel(const DevState* st, const RoundInfo* ri, const float* part, int len,
                                                                  float* dst, size_t d_pad, int chunk_rows, int RBp) {
  grid_dependency_sync();
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  const int per = RBp / chunk_rows, q0 = i * per;
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= len) return;
  float tot = 0.f;
  for (int q = 0; q < per; ++q) tot += part[(size_t)(q0 + q) * len + j];
  dst[(size_t)i * d_pad + j] += tot;
}

// After step u (Eq. 2 unrolled): w_i^{u+1} = w_i^0 - eta / B * (sum of the gradient sums so far), written
// as the copy the next step reads (skipped after the last step); block (0, i) also adds the
// step's mean loss and, after the last step, writes the uploaded loss (the average of the U mean
// minibatch losses; Algorithm 1, last worker line) or else the row layout of step u + 1.
template <typename T>
__global__ void __launch_bounds__(256) local_step_kernel(Args a, int u) {
  grid_dependency_sync();
  __shared__ float red[8];
  const DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.y;
  if (i >= ri->K) return;
  const int B = st->B;
  const int last = u == a.U - 1;
  if (!last) {
    if (blockIdx.x == 0) write_layout(a, st, i, u + 1);
    const float step = __fdiv_rn(a.lr, (float)B);
    const int slot = (ri->t - a.sel_tau[i]) % (st->S + 1);
    const T* w0 = (const T*)a.ring + (size_t)slot * a.d_pad;
    T* w = (T*)a.priv + (size_t)i * a.d_pad;
    const float4* gs = reinterpret_cast<const float4*>(a.gsum + (size_t)i * a.d_pad);
    const size_t n4 = a.d_pad / 4;
    for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (size_t)gridDim.x * blockDim.x) {
      const float4 g = gs[v];
      float4 m;
      if (sizeof(T) == 4) {
        m = reinterpret_cast<const float4*>(w0)[v];
      } else {
        const uint2 pk = reinterpret_cast<const uint2*>(w0)[v];
        const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.x));
        const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.y));
        m = make_float4(f0.x, f0.y, f1.x, f1.y);
      }
      m.x = fmaf(-step, g.x, m.x); m.y = fmaf(-step, g.y, m.y);
      m.z = fmaf(-step, g.z, m.z); m.w = fmaf(-step, g.w, m.w);
      if (sizeof(T) == 4) {
        reinterpret_cast<float4*>(w)[v] = m;
      } else {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(m.x, m.y), hi = __floats2bfloat162_rn(m.z, m.w);
        uint2 pk;
        pk.x = *reinterpret_cast<const unsigned*>(&lo);
        pk.y = *reinterpret_cast<const unsigned*>(&hi);
        reinterpret_cast<uint2*>(w)[v] = pk;
      }
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
