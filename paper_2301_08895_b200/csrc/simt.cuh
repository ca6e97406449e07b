// FP32-FMA gradient kernels: every model kind and both storage types.  They serve the fp32
// configurations, the narrow last layer of the bf16 networks and the least-squares model.
// Worker uploads are Eq. 2 with U = 1, evaluated at the ring slot of the model version the
// worker holds; Eq. 3 only needs the sum over the selected workers, so weight gradients are
// reduced over all gradient rows of the round and never stored per worker.
#pragma once
#include "common.cuh"
#include "ctl.cuh"

namespace absb {


constexpr int TM = 64, TN = 64, TK = 16;

// acc[4][4] += sum_k fa(k, m) * fb(k, n) over k in [k_begin, k_end) for a 64x64 tile;
// thread (ty, tx) owns rows ty*4.., columns tx*4...  fa/fb return 0 outside their range.
template <bool A_KCONTIG, bool B_KCONTIG, class FA, class FB>
__device__ __forceinline__ void tile_fma(float (&acc)[4][4], int k_begin, int k_end, FA fa, FB fb,
                                         float (*As)[TM + 4], float (*Bs)[TN + 4]) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  for (int k0 = k_begin; k0 < k_end; k0 += TK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int id = tid + e * 256;
      const int kk = A_KCONTIG ? (id & 15) : (id >> 6);
      const int mm = A_KCONTIG ? (id >> 4) : (id & 63);
      As[kk][mm] = (k0 + kk < k_end) ? fa(k0 + kk, mm) : 0.f;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int id = tid + e * 256;
      const int kk = B_KCONTIG ? (id & 15) : (id >> 6);
      const int nn = B_KCONTIG ? (id >> 4) : (id & 63);
      Bs[kk][nn] = (k0 + kk < k_end) ? fb(k0 + kk, nn) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
}

struct LayerArgs {
  const DevState* st;
  const RoundInfo* ri;
  const int* tile_slot;     // ring slot per RB-row tile
  const int* row_idx;       // sample index per row (-1: padding)
  const void* ring;         // model versions, storage type, [S+1][slot_stride]
  size_t slot_stride;       // elements
  size_t w_off;             // element offset of this layer's W[in][out]; bias follows at w_off + in*out
  int in, out;
  int gather;               // 1: input rows are X[row_idx[r]], else act_in[r]
  const void* act_in;       // [rows][in]   (or X when gather)
  void* act_out;            // fwd: [rows][out] storage type (hidden) or float logits (last)
  const void* delta_out;    // bwd: [rows][out] deltas of this layer's output
  void* delta_in;           // dgrad result [rows][in]
  float* G;                 // wgrad partials [P][slot_stride]
  int P;                    // 0: one split per selected worker (its rows), added to G[worker]
};

// Forward of one affine layer for all rows of the round: act_out = [relu](act_in W_s + b_s).
template <typename T, bool LAST>
__global__ void __launch_bounds__(256) simt_fwd_kernel(LayerArgs a) {
  grid_dependency_sync();
  __shared__ float As[TK][TM + 4], Bs[TK][TN + 4];
  const DevState* st = a.st;
  const RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  if (r0 >= ri->n_rows) return;
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  const T* bias = Wm + (size_t)a.in * a.out;
  const T* src = (const T*)a.act_in;
  const int in = a.in, out = a.out, gather = a.gather;
  const int* row_idx = a.row_idx;
  float acc[4][4] = {};
  auto fa = [&](int k, int mm) -> float {
    const int r = r0 + mm;
    if (gather) {
      const int s = row_idx[r];
      return s < 0 ? 0.f : ldf(src, (size_t)s * in + k);
    }
    return ldf(src, (size_t)r * in + k);
  };
  auto fb = [&](int k, int nn) -> float {
    const int n = n0 + nn;
    return n < out ? ldf(Wm, (size_t)k * out + n) : 0.f;
  };
  tile_fma<true, false>(acc, 0, in, fa, fb, As, Bs);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < out) {
        const float v = acc[i][j] + ldf(bias, n);
        if (LAST) ((float*)a.act_out)[(size_t)r * out + n] = v;
        else stf((T*)a.act_out, (size_t)r * out + n, fmaxf(v, 0.f));
      }
    }
  }
}

// Back-propagation through one affine layer and the ReLU before it:
// delta_in[r][m] = (sum_n delta_out[r][n] W_s[m][n]) * [act_in[r][m] > 0].
template <typename T>
__global__ void __launch_bounds__(256) simt_dgrad_kernel(LayerArgs a) {
  grid_dependency_sync();
  __shared__ float As[TK][TM + 4], Bs[TK][TN + 4];
  const DevState* st = a.st;
  const RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.y * TM, m0 = blockIdx.x * TN;
  if (r0 >= ri->n_rows) return;
  const int slot = a.tile_slot[r0 / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  const T* dl = (const T*)a.delta_out;
  const T* hin = (const T*)a.act_in;
  const int in = a.in, out = a.out;
  float acc[4][4] = {};
  auto fa = [&](int k, int mm) -> float { return ldf(dl, (size_t)(r0 + mm) * out + k); };
  auto fb = [&](int k, int nn) -> float {
    const int m = m0 + nn;
    return m < in ? ldf(Wm, (size_t)m * out + k) : 0.f;
  };
  tile_fma<true, true>(acc, 0, out, fa, fb, As, Bs);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + tx * 4 + j;
      if (m < in) {
        const float h = ldf(hin, (size_t)r * in + m);
        stf((T*)a.delta_in, (size_t)r * in + m, h > 0.f ? acc[i][j] : 0.f);
      }
    }
  }
}

// Weight and bias gradient of one layer summed over all rows of the round (the inner sums of
// Eq. 3): G_p[m][n] = sum_{r in chunk p} act_in[r][m] delta_out[r][n]; row m = `in` of the
// result is the bias gradient (an implicit input of ones).
template <typename T>
__global__ void __launch_bounds__(256) simt_wgrad_kernel(LayerArgs a) {
  grid_dependency_sync();
  __shared__ float As[TK][TM + 4], Bs[TK][TN + 4];
  const DevState* st = a.st;
  const RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN, p = blockIdx.z;
  const int n_rows = ri->n_rows;
  const int P = a.P > 0 ? a.P : ri->K;        // P = 0: one split per selected worker (its own rows)
  if (p >= P) return;
  const int chunk = round_up((n_rows + P - 1) / P, TK);
  const int k_begin = min(n_rows, p * chunk), k_end = min(n_rows, (p + 1) * chunk);
  const T* src = (const T*)a.act_in;
  const T* dl = (const T*)a.delta_out;
  const int in = a.in, out = a.out, gather = a.gather;
  const int* row_idx = a.row_idx;
  float acc[4][4] = {};
  auto fa = [&](int r, int mm) -> float {
    const int m = m0 + mm;
    if (m > in) return 0.f;
    if (m == in) return 1.f;
    if (gather) {
      const int s = row_idx[r];
      return s < 0 ? 0.f : ldf(src, (size_t)s * in + m);
    }
    return ldf(src, (size_t)r * in + m);
  };
  auto fb = [&](int r, int nn) -> float {
    const int n = n0 + nn;
    return n < out ? ldf(dl, (size_t)r * out + n) : 0.f;
  };
  tile_fma<false, false>(acc, k_begin, k_end, fa, fb, As, Bs);
  float* G = a.G + (size_t)p * a.slot_stride + a.w_off;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (m <= in && n < out) {
        if (a.P == 0) G[(size_t)m * out + n] += acc[i][j];      // per-worker split: adds to the worker's upload
        else G[(size_t)m * out + n] = acc[i][j];
      }
    }
  }
}

struct LossArgs {
  DevState* st;
  RoundInfo* ri;
  const int* tile_slot;   // ring slot of every row tile (RB rows)
  const int* row_idx;
  const int* labels;      // [n_samples]
  const float* logits;    // [rows][C]
  void* delta;            // [rows][C] storage type
  float* row_loss;        // [rows]
  int C;
};

// Soft-max cross-entropy per gradient row: loss = log sum exp(z - max) - (z_y - max),
// delta = softmax(z) - onehot(y).  Padding rows get zero delta so they add nothing to Eq. 3.
template <typename T>
__global__ void __launch_bounds__(256) net_loss_kernel(LossArgs a) {
  grid_dependency_sync();
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= ri->n_rows) return;
  const int C = a.C;
  T* d = (T*)a.delta + (size_t)r * C;
  const int s = a.row_idx[r];
  if (s < 0) {
    for (int c = 0; c < C; ++c) stf(d, c, 0.f);
    a.row_loss[r] = 0.f;
    return;
  }
  const float* z = a.logits + (size_t)r * C;
  const int y = a.labels[s];
  float zmax = z[0];
  for (int c = 1; c < C; ++c) zmax = fmaxf(zmax, z[c]);
  float se = 0.f;
  for (int c = 0; c < C; ++c) se += expf(z[c] - zmax);
  const float inv = 1.f / se;
  const float sa = sa_slot_weight(st, ri->t, a.tile_slot[r / st->RB]);   // staleness-aware step size
  for (int c = 0; c < C; ++c) stf(d, c, (expf(z[c] - zmax) * inv - (c == y ? 1.f : 0.f)) * sa);
  const float loss = logf(se) - (z[y] - zmax);
  a.row_loss[r] = loss;
  if (!isfinite(loss)) ri->diverged = 1;
}

struct LsqArgs {
  DevState* st;
  RoundInfo* ri;
  const int* sel; const int* job;
  const int* sel_tau; const int* sel_row0; const int* row_idx;
  const void* X; const float* y;
  const void* ring; size_t slot_stride;
  float* loss;            // [W]
  float* G;               // [W][slot_stride] one partial per selected worker
  int d;
};

// Least squares, one CTA per selected worker: residuals r_b = x_b . w_v - y_b at the worker's
// model version v, loss = mean 1/2 r^2, partial gradient g = sum_b r_b x_b.
template <typename T>
__global__ void __launch_bounds__(256) lsq_grad_kernel(LsqArgs a) {
  grid_dependency_sync();
  __shared__ float res[1024];
  __shared__ int sidx[1024];
  __shared__ float red[8];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int i = blockIdx.x;
  if (i >= ri->K) return;
  const int B = st->B, d = a.d;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int slot = (ri->t - a.sel_tau[i]) % (st->S + 1);
  const T* w = (const T*)a.ring + (size_t)slot * a.slot_stride;
  const T* X = (const T*)a.X;
  {
    // minibatch of the worker's job in flight: draw b = word b%4 of Philox block (n, j, 1, b/4),
    // mapped into the worker's shard [n M / N, (n+1) M / N)
    const int wn = a.sel[i], j = a.job[wn], W = st->W;
    const i64 M = st->n_samples;
    const i64 lo = ((i64)wn * M) / W, hi = ((i64)(wn + 1) * M) / W;
    const u64 len = (u64)(hi - lo);
    for (int blk = tid; blk < ((B + 3) >> 2); blk += 256) {
      uint32_t w4[4];
      philox4x32_10((uint32_t)wn, (uint32_t)j, 1u, (uint32_t)blk, st->key0, st->key1, w4);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (blk * 4 + q < B) sidx[blk * 4 + q] = (int)lo + (int)(((u64)w4[q] * len) >> 32);
    }
  }
  __syncthreads();
  for (int b = warp; b < B; b += 8) {
    const T* x = X + (size_t)sidx[b] * d;
    float acc = 0.f;
    for (int j = lane; j < d; j += 32) acc = fmaf(ldf(x, j), ldf(w, j), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) res[b] = acc - a.y[sidx[b]];
  }
  __syncthreads();
  float part = 0.f;
  for (int b = tid; b < B; b += 256) part += 0.5f * res[b] * res[b];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0) red[warp] = part;
  __syncthreads();
  if (tid == 0) {
    float tot = 0.f;
    for (int q = 0; q < 8; ++q) tot += red[q];
    const float loss = __fdiv_rn(tot, (float)B);
    a.loss[i] = loss;
    if (!isfinite(loss)) ri->diverged = 1;
  }
  float* g = a.G + (size_t)i * a.slot_stride;
  const float sa = st->sa_penalty ? sa_weight(a.sel_tau[i]) : 1.f;   // staleness-aware step size
  for (int j = tid; j < d; j += 256) {
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc = fmaf(res[b], ldf(X, (size_t)sidx[b] * d + j), acc);
    g[j] = acc * sa;
  }
}

struct UpdateArgs {
  const DevState* st;
  const RoundInfo* ri;
  const int* job; u64* next_dur; int* dur_job;   // duration look-ahead (see refresh_next_durations)
  float* master;          // [d_pad]
  void* ring;             // [S+1][d_pad] storage type
  const float* G;         // [P][d_pad]
  size_t d_pad;
  int P;                  // partial count, or 0: one partial per selected worker (K^t)
  const int* sel_tau;     // [K^t] staleness of each selected worker's upload (read when the staleness-aware
                          // step size is applied to whole uploads: DevState::sa_penalty == 2, P == 0)
  float lr;
  // Parts of the gradient that are still per-chunk partial sums (the output layer's block left by the fused
  // output kernels; bias gradients left as column sums per 32 rows by the back-propagation GEMM): blocks
  // [n_main_blocks, gridDim.x) add the chunks of 32 parameters each in a fixed order and apply Eq. 3 to those
  // parameters; the streaming blocks skip the ranges.
  struct Region {
    const float* part;    // [chunks][len]
    int len;              // parameters
    int chunk_rows;       // gradient rows per chunk
    size_t off;           // element offset inside the parameter vector (multiple of 4; len too, unless it ends a layer)
    int first_block;      // first of its (len + 31) / 32 blocks, counted from n_main_blocks
  };
  static constexpr int MAX_REGIONS = 3;
  Region region[MAX_REGIONS];
  int n_regions;
  int n_main_blocks;
};

// Eq. 3 and the ring write: w^{t+1} = w^t - eta / (K^t B) * sum_p G_p, stored as the fp32
// master and, in storage type, as ring slot (t+1) mod (S+1).  One pass, 16-byte accesses.
// LOOK: the first warps also prepare the next job durations (latency-bound models, one stream); the
// bandwidth-bound networks keep that in a kernel of its own so that this one stays a pure stream.
template <typename T, bool LOOK>
__global__ void __launch_bounds__(256, 4) update_kernel(UpdateArgs a) {
  grid_dependency_sync();
  const DevState* st = a.st;
  const RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  // duration look-ahead for the workers whose job index moved (first warp of the first ceil(N/32) blocks)
  if (LOOK && threadIdx.x < 32 && (int)blockIdx.x * 32 < st->W)
    refresh_next_durations(st, a.job, a.next_dur, a.dur_job, (int)blockIdx.x * 32 + (int)threadIdx.x);
  if (ri->diverged) return;
  const int K = ri->K;
  const int P = a.P > 0 ? a.P : K;
  const float step = __fdiv_rn(a.lr, (float)(K * st->B));
  const int slot = (ri->t + 1) % (st->S + 1);
  T* dst = (T*)a.ring + (size_t)slot * a.d_pad;
  if ((int)blockIdx.x >= a.n_main_blocks) {
    // lane w adds chunks w, w + 8, ... in order, then the 8 lanes are added in order
    __shared__ float red[8][33];
    const int rb = (int)blockIdx.x - a.n_main_blocks;
    int ri_ = 0;
#pragma unroll
    for (int q = 1; q < UpdateArgs::MAX_REGIONS; ++q)
      if (q < a.n_regions && rb >= a.region[q].first_block) ri_ = q;
    const UpdateArgs::Region& R = a.region[ri_];
    const int n_chunks = ri->n_rows / R.chunk_rows;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int j = (rb - R.first_block) * 32 + lane;
    float acc = 0.f;
    if (j < R.len) {
#pragma unroll 8
      for (int q = w; q < n_chunks; q += 8) acc += R.part[(size_t)q * R.len + j];
    }
    red[w][lane] = acc;
    __syncthreads();
    if (w == 0 && j < R.len) {
      float tot = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) tot += red[q][lane];
      const size_t e = R.off + (size_t)j;
      const float m = fmaf(-step, tot, a.master[e]);
      a.master[e] = m;
      stf(dst, e, m);
    }
    return;
  }
  const size_t n4 = a.d_pad / 4;
  // float4 ranges done by the reduce blocks (32-bit: the vector has fewer than 2^34 parameters)
  unsigned lo4[UpdateArgs::MAX_REGIONS], hi4[UpdateArgs::MAX_REGIONS];
#pragma unroll
  for (int q = 0; q < UpdateArgs::MAX_REGIONS; ++q) {
    lo4[q] = q < a.n_regions ? (unsigned)(a.region[q].off / 4) : 0xffffffffu;
    hi4[q] = q < a.n_regions ? (unsigned)((a.region[q].off + (size_t)a.region[q].len + 3) / 4) : 0xffffffffu;
  }
  const int n_blocks = a.n_main_blocks;
  const size_t stride = (size_t)n_blocks * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  auto finish = [&](size_t i, float4 g, float4 m) {
    bool skip = false;
#pragma unroll
    for (int q = 0; q < UpdateArgs::MAX_REGIONS; ++q) skip |= (unsigned)i - lo4[q] < hi4[q] - lo4[q];
    if (skip) return;                              // done by the reduce blocks
    m.x = fmaf(-step, g.x, m.x); m.y = fmaf(-step, g.y, m.y);
    m.z = fmaf(-step, g.z, m.z); m.w = fmaf(-step, g.w, m.w);
    reinterpret_cast<float4*>(a.master)[i] = m;
    if (sizeof(T) == 4) {
      reinterpret_cast<float4*>(dst)[i] = m;
    } else {
      __nv_bfloat162 lo = __floats2bfloat162_rn(m.x, m.y), hi = __floats2bfloat162_rn(m.z, m.w);
      uint2 pk;
      pk.x = *reinterpret_cast<unsigned*>(&lo);
      pk.y = *reinterpret_cast<unsigned*>(&hi);
      reinterpret_cast<uint2*>(dst)[i] = pk;
    }
  };
  // few partials (the split counts of the weight-gradient GEMMs): two vectors per thread and
  // iteration, all loads of both issued before the first use (same sums, same order per element)
  const bool weigh = a.P == 0 && st->sa_penalty == 2;
  if (P <= 4 && !weigh) {
    for (; i + stride < n4; i += 2 * stride) {
      const size_t j = i + stride;
      float4 ga[4], gb[4];
#pragma unroll
      for (int p = 0; p < 4; ++p)
        if (p < P) {
          ga[p] = reinterpret_cast<const float4*>(a.G + (size_t)p * a.d_pad)[i];
          gb[p] = reinterpret_cast<const float4*>(a.G + (size_t)p * a.d_pad)[j];
        }
      const float4 ma = reinterpret_cast<float4*>(a.master)[i], mb = reinterpret_cast<float4*>(a.master)[j];
      float4 g = ga[0], h = gb[0];
#pragma unroll
      for (int p = 1; p < 4; ++p)
        if (p < P) {
          g.x += ga[p].x; g.y += ga[p].y; g.z += ga[p].z; g.w += ga[p].w;
          h.x += gb[p].x; h.y += gb[p].y; h.z += gb[p].z; h.w += gb[p].w;
        }
      finish(i, g, ma);
      finish(j, h, mb);
    }
  }
  for (; i < n4; i += stride) {
    float4 g = reinterpret_cast<const float4*>(a.G)[i];
    if (weigh) {
      // staleness-aware step size on whole uploads: upload p counts with weight 1 / max(1, tau_p)
      const float w0 = sa_weight(a.sel_tau[0]);
      g.x *= w0; g.y *= w0; g.z *= w0; g.w *= w0;
      for (int p = 1; p < P; ++p) {
        const float4 q = reinterpret_cast<const float4*>(a.G + (size_t)p * a.d_pad)[i];
        const float wp = sa_weight(a.sel_tau[p]);
        g.x = fmaf(wp, q.x, g.x); g.y = fmaf(wp, q.y, g.y); g.z = fmaf(wp, q.z, g.z); g.w = fmaf(wp, q.w, g.w);
      }
    } else {
      for (int p = 1; p < P; ++p) {
        const float4 q = reinterpret_cast<const float4*>(a.G + (size_t)p * a.d_pad)[i];
        g.x += q.x; g.y += q.y; g.z += q.z; g.w += q.w;
      }
    }
    finish(i, g, reinterpret_cast<float4*>(a.master)[i]);
  }
}

// Initial model: master = w0 (already in place), ring slot 0 = storage-type copy.
template <typename T>
__global__ void ring_init_kernel(const float* master, void* ring, size_t d_pad) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < d_pad;
       i += (size_t)gridDim.x * blockDim.x)
    stf((T*)ring, i, master[i]);
}

}  // namespace absb
