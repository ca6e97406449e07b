// The two convolution blocks in front of the fully connected layers of the paper's model class
// (Sec. V-A: "two convolutional layers and three fully connected layers" on 32 x 32 x 3 images).
// A block is a k x k convolution (stride 1, no padding), ReLU, and a 2 x 2 max-pool of stride 2.
//
//   forward   a[y][x][co] = relu( b[co] + sum_{dy,dx,ci} in[y+dy][x+dx][ci] W_s[dy][dx][ci][co] )   (stored rounded)
//             p[py][px][co] = max of the 2 x 2 window of a, arg = position of its first maximum
//   backward  the delta of p goes to the window position `arg` (it arrives already zeroed where
//             p is not positive, i.e. where the ReLU was inactive);
//             G[dy][dx][ci][co] = sum over rows and pooled pixels of in[2py+ay+dy][2px+ax+dx][ci] dp[py][px][co]
//             d_in[y][x][ci]    = ( sum_{dy,dx,co} dz[y-dy][x-dx][co] W_s[dy][dx][ci][co] ) [in[y][x][ci] > 0]
// (Eq. 2 with U = 1 at the model version s the row's worker holds; Eq. 3 needs only the sum of G
// over all rows.)  Maps are stored [row][y][x][channel] in the storage type; the images of the
// first block are dataset rows fetched by sample index.  The channel counts of this model class
// are far below a tensor-core tile (3 -> 6 -> 16 in the benchmark network), so these are FP32-FMA
// kernels: one CTA per gradient row (forward, input delta) or per small chunk of rows (weight gradient),
// everything the CTA needs staged in shared memory, fixed summation orders.
#pragma once
#include "common.cuh"
#include "simt.cuh"

namespace absb {
namespace conv {

constexpr int THREADS = 256;
constexpr int MAX_CHUNK = 16;    // most gradient rows per CTA of the weight-gradient kernel

struct Args {
  DevState* st;
  RoundInfo* ri;
  const int* tile_slot;     // ring slot per RB-row tile
  const int* row_idx;       // sample index per gradient row (-1: padding)
  const void* ring; size_t slot_stride;
  size_t w_off;             // element offset of W[k][k][Ci][Co]; the bias b[Co] follows it
  int Hi, Wi, Ci, k, Co;    // input map, kernel size, output channels
  const void* in;           // input maps [rows][Hi][Wi][Ci], or the dataset when from_dataset
  int from_dataset;         // 1: row r reads X[row_idx[r]]
  void* pooled;             // [rows][Ph][Pw][Co] pooled ReLU outputs (storage type)
  unsigned char* arg;       // [rows][Ph][Pw][Co] window position (0..3 = (wy, wx) row-major) of the first maximum
  const void* d_pooled;     // backward: [rows][Ph][Pw][Co] delta of the pooled maps
  void* d_in;               // backward: [rows][Hi][Wi][Ci] delta of the input maps (second block)
  float* part;              // backward: [chunks][k k Ci Co + Co] per-chunk sums of the weight and bias gradient
  int chunk;                // gradient rows per CTA of the weight-gradient kernel: a power of two (divides the row
                            // padding unit, so a chunk never straddles two model versions), chosen by the host so
                            // that a round with every worker selected gives every SM at least four CTAs
};

inline size_t fwd_smem_bytes(int Hi, int Wi, int Ci, int k, int Co) {
  return sizeof(float) * ((size_t)Hi * Wi * Ci + (size_t)k * k * Ci * Co + Co);
}
inline size_t wgrad_smem_bytes(int Hi, int Wi, int Ci, int k, int Co) {
  const int Ho = Hi - k + 1, Wo = Wi - k + 1;
  return sizeof(float) * ((size_t)Hi * Wi * Ci + (size_t)(Ho / 2) * (Wo / 2) * Co) + (size_t)(Ho / 2) * (Wo / 2) * Co + 16;
}
inline size_t dgrad_smem_bytes(int Hi, int Wi, int Ci, int k, int Co) {
  const int Ho = Hi - k + 1, Wo = Wi - k + 1;
  return sizeof(float) * ((size_t)k * k * Ci * Co + (size_t)Ho * Wo * Co);
}
inline size_t bwd_smem_bytes(int Hi, int Wi, int Ci, int k, int Co) {
  return wgrad_smem_bytes(Hi, Wi, Ci, k, Co) > dgrad_smem_bytes(Hi, Wi, Ci, k, Co) ? wgrad_smem_bytes(Hi, Wi, Ci, k, Co)
                                                                                   : dgrad_smem_bytes(Hi, Wi, Ci, k, Co);
}

template <typename T>
__device__ __forceinline__ float as_stored_value(float v) { return v; }
template <>
__device__ __forceinline__ float as_stored_value<__nv_bfloat16>(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// One block forward for every gradient row of the round; CTA = row.
template <typename T>
__global__ void __launch_bounds__(THREADS) conv_block_fwd_kernel(Args a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) float csm[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r = blockIdx.x;
  if (r >= ri->n_rows) return;
  const int Hi = a.Hi, Wi = a.Wi, Ci = a.Ci, k = a.k, Co = a.Co;
  const int Ho = Hi - k + 1, Wo = Wi - k + 1, Ph = Ho >> 1, Pw = Wo >> 1;
  const int n_in = Hi * Wi * Ci, n_w = k * k * Ci * Co, n_out = Ph * Pw * Co;
  T* out = (T*)a.pooled + (size_t)r * n_out;
  unsigned char* arg = a.arg + (size_t)r * n_out;
  const int s = a.row_idx[r];
  if (s < 0) {                               // padding row: its deltas are zero, its maps only have to be finite
    for (int i = threadIdx.x; i < n_out; i += THREADS) { stf(out, i, 0.f); arg[i] = 0; }
    return;
  }
  float* img = csm;                          // [Hi][Wi][Ci]
  float* wk = img + n_in;                    // [k][k][Ci][Co]
  float* bias = wk + n_w;                    // [Co]
  const int slot = a.tile_slot[r / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  const T* src = (const T*)a.in + (size_t)(a.from_dataset ? s : r) * n_in;
  for (int i = threadIdx.x; i < n_in; i += THREADS) img[i] = ldf(src, i);
  for (int i = threadIdx.x; i < n_w + Co; i += THREADS) wk[i] = ldf(Wm, i);     // the bias follows the weights
  __syncthreads();
  // A thread computes the four window positions of CT neighbouring output channels of one pooled pixel: per
  // (dy, ci) the two image rows slide along dx, so an image value is read once for 2 CT FMAs and a weight once
  // for four.
  constexpr int CT = 2;
  const int cgs = (Co + CT - 1) / CT;
  for (int item = threadIdx.x; item < Ph * Pw * cgs; item += THREADS) {
    const int co0 = (item % cgs) * CT, px = (item / cgs) % Pw, py = item / (cgs * Pw);
    const int nco = min(CT, Co - co0);
    float acc4[CT][4];
#pragma unroll
    for (int c = 0; c < CT; ++c)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc4[c][q] = 0.f;
    for (int dy = 0; dy < k; ++dy)
      for (int ci = 0; ci < Ci; ++ci) {
        const float* r0 = img + ((2 * py + dy) * Wi + 2 * px) * Ci + ci;
        const float* r1 = r0 + Wi * Ci;
        const float* wp = wk + ((dy * k) * Ci + ci) * Co + co0;
        float p0 = r0[0], p1 = r1[0];
        for (int dx = 0; dx < k; ++dx) {
          const float n0 = r0[(dx + 1) * Ci], n1 = r1[(dx + 1) * Ci];
#pragma unroll
          for (int c = 0; c < CT; ++c) {
            const float w = c < nco ? wp[dx * Ci * Co + c] : 0.f;
            acc4[c][0] = fmaf(p0, w, acc4[c][0]);
            acc4[c][1] = fmaf(n0, w, acc4[c][1]);
            acc4[c][2] = fmaf(p1, w, acc4[c][2]);
            acc4[c][3] = fmaf(n1, w, acc4[c][3]);
          }
          p0 = n0;
          p1 = n1;
        }
      }
#pragma unroll
    for (int c = 0; c < CT; ++c) {
      if (c >= nco) break;
      const int co = co0 + c, e = (py * Pw + px) * Co + co;
      float best = 0.f;
      int where = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float v = as_stored_value<T>(fmaxf(acc4[c][q] + bias[co], 0.f));  // the stored ReLU output
        if (q == 0 || v > best) { best = v; where = q; }                         // first maximum wins a tie
      }
      stf(out, e, best);
      arg[e] = (unsigned char)where;
    }
  }
}

// Weight and bias gradient of one block over `chunk` consecutive gradient rows: this CTA's share of
// the sum of Eq. 3 (a fixed-order reduction over the CTAs follows).  Only the window position that
// supplied a pooled maximum carries a delta, so the sum runs over pooled pixels.
template <typename T>
__global__ void __launch_bounds__(THREADS) conv_block_wgrad_kernel(Args a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) float csm[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int CHUNK = a.chunk;
  const int r0 = blockIdx.x * CHUNK;
  if (r0 >= ri->n_rows) return;
  const int Hi = a.Hi, Wi = a.Wi, Ci = a.Ci, k = a.k, Co = a.Co;
  const int Ho = Hi - k + 1, Wo = Wi - k + 1, Ph = Ho >> 1, Pw = Wo >> 1;
  const int n_in = Hi * Wi * Ci, n_w = k * k * Ci * Co, n_out = Ph * Pw * Co;
  float* img = csm;                          // [Hi][Wi][Ci] input maps of the current row
  float* dp = img + n_in;                    // [Ph][Pw][Co] delta of the pooled maps
  unsigned char* ag = reinterpret_cast<unsigned char*>(dp + n_out);   // [Ph][Pw][Co]
  // A thread takes a unit (tap (dy, dx), output channel co) and up to DG input channels of it: per pooled pixel
  // the pool position and the delta are read once and feed DG FMAs on neighbouring image values.  The sums of a
  // row are added to this CTA's block of `part` by the thread that owns the elements (same thread every row).
  constexpr int DG = 8;
  const int n_units = k * k * Co, n_groups = (Ci + DG - 1) / DG;
  float* dst = a.part + (size_t)blockIdx.x * (size_t)(n_w + Co);
  bool first = true;
  const int n_rows = ri->n_rows;
  for (int rr = 0; rr < CHUNK && r0 + rr < n_rows; ++rr) {
    const int r = r0 + rr;
    const int s = a.row_idx[r];
    if (s < 0) continue;                     // padding row: zero deltas (same decision in every thread)
    __syncthreads();                         // the previous row's maps are no longer read
    const T* src = (const T*)a.in + (size_t)(a.from_dataset ? s : r) * n_in;
    const T* dps = (const T*)a.d_pooled + (size_t)r * n_out;
    const unsigned char* args = a.arg + (size_t)r * n_out;
    for (int i = threadIdx.x; i < n_in; i += THREADS) img[i] = ldf(src, i);
    for (int i = threadIdx.x; i < n_out; i += THREADS) { dp[i] = ldf(dps, i); ag[i] = args[i]; }
    __syncthreads();
    for (int item = threadIdx.x; item < n_units * n_groups; item += THREADS) {
      const int u = item % n_units, grp = item / n_units;
      const int co = u % Co, tap = u / Co, dx = tap % k, dy = tap / k;
      const int ci0 = grp * DG, nch = min(DG, Ci - ci0);
      float sum[DG];
#pragma unroll
      for (int j = 0; j < DG; ++j) sum[j] = 0.f;
      for (int py = 0; py < Ph; ++py)
        for (int px = 0; px < Pw; ++px) {
          const int o = (py * Pw + px) * Co + co;
          const int q = ag[o];
          const float d = dp[o];
          const float* ip = img + ((2 * py + (q >> 1) + dy) * Wi + 2 * px + (q & 1) + dx) * Ci + ci0;
#pragma unroll
          for (int j = 0; j < DG; ++j)
            if (j < nch) sum[j] = fmaf(ip[j], d, sum[j]);
        }
#pragma unroll
      for (int j = 0; j < DG; ++j)
        if (j < nch) {
          const int e = (tap * Ci + ci0 + j) * Co + co;
          dst[e] = first ? sum[j] : dst[e] + sum[j];
        }
    }
    if (threadIdx.x < Co) {                  // bias sums
      float sum = 0.f;
      for (int o = threadIdx.x; o < n_out; o += Co) sum += dp[o];
      dst[n_w + threadIdx.x] = first ? sum : dst[n_w + threadIdx.x] + sum;
    }
    first = false;
  }
  if (first)                                 // no row with a gradient in this chunk
    for (int e = threadIdx.x; e < n_w + Co; e += THREADS) dst[e] = 0.f;
}

// Delta of a block's input maps (second block only), CTA = gradient row: the pooled delta is put
// back at the window positions that supplied the maxima (dense map in shared memory), then every
// input element adds up the taps of the output pixels that cover it, masked by the ReLU that
// produced the input (it is a pooled ReLU output: positive where active).
template <typename T>
__global__ void __launch_bounds__(THREADS) conv_block_dgrad_kernel(Args a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) float csm[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r = blockIdx.x;
  if (r >= ri->n_rows) return;
  const int Hi = a.Hi, Wi = a.Wi, Ci = a.Ci, k = a.k, Co = a.Co;
  const int Ho = Hi - k + 1, Wo = Wi - k + 1, Ph = Ho >> 1, Pw = Wo >> 1;
  const int n_in = Hi * Wi * Ci, n_w = k * k * Ci * Co, n_out = Ph * Pw * Co, n_z = Ho * Wo * Co;
  T* din = (T*)a.d_in + (size_t)r * n_in;
  const int s = a.row_idx[r];
  if (s < 0) {                               // padding row: zero deltas
    for (int i = threadIdx.x; i < n_in; i += THREADS) stf(din, i, 0.f);
    return;
  }
  float* wk = csm;                           // [k][k][Ci][Co]
  float* dz = wk + n_w;                      // [Ho][Wo][Co] delta before the pool, dense
  const int slot = a.tile_slot[r / st->RB];
  const T* Wm = (const T*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  const T* dps = (const T*)a.d_pooled + (size_t)r * n_out;
  const unsigned char* args = a.arg + (size_t)r * n_out;
  const T* src = (const T*)a.in + (size_t)r * n_in;
  for (int i = threadIdx.x; i < n_w; i += THREADS) wk[i] = ldf(Wm, i);
  for (int i = threadIdx.x; i < n_z; i += THREADS) dz[i] = 0.f;
  __syncthreads();
  for (int e = threadIdx.x; e < n_out; e += THREADS) {
    const int co = e % Co, px = (e / Co) % Pw, py = e / (Co * Pw);
    const int q = args[e];
    dz[((2 * py + (q >> 1)) * Wo + 2 * px + (q & 1)) * Co + co] = ldf(dps, e);
  }
  __syncthreads();
  // a thread takes one input pixel and up to DG of its channels: a delta read from shared memory is used for
  // DG FMAs (the weights of the DG channels for one tap and output channel are DG reads)
  constexpr int DG = 8;
  const int n_groups = (Ci + DG - 1) / DG;
  for (int item = threadIdx.x; item < Hi * Wi * n_groups; item += THREADS) {
    const int grp = item % n_groups, pix = item / n_groups;
    const int x = pix % Wi, y = pix / Wi;
    const int ci0 = grp * DG, nch = min(DG, Ci - ci0);
    float sum[DG];
#pragma unroll
    for (int j = 0; j < DG; ++j) sum[j] = 0.f;
    for (int dy = 0; dy < k; ++dy) {
      const int oy = y - dy;
      if (oy < 0 || oy >= Ho) continue;
      for (int dx = 0; dx < k; ++dx) {
        const int ox = x - dx;
        if (ox < 0 || ox >= Wo) continue;
        const float* zp = dz + (oy * Wo + ox) * Co;
        const float* wp = wk + ((dy * k + dx) * Ci + ci0) * Co;
        for (int co = 0; co < Co; ++co) {
          const float z = zp[co];
#pragma unroll
          for (int j = 0; j < DG; ++j)
            if (j < nch) sum[j] = fmaf(z, wp[j * Co + co], sum[j]);
        }
      }
    }
    const int e0 = pix * Ci + ci0;
#pragma unroll
    for (int j = 0; j < DG; ++j)
      if (j < nch) stf(din, e0 + j, ldf(src, e0 + j) > 0.f ? sum[j] : 0.f);
  }
}

}  // namespace conv
}  // namespace absb
