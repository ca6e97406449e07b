// The narrow output layer of a bf16 network in one pass over 64 gradient rows per CTA, with its
// three small contractions on the warp-level tensor-core instruction (mma.sync m16n8k16, bf16
// operands, fp32 accumulation):
//   logits  Z[r][c]   = sum_m H[r][m] W_s[m][c] + b_s[c]       soft-max cross-entropy loss and
//                                                              delta D = softmax(Z) - onehot(y)
//   weights G[m][c]   = sum_r H[r][m] D[r][c]  (+ bias row)    this CTA's share, Eq. 3 adds them up
//   below   Dl[r][m]  = (sum_c D[r][c] W_s[m][c]) [H[r][m] > 0]
// (Eq. 2 with U = 1 for the rows' model version s; D is rounded to bf16 like every stored delta.)
// The 64 input rows stay in shared memory for all three; the class count is padded to 16 with
// zero weights.  The work per CTA is a few hundred tensor-core instructions, so the kernel is
// bound by the round trip of its loads and stores: one wave of CTAs, every phase short.
#pragma once
#include "common.cuh"
#include "narrow.cuh"

namespace absb {
namespace outl {

constexpr int ROWS = 64;          // gradient rows per CTA
constexpr int THREADS = 256;
constexpr int CP = 16;            // padded class count
constexpr int WP = 24;            // shared-memory pitch (elements) of the [.][16] class rows: 48 bytes,
                                  // which spreads eight consecutive rows over all banks

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// d += a (16 x 16, row) * b (16 x 8, col), bf16 in, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

inline size_t smem_bytes(int in, int C) {
  return (size_t)ROWS * (in + 8) * 2 + (size_t)(in + 8) * WP * 2 + (size_t)ROWS * WP * 2 + (size_t)4 * 32 * 8 * 4 +
         ((size_t)(in + 1) * C * 2 + 15) / 16 * 16 + 64;
}

// NT = in / 128: feature tiles (16 wide) per warp of the weight-gradient phase.
// part[cta][(in + 1) * C]: this CTA's share of the layer's gradient block (row `in` = bias sums).
template <int NT>
__global__ void __launch_bounds__(THREADS) out_layer_mma_kernel(NarrowArgs a, float* part, int has_dgrad) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char osm_raw[];
  DevState* st = a.st;
  RoundInfo* ri = a.ri;
  if (st->status != ST_OK) return;
  const int r0 = blockIdx.x * ROWS;
  if (r0 >= ri->n_rows) return;
  constexpr int IN = NT * 128;
  constexpr int HP = IN + 8;                    // row pitch of the input rows (elements): 16 bytes of padding
  const int C = a.C;
  __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(osm_raw);          // [ROWS][HP] input rows, later Dl
  __nv_bfloat16* ws = hs + (size_t)ROWS * HP;                             // [IN + 1 (+7)][WP] weights, row IN = bias
  __nv_bfloat16* d3s = ws + (size_t)(IN + 8) * WP;                        // [ROWS][WP] deltas of this layer
  float* lp = reinterpret_cast<float*>(d3s + (size_t)ROWS * WP);          // [4][32][8] logit partial sums
  __nv_bfloat16* wraw = reinterpret_cast<__nv_bfloat16*>(lp + 4 * 32 * 8);  // [IN + 1][C] weights + bias as stored
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;

  // ---- loads: the 64 input rows (asynchronous 16-byte copies), the weights of the rows' version
  const __nv_bfloat16* src = (const __nv_bfloat16*)a.act_in + (size_t)r0 * IN;
  for (int item = tid; item < ROWS * (IN / 8); item += THREADS) {
    const int rr = item / (IN / 8), v = item - rr * (IN / 8);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_u32(hs + (size_t)rr * HP + v * 8)),
                 "l"(src + (size_t)rr * IN + v * 8) : "memory");
  }
  const int slot = a.tile_slot[r0 / st->RB];
  const float sa = sa_slot_weight(st, ri->t, slot);     // staleness-aware step size: weight of these rows in Eq. 3
  const __nv_bfloat16* Wm = (const __nv_bfloat16*)a.ring + (size_t)slot * a.slot_stride + a.w_off;
  {
    // weights + bias are contiguous and start on a 128-byte boundary: whole 16-byte pieces
    const int n16 = (int)(((size_t)(IN + 1) * C * 2 + 15) / 16);
    for (int i = tid; i < n16; i += THREADS)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_u32(wraw + 8 * i)), "l"(Wm + 8 * i) : "memory");
  }
  // labels of the two rows whose soft-max this thread takes part in (warps 0..3)
  int lab[2] = {-1, -1};
  if (warp < 4) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int s = a.row_idx[r0 + 16 * warp + g + 8 * h];
      lab[h] = s < 0 ? -1 : a.labels[s];
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  for (int i = tid; i < (IN + 1) * CP; i += THREADS) {      // class rows padded to 16 with zeros
    const int k = i >> 4, c = i & 15;
    ws[k * WP + c] = c < C ? wraw[k * C + c] : __float2bfloat16_rn(0.f);
  }
  __syncthreads();

  // ---- logits: warp = (row tile mt, half of the features kh)
  {
    const int mt = warp & 3, kh = warp >> 2;
    float acc[2][4];
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;
    const uint32_t a_base = s_u32(hs + (size_t)(16 * mt + (lane & 15)) * HP + (lane >> 4) * 8);
    const uint32_t b_base = s_u32(ws + (size_t)((lane & 7) + ((lane >> 3) & 1) * 8) * WP + (lane >> 4) * 8);
#pragma unroll 4
    for (int k0 = kh * (IN / 2); k0 < (kh + 1) * (IN / 2); k0 += 16) {
      uint32_t af[4], bf[4];
      ldsm4(a_base + k0 * 2, af);
      ldsm4t(b_base + k0 * WP * 2, bf);
      mma16816(acc[0], af, bf[0], bf[1]);
      mma16816(acc[1], af, bf[2], bf[3]);
    }
    if (kh == 1) {
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) lp[(mt * 32 + lane) * 8 + n * 4 + i] = acc[n][i];
    }
    __syncthreads();
    if (kh == 0) {
      // thread: rows g and g + 8 of the tile, classes 2t, 2t+1, 8+2t, 8+2t+1
      bool bad = false;
      uint32_t dpk[2][2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float z[4];
        int cls[4];
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = 8 * n + 2 * t + j;
            cls[2 * n + j] = c;
            z[2 * n + j] = acc[n][2 * h + j] + lp[(mt * 32 + lane) * 8 + n * 4 + 2 * h + j] +
                           __bfloat162float(ws[IN * WP + c]);
          }
        float zmax = -3.0e38f;
#pragma unroll
        for (int i = 0; i < 4; ++i) if (cls[i] < C) zmax = fmaxf(zmax, z[i]);
        zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 1));
        zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 2));
        const int y = lab[h];
        float se = 0.f, zy = 0.f, e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          e[i] = cls[i] < C ? expf(z[i] - zmax) : 0.f;
          se += e[i];
          if (cls[i] == y) zy = z[i];
        }
        se += __shfl_xor_sync(0xffffffffu, se, 1);
        se += __shfl_xor_sync(0xffffffffu, se, 2);
        zy += __shfl_xor_sync(0xffffffffu, zy, 1);
        zy += __shfl_xor_sync(0xffffffffu, zy, 2);
        const float inv = 1.f / se;
        float d[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          d[i] = (y >= 0 && cls[i] < C) ? (e[i] * inv - (cls[i] == y ? 1.f : 0.f)) * sa : 0.f;   // padding rows add nothing to Eq. 3
        dpk[h][0] = pack_bf16(d[0], d[1]);
        dpk[h][1] = pack_bf16(d[2], d[3]);
        const int rr = 16 * mt + g + 8 * h;
        *reinterpret_cast<uint32_t*>(d3s + rr * WP + 2 * t) = dpk[h][0];
        *reinterpret_cast<uint32_t*>(d3s + rr * WP + 8 + 2 * t) = dpk[h][1];
        if (t == 0) {
          const float loss = y >= 0 ? logf(se) - (zy - zmax) : 0.f;
          a.row_loss[r0 + rr] = loss;
          bad |= !isfinite(loss);
        }
      }
      if (bad) ri->diverged = 1;
    }
    __syncthreads();
  }

  // ---- this CTA's share of the weight and bias gradient: warp w owns feature tiles w, w + 8, ...
  {
    float acc[NT][2][4];
#pragma unroll
    for (int m = 0; m < NT; ++m)
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[m][n][i] = 0.f;
    const uint32_t b_base = s_u32(d3s + (size_t)((lane & 7) + ((lane >> 3) & 1) * 8) * WP + (lane >> 4) * 8);
    const uint32_t a_base = s_u32(hs + (size_t)((lane & 7) + ((lane >> 4) & 1) * 8) * HP + ((lane >> 3) & 1) * 8);
#pragma unroll
    for (int ks = 0; ks < ROWS / 16; ++ks) {
      uint32_t bf[4];
      ldsm4t(b_base + ks * 16 * WP * 2, bf);
#pragma unroll
      for (int m = 0; m < NT; ++m) {
        uint32_t af[4];
        ldsm4t(a_base + (uint32_t)(ks * 16 * HP + (warp + 8 * m) * 16) * 2, af);
        mma16816(acc[m][0], af, bf[0], bf[1]);
        mma16816(acc[m][1], af, bf[2], bf[3]);
      }
    }
    float* dst = part + (size_t)blockIdx.x * (size_t)(IN + 1) * C;
#pragma unroll
    for (int m = 0; m < NT; ++m)
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int f = (warp + 8 * m) * 16 + g + 8 * (i >> 1), c = 8 * n + 2 * t + (i & 1);
          if (c < C) dst[(size_t)f * C + c] = acc[m][n][i];
        }
    if (tid < C) {
      float tot = 0.f;
      for (int rr = 0; rr < ROWS; ++rr) tot += __bfloat162float(d3s[rr * WP + tid]);
      dst[(size_t)IN * C + tid] = tot;
    }
  }
  if (!has_dgrad) return;
  __syncthreads();            // all reads of the input rows by the gradient phase are done

  // ---- delta of the layer below, written over the input rows: warp w owns features [w*IN/8, (w+1)*IN/8)
  {
    uint32_t af[ROWS / 16][4];
#pragma unroll
    for (int mt = 0; mt < ROWS / 16; ++mt)
      ldsm4(s_u32(d3s + (size_t)(16 * mt + (lane & 15)) * WP + (lane >> 4) * 8), af[mt]);
    const uint32_t b_base = s_u32(ws + (size_t)((lane & 7) + ((lane >> 4) & 1) * 8) * WP + ((lane >> 3) & 1) * 8);
#pragma unroll 2
    for (int f0 = warp * (IN / 8); f0 < (warp + 1) * (IN / 8); f0 += 16) {
      uint32_t bf[4];
      ldsm4(b_base + f0 * WP * 2, bf);
#pragma unroll
      for (int mt = 0; mt < ROWS / 16; ++mt)
#pragma unroll
        for (int n = 0; n < 2; ++n) {
          float d[4] = {0.f, 0.f, 0.f, 0.f};
          mma16816(d, af[mt], bf[2 * n], bf[2 * n + 1]);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t* hp = reinterpret_cast<uint32_t*>(hs + (size_t)(16 * mt + g + 8 * h) * HP + f0 + 8 * n + 2 * t);
            const float2 hv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(hp));
            *hp = pack_bf16(hv.x > 0.f ? d[2 * h] : 0.f, hv.y > 0.f ? d[2 * h + 1] : 0.f);
          }
        }
    }
  }
  __syncthreads();
  __nv_bfloat16* out = (__nv_bfloat16*)a.delta_in + (size_t)r0 * IN;
  for (int item = tid; item < ROWS * (IN / 8); item += THREADS) {
    const int rr = item / (IN / 8), v = item - rr * (IN / 8);
    *reinterpret_cast<uint4*>(out + (size_t)rr * IN + v * 8) = *reinterpret_cast<const uint4*>(hs + (size_t)rr * HP + v * 8);
  }
}

}  // namespace outl
}  // namespace absb
