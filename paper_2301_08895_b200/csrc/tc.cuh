// Grouped bf16 GEMMs of the hidden layers on the 5th-generation tensor cores (tcgen05, accumulators
// in tensor memory, operands staged by TMA into 128-byte-swizzled shared memory).
//
// One persistent, warp-specialised kernel serves the three contractions of Eq. 2 / Eq. 3:
//   FWD    H[r][n]  = relu( sum_k A[r][k] W_s[k][n] + b_s[n] )          rows grouped by model version
//   DGRAD  D[r][m]  = ( sum_n Dl[r][n] W_s[m][n] ) * [H[r][m] > 0]
//   WGRAD  G_p[m][n] = sum_{r in chunk p} A[r][m] Dl[r][n]               summed over ALL selected workers
// (DGRAD can also leave the column sums of D over each group of 32 rows: they add up to the bias gradient of the
// layer below, whose WGRAD then needs no row of ones.)
// "s" is the ring slot of the row tile's model version (all rows of a 128-row tile share it).
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns the tensor-memory allocation),
// warps 2..9 = epilogue (tensor memory -> registers -> global; two warps per tensor-memory lane
// quarter, each draining one half of the tile's columns).  Two accumulators alternate so the
// epilogue of one tile overlaps the main loop of the next.  Every mbarrier wait is bounded (WAIT_LIMIT_NS); on
// expiry the CTA raises ST_TIMEOUT, drains its own copies, frees tensor memory and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace absb {
namespace tc {

constexpr int BM = 128;      // tile rows (UMMA M)
constexpr int BK = 64;       // k elements per stage = one 128-byte swizzle row of bf16
constexpr int UK = 16;       // k per tcgen05.mma of kind::f16
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;

enum Mode : int { FWD = 0, DGRAD = 1, WGRAD = 2 };

struct Params {
  DevState* st;
  RoundInfo* ri;
  const int* tile_slot;
  int mode;
  int M_total;             // WGRAD: in + 1 (weight rows and the bias row of G); FWD/DGRAD: unused
  int N_total;             // FWD: out, DGRAD: in, WGRAD: out
  int K_total;             // FWD: in,  DGRAD: out, WGRAD: unused (rows come from the device state)
  int P;                   // WGRAD split count; 0: one split per selected worker, added to its upload
  const __nv_bfloat16* ring; size_t slot_stride; size_t b_off;   // FWD bias: ring + slot*stride + b_off
  const __nv_bfloat16* mask_src;   // DGRAD: H[r][N_total] (used when mask_bits is null)
  const uint32_t* mask_bits;       // DGRAD: word [r][n/32] holds (H[r][n] > 0) for its 32 columns, column j of
                                   // the word at bit (j >> 1) + 16 * (j & 1) (even columns low half, odd high)
  uint32_t* relu_bits;             // FWD: the same bits for this layer's output (may be null)
  int mask_words;                  // words per row of mask_bits / relu_bits = ceil(N_total / 32)
  __nv_bfloat16* out_bf16;         // FWD/DGRAD result [rows][N_total]
  float* out_f32;                  // WGRAD: G + w_off, partial p at + p*slot_stride, row pitch N_total
  float* colsum;                   // DGRAD: [rows / 32][N_total] column sums of the stored result over each group of 32
                                   // rows (they add up to the bias gradient of the layer below), or null
  int no_bias_tile;                // WGRAD: the bias gradient comes from such column sums: no extra row tile
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint32_t mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Longest time a kernel of the round loop waits on a barrier or a counter: 100 ms, thousands of
// times the longest tile, and short enough that a wait that can never end costs a shared GPU
// next to nothing.
constexpr unsigned long long WAIT_LIMIT_NS = 100000000ull;
// Bounded wait (limit_ns, and never more than 2^28 polls).  False = gave up, or another role of
// this CTA already gave up; *abort is the CTA-wide flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort,
                                          unsigned long long limit_ns = WAIT_LIMIT_NS) {
  if (mbar_test(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t i = 1; i < (1u << 28); ++i) {
    if (mbar_test(bar, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort) return false;
      if (global_ns() - t0 > limit_ns) break;
    }
  }
  *abort = 1;
  return false;
}

__device__ __forceinline__ void prefetch_map(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// Shared-memory matrix descriptor of a 128-byte-swizzled bf16 operand tile:
// bits [0,14) start >> 4, [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4,
// [46,48) descriptor version 1, [61,64) layout 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, majors, N >> 3, M >> 4.
__host__ __device__ constexpr uint32_t instr_desc(int a_mn_major, int b_mn_major, int n, int m = BM) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// ---- two-CTA form (cta_group::2): one MMA spans the tensor cores of a CTA pair; M = 256 (128 rows
// per CTA), each CTA supplies its A tile and its half of the B tile from its own shared memory.
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {   // same offset in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma2_load_2d(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void umma2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  const uint32_t z = 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
__device__ __forceinline__ void umma2_commit_both(uint64_t* bar) {   // arrives on `bar` in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int BN, int CG = 1> struct Cfg {
  static constexpr int STAGES = (BN == 256 && CG == 1) ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = (BN / CG) * BK * 2;     // with a CTA pair each CTA holds half of the B tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int OUT_BYTES = EPI_WARPS * 4096;   // epilogue staging: one box of 32 rows x 128 B per warp
  static constexpr size_t SMEM_BYTES =
      (size_t)STAGES * STAGE_BYTES + OUT_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + 2 * BN * 2 /*bias*/;
};

struct TileCoord { int which, rt, a_row, b_col, slot, k_begin, n_kb, split, bias_tile; };
// Tiling of one problem of a launch.
struct Prob { int mode, n_ct, n_mt_w, n_mt, n_tiles, chunk; };

// A launch serves one problem (p0), or two independent ones (p1.mode >= 0): a layer's weight
// gradient (p0) next to its delta back-propagation (p1).  Both are short (one or two tiles per
// CTA), so sharing one launch halves their fixed costs; the weight gradient's few long tiles go to
// the first CTAs, the remaining CTAs split the many short tiles of the back-propagation.
// CG = 1: one CTA per tile of 128 x BN.  CG = 2: a cluster of two CTAs per tile of 256 x BN; the
// leader (cluster rank 0) issues the MMAs for both, every CTA loads its own A rows and its half of
// B and drains its own half of the accumulator.
template <int BN, int CG>
__global__ void __launch_bounds__(THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_b0,
               const __grid_constant__ CUtensorMap map_ones, const __grid_constant__ CUtensorMap map_out0,
               const Params p0,
               const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ CUtensorMap map_out1, const Params p1) {
  // The kernel in front of this one may still be running (programmatic stream serialization): the
  // kernel behind this one may be scheduled as early, and everything that does not read the
  // predecessors' results -- barriers, the tensor-memory allocation, descriptor prefetch -- is done
  // before the wait for them.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using C = Cfg<BN, CG>;
  constexpr int TM_ROWS = BM * CG;              // rows of one tile
  extern __shared__ uint8_t smem_raw[];
  const int rank = (CG == 2) ? (int)cluster_rank() : 0;
  const int unit = (int)blockIdx.x / CG;        // tile-processing unit (CTA or CTA pair)
  const int n_units = (int)gridDim.x / CG;
  DevState* st = p0.st;
  RoundInfo* ri = p0.ri;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* stage_out = smem + (size_t)C::STAGES * C::STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(stage_out + C::OUT_BYTES);
  uint64_t* full = bars;                     // [STAGES] TMA bytes landed
  uint64_t* empty = bars + C::STAGES;        // [STAGES] MMAs that read the stage are done
  uint64_t* acc_full = bars + 2 * C::STAGES; // [2] accumulator complete
  uint64_t* acc_empty = acc_full + 2;        // [2] accumulator drained by the epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  __nv_bfloat16* bias_s = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<uint8_t*>(bars) + 256);   // [2][BN]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS * CG); }
    *abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_map(&map_a0); prefetch_map(&map_b0); prefetch_map(&map_out0);
    if (p1.mode >= 0) { prefetch_map(&map_a1); prefetch_map(&map_b1); prefetch_map(&map_out1); }
  }
  if (warp == 1) {
    if (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();              // the peer's barriers exist before anything signals them
  tc_fence_after();
  // barriers that live in the leader CTA, as addresses valid from either CTA of the pair
  const uint32_t full0_addr = (CG == 2) ? map_to_cta(smem_u32(&full[0]), 0) : smem_u32(&full[0]);
  const uint32_t acc_empty0_addr = (CG == 2) ? map_to_cta(smem_u32(&acc_empty[0]), 0) : smem_u32(&acc_empty[0]);
  const uint32_t tmem_base = *tmem_slot;

  // from here on the kernel reads what its predecessors wrote (device state, layouts, operands)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const bool running = st->status == ST_OK;
  const int n_rows = running ? ri->n_rows : 0;
  const int n_row_tiles = n_rows / TM_ROWS;
  auto make_prob = [&](const Params& q) -> Prob {
    Prob r;
    r.mode = q.mode;
    r.n_ct = (q.N_total + BN - 1) / BN;
    // WGRAD: one extra row tile multiplies a column of ones with the deltas, which yields the bias
    // gradient (row `in` of the [in + 1][out] gradient block) on the tensor cores for free
    r.n_mt_w = (q.M_total - 1 + TM_ROWS - 1) / TM_ROWS;
    r.n_mt = (q.mode == WGRAD) ? r.n_mt_w + (q.no_bias_tile ? 0 : 1) : n_row_tiles;
    const int n_splits = max(1, q.P > 0 ? q.P : ri->K);   // P = 0: one split per selected worker (its own rows)
    r.n_tiles = (q.mode == WGRAD) ? r.n_mt * r.n_ct * n_splits : n_row_tiles * r.n_ct;
    r.chunk = (q.mode == WGRAD) ? round_up((n_rows + n_splits - 1) / n_splits, BK) : 0;
    return r;
  };
  const Prob P0 = make_prob(p0);
  Prob P1 = P0;
  P1.n_tiles = 0;
  if (p1.mode >= 0) P1 = make_prob(p1);
  const int T0 = P0.n_tiles, T1 = P1.n_tiles;
  // i-th tile of this unit, or -1.  Two problems with fewer long tiles than units: units [0, T0)
  // take one tile of problem 0 each, the others stride over problem 1; otherwise all units stride
  // over the concatenated tiles.  Weight gradient + back-propagation: a long tile costs about as
  // much as `lead` short ones (k-blocks at 0.34 us plus about 3.5 us of fixed cost per tile), so
  // the other units take `lead` short tiles each and what is left is strided over ALL units.
  const bool split_units = T1 > 0 && T0 < n_units;
  const int R_units = n_units - T0;
  int lead = 1 << 20;
  if (split_units && p0.mode == WGRAD && p1.mode == DGRAD) {
    const float long_t = (float)(P0.chunk / BK) * 0.34f + 3.5f;
    const float short_t = (float)((p1.K_total + BK - 1) / BK) * 0.34f + 3.5f;
    lead = max(1, (int)(long_t / short_t + 0.5f));
  }
  const int n_lead = split_units ? min(T1, lead * R_units) : 0;      // short tiles handed out before the long-tile units join
  auto tile_at = [&](int i) -> int {
    if (split_units) {
      if (unit < T0) {
        if (i == 0) return unit;
        const int t1 = n_lead + unit + (i - 1) * n_units;
        return t1 < T1 ? T0 + t1 : -1;
      }
      if (i < lead) {
        const int t1 = (unit - T0) + i * R_units;
        return t1 < n_lead ? T0 + t1 : -1;
      }
      const int t1 = n_lead + unit + (i - lead) * n_units;
      return t1 < T1 ? T0 + t1 : -1;
    }
    const int t = unit + i * n_units;
    return t < T0 + T1 ? t : -1;
  };
  // a CTA (pair) without work, or a run that has ended, goes straight to the teardown (same
  // decision in both CTAs of a pair)
  const bool has_work = running && tile_at(0) >= 0;
  const int RB = st->RB;

  auto tile_coord = [&](int gtile) -> TileCoord {
    TileCoord c;
    c.which = gtile >= T0 ? 1 : 0;
    const int tile = c.which ? gtile - T0 : gtile;
    const Prob& P = c.which ? P1 : P0;
    const Params& q = c.which ? p1 : p0;
    if (P.mode == WGRAD) {
      const int per_split = P.n_mt * P.n_ct;
      c.split = tile / per_split;
      const int rem = tile - c.split * per_split;
      const int mt = rem / P.n_ct;
      c.bias_tile = (mt == P.n_mt_w);
      c.rt = mt;
      c.a_row = mt * TM_ROWS + rank * BM;    // m0 of this CTA
      c.b_col = (rem % P.n_ct) * BN;         // n0
      c.slot = 0;
      c.k_begin = min(n_rows, c.split * P.chunk);
      const int k_end = min(n_rows, (c.split + 1) * P.chunk);
      c.n_kb = (k_end - c.k_begin) / BK;
    } else {
      const int rt = tile / P.n_ct;
      c.rt = rt;
      c.split = 0;
      c.bias_tile = 0;
      c.a_row = rt * TM_ROWS + rank * BM;
      c.b_col = (tile - rt * P.n_ct) * BN;
      c.slot = q.tile_slot[(rt * TM_ROWS) / RB];
      c.k_begin = 0;
      c.n_kb = (q.K_total + BK - 1) / BK;
    }
    return c;
  };

  if (!has_work) {
    // nothing to do
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    int armed[C::STAGES];
    for (int s = 0; s < C::STAGES; ++s) armed[s] = -1;
    bool ok = true;
    // loads complete on the leader's "full" barrier (own barrier when CG == 1)
    auto ld2 = [&](void* dst, const CUtensorMap* map, int st_, int x, int y) {
      if (CG == 2) tma2_load_2d(dst, map, full0_addr + 8u * (uint32_t)st_, x, y);
      else tma_load_2d(dst, map, &full[st_], x, y);
    };
    auto ld3 = [&](void* dst, const CUtensorMap* map, int st_, int x, int y, int z) {
      if (CG == 2) tma2_load_3d(dst, map, full0_addr + 8u * (uint32_t)st_, x, y, z);
      else tma_load_3d(dst, map, &full[st_], x, y, z);
    };
    constexpr int BH = BN / CG;                  // B columns (rows of the B tile) this CTA loads
    // one elected lane: the stage ring is shallow, so nothing may sit between a stage being
    // released and its next loads being issued
    if (lane == 0) {
      for (int it = 0; ok; ++it) {
        const int tile = tile_at(it);
        if (tile < 0) break;
        const TileCoord c = tile_coord(tile);
        const int mode = c.which ? p1.mode : p0.mode;
        const CUtensorMap& map_a = c.which ? map_a1 : map_a0;
        const CUtensorMap& map_b = c.which ? map_b1 : map_b0;
        const int b0 = c.b_col + rank * BH;
        for (int kb = 0; kb < c.n_kb; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1u, abort)) { ok = false; break; }
          uint8_t* sa = smem + (size_t)stage * C::STAGE_BYTES;
          uint8_t* sb = sa + C::A_BYTES;
          if (rank == 0) {                     // the leader arms the barrier for the bytes of the whole pair
            mbar_expect_tx(&full[stage], CG * C::STAGE_BYTES);
            armed[stage] = (int)phase;
          }
          const int k0 = c.k_begin + kb * BK;
          if (mode == FWD) {
            ld2(sa, &map_a, stage, k0, c.a_row);
            for (int j = 0; j < BH / 64; ++j) ld3(sb + j * 8192, &map_b, stage, b0 + 64 * j, k0, c.slot);
          } else if (mode == DGRAD) {
            ld2(sa, &map_a, stage, k0, c.a_row);
            ld3(sb, &map_b, stage, k0, b0, c.slot);
          } else {
            if (c.bias_tile) {   // only column 0 of the 64-wide ones matrix is non-zero; the rest is zero fill
              for (int j = 0; j < BM / 64; ++j) ld2(sa + j * 8192, &map_ones, stage, rank * BM + 64 * j, k0);
            } else {
              for (int j = 0; j < BM / 64; ++j) ld2(sa + j * 8192, &map_a, stage, c.a_row + 64 * j, k0);
            }
            for (int j = 0; j < BH / 64; ++j) ld2(sb + j * 8192, &map_b, stage, b0 + 64 * j, k0);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
    // tail: every stage's release (an asynchronous arrive from the tensor core) must have landed
    // before this CTA's shared memory goes away
    if (lane == 0) {
      for (int s = 0; s < C::STAGES && ok; ++s) {
        if (!mbar_wait(&empty[stage], phase ^ 1u, abort)) ok = false;
        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        // let this CTA's copies in flight land before the shared memory is released
        for (int s = 0; s < C::STAGES; ++s)
          if (armed[s] >= 0) {
            const unsigned long long t0 = global_ns();
            while (!mbar_test(&full[s], (uint32_t)armed[s]) && global_ns() - t0 < WAIT_LIMIT_NS) {}
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {            // with a CTA pair only the leader issues MMAs
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int it = 0; ok; ++it) {
        const int tile = tile_at(it);
        if (tile < 0) break;
        const TileCoord c = tile_coord(tile);
        if (c.n_kb == 0) continue;
        const int mode = c.which ? p1.mode : p0.mode;
        const bool a_mn = (mode == WGRAD), b_mn = (mode != DGRAD);
        const uint32_t idesc = instr_desc(a_mn ? 1 : 0, b_mn ? 1 : 0, BN, TM_ROWS);
        // K-major tile: rows of 128 B, 8-row groups 1024 B apart; a k step of 16 elements is 32 B.
        // MN-major tile: 64-wide boxes 8192 B apart (leading offset), 8-k groups 1024 B apart;
        // a k step of 16 rows is 2048 B.
        const uint32_t a_lbo = a_mn ? 8192u : 16u, b_lbo = b_mn ? 8192u : 16u;
        const uint32_t a_kstep = a_mn ? 2048u : 32u, b_kstep = b_mn ? 2048u : 32u;
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < c.n_kb; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + (uint32_t)stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / UK; ++kk) {
            const uint64_t da = smem_desc(sa + kk * a_kstep, a_lbo, 1024u);
            const uint64_t db = smem_desc(sb + kk * b_kstep, b_lbo, 1024u);
            if (CG == 2) umma2(d_tmem, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
            else umma(d_tmem, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          if (CG == 2) umma2_commit_both(&empty[stage]);      // frees the stage in both CTAs
          else umma_commit(&empty[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (CG == 2) umma2_commit_both(&acc_full[acc]);       // wakes both epilogues
        else umma_commit(&acc_full[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps)
    // Results leave through per-warp staging boxes (32 rows x 128 bytes, 128-byte swizzle) and one
    // bulk tensor store per box, so global memory sees whole rows instead of 32 scattered 16-byte
    // pieces per store instruction and a warp never waits for another warp.
    const int q = warp & 3;                    // tensor-memory lane quarter this warp may read
    const int half = (warp - 2) >> 2;          // which half of the tile's columns this warp drains
    constexpr int N_HALF = (BN >= 128) ? 2 : 1;      // a 64-column tile is drained by four warps only
    constexpr int HALF_COLS = BN / N_HALF;
    const bool works = half < N_HALF;
    const int row_in_tile = q * 32 + lane;
    const bool issuer = lane == 0;             // issues and tracks this warp's bulk stores
    const int sw = lane & 7;
    uint8_t* my_box = stage_out + ((warp - 2) << 12);
    uint8_t* my_row = my_box + lane * 128;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int it = 0; ; ++it) {
      const int tile = tile_at(it);
      if (tile < 0) break;
      const TileCoord c = tile_coord(tile);
      const Params& p = c.which ? p1 : p0;
      const int mode = p.mode;
      const CUtensorMap& map_out = c.which ? map_out1 : map_out0;
      const int box_cols = (mode == WGRAD) ? 32 : 64;
      const bool have = c.n_kb > 0;
      // output row (FWD/DGRAD) or gradient row m (WGRAD; the bias tile's row 0 is row `in`)
      const int r = (mode == WGRAD && c.bias_tile) ? (p.M_total - 1) + rank * BM + row_in_tile : c.a_row + row_in_tile;
      // fetch what the epilogue needs from global memory before waiting for the accumulator
      uint32_t mw[BN / 32];
      __nv_bfloat16* bias_t = bias_s + acc * BN;
      if (mode == FWD) {
        const __nv_bfloat16* bias = p.ring + (size_t)c.slot * p.slot_stride + p.b_off;
        for (int i = (int)threadIdx.x - 64; i < BN; i += 32 * EPI_WARPS) {
          const int n = c.b_col + i;
          bias_t[i] = n < p.N_total ? bias[n] : __float2bfloat16_rn(0.f);
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * EPI_WARPS) : "memory");
      } else if (mode == DGRAD) {
#pragma unroll
        for (int i = 0; i < BN / 32; ++i) {
          const int w = c.b_col / 32 + i;
          if (i * 32 / HALF_COLS != half) { mw[i] = 0u; continue; }
          if (p.mask_bits != nullptr) {
            mw[i] = w < p.mask_words ? p.mask_bits[(size_t)r * p.mask_words + w] : 0u;
          } else {                               // no stored sign bits: derive them from the activations
            uint32_t bits = 0u;
            for (int j = 0; j < 32; ++j) {
              const int n = w * 32 + j;
              if (n < p.N_total && __bfloat162float(p.mask_src[(size_t)r * p.N_total + n]) > 0.f)
                bits |= 1u << ((j >> 1) + 16 * (j & 1));
            }
            mw[i] = bits;
          }
        }
      }
      if (have) {
        if (!mbar_wait(&acc_full[acc], acc_phase, abort)) break;
        tc_fence_after();
      }
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c0 = half * HALF_COLS; c0 < (half + 1) * HALF_COLS && works; c0 += box_cols) {
        const int n0 = c.b_col + c0;
        if (n0 >= p.N_total) break;            // uniform in the warp
        uint32_t v[32];
        if (mode == WGRAD) {
          if (have) tmem_ld32(t_row + (uint32_t)c0, v);
          else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;
          }
          // the staging box is free once the bulk store issued from it has read it
          if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
          if (c.bias_tile) {                   // a single useful row: plain stores
            if (row_in_tile == 0 && rank == 0) {
              float* dst = p.out_f32 + (size_t)c.split * p.slot_stride + (size_t)r * p.N_total + n0;
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                if (n0 + i < p.N_total) {
                  uint4 o = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                  if (p.P == 0) {              // per-worker splits add to the worker's upload
                    const float4 old = *reinterpret_cast<const float4*>(dst + i);
                    o.x = __float_as_uint(old.x + __uint_as_float(o.x));
                    o.y = __float_as_uint(old.y + __uint_as_float(o.y));
                    o.z = __float_as_uint(old.z + __uint_as_float(o.z));
                    o.w = __float_as_uint(old.w + __uint_as_float(o.w));
                  }
                  *reinterpret_cast<uint4*>(dst + i) = o;
                }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<uint4*>(my_row + ((j ^ sw) << 4)) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          }
        } else {
#pragma unroll
          for (int hlf = 0; hlf < 2; ++hlf) {
            const int cc = c0 + 32 * hlf;       // column offset inside the tile
            if (c.b_col + cc >= p.N_total) break;
            if (have) tmem_ld32(t_row + (uint32_t)cc, v);
            else {
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = 0u;
            }
            if (hlf == 0) {                     // the staging box is free once its last store has read it
              if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
              __syncwarp();
            }
            uint32_t bits = 0u;
            if (mode == DGRAD) {
#pragma unroll
              for (int i = 0; i < BN / 32; ++i) bits = (i == (cc >> 5)) ? mw[i] : bits;
            }
            uint32_t relu = 0u;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint4 o;
              __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int i = 8 * j + 2 * e;    // columns i, i + 1 = pair i / 2 of the 32-column word
                float x = __uint_as_float(v[i]), y = __uint_as_float(v[i + 1]);
                if (mode == FWD) {
                  const float2 bf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(bias_t + cc + i));
                  x = fmaxf(x + bf.x, 0.f);
                  y = fmaxf(y + bf.y, 0.f);
                }
                o2[e] = __floats2bfloat162_rn(x, y);
                uint32_t& u = *reinterpret_cast<uint32_t*>(&o2[e]);
                if (mode == FWD) {
                  // The bit records the sign of the STORED activation.  Stored values are >= 0, so
                  // "positive" = "magnitude bits non-zero": adding 0x7fff carries into bit 15 of each
                  // half exactly then.  After 16 pairs the flags of pair q sit at bits q and 16 + q.
                  relu = (relu >> 1) | (((u & 0x7fff7fffu) + 0x7fff7fffu) & 0x80008000u);
                } else {
                  u &= ((bits >> (i >> 1)) & 0x00010001u) * 0xffffu;
                }
              }
              *reinterpret_cast<uint4*>(my_row + (((4 * hlf + j) ^ sw) << 4)) = o;
            }
            if (mode == FWD && p.relu_bits != nullptr)
              p.relu_bits[(size_t)r * p.mask_words + ((c.b_col + cc) >> 5)] = relu;
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (mode == DGRAD && p.colsum != nullptr) {
          // column sums of the warp's 32 x 64 box of stored (rounded, masked) deltas: lane l adds columns
          // 2l, 2l + 1 over the 32 rows in order, reading the swizzled staging box row by row
          float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
          for (int rr = 0; rr < 32; ++rr) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(my_box + rr * 128 + ((((lane >> 2) ^ (rr & 7))) << 4) + ((lane & 3) << 2));
            s0 += __uint_as_float(w << 16);
            s1 += __uint_as_float(w & 0xffff0000u);
          }
          const int n = n0 + 2 * lane;
          if (n < p.N_total)
            *reinterpret_cast<float2*>(p.colsum + (size_t)((c.a_row + q * 32) >> 5) * p.N_total + n) = make_float2(s0, s1);
        }
        if (issuer && !(mode == WGRAD && c.bias_tile)) {
          if (mode == WGRAD && p.P == 0)       // one split per worker: the tile adds to that worker's upload
            asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(smem_u32(my_box)), "r"(n0), "r"(c.a_row + q * 32), "r"(c.split)
                         : "memory");
          else if (mode == WGRAD)
            asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(smem_u32(my_box)), "r"(n0), "r"(c.a_row + q * 32), "r"(c.split)
                         : "memory");
          else
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(smem_u32(my_box)), "r"(n0), "r"(c.a_row + q * 32)
                         : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      if (have) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {                       // the accumulator barrier lives in the leader CTA
          if (CG == 2) mbar_arrive_cluster(acc_empty0_addr + 8u * (uint32_t)acc);
          else mbar_arrive(&acc_empty[acc]);
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
    // shared memory may be released once the stores have read it; their global writes complete
    // with the grid
    if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();              // neither CTA leaves while the pair still uses its memory
  if (warp == 1) {
    tc_fence_after();
    if (CG == 2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::TMEM_COLS) : "memory");
  }
  if (threadIdx.x == 0 && *abort) {
    st->timeout_where = 100 + p0.mode;
    st->status = ST_TIMEOUT;
  }
}

// Self-test of the bounded wait: one warp initialises a barrier that expects one arrival, nobody
// ever arrives, and lane 0 waits on it with the given limit.  The wait must give up, and the
// kernel then reports it the way the round-loop kernels do (status word + site), and returns.
constexpr int TIMEOUT_SITE_SELFTEST = 900;
__global__ void wait_selftest_kernel(DevState* st, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait(&bar, 0u, &abort_flag, limit_ns)) {
    st->timeout_where = TIMEOUT_SITE_SELFTEST;
    st->status = ST_TIMEOUT;
  }
}

}  // namespace tc
}  // namespace absb
