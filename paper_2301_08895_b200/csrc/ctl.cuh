// Server-side integer engine of Algorithm 1: arrival selection, Eq. 4-6 bookkeeping,
// Philox job durations and minibatch indices.  One CTA of 1024 threads; every result is an
// integer decided by exact arithmetic, so the trace is reproducible bit for bit.
#pragma once
#include "common.cuh"

namespace absb {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies, with the key
// advanced by Weyl constants between rounds.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi_a = __umulhi(0xD2511F53u, c0), lo_a = 0xD2511F53u * c0;
    const uint32_t hi_b = __umulhi(0xCD9E8D57u, c2), lo_b = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi_b ^ c1 ^ k0, n2 = hi_a ^ c3 ^ k1;
    c0 = n0; c1 = lo_b; c2 = n2; c3 = lo_a;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Series logarithm that defines the exponential job times: u = m 2^e with m in [sqrt(1/2),
// sqrt(2)), s = (m-1)/(m+1), ln u = e ln2 + 2s(1 + s^2/3 + ... + s^22/23).  Each step is one
// binary64 operation rounded to nearest (the _rn intrinsics are never contracted into FMAs).
__device__ __forceinline__ double ln_series(double u) {
  const u64 bits = (u64)__double_as_longlong(u);
  int e = (int)((bits >> 52) & 0x7FF) - 1023;
  double m = __longlong_as_double((i64)((bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull));
  if (m >= 1.4142135623730951) { m = __dmul_rn(m, 0.5); e += 1; }
  const double s = __ddiv_rn(__dadd_rn(m, -1.0), __dadd_rn(m, 1.0));
  const double s2 = __dmul_rn(s, s);
  // the coefficients 1 / (2k + 1) are correctly rounded quotients of constants: compile-time values
  constexpr double INV_ODD[12] = {1.0 / 1.0,  1.0 / 3.0,  1.0 / 5.0,  1.0 / 7.0,  1.0 / 9.0,  1.0 / 11.0,
                                  1.0 / 13.0, 1.0 / 15.0, 1.0 / 17.0, 1.0 / 19.0, 1.0 / 21.0, 1.0 / 23.0};
  double p = INV_ODD[11];
#pragma unroll
  for (int k = 10; k >= 0; --k) {
    p = __dmul_rn(p, s2);
    p = __dadd_rn(p, INV_ODD[k]);
  }
  const double head = __dmul_rn((double)e, 0.6931471805599453);
  const double tail = __dmul_rn(__dmul_rn(2.0, s), p);
  return __dadd_rn(head, tail);
}

// Duration of job j of worker n in ticks (2^20 per time unit); 0 signals "out of range".
__device__ __forceinline__ u64 job_ticks(const TimeDist& d, uint32_t k0, uint32_t k1, int n, int j) {
  uint32_t w[4];
  philox4x32_10((uint32_t)n, (uint32_t)j, 0u, 0u, k0, k1, w);
  const double u = __dmul_rn(__dadd_rn((double)w[0], 0.5), 2.3283064365386963e-10);  // 2^-32
  double dur;
  if (d.kind == ABS_T_GAMMA) {
    // sum of `shape` exponential draws, left to right; draw i uses word i % 4 of block i / 4
    double total = -ln_series(u);
    for (int i = 1; i < d.shape; ++i) {
      if ((i & 3) == 0) philox4x32_10((uint32_t)n, (uint32_t)j, 0u, (uint32_t)(i >> 2), k0, k1, w);
      const uint32_t wi = (i & 3) == 0 ? w[0] : (i & 3) == 1 ? w[1] : (i & 3) == 2 ? w[2] : w[3];
      const double ui = __dmul_rn(__dadd_rn((double)wi, 0.5), 2.3283064365386963e-10);
      total = __dadd_rn(total, -ln_series(ui));
    }
    dur = __dadd_rn(d.shift, __ddiv_rn(total, d.rate));
  } else if (d.kind == ABS_T_CONST) dur = d.shift;
  else if (d.kind == ABS_T_EXP) dur = __ddiv_rn(-ln_series(u), d.rate);
  else if (d.kind == ABS_T_SHIFTED_EXP) dur = __dadd_rn(d.shift, __ddiv_rn(-ln_series(u), d.rate));
  else dur = __ddiv_rn(d.scale, __dsqrt_rn(u));
  if (d.slow_mod > 0 && n % d.slow_mod == d.slow_rem) dur = __dmul_rn(dur, d.slow_factor);
  const double scaled = __dmul_rn(dur, 1048576.0);
  if (!(scaled < 9007199254740992.0)) return 0ull;
  const u64 ticks = __double2ull_rd(scaled);
  return ticks < 1ull ? 1ull : ticks;
}

// The double-precision pipe of one SM is narrow, so the control CTA does not compute durations
// itself: the duration of the job a worker will start NEXT depends only on (worker, job index)
// and is prepared ahead of time by one warp of each of the first ceil(N/32) CTAs of a wide
// kernel that runs between two control kernels.  Only workers whose job index moved are redone.
__device__ __forceinline__ void refresh_next_durations(const DevState* st, const int* job, u64* next_dur,
                                                       int* dur_job, int n) {
  if (n >= st->W) return;
  const int j = job[n] + 1;
  if (dur_job[n] != j) {
    next_dur[n] = job_ticks(st->dist, st->key0, st->key1, n, j);
    dur_job[n] = j;
  }
}

// ---------------------------------------------------------------------------------------------
// Sort of up to 1024 distinct 64-bit keys, one per thread, by ranking: inside a warp every key
// counts the smaller keys of its warp (31 shuffles, no dependent chain); sorted runs are then
// merged pairwise, each key finding its place in the sibling run by binary search.  All steps
// are short and independent per thread, which matters because one CTA does this alone.
// Returns the buffer (A or B) that holds the sorted keys.
__device__ __forceinline__ u64* rank_merge_sort(u64 key, u64* A, u64* B, int n_pow2) {
  const int tid = threadIdx.x, lane = tid & 31;
  const bool active = tid < n_pow2;            // whole warps: n_pow2 is a multiple of 32
  if (active) {
    int rank = 0;
#pragma unroll
    for (int l = 0; l < 32; ++l) rank += (__shfl_sync(0xffffffffu, key, l) < key) ? 1 : 0;
    A[(tid - lane) + rank] = key;
  }
  __syncthreads();
  u64* src = A;
  u64* dst = B;
  for (int L = 32; L < n_pow2; L <<= 1) {
    if (active) {
      const u64 k = src[tid];
      const int pair_base = tid & ~(2 * L - 1);
      const int idx = tid - pair_base;
      const int own = idx & (L - 1);
      const u64* other = src + pair_base + ((idx < L) ? L : 0);
      int lo = 0, hi = L;
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (other[mid] < k) lo = mid + 1; else hi = mid;
      }
      dst[pair_base + own + lo] = k;
    }
    __syncthreads();
    u64* tmp = src; src = dst; dst = tmp;
  }
  return src;
}

__device__ __forceinline__ i64 floor_div(i64 a, i64 b) {  // b > 0
  i64 q = a / b;
  if ((a % b != 0) && (a < 0)) --q;
  return q;
}

struct CtlShared {
  u64 keysA[1024], keysB[1024];
  unsigned short wcnt[32][MAX_TAU];   // per-warp count of selected workers per staleness
  int cnt[MAX_TAU];                    // selected workers per staleness
  int grow0[MAX_TAU];                  // first row of each staleness group
  unsigned char flag[1024];            // selected marker per worker id
  int row0[1024];                      // first gradient row of each selected worker
  float lossv[1024];                   // mean minibatch loss of each selected worker
  int version[1024], job[1024];        // per-worker state after the round's bookkeeping
  int sel_n[1024];                     // worker id of each arrival, in arrival order
  int shard_lo[1024];
  unsigned shard_len[1024];
  float redf[32];
  int warp_tot[32];
  int scalar[8];
};

// Completes the open round (Eq. 5, Eq. 4, Eq. 6, trace row), then selects the arrivals of the
// next round and lays out its gradient rows.
//   do_finish: complete the open round if there is one
//   do_select: open the next round
// A dependent global-memory access costs this lone CTA close to a microsecond, so everything it
// needs is loaded up front in one wave and later phases work from registers and shared memory.
//   t_sel:     index of the round that follows the open one (the host counts rounds; parity of
//              t_sel - 1 / t_sel picks the layout copy of the open / the new round)
//   look_here: the workers that were renewed also get the duration of the job AFTER the one they
//              start now prepared here, at the end of the step (see refresh_next_durations), for
//              callers that have no other kernel between two control steps to do it
//   late_status: when the step runs next to the Eq. 3 kernel of the round it finishes, a status it
//              raises must not be seen by that kernel's blocks (they would skip a valid step):
//              the status is left in *late_status (shared memory) for the caller to publish later
template <int NT>
__device__ __forceinline__ int ctl_round(const CtlArgs& a, CtlShared& sh, int do_finish, int do_select, int t_sel,
                                         int look_here = 0, int* late_status = nullptr) {
  DevState* st = a.st;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto raise = [&](int code) {
    if (late_status != nullptr) *late_status = code;
    else st->status = code;
  };
  // ---- one wave of loads
  const int W = st->W, S = st->S, B = st->B, RB = st->RB, K0 = st->K0;
  const int po = (t_sel - 1) & 1, pn = t_sel & 1;     // layout copy of the open / of the new round
  const int status0 = st->status, open0 = st->open, diverged0 = a.ri[po].diverged;
  const int k_mode = st->k_mode, bound_mode = st->bound_mode, max_rounds = st->max_rounds;
  const int bound_offset = st->bound_offset, Scap = st->theta_cap, literal = st->literal_eq6;
  const int no_restart = st->no_restart;
  const uint32_t key0 = st->key0, key1 = st->key1;
  const i64 n_samples = st->n_samples;
  const u64 T_end0 = st->T_end;
  const float L0_prev = st->L0;
  const i64 sel_off = st->sel_total, rst_off = st->rst_total;
  const u64 comm0 = st->comm;
  int t = st->t, K = st->K;
  const bool net = a.row_loss != nullptr;
  const bool fin = do_finish && open0;
  u64 my_c = 0;
  int my_version = 0, my_job = 0, my_dur_job = -1;
  u64 my_next_dur = 0;
  if (tid < W) {
    my_c = a.c[tid]; my_version = a.version[tid]; my_job = a.job[tid];
    my_dur_job = a.dur_job[tid]; my_next_dur = a.next_dur[tid];
  }
  int my_sel = 0, my_tau = 0, my_row0 = 0;
  float my_loss = 0.f;
  if (fin && tid < K) {
    my_sel = a.sel[po][tid]; my_tau = a.sel_tau[po][tid]; my_row0 = a.sel_row0[po][tid];
    if (!net && a.loss_part == nullptr) my_loss = a.loss[tid];
    if (!net && a.loss_part != nullptr) {
      // the least-squares pipeline leaves per-group sums; same order and rounding as its Eq. 3 kernel
      float s = 0.f;
      for (int g = 0; g < a.loss_groups; ++g) s += a.loss_part[(size_t)tid * a.loss_groups + g];
      my_loss = __fdiv_rn(s, (float)B);
    }
  }
  if (status0 != ST_OK) return 1;

  int renewed = 0;          // this thread's worker started a new job in the finish step
  // ------------------------------------------------------------------ finish round t
  if (fin) {
    const u64 T_end = T_end0;
    if (net) {
      // per-worker mean of the per-sample losses: TPW neighbouring threads share a worker, each
      // adds every TPW-th row (independent loads), then the TPW partial sums are added by a
      // fixed shuffle tree
      sh.row0[tid] = my_row0;
      __syncthreads();
      int kp = 32;
      while (kp < K) kp <<= 1;
      const int tpw = min(32, NT / kp);
      const int i = tid / tpw, sub = tid - i * tpw;
      float acc = 0.f;
      if (i < K) {
        const float* rl = a.row_loss + sh.row0[i];
#pragma unroll 8
        for (int b = sub; b < B; b += tpw) acc += rl[b];
      }
      for (int o = tpw >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (i < K && sub == 0) sh.lossv[i] = __fdiv_rn(acc, (float)B);
      __syncthreads();
      if (tid < K) my_loss = sh.lossv[tid];
    }
    const int bad = __syncthreads_or((tid < K) && !isfinite(my_loss)) || diverged0;
    if (bad) {
      if (tid == 0) { raise(ST_DIVERGED); st->open = 0; }
      return 1;
    }
    // loss estimate: adjacent-pair tree sum in binary32 over 1024 leaves, /K in binary32
    float v = (tid < K) ? my_loss : 0.f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) v = __fadd_rn(v, __shfl_down_sync(0xffffffffu, v, o));
    if (lane == 0) sh.redf[warp] = v;
    sh.flag[tid] = 0;
    __syncthreads();
    if (warp == 0) {
      float x = (lane < NT / 32) ? sh.redf[lane] : 0.f;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) x = __fadd_rn(x, __shfl_down_sync(0xffffffffu, x, o));
      if (lane == 0) {
        const float Lt0 = __fdiv_rn(x, (float)K);
        const float L00 = (t == 0) ? Lt0 : L0_prev;
        // Eq. 5 as an exact integer rule: largest k with k^2 Lt <= K0^2 L0 (binary64 products of a
        // 20-bit integer and a binary32 value are exact).  A binary32 estimate of K0 sqrt(L0/Lt)
        // is corrected with the exact test, so only a handful of double operations are issued.
        int kr = 0;
        if (k_mode == ABS_K_ADAPTIVE) {
          if (Lt0 <= 0.f) {
            kr = W;
          } else {
            const double rhs = __dmul_rn((double)(K0 * K0), (double)L00);
            const double lt = (double)Lt0;
            const float est = (float)K0 * sqrtf(L00 / Lt0);
            int k = (est >= (float)W) ? W : ((est >= 1.f) ? (int)est : 1);
            while (k < W && __dmul_rn((double)((k + 1) * (k + 1)), lt) <= rhs) ++k;
            while (k >= 1 && !(__dmul_rn((double)(k * k), lt) <= rhs)) --k;
            kr = k;
          }
        }
        sh.redf[0] = Lt0;
        sh.redf[1] = L00;
        sh.scalar[2] = kr;
      }
    }
    if (tid < K) sh.flag[my_sel] = 1;
    __syncthreads();
    const float Lt = sh.redf[0];
    const float L0 = sh.redf[1];
    int K_next = K;
    if (k_mode == ABS_K_ADAPTIVE) K_next = min(W, max(K, sh.scalar[2]));
    // Eq. 4 with a = S - N/K0, in integers
    int theta = Scap;
    if (bound_mode == ABS_BOUND_ADAPTIVE) {
      const i64 fl = floor_div((i64)W * (i64)(K0 - K_next), (i64)K_next * (i64)K0);
      i64 th = (i64)Scap + fl;
      if (th < 1) th = 1;
      if (th > Scap) th = Scap;
      theta = (int)th;
    } else if (bound_mode == ABS_BOUND_OFFSET) {     // Eq. 4 with a given: floor(N/K + a) = floor(N/K) + a
      int th = W / K_next + bound_offset;
      if (th < 1) th = 1;
      if (th > Scap) th = Scap;
      theta = th;
    }
    // Eq. 6 in Algorithm 1's order: arrivals and over-stale workers get w^{t+1}
    int restart = 0, renew = 0;
    if (tid < W) {
      const int sel_me = sh.flag[tid];
      restart = (!sel_me) && !no_restart && ((t + 1 - literal - my_version) > theta);
      renew = sel_me || restart;
    }
    int range_err = 0;
    if (renew) {
      const int j = my_job + 1;
      const u64 dt = (my_dur_job == j) ? my_next_dur : job_ticks(st->dist, key0, key1, tid, j);
      const u64 cn = T_end + dt;
      if (dt == 0ull || cn >= (1ull << 53)) range_err = 1;
      my_job = j; my_version = t + 1; my_c = cn;
      renewed = 1;
      a.job[tid] = j;
      a.version[tid] = t + 1;
      a.c[tid] = cn;
    }
    // ascending list of restarted ids
    const unsigned rb = __ballot_sync(0xffffffffu, restart);
    if (lane == 0) sh.warp_tot[warp] = __popc(rb);
    range_err = __syncthreads_or(range_err);
    int base = 0, R = 0;
    for (int w = 0; w < NT / 32; ++w) { const int c = sh.warp_tot[w]; if (w < warp) base += c; R += c; }
    if (restart) a.tr_rst_id[rst_off + base + __popc(rb & ((1u << lane) - 1u))] = tid;
    if (tid < K) {
      a.tr_sel_id[sel_off + tid] = my_sel;
      a.tr_sel_tau[sel_off + tid] = my_tau;
      a.tr_sel_loss[sel_off + tid] = my_loss;
    }
    const u64 comm = comm0 + (u64)(K + R);
    if (tid == 0) {
      a.tr_K[t] = K; a.tr_R[t] = R; a.tr_theta[t] = theta; a.tr_T[t] = T_end;
      a.tr_loss[t] = Lt; a.tr_comm[t] = comm;
      a.tr_sel_off[t] = sel_off; a.tr_rst_off[t] = rst_off;
      a.tr_sel_off[t + 1] = sel_off + K; a.tr_rst_off[t + 1] = rst_off + R;
      st->sel_total = sel_off + K; st->rst_total = rst_off + R; st->comm = comm;
      st->L0 = L0; st->theta = theta; st->K = K_next; st->t = t + 1; st->open = 0;
      if (range_err) raise(ST_RANGE);
    }
    if (range_err) return 1;
    t = t + 1;
    K = K_next;
    __syncthreads();
  }

  // duration of the job after the one just started, for the next control step to look up
  if (look_here && renewed) {
    a.next_dur[tid] = job_ticks(st->dist, key0, key1, tid, my_job + 1);
    a.dur_job[tid] = my_job + 1;
  }
  // ------------------------------------------------------------------ select round t
  if (!do_select) return 1;
  if (t != t_sel) {                      // host and device disagree on the round index
    if (tid == 0) raise(ST_INTERNAL);
    return 1;
  }
  if (t >= max_rounds) {
    if (tid == 0) raise(ST_NOSPACE);
    return 1;
  }
  {
    sh.version[tid] = my_version;
    sh.job[tid] = my_job;
    if (net) for (int i = tid; i < 32 * MAX_TAU; i += NT) (&sh.wcnt[0][0])[i] = 0;
    // arrivals: the K smallest (completion tick, worker id) keys; unused slots get distinct
    // keys above every real one
    int n_pow2 = 32;
    while (n_pow2 < W) n_pow2 <<= 1;
    const u64 key_in = (tid < W) ? ((my_c << 10) | (u64)tid) : (0xFFFFFFFFFFFFFC00ull | (u64)tid);
    const u64* sorted = rank_merge_sort(key_in, sh.keysA, sh.keysB, n_pow2);
    const u64 T_end = sorted[K - 1] >> 10;
    int n = -1, tau = -1;
    if (tid < K) {
      n = (int)(sorted[tid] & 1023ull);
      tau = t - sh.version[n];
    }
    const int tau_bad = __syncthreads_or(tid < K && (tau < 0 || tau > S));
    if (tau_bad) {
      // with forced restarts this cannot happen (consumed staleness <= threshold <= S); without
      // them the arrival's model version may have left the ring: the run ends here, before any
      // kernel reads the slot that was overwritten
      if (tid == 0) raise(no_restart ? ST_STALE : ST_INTERNAL);
      return 1;
    }
    // network models: group the arrivals by staleness (all members of a group read the same
    // ring slot); inside a group keep arrival order.  Least squares needs no row layout.
    int row0_me = tid * B;
    if (net) {
      const unsigned peers = __match_any_sync(0xffffffffu, tau);
      const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
      if (tau >= 0 && rank_in_warp == 0) sh.wcnt[warp][tau] = (unsigned short)__popc(peers);
      __syncthreads();
      if (tid <= S) {
        int c = 0;
        for (int w = 0; w < 32; ++w) { const int x = sh.wcnt[w][tid]; sh.wcnt[w][tid] = (unsigned short)c; c += x; }
        sh.cnt[tid] = c;
      }
      __syncthreads();
      if (tid <= S) {
        int r0 = 0, g = 0;
        for (int q = 0; q < tid; ++q) { r0 += round_up(sh.cnt[q] * B, RB); g += sh.cnt[q] > 0; }
        sh.grow0[tid] = r0;
        if (tid == S) {
          sh.scalar[0] = r0 + round_up(sh.cnt[S] * B, RB);
          sh.scalar[1] = g + (sh.cnt[S] > 0);
        }
      }
      __syncthreads();
      if (tid < K) row0_me = sh.grow0[tau] + ((int)sh.wcnt[warp][tau] + rank_in_warp) * B;
    }
    const int n_rows = net ? sh.scalar[0] : K * B;
    const int n_groups = net ? sh.scalar[1] : 0;
    if (tid < K) {
      const int row0 = row0_me;
      a.sel[pn][tid] = n;
      a.sel_tau[pn][tid] = tau;
      a.sel_row0[pn][tid] = row0;
      sh.row0[tid] = row0;
      sh.sel_n[tid] = n;
      sh.flag[tid] = 0;
      if (net) {
        const i64 lo = ((i64)n * n_samples) / W, hi = ((i64)(n + 1) * n_samples) / W;
        sh.shard_lo[tid] = (int)lo;
        sh.shard_len[tid] = (unsigned)(hi - lo);
      }
    }
    if (tid == 0) {
      st->T_end = T_end;
      st->n_rows = n_rows;
      st->n_row_tiles = n_rows / RB;
      st->n_groups = n_groups;
      st->open = 1;
      RoundInfo info;
      info.n_rows = n_rows; info.K = K; info.t = t; info.diverged = 0;
      a.ri[pn] = info;
      sh.scalar[4] = K; sh.scalar[5] = t;
    }
    if (!net) return 0;           // least squares: no row tiles, minibatches drawn by its own kernel
    __syncthreads();
    // ring slot of every row tile and padding rows
    {
      const int n_tiles = n_rows / RB;
      for (int q = tid; q < n_tiles; q += NT) {
        const int r = q * RB;
        int g = 0;                                  // last non-empty group starting at or before r
        for (int u = 0; u <= S; ++u) if (sh.cnt[u] > 0 && sh.grow0[u] <= r) g = u;
        a.tile_slot[pn][q] = (t - g) % (S + 1);
      }
      for (int g = 0; g <= S; ++g) {
        const int c = sh.cnt[g];
        if (c == 0) continue;
        const int p0 = sh.grow0[g] + c * B, p1 = sh.grow0[g] + round_up(c * B, RB);
        for (int r = p0 + tid; r < p1; r += NT) a.row_idx[pn][r] = -1;
      }
    }
    // minibatch draws: sample b of job (n, j) = word b%4 of Philox block (n, j, 1, b/4),
    // mapped into the worker's shard [n M / N, (n+1) M / N)
    const int blocks_per = (B + 3) >> 2;
    for (int item = tid; item < K * blocks_per; item += NT) {
      const int i = item / blocks_per, blk = item - i * blocks_per;
      const int wn = (int)(sorted[i] & 1023ull);
      uint32_t w4[4];
      philox4x32_10((uint32_t)wn, (uint32_t)sh.job[wn], 1u, (uint32_t)blk, key0, key1, w4);
      const int lo = sh.shard_lo[i], row0 = sh.row0[i];
      const u64 len = (u64)sh.shard_len[i];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int b = blk * 4 + q;
        if (b < B) a.row_idx[pn][row0 + b] = lo + (int)(((u64)w4[q] * len) >> 32);
      }
    }
  }
  return 0;
}

// pdl = 0: the step waits for the kernel in front of it before it starts.  pdl = 1: the kernel in
// front is the Eq. 3 step of the round being finished, which this step does not depend on (it reads
// the uploaded losses, which were complete before the Eq. 3 kernel passed its own wait, and it
// prepares the job durations itself): the two run side by side, and this kernel waits for the
// Eq. 3 kernel only at its end, so that whatever follows in the stream sees both complete.
// look: see ctl_round (the Eq. 3 kernel then does not touch the prepared durations).
__global__ void __launch_bounds__(1024, 1) abs_ctl_kernel(CtlArgs a, int do_finish, int do_select, int t_sel, int pdl, int look) {
  if (pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  else grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char ctl_smem[];
  CtlShared& sh = *reinterpret_cast<CtlShared*>(ctl_smem);
  __shared__ int late;
  if (threadIdx.x == 0) late = ST_OK;
  ctl_round<1024>(a, sh, do_finish, do_select, t_sel, look, pdl ? &late : nullptr);
  if (pdl) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0 && late != ST_OK) a.st->status = late;      // the Eq. 3 kernel is done: publish
  }
}

// The same step with 256 threads for runs of at most 256 workers (one thread per worker is all the
// step needs; its block-wide barriers are cheaper with 8 warps than with 32).
__global__ void __launch_bounds__(256, 1) abs_ctl_small_kernel(CtlArgs a, int do_finish, int do_select, int t_sel, int pdl, int look) {
  if (pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  else grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char ctl_smem[];
  CtlShared& sh = *reinterpret_cast<CtlShared*>(ctl_smem);
  __shared__ int late;
  if (threadIdx.x == 0) late = ST_OK;
  ctl_round<256>(a, sh, do_finish, do_select, t_sel, look, pdl ? &late : nullptr);
  if (pdl) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0 && late != ST_OK) a.st->status = late;      // the Eq. 3 kernel is done: publish
  }
}

// Duration look-ahead (see refresh_next_durations): one warp per 32 workers.
__global__ void abs_times_kernel(const DevState* st, const int* job, u64* next_dur, int* dur_job) {
  grid_dependency_sync();
  if (st->status != ST_OK) return;
  refresh_next_durations(st, job, next_dur, dur_job, blockIdx.x * 32 + threadIdx.x);
}

// Algorithm 1, initialisation: every worker holds w^0 and starts job 0 at tick 0.
__global__ void abs_init_state_kernel(CtlArgs a) {
  DevState* st = a.st;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (tid < st->W) {
    const u64 dt = job_ticks(st->dist, st->key0, st->key1, tid, 0);
    if (dt == 0ull) st->status = ST_RANGE;
    a.c[tid] = dt;
    a.version[tid] = 0;
    a.job[tid] = 0;
    a.next_dur[tid] = job_ticks(st->dist, st->key0, st->key1, tid, 1);
    a.dur_job[tid] = 1;
  }
}

}  // namespace absb
