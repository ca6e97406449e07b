// Shared device/host declarations of the ABS round loop.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/abs_b200.h"

namespace absb {

typedef unsigned long long u64;
typedef long long i64;

// Device status words (DevState::status).  0 = running.
enum : int {
  ST_OK = 0,
  ST_DIVERGED = 1,   // a non-finite loss was uploaded in round `t`
  ST_RANGE = 2,      // a completion tick left the 2^53 range
  ST_NOSPACE = 3,    // round index reached the trace capacity
  ST_INTERNAL = 4,   // an invariant failed (consumed staleness above the bound)
  ST_TIMEOUT = 5,    // a bounded wait inside a kernel expired
  ST_STALE = 6,      // runs without forced restarts: an arrival is older than the model versions kept
};

constexpr int MAX_W = ABS_MAX_WORKERS;
constexpr int MAX_TAU = ABS_MAX_BOUND + 1;

struct TimeDist {
  int kind;
  double shift, rate, scale;
  int slow_mod, slow_rem;
  double slow_factor;
  int shape;
};

// Scalars of Algorithm 1 that live on the device between rounds.
struct DevState {
  // constants of the run
  int W, K0, S, B, RB;            // S: the ring keeps S + 1 model versions; RB: every version group's rows are
                                  // padded to a multiple of RB
  int k_mode, bound_mode, max_rounds;
  int bound_offset;               // the constant a of Eq. 4 (ABS_BOUND_OFFSET)
  int theta_cap;                  // largest threshold = the caller's staleness bound
  int literal_eq6;                // 1: the restart test reads the age before its increment (Eq. 6 as printed);
                                  // S is then the caller's bound + 1 (oldest model version still in use)
  int no_restart;                 // 1: Eq. 6 never forces a restart (AdaSync / K-async SGD, Sec. II-B); an arrival
                                  // older than S rounds ends the run with ST_STALE
  int sa_penalty;                 // staleness-aware step size (Sec. I): 0 off; 1 the gradient kernels scale the
                                  // rows of a tile by the weight of the tile's staleness; 2 the Eq. 3 kernel
                                  // weights each selected worker's upload (runs with local steps on networks)
  i64 n_samples;
  uint32_t key0, key1;            // Philox key = (seed low, seed high)
  TimeDist dist;
  // server state
  int t;                          // round index of the next round to select
  int K;                          // K^t
  int theta;                      // threshold of the last restart test
  int status;                     // ST_*
  int diverged;                   // set by the loss kernels of the open round
  int open;                       // 1 between selection and completion of a round
  float L0;                       // loss estimate of round 0, f(w^0) in Eq. 5
  u64 T_end;                      // end tick of the open round
  int n_rows;                     // padded gradient rows of the open round
  int n_row_tiles;                // n_rows / RB
  int n_groups;
  i64 sel_total, rst_total;       // flat trace fill
  u64 comm;                       // communication-round counter (Sec. V-B)
  int timeout_where;
};

// What the gradient kernels of one round need to know about it.  Two copies alternate by round
// parity: the control kernel lays out round t+1 while the backward kernels of round t still run.
struct RoundInfo {
  int n_rows;       // padded gradient rows
  int K;            // K^t
  int t;            // round index
  int diverged;     // set by the loss kernels of the round
};

// Pointers the control kernel works on (all device memory inside the workspace).
struct CtlArgs {
  DevState* st;
  RoundInfo* ri;       // [2] by round parity
  u64* c;              // [W] completion tick of each worker's job in flight
  int* version;        // [W] round index of the model the worker holds
  int* job;            // [W] index of the job in flight
  // per-round layout, two copies by round parity
  int* sel[2];         // [W] selected worker ids of the round, arrival order
  int* sel_tau[2];     // [W]
  int* sel_row0[2];    // [W] first gradient row of each selected worker
  float* loss;         // [W] mean minibatch loss of each selected worker
  float* row_loss;     // [rows_cap] per-sample losses (network models), else null
  int* row_idx[2];     // [rows_cap] sample index of each gradient row, -1 for padding
  int* tile_slot[2];   // [rows_cap / RB] ring slot of each row tile
  u64* next_dur;       // [W] duration of the job each worker starts next, computed ahead of time
  int* dur_job;        // [W] job index next_dur[n] belongs to
  const float* loss_part;  // least-squares pipeline: per (selected worker, row group) sums of 1/2 r^2, or null;
  int loss_groups;         // the upload's loss is their sum over the groups divided by B
  // trace
  int* tr_K; int* tr_R; int* tr_theta; u64* tr_T; float* tr_loss; u64* tr_comm;
  i64* tr_sel_off; i64* tr_rst_off;
  int* tr_sel_id; int* tr_sel_tau; float* tr_sel_loss; int* tr_rst_id;
};

__device__ __forceinline__ float ldf(const float* p, size_t i) { return p[i]; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void stf(float* p, size_t i, float v) { p[i] = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

// First statement of every kernel of the round loop.  The kernels are launched with programmatic
// stream serialization, so a kernel's CTAs may be resident before the kernel in front of it has
// finished: wait until that kernel has completed (its writes are then visible), then allow the
// kernel behind this one to be scheduled early in the same way.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Staleness-aware step size (Sec. I: the step size of a stale gradient is penalised linearly in its
// delay): weight of a gradient of staleness tau in the sum of Eq. 3.
__device__ __forceinline__ float sa_weight(int tau) { return tau > 1 ? __fdiv_rn(1.f, (float)tau) : 1.f; }
// Weight of the gradient rows of a tile that reads ring slot `slot` in round t: a consumed gradient
// is at most S rounds old, so its staleness is (t - slot) mod (S + 1) (slot = version mod (S + 1)
// and version <= t, so t - slot is never negative).
__device__ __forceinline__ float sa_slot_weight(const DevState* st, int t, int slot) {
  return st->sa_penalty == 1 ? sa_weight((t - slot) % (st->S + 1)) : 1.f;
}

__host__ __device__ inline int round_up(int a, int b) { return (a + b - 1) / b * b; }
__host__ __device__ inline size_t round_up_sz(size_t a, size_t b) { return (a + b - 1) / b * b; }

}  // namespace absb
