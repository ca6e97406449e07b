// Stand-alone operation of the round loop: minibatch gradients of the least-squares model for
// several workers at one model, and their mean (Eq. 2 with U = 1, then the sum of Eq. 3).
#include <cstdarg>
#include <cstdio>
#include <mutex>
#include <string>

#include "common.cuh"

using namespace absb;

namespace absb {
void set_last_error(const char* text);   // abs_api.cu: text returned by abs_last_error()
}

namespace {

int op_fail(int code, const char* fmt, ...) {
  char buf[384];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  set_last_error(buf);
  return code;
}

// One CTA per worker i: residuals r_b = x_b . w - y_b over its B sampled rows, loss[i] = mean
// 1/2 r^2, partial[i][j] = sum_b r_b x_b[j].
template <typename T>
__global__ void __launch_bounds__(256) op_lsq_partial_kernel(const T* X, const float* y, const T* w, const int* idx,
                                                             int B, int d, float* partial, float* loss) {
  __shared__ float res[1024];
  __shared__ int sidx[1024];
  __shared__ float red[8];
  const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int b = tid; b < B; b += 256) sidx[b] = idx[(size_t)i * B + b];
  __syncthreads();
  for (int b = warp; b < B; b += 8) {
    const T* x = X + (size_t)sidx[b] * d;
    float acc = 0.f;
    for (int j = lane; j < d; j += 32) acc = fmaf(ldf(x, j), ldf(w, j), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) res[b] = acc - y[sidx[b]];
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
    loss[i] = __fdiv_rn(tot, (float)B);
  }
  float* g = partial + (size_t)i * d;
  for (int j = tid; j < d; j += 256) {
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc = fmaf(res[b], ldf(X, (size_t)sidx[b] * d + j), acc);
    g[j] = acc;
  }
}

// g[j] = (1 / (n B)) sum_i partial[i][j], workers added in index order.
__global__ void __launch_bounds__(256) op_lsq_reduce_kernel(const float* partial, int n, int B, int d, float* g) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= d) return;
  float acc = 0.f;
  for (int i = 0; i < n; ++i) acc += partial[(size_t)i * d + j];
  g[j] = acc / (float)((long long)n * B);
}

int check_args(const void* X, const float* y, const void* w, const int* idx, int n, int B, int d, int dtype,
               const float* g_out, const float* loss_out) {
  if (!X || !y || !w || !idx || !g_out || !loss_out) return op_fail(ABS_EINVAL, "null pointer argument");
  if (n < 1 || n > ABS_MAX_WORKERS) return op_fail(ABS_EINVAL, "n %d outside [1, %d]", n, ABS_MAX_WORKERS);
  if (B < 1 || B > 1024) return op_fail(ABS_EINVAL, "B %d outside [1, 1024]", B);
  if (d < 1 || d > (1 << 20)) return op_fail(ABS_EINVAL, "d %d outside [1, 2^20]", d);
  if (dtype != ABS_FP32 && dtype != ABS_BF16_FP32MASTER) return op_fail(ABS_EUNSUPPORTED, "unknown dtype %d", dtype);
  return ABS_OK;
}

int run(const void* X, const float* y, const void* w, const int* idx, int n, int B, int d, int dtype, float* scratch,
        float* g_out, float* loss_out, cudaStream_t s) {
  if (dtype == ABS_FP32)
    op_lsq_partial_kernel<float><<<n, 256, 0, s>>>((const float*)X, y, (const float*)w, idx, B, d, scratch, loss_out);
  else
    op_lsq_partial_kernel<__nv_bfloat16><<<n, 256, 0, s>>>((const __nv_bfloat16*)X, y, (const __nv_bfloat16*)w, idx, B,
                                                          d, scratch, loss_out);
  op_lsq_reduce_kernel<<<(d + 255) / 256, 256, 0, s>>>(scratch, n, B, d, g_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return op_fail(ABS_ECUDA, "kernel launch: %s", cudaGetErrorString(e));
  return ABS_OK;
}

}  // namespace

extern "C" int abs_lsq_gradient(const void* X, const float* y, const void* w, const int* idx, int n, int B, int d,
                                int dtype, float* scratch, size_t scratch_floats, float* g_out, float* loss_out,
                                void* stream) {
  const int rc = check_args(X, y, w, idx, n, B, d, dtype, g_out, loss_out);
  if (rc != ABS_OK) return rc;
  if (!scratch) return op_fail(ABS_EINVAL, "scratch is null");
  if (scratch_floats < (size_t)n * d)
    return op_fail(ABS_ENOSPACE, "scratch holds %zu floats, n*d = %zu needed", scratch_floats, (size_t)n * d);
  return run(X, y, w, idx, n, B, d, dtype, scratch, g_out, loss_out, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate device memory.  The per-worker partial sums live in a
// fixed array that is part of the loaded library image on every GPU (4 MiB, held until exit).
namespace {

constexpr size_t NOALLOC_MAX_FLOATS = 1u << 20;          // n * d limit of the no-allocation variant
static __device__ __align__(256) float g_noalloc_partials[NOALLOC_MAX_FLOATS];

constexpr int MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
float* g_noalloc_ptr[MAX_DEVICES] = {};                  // device address of the array, per device

// Device address of the array on the current device.  In host code the array's name is only a
// handle; the address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
int noalloc_scratch(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return op_fail(ABS_ECUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= MAX_DEVICES) return op_fail(ABS_EUNSUPPORTED, "device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    float* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_noalloc_partials);
    if (e != cudaSuccess || !p)
      return op_fail(ABS_ECUDA, "cudaGetSymbolAddress(partials): %s", cudaGetErrorString(e));
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return ABS_OK;
}

}  // namespace

extern "C" int abs_lsq_gradient_noalloc(const void* X, const float* y, const void* w, const int* idx, int n, int B,
                                        int d, int dtype, float* g_out, float* loss_out, void* stream) {
  const int rc = check_args(X, y, w, idx, n, B, d, dtype, g_out, loss_out);
  if (rc != ABS_OK) return rc;
  if ((size_t)n * (size_t)d > NOALLOC_MAX_FLOATS)
    return op_fail(ABS_ENOSPACE, "n*d = %zu exceeds the built-in limit of %zu floats; use abs_lsq_gradient with "
                   "caller scratch", (size_t)n * d, NOALLOC_MAX_FLOATS);
  float* scratch = nullptr;
  const int rs = noalloc_scratch(&scratch);
  if (rs != ABS_OK) return rs;
  // every partial that the reduction reads is written by the first kernel of this call, so the
  // previous call's leftovers in the shared array never need clearing
  return run(X, y, w, idx, n, B, d, dtype, scratch, g_out, loss_out, (cudaStream_t)stream);
}
