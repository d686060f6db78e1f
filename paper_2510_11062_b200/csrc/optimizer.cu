// Parameter update of one policy's LM head: theta_m <- theta_m - eta * grad L (Sec. 3) with the
// optimiser of App. "Training Details": global-norm gradient clipping, then Adam with decoupled
// weight decay.  Two memory-bound kernels: a fixed-order sum of squares of the gradient, and one
// fused pass that reads gradient, fp32 master weight and both moments and writes them back
// together with the bf16 weight the LM-head kernels consume (30 bytes per parameter with an fp32
// gradient).
#include <cuda_bf16.h>
#include "internal.h"

namespace atgrpo {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 148 * 8;

__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  x[0] = a.x, x[1] = a.y, x[2] = a.z, x[3] = a.w, x[4] = b.x, x[5] = b.y, x[6] = b.z, x[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(h[i]);
    x[2 * i] = f.x, x[2 * i + 1] = f.y;
  }
}
__device__ __forceinline__ void store8(float* p, const float (&x)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(x[0], x[1], x[2], x[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(x[4], x[5], x[6], x[7]);
}

// Sum of squares: per-thread strided partial in fp64, fixed tree in the block, the last block
// adds the per-block partials with a fixed strided assignment and a fixed tree.
template <class G>
__global__ void __launch_bounds__(kThreads)
k_sumsq(const G* __restrict__ g, int64_t n, double* __restrict__ partial, unsigned* done,
        double* __restrict__ out) {
  __shared__ double red[kThreads];
  __shared__ bool s_last;
  double acc = 0.0;
  const int64_t n8 = n >> 3;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x; q < n8; q += stride) {
    float x[8];
    load8(g + 8 * q, x);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s = fmaf(x[i], x[i], s);
    acc += (double)s;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0)
    for (int64_t j = 8 * n8; j < n; ++j) acc += (double)((float)g[j] * (float)g[j]);
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  double v = 0.0;
  for (unsigned b = threadIdx.x; b < gridDim.x; b += kThreads) v += partial[b];
  red[threadIdx.x] = v;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *out = red[0];
    *done = 0;
  }
}

struct AdamArgs {
  float lr, beta1, beta2, eps, decay_factor;   // decay_factor = 1 - lr*weight_decay
  float inv_bc1, inv_bc2;                      // 1/(1-beta1^t), 1/(1-beta2^t)
  float max_norm;
};

__device__ __forceinline__ float clip_scale(const double* sumsq, float max_norm) {
  if (sumsq == nullptr || !(max_norm > 0.f)) return 1.f;
  const double s = (double)max_norm / (sqrt(*sumsq) + 1e-6);
  return (float)(s < 1.0 ? s : 1.0);
}

__device__ __forceinline__ void adam_one(float g, float& th, float& m, float& v, const AdamArgs& a) {
  m = a.beta1 * m + (1.f - a.beta1) * g;
  v = a.beta2 * v + (1.f - a.beta2) * g * g;
  th = th * a.decay_factor - a.lr * (m * a.inv_bc1) / (sqrtf(v * a.inv_bc2) + a.eps);
}

template <class G>
__global__ void __launch_bounds__(kThreads)
k_adamw(const G* __restrict__ grad, float* __restrict__ master, float* __restrict__ m,
        float* __restrict__ v, __nv_bfloat16* __restrict__ w_out, int64_t n,
        const double* __restrict__ sumsq, AdamArgs a) {
  const float scale = clip_scale(sumsq, a.max_norm);
  const int64_t n8 = n >> 3;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x; q < n8; q += stride) {
    float g[8], th[8], mm[8], vv[8];
    load8(grad + 8 * q, g);
    load8(master + 8 * q, th);
    load8(m + 8 * q, mm);
    load8(v + 8 * q, vv);
#pragma unroll
    for (int i = 0; i < 8; ++i) adam_one(g[i] * scale, th[i], mm[i], vv[i], a);
    store8(master + 8 * q, th);
    store8(m + 8 * q, mm);
    store8(v + 8 * q, vv);
    if (w_out) {
      uint4 u;
      __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
      for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(th[2 * i], th[2 * i + 1]);
      *reinterpret_cast<uint4*>(w_out + 8 * q) = u;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    for (int64_t j = 8 * n8; j < n; ++j) {
      float th = master[j], mm = m[j], vv = v[j];
      adam_one((float)grad[j] * scale, th, mm, vv, a);
      master[j] = th, m[j] = mm, v[j] = vv;
      if (w_out) w_out[j] = __float2bfloat16_rn(th);
    }
  }
}

int grid_for(int64_t n) {
  int64_t g = ((n >> 3) + kThreads - 1) / kThreads;
  if (g < 1) g = 1;
  if (g > kMaxBlocks) g = kMaxBlocks;
  return (int)g;
}

}  // namespace

size_t grad_sumsq_workspace_bytes() {
  Carver c(nullptr);
  c.take<double>(kMaxBlocks);
  c.take<unsigned>(1);
  return c.off;
}

int grad_sumsq_launch(const void* grad, int grad_dtype, int64_t n, double* sumsq_out, void* workspace,
                      cudaStream_t st) {
  Carver c(workspace);
  double* partial = c.take<double>(kMaxBlocks);
  unsigned* done = c.take<unsigned>(1);
  ATGRPO_CUDA_OK(cudaMemsetAsync(done, 0, sizeof(unsigned), st));
  const int g = grid_for(n);
  if (grad_dtype == ATGRPO_BF16)
    k_sumsq<<<g, kThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(grad), n, partial, done, sumsq_out);
  else
    k_sumsq<<<g, kThreads, 0, st>>>(static_cast<const float*>(grad), n, partial, done, sumsq_out);
  return launch_ok();
}

int adamw_launch(const void* grad, int grad_dtype, float* master, float* m, float* v, void* w_bf16,
                 int64_t n, const double* sumsq, float lr, float beta1, float beta2, float eps,
                 float weight_decay, float max_norm, int step, cudaStream_t st) {
  AdamArgs a;
  a.lr = lr, a.beta1 = beta1, a.beta2 = beta2, a.eps = eps;
  a.decay_factor = (float)(1.0 - (double)lr * (double)weight_decay);
  a.inv_bc1 = (float)(1.0 / (1.0 - pow((double)beta1, (double)step)));
  a.inv_bc2 = (float)(1.0 / (1.0 - pow((double)beta2, (double)step)));
  a.max_norm = max_norm;
  const int g = grid_for(n);
  if (grad_dtype == ATGRPO_BF16)
    k_adamw<<<g, kThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(grad), master, m, v,
                                    static_cast<__nv_bfloat16*>(w_bf16), n, sumsq, a);
  else
    k_adamw<<<g, kThreads, 0, st>>>(static_cast<const float*>(grad), master, m, v,
                                    static_cast<__nv_bfloat16*>(w_bf16), n, sumsq, a);
  return launch_ok();
}

}  // namespace atgrpo
