// ada_ldlp_eval_static: the length predictor (class-logit form) for callers that cannot allocate.
//
// Every other entry point works inside a workspace the caller allocated.  Some callers have no way
// to get one: code that runs after the process has handed all device memory to another allocator,
// plugins called from inside a host framework that forbids cudaMalloc on its threads, or anything
// running where an allocation would synchronise the device at a bad moment.  For them this one
// call keeps its scratch (the predictor's hidden activations) in a fixed array that is part of the
// library image: ADA_STATIC_MAX_HIDDEN floats (16 KiB) on every GPU that loads the library, held
// until the process exits.
//
// The array is shared by all calls on a device and keeps what the last call wrote.  Nothing in it has
// to start at zero: a call overwrites every entry it later reads.  Two calls that overlap on the
// GPU (different streams, or threads racing on one device) use the same array and corrupt each
// other; callers must order them.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "ada.h"

namespace {

static __device__ __align__(256) float g_ldlp_hidden[ADA_STATIC_MAX_HIDDEN];

// In host code the name above is only a handle; the device address is looked up once per device.
constexpr int kMaxDevices = 64;
std::atomic<float *> g_scratch_addr[kMaxDevices];   // (zero-initialised; threads racing on the first call store the same address)

__device__ __forceinline__ float warp_total(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// hidden[u] = ReLU(W1[u] . [e ; f] + b1[u]); one warp per hidden unit
__global__ void k_static_hidden(const __nv_bfloat16 *w1, const __nv_bfloat16 *b1, const __nv_bfloat16 *e,
                                const float *f, int d, int hid, float *hidden) {
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (u >= hid) return;
  const __nv_bfloat16 *w = w1 + (size_t)u * 2 * d;
  float s = 0.f;
  for (int i = lane; i < d; i += 32) s += __bfloat162float(w[i]) * __bfloat162float(e[i]);
  for (int i = lane; i < d; i += 32) s += __bfloat162float(w[d + i]) * f[i];
  s = warp_total(s);
  if (lane == 0) hidden[u] = fmaxf(s + __bfloat162float(b1[u]), 0.f);
}

// z = W2 hidden + b2; n = argmax + 1, lowest index among equals; one warp
__global__ void k_static_out(const float *hidden, const __nv_bfloat16 *w2, const __nv_bfloat16 *b2, int hid, int nmax,
                             int *n_out, float *z_out) {
  const int lane = threadIdx.x;
  float best = -INFINITY;
  int bi = 0;
  for (int c = 0; c < nmax; ++c) {
    float s = 0.f;
    for (int i = lane; i < hid; i += 32) s += __bfloat162float(w2[(size_t)c * hid + i]) * hidden[i];
    s = warp_total(s) + __bfloat162float(b2[c]);
    if (lane == 0 && z_out) z_out[c] = s;
    if (s > best) { best = s; bi = c; }
  }
  if (lane == 0) *n_out = bi + 1;
}

}  // namespace

extern "C" int ada_ldlp_eval_static(const void *d_w1, const void *d_b1, const void *d_w2, const void *d_b2,
                                    const void *d_embed_row, const float *d_feature, int32_t d_model, int32_t hidden,
                                    int32_t n_max, int32_t *d_n, float *d_z, void *cuda_stream) {
  if (!d_w1 || !d_b1 || !d_w2 || !d_b2 || !d_embed_row || !d_feature || !d_n) return ADA_ERR_NULL;
  if (hidden > ADA_STATIC_MAX_HIDDEN) return ADA_ERR_TOO_LARGE;
  if (d_model < 1 || hidden < 1 || n_max < 1 || n_max > ADA_MAX_NMAX) return ADA_ERR_RANGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ADA_ERR_CUDA;
  float *scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {  // first call on this device (it is the current one): look the array up
    if (cudaGetSymbolAddress((void **)&scratch, g_ldlp_hidden) != cudaSuccess || !scratch) return ADA_ERR_CUDA;
    g_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  k_static_hidden<<<(hidden + 7) / 8, 256, 0, st>>>((const __nv_bfloat16 *)d_w1, (const __nv_bfloat16 *)d_b1,
                                                    (const __nv_bfloat16 *)d_embed_row, d_feature, d_model, hidden,
                                                    scratch);
  k_static_out<<<1, 32, 0, st>>>(scratch, (const __nv_bfloat16 *)d_w2, (const __nv_bfloat16 *)d_b2, hidden, n_max, d_n,
                                 d_z);
  return cudaGetLastError() == cudaSuccess ? ADA_OK : ADA_ERR_CUDA;
}
