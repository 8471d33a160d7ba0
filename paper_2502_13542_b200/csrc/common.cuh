// Shared device / host helpers of the ActQKV CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "actqkv.h"

namespace actqkv {

struct Batch {
  int n_seq, n_layers, layer0;
  __host__ __device__ int units() const { return n_seq * n_layers; }
};

inline Batch get_batch(const actqkv_batch* b) {
  Batch r{1, 1, 0};
  if (b) { r.n_seq = b->n_seq; r.n_layers = b->n_layers; r.layer0 = b->layer0; }
  return r;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Host-side validation shared by every entry point; returns ACTQKV_OK or a negative code.
inline int check_config(const actqkv_config* c, const Batch& b) {
  if (!c) return ACTQKV_ERR_NULL;
  if (c->dtype != ACTQKV_F32 && c->dtype != ACTQKV_BF16) return ACTQKV_ERR_DTYPE;
  if (c->out_dtype != ACTQKV_F32 && c->out_dtype != ACTQKV_BF16) return ACTQKV_ERR_DTYPE;
  if (c->probe_mode != ACTQKV_PROBE_ACTIVATION && c->probe_mode != ACTQKV_PROBE_MEAN_POOL) return ACTQKV_ERR_SHAPE;
  if (c->attention_kernel < ACTQKV_ATTN_AUTO || c->attention_kernel > ACTQKV_ATTN_CLUSTER4) return ACTQKV_ERR_SHAPE;
  if (c->head_dim != 64 && c->head_dim != 128) return ACTQKV_ERR_SHAPE;
  if (c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->n_q_heads % c->n_kv_heads) return ACTQKV_ERR_SHAPE;
  if (c->n_q_heads / c->n_kv_heads > 8) return ACTQKV_ERR_SHAPE;
  if (c->page_tokens <= 0 || c->block <= 0 || c->n_repr <= 0) return ACTQKV_ERR_SHAPE;
  if (c->block % c->page_tokens || c->block % c->n_repr || c->n_init % c->page_tokens) return ACTQKV_ERR_SHAPE;
  if (c->n_init < 0 || c->n_local_prev < 0 || c->window <= 0) return ACTQKV_ERR_SHAPE;
  if (c->cap_blocks < 0 || c->k_blocks < 0 || c->n_cap < 0 || c->n_layers <= 0) return ACTQKV_ERR_SHAPE;
  if (b.n_seq <= 0 || b.n_layers <= 0 || b.layer0 < 0 || b.layer0 + b.n_layers > c->n_layers)
    return ACTQKV_ERR_SHAPE;
  return ACTQKV_OK;
}

inline size_t elt_size(const actqkv_config* c) { return c->dtype == ACTQKV_BF16 ? 2 : 4; }

#define ACTQKV_REQUIRE_PTR(p)                      \
  do {                                             \
    if (!(p)) return ACTQKV_ERR_NULL;              \
    if (!actqkv::aligned16(p)) return ACTQKV_ERR_ALIGN; \
  } while (0)
#define ACTQKV_OPTIONAL_PTR(p)                            \
  do {                                                    \
    if ((p) && !actqkv::aligned16(p)) return ACTQKV_ERR_ALIGN; \
  } while (0)

// Every kernel of the library asks for the largest shared-memory carve-out, as the attention
// kernels need: consecutive kernels of a step then run under one L1 / shared-memory split and
// the SMs are not reconfigured between them.
template <typename Kernel>
inline void prefer_max_shared(Kernel kern) {
  (void)cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, int(cudaSharedmemCarveoutMaxShared));
}

// Programmatic dependent launch: a kernel launched with this attribute may start while the kernel
// before it in the stream is still running, as soon as every CTA of that kernel has executed
// grid_launch_dependents() (or has left).  It must execute grid_dependency_wait() -- which returns
// once the kernel before it has completed and its writes are visible -- before it WRITES anything
// and before it reads anything that a kernel of the library writes.  The short kernels of a step
// (bias + probe, score, density, cut-off, selection) let their successor start at once and wait
// right after, so the whole chain of a step is resident early and each link starts the moment its
// predecessor ends; since every link waits for its predecessor before it writes, the wait of the
// last link still orders it after all of them.  What a kernel does BEFORE its wait may therefore
// overlap any earlier kernel of the chain: it may read only what none of them writes (the step's
// Q / K / V, positions, the page table, cache pages and table rows of past tokens).  Kernels that
// write those (the append) neither start early nor let their successor start before they end.
// Without the attribute the wait is a no-op.
inline void allow_early_launch(cudaLaunchAttribute& a) {
  a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  a.val.programmaticStreamSerializationAllowed = 1;
}

// A kernel that needs more than 48 KiB of dynamic shared memory must opt in, and the opt-in
// belongs to the device that was current when it was made.  `done` is a per-kernel table with one
// flag per device ordinal; two host threads that race on a device's first launch both make the
// (idempotent) call.
constexpr int kMaxDevices = 64;
template <typename Kernel>
inline bool opt_in_shared_memory(Kernel kern, int bytes, std::atomic<bool> (&done)[kMaxDevices]) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return false;
  const bool tracked = dev < kMaxDevices;
  if (tracked && done[dev].load(std::memory_order_acquire)) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  if (tracked) done[dev].store(true, std::memory_order_release);
  return true;
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? ACTQKV_OK : ACTQKV_ERR_LAUNCH; }

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream become resident (it still waits for this one to end).
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void set_status(int32_t* status, int bit) {
  if (status) atomicOr(status, bit);
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// 16-byte vector of T converted to fp32: 4 floats or 8 bf16.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void unpack(const uint4& v, float (&out)[4]) {
    out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
    out[2] = __uint_as_float(v.z); out[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ void load(const float* p, float (&out)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
  __device__ static __forceinline__ void load_nc(const float* p, float (&out)[4]) {
    float4 v = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float (&out)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&out)[8]) {
    unpack(*reinterpret_cast<const uint4*>(p), out);
  }
  __device__ static __forceinline__ void load_nc(const __nv_bfloat16* p, float (&out)[8]) {
    unpack(__ldg(reinterpret_cast<const uint4*>(p)), out);
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Key-set geometry of one step (device and host): the past splits into
// [0, init_len) | n candidate blocks | [local_start, p0).
struct Geometry {
  int64_t p0;
  int init_len;
  int n_cand;
  int64_t local_start;
};
__host__ __device__ inline Geometry make_geometry(int64_t p0, int n_init, int block, int n_local_prev) {
  Geometry g;
  g.p0 = p0;
  if (p0 <= n_init) {
    g.init_len = 0; g.n_cand = 0; g.local_start = 0;
  } else {
    int64_t n = (p0 - n_local_prev - n_init) / block;
    if (p0 - n_local_prev - n_init < 0) n = 0;
    g.init_len = n_init;
    g.n_cand = static_cast<int>(n);
    g.local_start = n_init + n * block;
  }
  return g;
}

}  // namespace actqkv
