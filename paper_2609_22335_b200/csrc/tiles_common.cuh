// Shared pieces of the tile bodies.  Each body is executed by one worker group of WORKER_THREADS
// threads: either a whole CTA of an ordinary kernel or one worker group inside
// the persistent co-scheduling kernel.  Bodies synchronise with the worker's
// named barrier only (never __syncthreads) and use the shared-memory slab they
// are handed, so the same code, tile shapes and reduction orders run in every
// mode -- which is what makes the modes bit-identical.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "vla_types.h"

namespace vla {

struct TileCtx {
  char* arena;
  uint64_t slot_base;   // arena offset of this frame slot's buffers
  char* smem;           // this tile's shared-memory slab (1024-byte aligned): operand stages, staging tiles
  char* ctl;            // this worker's 1 KB control block (mbarriers, row scales): outside the slab, so tile
                        // slabs are whole powers-of-two-friendly sizes (64 KB, 72 KB, 48 KB)
  uint32_t tmem;        // this worker's tensor-memory column base
  int tid;              // 0 .. WORKER_THREADS-1
  int bar_id;           // named barrier of this worker
  uint64_t deadline;    // %globaltimer value after which bounded waits give up
  unsigned int* error;  // sticky device error word
  const uint64_t* inputs;  // this frame slot's input pointer table
  const void* tmaps;    // tensor-map table (128 bytes per entry)
  int amap_base;        // index of this frame slot's first activation map
  int drop_loads;       // test hook of the stand-alone operators: the TMA producer issues nothing, so the consumers'
                        // bounded waits run out (0 everywhere else)
};

template <typename T>
__device__ __forceinline__ T* resolve(const TileCtx& c, Ref r) {
  if (r == 0) return nullptr;
  if (r & REF_INPUT) {
    const unsigned long long p = __ldcg(reinterpret_cast<const unsigned long long*>(c.inputs) + ((r >> 56) & 0xF));
    return reinterpret_cast<T*>(p + (r & ((1ull << 56) - 1)));
  }
  return reinterpret_cast<T*>(c.arena + (r & ~REF_SLOT) + ((r & REF_SLOT) ? c.slot_base : 0ull));
}

__device__ __forceinline__ void worker_sync(const TileCtx& c) {
  asm volatile("bar.sync %0, %1;" ::"r"(c.bar_id), "r"(WORKER_THREADS) : "memory");
}

// Activations are produced by other SMs during the same kernel: read them through L2.
__device__ __forceinline__ float ld_act(const float* p) { return __ldcg(p); }
__device__ __forceinline__ uint4 ld_act(const uint4* p) { return __ldcg(p); }
__device__ __forceinline__ unsigned short ld_act(const unsigned short* p) { return __ldcg(p); }
__device__ __forceinline__ int ld_act(const int* p) { return __ldcg(p); }

__device__ __forceinline__ float bf16_bits_to_f32(unsigned short b) { return __uint_as_float(((unsigned int)b) << 16); }
__device__ __forceinline__ unsigned short f32_to_bf16_bits(float f) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

// Activations use the hardware approximations (tanh.approx, ex2.approx): their error (~2^-11 relative)
// is below the bf16 rounding of the values they produce.
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_tanh_f(float x) {
  const float c = 0.7978845608028654f;
  return 0.5f * x * (1.0f + tanh_fast(c * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu_f(float x) { return __fdividef(x, 1.0f + __expf(-x)); }
template <int ACT>
__device__ __forceinline__ float apply_act_t(float v) {
  return ACT == ACT_GELU ? gelu_tanh_f(v) : (ACT == ACT_SILU ? silu_f(v) : v);
}
__device__ __forceinline__ float apply_act(int act, float v) {
  return act == ACT_GELU ? gelu_tanh_f(v) : (act == ACT_SILU ? silu_f(v) : v);
}

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

// ------------------------------------------------------------------ GEMM epilogue (one output element)
struct GemmPtrs {
  const float* X; const float* vec; const float* tab; const float* tab2; const float* bias;
  float* out32; unsigned short* out16; unsigned short* outT;
};
__device__ __forceinline__ GemmPtrs gemm_ptrs(const TileCtx& c, const GemmArgs& g) {
  GemmPtrs p;
  p.X = resolve<const float>(c, g.X); p.vec = resolve<const float>(c, g.vec);
  p.tab = resolve<const float>(c, g.tab); p.tab2 = resolve<const float>(c, g.tab2);
  p.bias = resolve<const float>(c, g.bias);
  p.out32 = resolve<float>(c, g.out32); p.out16 = resolve<unsigned short>(c, g.out16);
  p.outT = resolve<unsigned short>(c, g.outT);
  return p;
}
}  // namespace vla
