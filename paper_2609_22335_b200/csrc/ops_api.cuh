// Stand-alone operator entry points: the GEMM and fused-attention tile bodies of the
// engine, launched as ordinary kernels on caller-owned device tensors.  They exist so the
// tile bodies can be checked operator by operator against the CPU oracle, and for callers
// that want the kernels without the frame pipeline.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/vla.h"
#include "dispatch.cuh"

namespace vla {

struct OpMaps {
  alignas(64) CUtensorMap m[4];
};

typedef CUresult (*OpEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline OpEncodeFn op_encoder() {
  static OpEncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<OpEncodeFn>(p);
  }
  return fn;
}

// 2-D bf16 row-major tensor, 64-column boxes, 128-byte swizzle, zero fill outside.
inline bool op_encode(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  OpEncodeFn enc = op_encoder();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)GEMM_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Bound of the operators' device-side waits, and the test hook that makes one run out (vla_debug_op_fault).
struct OpFault {
  unsigned long long wait_limit_ns;
  int drop_loads;
};
inline OpFault& op_fault() {
  static OpFault f = {2000000000ull, 0};
  return f;
}

__device__ __forceinline__ TileCtx op_tile_ctx(char* smem, char* ctl, uint32_t tmem, const void* maps, unsigned* err,
                                               OpFault fault) {
  TileCtx tc;
  tc.arena = nullptr;          // Refs of the stand-alone operators are absolute device addresses
  tc.slot_base = 0;
  tc.smem = smem;
  tc.ctl = ctl;
  tc.tmem = tmem;
  tc.tid = threadIdx.x;
  tc.bar_id = 1;
  tc.error = err;
  tc.tmaps = maps;
  tc.inputs = nullptr;
  tc.amap_base = 0;
  tc.drop_loads = fault.drop_loads;
  tc.deadline = gtimer() + fault.wait_limit_ns;
  return tc;
}

__global__ void __launch_bounds__(WORKER_THREADS) vla_op_attention_kernel(AttnArgs a, const __grid_constant__ OpMaps maps,
                                                                          int tmem_cols, unsigned* err, OpFault fault) {
  extern __shared__ __align__(1024) char smem_raw[];
  __shared__ uint32_t tmem_base_s;
  __shared__ __align__(16) char ctl_block[1024];
  if (threadIdx.x < 32) tmem_alloc(&tmem_base_s, (uint32_t)tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  TileCtx tc = op_tile_ctx(smem_raw, ctl_block, tmem_base_s, &maps, err, fault);
  tile_attention(tc, a, (int)blockIdx.x);
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(tmem_base_s, (uint32_t)tmem_cols);
}

__global__ void __launch_bounds__(WORKER_THREADS) vla_op_linear_kernel(GemmArgs g, const __grid_constant__ OpMaps maps,
                                                                       int tmem_cols, unsigned* err, OpFault fault) {
  extern __shared__ __align__(1024) char smem_raw[];
  __shared__ uint32_t tmem_base_s;
  __shared__ __align__(16) char ctl_block[1024];
  if (threadIdx.x < 32) tmem_alloc(&tmem_base_s, (uint32_t)tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  TileCtx tc = op_tile_ctx(smem_raw, ctl_block, tmem_base_s, &maps, err, fault);
  tile_gemm(tc, g, (int)blockIdx.x);
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(tmem_base_s, (uint32_t)tmem_cols);
}

// vt[c][t] = v[t][c] for a bf16 matrix v [rows, cols] (row pitch ldv), vt row pitch ldt.
__global__ void vla_op_transpose_kernel(const unsigned short* v, unsigned short* vt, int rows, int cols, int ldv, int ldt) {
  __shared__ unsigned short tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int r = r0 + i, c = c0 + threadIdx.x;
    tile[i][threadIdx.x] = (r < rows && c < cols) ? v[(size_t)r * ldv + c] : (unsigned short)0;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int c = c0 + i, r = r0 + threadIdx.x;
    if (c < cols && r < rows) vt[(size_t)c * ldt + r] = tile[threadIdx.x][i];
  }
}

constexpr size_t OP_ATTN_HEADER = 256;   // error word + padding in front of V^T

// Error word of vla_op_linear: one per device, in a fixed device array of the library, looked up on the first call
// made with that device current.  Calls on one device share it (see the header: check vla_op_status before
// launching another operator call that could overwrite it).
static __device__ __align__(256) unsigned g_op_linear_error[64];
inline unsigned* op_linear_error_word() {
  constexpr int kMax = 64;
  static std::atomic<unsigned*> ptr[kMax];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMax) return nullptr;
  unsigned* p = ptr[dev].load(std::memory_order_acquire);
  if (!p) {
    void* a = nullptr;
    if (cudaGetSymbolAddress(&a, g_op_linear_error) != cudaSuccess || !a) return nullptr;
    p = static_cast<unsigned*>(a);
    ptr[dev].store(p, std::memory_order_release);
  }
  return p;
}

// Reads an operator's error word back after the stream has drained.
inline int op_status_of(const unsigned* dev_word, cudaStream_t s) {
  if (cudaStreamSynchronize(s) != cudaSuccess) return VLA_ERR_CUDA;
  unsigned v = 0;
  if (cudaMemcpy(&v, dev_word, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return VLA_ERR_CUDA;
  return v == 0 ? VLA_OK : VLA_ERR_TIMEOUT;
}

inline int64_t op_pad(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

inline bool op_attention_shape_ok(int tq, int tkv, int hq, int hkv, int hd) {
  return tq >= 1 && tkv >= 1 && hq >= 1 && hkv >= 1 && hq % hkv == 0 && hd >= 16 && hd <= 256 && hd % 16 == 0;
}

inline size_t op_attention_scratch_bytes(int tkv, int hkv, int hd) {
  return OP_ATTN_HEADER + (size_t)hkv * hd * (size_t)op_pad(tkv, 64) * 2;
}

// Shared implementation of the two attention entry points: `scratch` holds an error word and V^T.
inline int op_attention_run(const void* q, const void* k, const void* v, void* out, int tq, int tkv, int hq, int hkv, int hd,
                            int causal, void* scratch, cudaStream_t s) {
  const int64_t tpad = op_pad(tkv, 64);
  unsigned* err = static_cast<unsigned*>(scratch);
  unsigned short* vt = reinterpret_cast<unsigned short*>(static_cast<char*>(scratch) + OP_ATTN_HEADER);
  if (cudaMemsetAsync(scratch, 0, OP_ATTN_HEADER, s) != cudaSuccess) return VLA_ERR_CUDA;
  dim3 tb(32, 8), tg((unsigned)((hkv * hd + 31) / 32), (unsigned)((tkv + 31) / 32));
  vla_op_transpose_kernel<<<tg, tb, 0, s>>>(static_cast<const unsigned short*>(v), vt, tkv, hkv * hd, hkv * hd, (int)tpad);

  AttnArgs a;
  memset(&a, 0, sizeof a);
  a.out = reinterpret_cast<Ref>(out);
  a.ldo = hq * hd;
  a.tq = tq; a.t0 = tkv; a.t1 = 0;
  a.hq = hq; a.hkv = hkv; a.hd = hd; a.hs = hd; a.causal = causal ? 1 : 0;
  a.bn = 64;
  a.q_blocks = (tq + 127) / 128;
  a.hpt = attn_fold(tq, hq, hkv, &a.rph);
  const int n_tiles = a.hpt > 1 ? hkv * (((hq / hkv) + a.hpt - 1) / a.hpt) : hq * a.q_blocks;
  a.scale_log2e = 1.4426950408889634f / sqrtf((float)hd);
  a.qmap = 0; a.k0map = 1; a.v0map = 2; a.k1map = 1; a.v1map = 2;
  OpMaps maps;
  memset(&maps, 0, sizeof maps);
  if (!op_encode(&maps.m[0], q, tq, (int64_t)hq * hd, (int64_t)hq * hd, a.hpt > 1 ? a.rph : 128) ||
      !op_encode(&maps.m[1], k, tkv, (int64_t)hkv * hd, (int64_t)hkv * hd, a.bn) ||
      !op_encode(&maps.m[2], vt, (int64_t)hkv * hd, tkv, tpad, hd))
    return VLA_ERR_CUDA;
  const int smem = attn_smem_bytes(hd);
  int tmem_cols = 32;
  while (tmem_cols < a.bn + hd) tmem_cols <<= 1;
  if (cudaFuncSetAttribute(vla_op_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return VLA_ERR_CUDA;
  vla_op_attention_kernel<<<n_tiles, WORKER_THREADS, smem, s>>>(a, maps, tmem_cols, err, op_fault());
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

}  // namespace vla

extern "C" {

int vla_op_attention_scratch_bytes(int32_t tkv, int32_t hkv, int32_t hd, size_t* out_bytes) {
  if (!out_bytes || tkv < 1 || hkv < 1 || hd < 16 || hd > 256 || hd % 16) return VLA_ERR_INVALID;
  *out_bytes = vla::op_attention_scratch_bytes(tkv, hkv, hd);
  return VLA_OK;
}

int vla_op_attention(const void* q, const void* k, const void* v, void* out, int32_t tq, int32_t tkv, int32_t hq, int32_t hkv,
                     int32_t hd, int32_t causal, void* scratch, size_t scratch_bytes, void* stream) {
  if (!q || !k || !v || !out || !scratch || !vla::op_attention_shape_ok(tq, tkv, hq, hkv, hd)) return VLA_ERR_INVALID;
  if (causal && tq != tkv) return VLA_ERR_INVALID;
  if (scratch_bytes < vla::op_attention_scratch_bytes(tkv, hkv, hd) || (reinterpret_cast<uintptr_t>(scratch) & 255))
    return VLA_ERR_NOMEM;
  return vla::op_attention_run(q, k, v, out, tq, tkv, hq, hkv, hd, causal, scratch, static_cast<cudaStream_t>(stream));
}

int vla_op_linear(const void* a, const void* w, float* out32, void* out16, int32_t m, int32_t n, int32_t k, int32_t act,
                  void* stream) {
  using namespace vla;
  if (!a || !w || (!out32 && !out16) || m < 1 || n < 1 || k < 8 || k % 8 || act < 0 || act > 2) return VLA_ERR_INVALID;
  GemmArgs g;
  memset(&g, 0, sizeof g);
  g.M = m; g.N = n; g.Kp = (int)op_pad(k, GEMM_BK);
  g.out32 = reinterpret_cast<Ref>(out32); g.ldo32 = n;
  g.out16 = reinterpret_cast<Ref>(out16); g.ldo16 = n;
  g.act = act; g.c_acc = 1.f; g.c_x = 1.f;
  g.tiles_t = (m + GEMM_MAX_BT - 1) / GEMM_MAX_BT;
  g.bt = (int)op_pad((m + g.tiles_t - 1) / g.tiles_t, 16);
  g.stages = gemm_stages(g.bt, g.Kp);
  g.wmap = 0; g.w2map = 0; g.amap = 1;
  OpMaps maps;
  memset(&maps, 0, sizeof maps);
  if (!op_encode(&maps.m[0], w, n, k, k, GEMM_BM) || !op_encode(&maps.m[1], a, m, k, k, g.bt)) return VLA_ERR_CUDA;
  const int smem = gemm_smem_bytes(g.bt, g.stages);
  int tmem_cols = 32;
  while (tmem_cols < g.bt) tmem_cols <<= 1;
  unsigned* err = op_linear_error_word();     // this device's word (a fixed device array: nothing is allocated)
  if (!err) return VLA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(err, 0, 4, s) != cudaSuccess) return VLA_ERR_CUDA;
  if (cudaFuncSetAttribute(vla_op_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return VLA_ERR_CUDA;
  vla_op_linear_kernel<<<((n + GEMM_BM - 1) / GEMM_BM) * g.tiles_t, WORKER_THREADS, smem, s>>>(g, maps, tmem_cols, err, op_fault());
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

int vla_debug_op_fault(int32_t drop_operand_loads, uint64_t wait_limit_ns) {
  vla::op_fault().drop_loads = drop_operand_loads ? 1 : 0;
  vla::op_fault().wait_limit_ns = wait_limit_ns ? wait_limit_ns : 2000000000ull;
  return VLA_OK;
}

}  // extern "C"
