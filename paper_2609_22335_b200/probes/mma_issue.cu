// How long does one thread take to issue tcgen05.mma instructions, and how long does the tensor pipe take to run them?
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr) {
  uint64_t d = 0; d |= (uint64_t)((saddr >> 4) & 0x3FFFu); d |= (uint64_t)1 << 16; d |= (uint64_t)(1024 >> 4) << 32; d |= (uint64_t)1 << 46; d |= (uint64_t)2 << 61; return d;
}
__device__ __forceinline__ uint32_t idesc_bf16(int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24); }
__device__ __forceinline__ void mma(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc));
}
__device__ __forceinline__ void commit(uint32_t bar) { asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__global__ void probe(int n, int count, int reps, long long* out, unsigned* err) {
  extern __shared__ __align__(1024) char sm[];
  __shared__ uint32_t tmem_base; __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x < 32) { asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(256u)); asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;"); }
  for (int i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(sm)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) { asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar))); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (threadIdx.x == 0) {
    const uint32_t a_s = smem_u32(sm), b_s = smem_u32(sm) + 16384, d = tmem_base, id = idesc_bf16(n), br = smem_u32(&bar);
    long long t_issue = 0, t_done = 0, t_wait_done = 0;
    for (int r = 0; r < reps; ++r) {
      long long t0 = clock64();
      for (int i = 0; i < count; ++i) mma(d, desc_sw128(a_s) + 2u * (i & 3), desc_sw128(b_s) + 2u * (i & 3), id, i != 0);
      commit(br);
      long long t1 = clock64();
      bool ok = false;
      for (int s = 0; s < 1000000 && !ok; ++s) ok = try_wait(br, (uint32_t)r & 1u);
      long long t2 = clock64();
      if (!ok) { atomicExch(err, 1u); break; }
      // a wait on a barrier whose phase has long completed
      bool ok2 = try_wait(br, (uint32_t)r & 1u);
      long long t3 = clock64();
      t_issue += t1 - t0; t_done += t2 - t0; t_wait_done += t3 - t2 + (ok2 ? 0 : 1000000);
    }
    out[0] = t_issue / reps; out[1] = t_done / reps; out[2] = t_wait_done / reps;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u));
}
int main() {
  long long* out; unsigned* err; cudaMalloc(&out, 64); cudaMalloc(&err, 4); cudaMemset(err, 0, 4);
  cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
  int ns[] = {16, 64, 128, 256}; int counts[] = {1, 4, 8, 16, 32};
  for (int n : ns) for (int c : counts) {
    probe<<<1, 128, 48 * 1024>>>(n, c, 50, out, err);
    cudaError_t e = cudaDeviceSynchronize();
    long long h[3]; unsigned he; cudaMemcpy(h, out, 24, cudaMemcpyDeviceToHost); cudaMemcpy(&he, err, 4, cudaMemcpyDeviceToHost);
    printf("N=%3d x %2d MMAs: issue+commit %5lld cycles (%.0f per MMA), issue->complete %5lld cycles (%.0f per MMA), wait on a completed barrier %lld cycles  err %u %s\n", n, c, h[0], (double)h[0] / c,
           h[1], (double)h[1] / c, h[2], he, cudaGetErrorString(e));
    if (e != cudaSuccess) return 1;
  }
  return 0;
}
