// Cost of mbarrier.try_wait on a barrier that completed a while ago: one thread, or all 128 threads of a block.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__global__ void probe(int mode, long long* out) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ long long tmax[4];
  const uint32_t br = smem_u32(&bar);
  long long acc = 0;
  for (int r = 0; r < 20; ++r) {
    if (threadIdx.x == 0) { asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(br)); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(br) : "memory");   // completes phase 0
    __syncthreads();
    long long t = clock64();
    while (clock64() - t < 3000) {}
    __syncthreads();
    long long t0 = clock64();
    bool ok = true;
    if (mode == 0) { if (threadIdx.x == 0) ok = try_wait(br, 0u); }
    else if (mode == 1) ok = try_wait(br, 0u);
    else if (mode == 2) ok = test_wait(br, 0u);
    else if (mode == 3) { if ((threadIdx.x & 31) == 0) ok = try_wait(br, 0u); __syncwarp(); }
    long long t1 = clock64();
    acc += (t1 - t0) + (ok ? 0 : 100000);
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(br) : "memory");
    __syncthreads();
  }
  // the slowest thread's average
  long long v = acc / 20;
  for (int o = 16; o > 0; o >>= 1) { long long w = __shfl_xor_sync(0xffffffffu, v, o); v = v > w ? v : w; }
  if ((threadIdx.x & 31) == 0) tmax[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) { long long m = 0; for (int i = 0; i < 4; ++i) m = m > tmax[i] ? m : tmax[i]; out[mode] = m; }
}
int main() {
  long long* out; cudaMalloc(&out, 64);
  const char* names[] = {"one thread try_wait", "128 threads try_wait", "128 threads test_wait", "lane 0 of each warp try_wait + syncwarp"};
  for (int mode = 0; mode < 4; ++mode) {
    probe<<<1, 128>>>(mode, out);
    cudaError_t e = cudaDeviceSynchronize();
    long long h[4]; cudaMemcpy(h, out, 32, cudaMemcpyDeviceToHost);
    printf("%-44s slowest thread: %lld cycles  %s\n", names[mode], h[mode], cudaGetErrorString(e));
  }
  return 0;
}
