// L2 -> shared-memory bulk-copy throughput probe: every CTA keeps S copies of CH bytes in flight from a region that fits L2.
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <cuda_runtime.h>
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__global__ void probe(const char* src, size_t region, int iters, int S, int CH, unsigned* err) {
  extern __shared__ __align__(1024) char sm[];
  __shared__ __align__(8) uint64_t bars[8];
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[s])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    size_t off = ((size_t)blockIdx.x * 2654435761u) % (region / CH) * CH;
    for (int it = 0; it < iters + S; ++it) {
      int s = it % S;
      uint32_t bar = smem_u32(&bars[s]);
      if (it >= S) {
        uint32_t ph = ((it / S) - 1) & 1u, ok = 0;
        for (int spin = 0; spin < 2000000 && !ok; ++spin)
          asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }" : "=r"(ok) : "r"(bar), "r"(ph) : "memory");
        if (!ok) { atomicExch(err, 1u); break; }
      }
      if (it < iters) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)CH) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(sm + (size_t)s * CH)),
                     "l"(src + off), "r"((uint32_t)CH), "r"(bar) : "memory");
        off += (size_t)CH * 37; if (off >= region) off -= region; off = off / CH * CH; if (off + CH > region) off = 0;
      }
    }
  }
}
int main(int argc, char** argv) {
  for (int mb : {16, 48}) {
  size_t region = (size_t)(argc > 1 ? atoi(argv[1]) : mb) << 20;
  char* src; unsigned* err;
  cudaMalloc(&src, region); cudaMemset(src, 1, region); cudaMalloc(&err, 4); cudaMemset(err, 0, 4);
  cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  int cfgs[][3] = {{1, 2, 32768}, {1, 4, 32768}, {1, 6, 32768}, {2, 2, 32768}, {3, 2, 32768}, {3, 2, 16384}, {3, 4, 16384}, {2, 3, 32768}, {4, 3, 16384}, {6, 2, 16384}};
  for (auto& c : cfgs) {
    int per_sm = c[0], S = c[1], CH = c[2], iters = 4000;
    int grid = 148 * per_sm; size_t smem = (size_t)S * CH;
    probe<<<grid, 32, smem>>>(src, region, 200, S, CH, err);
    cudaDeviceSynchronize();
    cudaEventRecord(e0);
    probe<<<grid, 32, smem>>>(src, region, iters, S, CH, err);
    cudaEventRecord(e1); cudaDeviceSynchronize();
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    unsigned h; cudaMemcpy(&h, err, 4, cudaMemcpyDeviceToHost);
    printf("region %zu MB ctas/sm %d stages %d chunk %d: %.2f TB/s (%.1f B/clk/SM @1.95GHz) in-flight/SM %d KB err %u %s\n", region >> 20, per_sm, S, CH,
           (double)grid * iters * CH / ms / 1e9, (double)per_sm * iters * CH / (ms * 1e-3 * 1.95e9), per_sm * S * CH / 1024, h, cudaGetErrorString(cudaGetLastError()));
  }
  cudaFree(src); cudaFree(err);
  if (argc > 1) break;
  }
  return 0;
}
