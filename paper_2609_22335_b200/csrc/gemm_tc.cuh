// GEMM tile on the 5th-generation tensor cores: operands staged by TMA into
// 128-byte-swizzled shared memory, tcgen05.mma accumulating in tensor memory,
// epilogue read back with tcgen05.ld.
//
// Tile: 128 output features (MMA M, one TMEM lane each) x bt tokens (MMA N,
// one TMEM column each), K walked in 64-element stages.  The weight tile is
// the MMA "A" operand and the activation tile the "B" operand, both K-major, so
// small token counts (the action head's 9..51 rows) still fill the 128-row
// datapath and stream each weight exactly once.  Gated MLPs run two MMAs per
// stage (gate and up weights against the same activation tile) into two
// accumulators.
//
// Roles inside the 128-thread worker: thread 0 of warp 0 issues TMA loads,
// thread 0 of warp 1 issues MMAs, all four warps run the epilogue (warp w reads
// TMEM lanes 32w..32w+31).  Every mbarrier wait is bounded; on expiry the worker
// records an error and leaves the tile.
#pragma once
#include "tiles_common.cuh"

namespace vla {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
  asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the deadline passed or another worker already reported an error.
__device__ __forceinline__ bool mbar_wait(const TileCtx& c, uint32_t bar, uint32_t parity) {
  unsigned spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 1023u) == 0) {
      if (*reinterpret_cast<volatile unsigned*>(c.error) != 0u) return false;
      uint64_t now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (now > c.deadline) {
        atomicCAS(c.error, 0u, (unsigned)DEV_ERR_WAIT_MBAR);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                 // descriptor version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(GEMM_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

constexpr int GEMM_BAR_BYTES = 1024;   // barrier block at the head of the slab (keeps the stages 1024-byte aligned)
constexpr int GEMM_W_STAGE_BYTES = GEMM_BM * GEMM_BK * 2;

__device__ void tile_gemm(const TileCtx& c, const GemmArgs& g, int tile) {
  const int ft = tile / g.tiles_t, tt = tile % g.tiles_t;
  const int f0 = ft * GEMM_BM, t0 = tt * g.bt;
  const int nt = min(g.bt, g.M - t0);
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int nkb = g.Kp / GEMM_BK;
  const int S = g.stages;
  const int a_bytes = g.bt * GEMM_BK * 2;
  const int stage_bytes = GEMM_W_STAGE_BYTES * (g.dual ? 2 : 1) + a_bytes;

  uint64_t* bars = reinterpret_cast<uint64_t*>(c.smem);          // full[S], empty[S], accum
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t stage0 = smem_u32(c.smem + GEMM_BAR_BYTES);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  const uint32_t accum_bar = bar0 + 8u * (2 * S);

  if (c.tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accum_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  worker_sync(c);

  const uint32_t tmem_d = c.tmem;                 // accumulator columns [0, bt) (and [bt, 2 bt) when dual)
#ifdef VLA_TILE_TIMING
  uint64_t tt0; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tt0));
#endif
  // Whole warps take a role: lanes 1..31 of the producer and MMA warps park at __syncwarp (they must not
  // spin on a barrier, which would stall the issuing lane of the same warp).
  if (warp == 0) {
    if (lane == 0) {
    // ---------------- TMA producer
    asm volatile("fence.proxy.async;" ::: "memory");   // operands were written by generic stores on other SMs
    const char* tm = reinterpret_cast<const char*>(c.tmaps);
    const void* wmap = tm + (size_t)g.wmap * 128;
    const void* w2map = tm + (size_t)g.w2map * 128;
    const void* amap = tm + (size_t)(c.amap_base + g.amap) * 128;
    for (int kb = 0; kb < nkb; ++kb) {
      const int s = kb % S;
      const uint32_t ph = (uint32_t)(kb / S) & 1u;
      if (!mbar_wait(c, empty_bar(s), ph ^ 1u)) break;
      mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
      const uint32_t dst = stage0 + (uint32_t)(s * stage_bytes);
      tma_load_2d(dst, wmap, full_bar(s), kb * GEMM_BK, f0);
      if (g.dual) tma_load_2d(dst + GEMM_W_STAGE_BYTES, w2map, full_bar(s), kb * GEMM_BK, f0);
      tma_load_2d(dst + GEMM_W_STAGE_BYTES * (g.dual ? 2 : 1), amap, full_bar(s), kb * GEMM_BK, t0);
    }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = umma_idesc_bf16(g.bt);
    bool ok = true;
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb % S;
      const uint32_t ph = (uint32_t)(kb / S) & 1u;
      ok = mbar_wait(c, full_bar(s), ph);
      if (!ok) break;
#ifdef VLA_TILE_TIMING
      if (kb == 0 && g.M > 512 && c.dbg) { uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); atomicAdd(c.dbg + 0, t - tt0); }
#endif
      tc_fence_after();
      const uint32_t wsm = stage0 + (uint32_t)(s * stage_bytes);
      const uint32_t asm_ = wsm + GEMM_W_STAGE_BYTES * (g.dual ? 2 : 1);
      const uint64_t wd = umma_desc_sw128(wsm), ad = umma_desc_sw128(asm_);
      const uint64_t w2d = umma_desc_sw128(wsm + GEMM_W_STAGE_BYTES);
#pragma unroll
      for (int k = 0; k < GEMM_BK / 16; ++k) {
        const uint32_t accumulate = (kb | k) != 0 ? 1u : 0u;
        umma_bf16(tmem_d, wd + 2u * k, ad + 2u * k, idesc, accumulate);          // 16 bf16 = 32 bytes per K step
        if (g.dual) umma_bf16(tmem_d + (uint32_t)g.bt, w2d + 2u * k, ad + 2u * k, idesc, accumulate);
      }
      umma_commit(empty_bar(s));        // stage reusable once these MMAs have read it
    }
    if (ok) umma_commit(accum_bar);     // accumulators complete
    }
    __syncwarp();
  }

  // ---------------- epilogue: warp w owns TMEM lanes 32w..32w+31 = features f0+32w..
  const bool ready = mbar_wait(c, accum_bar, 0u);
  __syncwarp();
  tc_fence_after();
#ifdef VLA_TILE_TIMING
  uint64_t tt1; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tt1));
#endif
  if (ready) {
    GemmPtrs ptrs = gemm_ptrs(c, g);
    const int f = f0 + warp * 32 + lane;
    const bool fok = f < g.N;
    const float vecf = (ptrs.vec && fok) ? ptrs.vec[f] : 0.f;
    const uint32_t lane_base = tmem_d + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < nt; c0 += 16) {
      float a[16], b[16];
      tmem_ld16(lane_base + (uint32_t)c0, a);
      if (g.dual) tmem_ld16(lane_base + (uint32_t)(g.bt + c0), b);
      if (!fok) continue;
      const int n = min(16, nt - c0), r0 = t0 + c0;
      if (g.dual) {
        if (g.act == ACT_SILU) gemm_store16<ACT_SILU, true>(g, ptrs, r0, n, f, vecf, a, b);
        else gemm_store16<ACT_GELU, true>(g, ptrs, r0, n, f, vecf, a, b);
      } else if (g.act == ACT_GELU) gemm_store16<ACT_GELU, false>(g, ptrs, r0, n, f, vecf, a, b);
      else if (g.act == ACT_SILU) gemm_store16<ACT_SILU, false>(g, ptrs, r0, n, f, vecf, a, b);
      else gemm_store16<ACT_NONE, false>(g, ptrs, r0, n, f, vecf, a, b);
    }
  }
  tc_fence_before();
  worker_sync(c);
#ifdef VLA_TILE_TIMING
  if (c.tid == 64 && g.M > 512 && c.dbg) {
    uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicAdd(c.dbg + 1, tt1 - tt0); atomicAdd(c.dbg + 2, t - tt1); atomicAdd(c.dbg + 3, 1ull); atomicAdd(c.dbg + 4, (unsigned long long)nkb);
  }
#endif
  if (c.tid == 0) {
    for (int s = 0; s < 2 * S + 1; ++s) mbar_inval(bar0 + 8u * s);
  }
}

}  // namespace vla
