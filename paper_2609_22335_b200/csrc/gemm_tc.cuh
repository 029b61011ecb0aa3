// GEMM tile on the 5th-generation tensor cores: operands staged by TMA into
// 128-byte-swizzled shared memory, tcgen05.mma accumulating in tensor memory,
// epilogue read back with tcgen05.ld.
//
// Tile: 128 output features (MMA M, one TMEM lane each) x bt tokens (MMA N,
// one TMEM column each), K walked in 64-element stages.  The weight tile is
// the MMA "A" operand and the activation tile the "B" operand, both K-major, so
// small token counts (the action head's 9..51 rows) still fill the 128-row
// datapath and stream each weight exactly once.  A gated MLP tile covers 64
// output features: rows 0..63 of its weight tile are gate rows and rows 64..127
// the matching up rows (two 64-row TMA boxes per stage), so it is one MMA stream
// and one accumulator like any other tile; the epilogue multiplies act(gate) by up.
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
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate));   // no memory clobber: the waits, fences and
                                                                           // commits around a batch of MMAs order it
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16-byte asynchronous copy global -> shared through L2 (the source was written by other SMs)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

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

__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Epilogue phase 1 (thread = output feature, the TMEM lane it owns): read the accumulators 16 token columns at a
// time, apply the row scale and the activation, and park the values in shared memory as [token][feature]; a
// feature of the V^T part of a q|k|v projection is written from here, 16 consecutive tokens per store pair.
struct Phase1Args {
  float* St; const float* rs; unsigned short* outT_row;
  float c_acc, c_x, bias; uint32_t lane_base; int bt, nt, tid, t0;
  bool x_staged;            // the residual rows already sit in St: accumulate on top of them
};
template <int ACT>
__device__ __forceinline__ void gemm_phase1(const Phase1Args& p) {
  for (int c0 = 0; c0 < p.nt; c0 += 16) {
    float a[16], v[16], sc[16];
    tmem_ld16(p.lane_base + (uint32_t)c0, a);
    if (p.rs) {                                        // 16 row scales in four broadcast 16-byte loads
#pragma unroll
      for (int j = 0; j < 16; j += 4) {
        const float4 r4 = *reinterpret_cast<const float4*>(p.rs + c0 + j);
        sc[j] = r4.x; sc[j + 1] = r4.y; sc[j + 2] = r4.z; sc[j + 3] = r4.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) sc[j] = 1.0f;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      v[j] = apply_act_t<ACT>(fmaf(a[j], sc[j], p.bias)) * p.c_acc;
    }
    if (p.outT_row) {
      unsigned short* op = p.outT_row + p.t0 + c0;
      uint32_t pk[8];
#pragma unroll
      for (int j = 0; j < 16; j += 2) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[j], v[j + 1]);
        pk[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
      }
      if (p.nt - c0 >= 16) {
        *reinterpret_cast<uint4*>(op) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4*>(op + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j < p.nt - c0) op[j] = (unsigned short)((j & 1) ? (pk[j >> 1] >> 16) : (pk[j >> 1] & 0xFFFFu));
      }
    }
    float* sp = p.St + (size_t)c0 * GEMM_BM + p.tid;
    if (p.x_staged) {
      float x[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) x[j] = sp[j * GEMM_BM];
#pragma unroll
      for (int j = 0; j < 16; ++j) sp[j * GEMM_BM] = fmaf(p.c_x, x[j], v[j]);
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) sp[j * GEMM_BM] = v[j];
    }
  }
}

// Epilogue phase 2, rows of the staged tile (warp = token row, lane = four consecutive features).  A template
// flag that is false removes that output or addend statically; one that is true is still checked per lane (a
// lane beyond the last feature, or one whose columns went to V^T, has a null pointer).  Branches cost a lone warp
// dearly, so the common shapes get straight-line code.
struct Phase2Args {
  const float* tab; const float* tab2; float* o32; unsigned short* o16; float* St;
  float4 vecv;
  size_t ldo32, ldo16, ldtab, ldtab2;
  int nt, t0, warp, lane, gf;
  bool fok, ss;
};
template <bool TAB, bool O32, bool O16, bool SS>
__device__ __forceinline__ void gemm_phase2_row(const Phase2Args& p, int tok, float4 w) {
  const int r = p.t0 + tok;
  if (TAB) {
    w.x += p.vecv.x; w.y += p.vecv.y; w.z += p.vecv.z; w.w += p.vecv.w;
    if (p.tab) {
      const float4 t = *reinterpret_cast<const float4*>(p.tab + (size_t)r * p.ldtab + p.gf);
      w.x += t.x; w.y += t.y; w.z += t.z; w.w += t.w;
    }
    if (p.tab2) {
      const float4 t = *reinterpret_cast<const float4*>(p.tab2 + (size_t)r * p.ldtab2 + p.gf);
      w.x += t.x; w.y += t.y; w.z += t.z; w.w += t.w;
    }
  }
  if (O32 && p.o32) *reinterpret_cast<float4*>(p.o32 + (size_t)r * p.ldo32 + p.gf) = w;
  if (O16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
    if (p.o16)
      *reinterpret_cast<uint2*>(p.o16 + (size_t)r * p.ldo16 + p.gf) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
  if (SS && p.ss) {
    // the lane's share of the row's sum of squares, parked in the row's first 32 words at a position rotated by
    // the row's slot so that the final per-row additions run without bank conflicts
    const float sq = p.fok ? (w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w) : 0.f;
    p.St[(size_t)tok * GEMM_BM + ((p.lane + (tok >> 2)) & 31)] = sq;
  }
}
template <bool TAB, bool O32, bool O16, bool SS>
__device__ __forceinline__ void gemm_phase2_rows(const Phase2Args& p) {
  constexpr int RP = 4;                              // token rows per pass
  int tok0 = p.warp;
  for (; tok0 + 4 * (RP - 1) < p.nt; tok0 += 4 * RP) {   // full passes: no per-row bound checks
    float4 v[RP];
#pragma unroll
    for (int q = 0; q < RP; ++q) v[q] = *reinterpret_cast<const float4*>(p.St + (size_t)(tok0 + 4 * q) * GEMM_BM + 4 * p.lane);
    if (SS) __syncwarp();                            // every lane has its part of the rows before partial sums overwrite them
#pragma unroll
    for (int q = 0; q < RP; ++q) gemm_phase2_row<TAB, O32, O16, SS>(p, tok0 + 4 * q, v[q]);
  }
  for (; tok0 < p.nt; tok0 += 4) {                   // ragged tail, one row at a time
    const float4 v = *reinterpret_cast<const float4*>(p.St + (size_t)tok0 * GEMM_BM + 4 * p.lane);
    if (SS) __syncwarp();
    gemm_phase2_row<TAB, O32, O16, SS>(p, tok0, v);
  }
}

// Rows of a gated tile: columns 0..63 of the staged row are gate values, 64..127 the up values of the same 64
// features.  Sixteen lanes cover a row (four features each), so a warp does two rows per pass.
template <int ACT>
__device__ __forceinline__ void gemm_phase2_rows_gated(const Phase2Args& p, float c_acc, int f0, int N) {
  const int sub = p.lane >> 4, l16 = p.lane & 15;
  const int gf = f0 + 4 * l16;
  const bool fok = gf < N;
  for (int tok0 = p.warp; tok0 < p.nt; tok0 += 8) {
    const int tok = tok0 + 4 * sub;
    if (tok < p.nt && fok) {
      const float4 gt = *reinterpret_cast<const float4*>(p.St + (size_t)tok * GEMM_BM + 4 * l16);
      const float4 up = *reinterpret_cast<const float4*>(p.St + (size_t)tok * GEMM_BM + GEMM_BM / 2 + 4 * l16);
      const float w0 = apply_act_t<ACT>(gt.x) * up.x * c_acc, w1 = apply_act_t<ACT>(gt.y) * up.y * c_acc;
      const float w2 = apply_act_t<ACT>(gt.z) * up.z * c_acc, w3 = apply_act_t<ACT>(gt.w) * up.w * c_acc;
      __nv_bfloat162 lo = __floats2bfloat162_rn(w0, w1), hi = __floats2bfloat162_rn(w2, w3);
      *reinterpret_cast<uint2*>(p.o16 + (size_t)(p.t0 + tok) * p.ldo16 + gf) =
          make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    }
  }
}

constexpr int GEMM_W_STAGE_BYTES = GEMM_BM * GEMM_BK * 2;

__device__ void tile_gemm(const TileCtx& c, const GemmArgs& g, int tile) {
  const int ft = tile / g.tiles_t, tt = tile % g.tiles_t;
  const int f0 = ft * (g.dual ? GEMM_BM / 2 : GEMM_BM), t0 = tt * g.bt;    // a gated tile covers 64 output features
  const int nt = min(g.bt, g.M - t0);
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int nkb = g.Kp / GEMM_BK;
  const int S = g.stages;
  const int a_bytes = g.bt * GEMM_BK * 2;
  const bool dual = g.dual != 0;            // arguments used inside the loops, out of global memory once
  const int bt = g.bt;
  const int stage_bytes = GEMM_W_STAGE_BYTES + a_bytes;

  uint64_t* bars = reinterpret_cast<uint64_t*>(c.ctl);           // full[S], empty[S], accum (the worker's control block)
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t stage0 = smem_u32(c.smem);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  const uint32_t accum_bar = bar0 + 8u * (2 * S);

  if (c.tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accum_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  worker_sync(c);

  // epilogue pointers and shape facts are resolved now, so their loads overlap the main loop
  const GemmPtrs ptrs = gemm_ptrs(c, g);
  const bool vec4 = (g.N % 4 == 0) && (!ptrs.X || g.ldx % 4 == 0) && (!ptrs.tab || g.ldtab % 4 == 0) &&
                    (!ptrs.tab2 || g.ldtab2 % 4 == 0) && (!ptrs.out32 || g.ldo32 % 4 == 0) && (!ptrs.out16 || g.ldo16 % 4 == 0);
  const int gf = f0 + 4 * lane;            // epilogue phase 2: this lane's four consecutive features
  const bool fok = gf < g.N;
  const uint32_t tmem_d = c.tmem;                 // accumulator columns [0, bt)
  float* rs_smem = reinterpret_cast<float*>(c.ctl + 256);        // [bt] row scales, in the control block
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
    for (int kb = 0; kb < nkb && !c.drop_loads; ++kb) {
      const int s = kb % S;
      const uint32_t ph = (uint32_t)(kb / S) & 1u;
      if (!mbar_wait(c, empty_bar(s), ph ^ 1u)) break;
      mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
      const uint32_t dst = stage0 + (uint32_t)(s * stage_bytes);
      tma_load_2d(dst, wmap, full_bar(s), kb * GEMM_BK, f0);      // 128 rows, or the 64 gate rows of a gated tile
      if (dual) tma_load_2d(dst + GEMM_W_STAGE_BYTES / 2, w2map, full_bar(s), kb * GEMM_BK, f0);   // its 64 up rows
      tma_load_2d(dst + GEMM_W_STAGE_BYTES, amap, full_bar(s), kb * GEMM_BK, t0);
    }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = umma_idesc_bf16(bt);
    bool ok = true;
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb % S;
      const uint32_t ph = (uint32_t)(kb / S) & 1u;
      ok = mbar_wait(c, full_bar(s), ph);
      if (!ok) break;
      tc_fence_after();
      const uint32_t wsm = stage0 + (uint32_t)(s * stage_bytes);
      const uint32_t asm_ = wsm + GEMM_W_STAGE_BYTES;
      const uint64_t wd = umma_desc_sw128(wsm), ad = umma_desc_sw128(asm_);
#pragma unroll
      for (int k = 0; k < GEMM_BK / 16; ++k) {
        const uint32_t accumulate = (kb | k) != 0 ? 1u : 0u;
        umma_bf16(tmem_d, wd + 2u * k, ad + 2u * k, idesc, accumulate);          // 16 bf16 = 32 bytes per K step
      }
      umma_commit(empty_bar(s));        // stage reusable once these MMAs have read it
    }
    if (ok) umma_commit(accum_bar);     // accumulators complete
    }
    __syncwarp();
  } else if (g.rs_d > 0) {
    // ---------------- folded RMSNorm: row scales from the stream's per-row partial sums of squares, summed in a
    // fixed order while the main loop runs (thread j: tokens j and j + 64)
    const float* ssp = resolve<const float>(c, g.ss_in);
    const int ss_nft = g.ss_nft;
    const float inv_d = (float)g.rs_d;
    for (int tkn = c.tid - 64; tkn < bt; tkn += 64) {
      float ssq = 0.f;
      if (tkn < nt)
        for (int q = 0; q < ss_nft; ++q) ssq += ld_act(ssp + (size_t)(t0 + tkn) * ss_nft + q);
      rs_smem[tkn] = 1.0f / sqrtf(ssq / inv_d + 1e-6f);
    }
  }

  // ---------------- epilogue in two phases.
  // Phase 1 (thread = output feature, the TMEM lane it owns): read the accumulators, apply the row scale and the
  // activation, and park the values in shared memory (the pipeline stages are free now) as [token][feature];
  // the V^T part of a q|k|v projection is written from here, 16 consecutive tokens per thread.
  // Phase 2 (warp = token row, lane = 4 consecutive features): add the residual / vectors / tables and store
  // whole 512-byte rows; the row's sum of squares over this tile's features goes to the stream's partials.
  const bool ready = mbar_wait(c, accum_bar, 0u);
  __syncwarp();
  tc_fence_after();
  float* St = reinterpret_cast<float*>(c.smem);   // [bt][128] fp32
  // The residual rows of this tile start their way into the staging area now (asynchronous 16-byte copies
  // through L2, no registers held), so their latency overlaps the accumulator read-out.
  const bool x_staged = vec4 && ptrs.X != nullptr;
  if (x_staged) {
    if (ready && fok)
      for (int tok = warp; tok < nt; tok += 4)
        cp_async16(smem_u32(St + (size_t)tok * GEMM_BM + 4 * lane), ptrs.X + (size_t)(t0 + tok) * g.ldx + gf);
    cp_async_wait_all();
  }
  if (g.rs_d > 0 || x_staged) worker_sync(c);     // row scales written by warps 2 and 3; residual rows landed
  if (ready) {
    Phase1Args p1;
    p1.St = St; p1.rs = g.rs_d > 0 ? rs_smem : nullptr; p1.c_acc = g.c_acc; p1.c_x = g.c_x; p1.x_staged = x_staged;
    p1.lane_base = tmem_d + ((uint32_t)(warp * 32) << 16);
    p1.bt = g.bt; p1.nt = nt; p1.tid = c.tid; p1.t0 = t0;
    const int f = f0 + c.tid;
    p1.bias = (ptrs.bias != nullptr && f < g.N) ? ptrs.bias[f] : 0.0f;      // this thread's output feature
    p1.outT_row = (ptrs.outT != nullptr && f >= g.t_col0 && f < g.N) ? ptrs.outT + (size_t)(f - g.t_col0) * g.ldoT : nullptr;
    if (dual) { p1.c_acc = 1.0f; gemm_phase1<ACT_NONE>(p1); }   // gate and up rows parked raw: phase 2 combines them
    else if (g.act == ACT_GELU) gemm_phase1<ACT_GELU>(p1);
    else if (g.act == ACT_SILU) gemm_phase1<ACT_SILU>(p1);
    else gemm_phase1<ACT_NONE>(p1);
  }
  worker_sync(c);
  if (ready) {
    float* ssq_out = resolve<float>(c, g.ss_out);
    if (vec4) {
      // the node's arguments live in global memory, which the stores below might alias as far as the compiler
      // knows: everything the row loop needs is taken into registers first
      const size_t ldo32 = (size_t)g.ldo32, ldo16 = (size_t)g.ldo16, ldtab = (size_t)g.ldtab, ldtab2 = (size_t)g.ldtab2;
      const size_t ss_ld = (size_t)g.ss_out_ld;
      const float* const tab = fok ? ptrs.tab : nullptr;
      const float* const tab2 = fok ? ptrs.tab2 : nullptr;
      float* const o32 = fok ? ptrs.out32 : nullptr;
      const bool skip16 = ptrs.outT != nullptr && gf >= g.t_col0;      // these columns went to V^T in phase 1
      unsigned short* const o16 = (fok && !skip16) ? ptrs.out16 : nullptr;
      Phase2Args p2;
      p2.vecv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (ptrs.vec && fok) p2.vecv = *reinterpret_cast<const float4*>(ptrs.vec + gf);
      p2.tab = tab; p2.tab2 = tab2; p2.o32 = o32; p2.o16 = o16; p2.St = St;
      p2.ldo32 = ldo32; p2.ldo16 = ldo16; p2.ldtab = ldtab; p2.ldtab2 = ldtab2;
      p2.nt = nt; p2.t0 = t0; p2.warp = warp; p2.lane = lane; p2.gf = gf; p2.fok = fok; p2.ss = ssq_out != nullptr;
      const bool has_tab = ptrs.tab || ptrs.tab2 || ptrs.vec;          // warp-uniform choices of the row code
      if (dual) {
        p2.o16 = ptrs.out16;
        if (g.act == ACT_SILU) gemm_phase2_rows_gated<ACT_SILU>(p2, g.c_acc, f0, g.N);
        else if (g.act == ACT_GELU) gemm_phase2_rows_gated<ACT_GELU>(p2, g.c_acc, f0, g.N);
        else gemm_phase2_rows_gated<ACT_NONE>(p2, g.c_acc, f0, g.N);
      } else if (!has_tab && !ptrs.out32 && !ssq_out) gemm_phase2_rows<false, false, true, false>(p2);      // bf16 only (q|k|v, MLP up)
      else if (!has_tab) gemm_phase2_rows<false, true, true, true>(p2);                                // residual stream
      else gemm_phase2_rows<true, true, true, true>(p2);
      if (ssq_out) {
        __syncwarp();
        const int tok = warp + 4 * lane;                 // this lane's row: slot `lane` of this warp
        if (tok < nt) {
          float sq = 0.f;
#pragma unroll 8
          for (int i = 0; i < 32; ++i) sq += St[(size_t)tok * GEMM_BM + ((i + lane) & 31)];   // lane order 0..31
          ssq_out[(size_t)(t0 + tok) * ss_ld + ft] = sq;
        }
      }
    } else {
      // odd widths (e.g. a 7-wide action output): one feature per lane and pass
      for (int tok = warp; tok < nt; tok += 4) {
        const int r = t0 + tok;
        float sq = 0.f;
        for (int q = lane; q < GEMM_BM; q += 32) {
          const int of = f0 + q;
          if (of >= g.N) continue;
          float v = St[(size_t)tok * GEMM_BM + q];
          if (ptrs.X) v = fmaf(g.c_x, ld_act(ptrs.X + (size_t)r * g.ldx + of), v);
          if (ptrs.vec) v += ptrs.vec[of];
          if (ptrs.tab) v += ptrs.tab[(size_t)r * g.ldtab + of];
          if (ptrs.tab2) v += ptrs.tab2[(size_t)r * g.ldtab2 + of];
          if (ptrs.out32) ptrs.out32[(size_t)r * g.ldo32 + of] = v;
          if (ptrs.out16 && !(ptrs.outT && of >= g.t_col0)) ptrs.out16[(size_t)r * g.ldo16 + of] = f32_to_bf16_bits(v);
          sq = fmaf(v, v, sq);
        }
        if (ssq_out) {
          sq = warp_sum(sq);
          if (lane == 0) ssq_out[(size_t)r * g.ss_out_ld + ft] = sq;
        }
      }
    }
  }
  tc_fence_before();
  worker_sync(c);
  if (c.tid == 0) {
    for (int s = 0; s < 2 * S + 1; ++s) mbar_inval(bar0 + 8u * s);
  }
}

}  // namespace vla
