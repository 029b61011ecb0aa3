// Fused attention tile on tcgen05 / tensor memory.
//
// One tile = one query head x 128 queries -- or, where few queries meet grouped KV heads (the action head's 9..51
// tokens), several query heads of one KV head side by side in the 128 rows.  Per block of bn keys:
//   S = Q K^T          tcgen05.mma, Q and K tiles K-major (head dim contiguous), S in TMEM
//   online softmax     one thread per query row reads its S row from TMEM (no shuffles),
//                      writes P as bf16 into 128-byte-swizzled shared memory
//   O += P V           tcgen05.mma, P from shared memory, V consumed from its transposed
//                      copy V^T [head dim, tokens] so that it too is K-major; O in TMEM,
//                      rescaled in place when a row maximum moves
// Keys come from up to two segments (cached prefix K/V, then the head's own K/V); blocks
// never straddle segments.  Head dims are handled in 16-wide K steps, so a head padded to
// a multiple of 16 (72 -> 80) costs only its padding.  All waits are bounded.
#pragma once
#include "gemm_tc.cuh"

namespace vla {

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t umma_idesc_bf16_n(int n) { return umma_idesc_bf16(n); }

constexpr int ATTN_BQ = 128;   // queries per tile (MMA M)
constexpr int ATTN_BN = 64;    // keys per block (MMA N of S, MMA K of P V; one 128-byte swizzle row of P)
constexpr float ATTN_RESCALE_LOG2 = 8.0f;   // the running row maximum may lag the true one by this much (log2 units)

// Barrier over the worker's threads that also ANDs a predicate, so every thread takes the same exit.
__device__ __forceinline__ bool worker_all(const TileCtx& c, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "barrier.cta.red.and.pred p, %1, %2, q;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(c.bar_id), "r"(WORKER_THREADS), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

__device__ __forceinline__ float exp2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Key blocks of a tile: segment 0 (cached prefix) then segment 1 (the head's own keys), 64 keys each,
// never straddling a segment; with a causal mask the walk stops at the diagonal.
struct KvBlock {
  int seg, kv0;
  bool valid;
};
template <typename A>
__device__ __forceinline__ KvBlock kv_first(const A& a) {
  KvBlock b;
  b.seg = a.t0 > 0 ? 0 : 1;
  b.kv0 = 0;
  b.valid = (a.t0 > 0 || a.t1 > 0);
  return b;
}
template <typename A>
__device__ __forceinline__ KvBlock kv_next(const A& a, KvBlock b, int q_last) {
  b.kv0 += ATTN_BN;
  const int L = b.seg == 0 ? a.t0 : a.t1;
  if (b.kv0 >= L) {
    if (b.seg == 0 && a.t1 > 0) { b.seg = 1; b.kv0 = 0; }
    else b.valid = false;
  }
  if (a.causal && b.kv0 > q_last) b.valid = false;
  return b;
}

__device__ void tile_attention(const TileCtx& c, const AttnArgs& a_in, int tile) {
  // The node's arguments live in global memory; the shared-memory stores and the asm statements of the block loop
  // would make the compiler fetch them again and again, so the ones the loop uses are copied into registers.
  struct { int32_t k0map, v0map, k1map, v1map, t0, t1, causal, hq, hkv, hs, hd, q_blocks, qmap, tq, ldo, hpt, rph, sfx; float scale_log2e; Ref out; } a;
  a.k0map = a_in.k0map; a.v0map = a_in.v0map; a.k1map = a_in.k1map; a.v1map = a_in.v1map; a.t0 = a_in.t0; a.t1 = a_in.t1;
  a.causal = a_in.causal; a.hq = a_in.hq; a.hkv = a_in.hkv; a.hs = a_in.hs; a.hd = a_in.hd; a.q_blocks = a_in.q_blocks;
  a.qmap = a_in.qmap; a.tq = a_in.tq; a.ldo = a_in.ldo; a.scale_log2e = a_in.scale_log2e; a.out = a_in.out;
  a.hpt = a_in.hpt > 1 ? a_in.hpt : 1; a.rph = a_in.rph; a.sfx = a_in.sfx;
  const int warp = c.tid >> 5, lane = c.tid & 31;
  // folded: tile -> (KV head g, first query head, heads in this tile); else tile -> (head, query block)
  const bool folded = a.hpt > 1;
  const int group = a.hq / a.hkv;
  const int tiles_per_group = folded ? (group + a.hpt - 1) / a.hpt : 1;
  const int head = folded ? (tile / tiles_per_group) * group + (tile % tiles_per_group) * a.hpt : tile / a.q_blocks;
  const int qb = folded ? 0 : tile % a.q_blocks;
  const int nh = folded ? min(a.hpt, group - (tile % tiles_per_group) * a.hpt) : 1;
  const int g = (head * a.hkv) / a.hq;
  const int q0 = qb * ATTN_BQ;
  const int hs = a.hs;
  const int nbox = (hs + 63) / 64;          // 64-column boxes covering one head
  const int kchunks = hs / 16;              // 16-wide K steps of Q K^T

  // shared-memory carve-up (all tile bases 1024-byte aligned)
  const uint32_t base = smem_u32(c.smem);
  const uint32_t bar0 = smem_u32(c.ctl);                       // the five barriers live in the worker's control block
  const uint32_t bar_q = bar0, bar_k = bar0 + 8, bar_v = bar0 + 16, bar_s = bar0 + 24, bar_o = bar0 + 32;
  const uint32_t Qs = base;
  const uint32_t Ks = Qs + (uint32_t)nbox * (ATTN_BQ * 128);
  const uint32_t Vs = Ks + (uint32_t)nbox * (ATTN_BN * 128);
  const uint32_t Ps = Vs + (uint32_t)(hs * 128);
  char* Ps_gen = c.smem + (Ps - base);

  if (c.tid == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_k, 1); mbar_init(bar_v, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  worker_sync(c);

  const uint32_t tmem_s = c.tmem;                            // S: columns [0, 64)
  const uint32_t tmem_o = c.tmem + (uint32_t)ATTN_BN;        // O: columns [64, 64 + hs)
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
  const char* tm = reinterpret_cast<const char*>(c.tmaps);
  auto map_ptr = [&](int idx) { return reinterpret_cast<const void*>(tm + (size_t)(c.amap_base + idx) * 128); };
  const uint32_t idesc_s = umma_idesc_bf16(ATTN_BN), idesc_o = umma_idesc_bf16(hs);
  const bool issuer = c.tid == 0;
  auto load_k = [&](const KvBlock& b) {
    mbar_expect_tx(bar_k, (uint32_t)nbox * (ATTN_BN * 128));
    const void* m = map_ptr(b.seg == 0 ? a.k0map : a.k1map);
    for (int i = 0; i < nbox; ++i) tma_load_2d(Ks + (uint32_t)i * (ATTN_BN * 128), m, bar_k, g * hs + i * 64, b.kv0);
  };
  auto load_v = [&](const KvBlock& b) {
    mbar_expect_tx(bar_v, (uint32_t)(hs * 128));
    tma_load_2d(Vs, map_ptr(b.seg == 0 ? a.v0map : a.v1map), bar_v, b.kv0, g * hs);
  };

  KvBlock cur = kv_first(a);
  const bool loads_on = !c.drop_loads;          // (test hook: with the loads off, the waits below run out)
  if (issuer && loads_on) {
    asm volatile("fence.proxy.async;" ::: "memory");
    if (!folded) {
      mbar_expect_tx(bar_q, (uint32_t)nbox * (ATTN_BQ * 128));
      for (int b = 0; b < nbox; ++b) tma_load_2d(Qs + (uint32_t)b * (ATTN_BQ * 128), map_ptr(a.qmap), bar_q, head * hs + b * 64, q0);
    } else {
      // head i of the tile: a box of rph rows (rows past tq are outside the tensor and arrive as zeros) at row i * rph
      // (a multiple of 8 rows = of one 1024-byte swizzle group); rows past the last head keep whatever the slab held --
      // every output row depends on its own query row only, and those rows are never stored
      mbar_expect_tx(bar_q, (uint32_t)(nh * nbox * a.rph * 128));
      for (int i = 0; i < nh; ++i)
        for (int b = 0; b < nbox; ++b)
          tma_load_2d(Qs + (uint32_t)b * (ATTN_BQ * 128) + (uint32_t)(i * a.rph * 128), map_ptr(a.qmap), bar_q, (head + i) * hs + b * 64, 0);
    }
    if (cur.valid) load_k(cur);
  }

  const int r_in = warp * 32 + lane;                    // this thread's row of the tile
  const int fold_h = folded ? r_in / a.rph : 0;         // which of the tile's heads the row belongs to
  const int row = folded ? r_in - fold_h * a.rph : q0 + r_in;   // this thread's query
  const bool row_ok = row < a.tq && fold_h < nh;
  float m_run = -INFINITY, l_run = 0.f;
  int blk = 0;
  bool ok = true;
  while (cur.valid) {
    const KvBlock nxt = kv_next(a, cur, q0 + ATTN_BQ - 1);
    const uint32_t ph = (uint32_t)blk & 1u;
    // ---- S = Q K^T of this block (issued by one lane; its warp mates park at the __syncwarp)
    if (warp == 0) {
      if (lane == 0) {
        bool go = (blk > 0 || mbar_wait(c, bar_q, 0u)) && mbar_wait(c, bar_k, ph);
        if (go) {
          tc_fence_after();
          for (int kc = 0; kc < kchunks; ++kc) {
            const uint64_t qd = umma_desc_sw128(Qs + (uint32_t)(kc >> 2) * (ATTN_BQ * 128)) + 2u * (kc & 3);
            const uint64_t kd = umma_desc_sw128(Ks + (uint32_t)(kc >> 2) * (ATTN_BN * 128)) + 2u * (kc & 3);
            umma_bf16(tmem_s, qd, kd, idesc_s, kc != 0 ? 1u : 0u);
          }
          umma_commit(bar_s);
        }
      }
      __syncwarp();
    }
    ok = worker_all(c, mbar_wait(c, bar_s, ph));
    tc_fence_after();
    if (!ok) break;
    // S(blk) complete implies P V(blk-1) complete: K, V^T and P buffers are free.  Fetch the next K and
    // this block's V^T now; both loads hide behind the softmax below.
    if (warp == 0) {
      if (lane == 0) {
        if (nxt.valid) load_k(nxt);
        load_v(cur);
      }
      __syncwarp();
    }
    // ---- softmax of this block: one thread per query row, the 64 scores held in registers
    const int L = cur.seg == 0 ? a.t0 : a.t1;
    const int valid = min(ATTN_BN, L - cur.kv0);
    int lim = a.causal ? min(valid, row - cur.kv0 + 1) : valid;   // keys [0, lim) of the block are visible to this row
    if (a.sfx > 0 && cur.seg == 1 && row < a.sfx) lim = min(lim, a.sfx - cur.kv0);   // blocked suffix: the leading own tokens
                                                                                    // see only one another in segment 1
    uint32_t sr[ATTN_BN];
    tmem_ld16_nowait(tmem_s + lane_off + 0u, sr + 0);
    tmem_ld16_nowait(tmem_s + lane_off + 16u, sr + 16);
    tmem_ld16_nowait(tmem_s + lane_off + 32u, sr + 32);
    tmem_ld16_nowait(tmem_s + lane_off + 48u, sr + 48);
    tmem_ld_wait();
    // full blocks (the common case) run without per-key predicates; four independent max / sum chains keep
    // the single warp a scheduler sees from waiting on its own results
    const bool full = __all_sync(0xffffffffu, lim >= ATTN_BN);
    float m4[4] = {m_run, -INFINITY, -INFINITY, -INFINITY};
    if (full) {
#pragma unroll
      for (int j = 0; j < ATTN_BN; ++j) m4[j & 3] = fmaxf(m4[j & 3], __uint_as_float(sr[j]));
    } else {
#pragma unroll
      for (int j = 0; j < ATTN_BN; ++j)
        if (j < lim) m4[j & 3] = fmaxf(m4[j & 3], __uint_as_float(sr[j]));
    }
    float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    const float sl2 = a.scale_log2e;
    // The running maximum only has to keep the exponentials in range, not to be exact: softmax does not depend on
    // the shift, and l and O are accumulated with the same one.  It follows the true maximum only when that has
    // moved by more than 8 in the exponent (p then stays below 2^8), so O is rescaled on few blocks instead of
    // on nearly every one (with 32 rows per warp some row's maximum moves in almost every block).
    float alpha;
    if (m_run == -INFINITY) alpha = 0.f;
    else if ((mx - m_run) * sl2 <= ATTN_RESCALE_LOG2) { mx = m_run; alpha = 1.0f; }
    else alpha = exp2_fast((m_run - mx) * sl2);
    const float mb = mx * sl2;
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
    char* prow = Ps_gen + (size_t)r_in * 128;
#pragma unroll
    for (int ch = 0; ch < ATTN_BN / 8; ++ch) {
      uint32_t pk[4];
#pragma unroll
      for (int j = 0; j < 8; j += 2) {
        const int jj = ch * 8 + j;
        float p0 = exp2_fast(fmaf(__uint_as_float(sr[jj]), sl2, -mb));
        float p1 = exp2_fast(fmaf(__uint_as_float(sr[jj + 1]), sl2, -mb));
        if (!full) { p0 = (jj < lim) ? p0 : 0.f; p1 = (jj + 1 < lim) ? p1 : 0.f; }
        __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
        s4[(j >> 1) & 3] += p0 + p1;
        pk[j >> 1] = *reinterpret_cast<uint32_t*>(&h2);
      }
      *reinterpret_cast<uint4*>(prow + ((ch ^ (r_in & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
    const float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    l_run = l_run * alpha + sum;
    m_run = mx;
    // rescale O where a row maximum moved (warp-uniform decision: the TMEM accesses are warp-wide)
    if (blk > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
      for (int c0 = 0; c0 < hs; c0 += 16) {
        float o[16];
        tmem_ld16(tmem_o + lane_off + (uint32_t)c0, o);
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j] *= alpha;
        tmem_st16(tmem_o + lane_off + (uint32_t)c0, o);
      }
      tmem_st_wait();
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P written by generic stores, read by the MMA
    tc_fence_before();
    worker_sync(c);
    // ---- O += P V
    if (warp == 0) {
      if (lane == 0) {
        if (mbar_wait(c, bar_v, ph)) {
          tc_fence_after();
          for (int kc = 0; kc < ATTN_BN / 16; ++kc) {
            const uint64_t pd = umma_desc_sw128(Ps) + 2u * kc;
            const uint64_t vd = umma_desc_sw128(Vs) + 2u * kc;
            umma_bf16(tmem_o, pd, vd, idesc_o, (blk | kc) != 0 ? 1u : 0u);
          }
          umma_commit(bar_o);
        }
      }
      __syncwarp();
    }
    cur = nxt;
    ++blk;
  }
  // ---- epilogue: O / l -> bf16 (after the last P V has landed)
  if (ok && blk > 0) ok = worker_all(c, mbar_wait(c, bar_o, (uint32_t)(blk - 1) & 1u));
  tc_fence_after();
  if (ok && blk > 0) {
    unsigned short* O = resolve<unsigned short>(c, a.out);
    const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
    for (int c0 = 0; c0 < hs; c0 += 16) {
      float o[16];
      tmem_ld16(tmem_o + lane_off + (uint32_t)c0, o);
      if (row_ok) {
        uint32_t pk[8];
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          __nv_bfloat162 v = __floats2bfloat162_rn(o[j] * inv, o[j + 1] * inv);
          pk[j >> 1] = *reinterpret_cast<uint32_t*>(&v);
        }
        unsigned short* dst = O + (size_t)row * a.ldo + (head + fold_h) * a.hd + c0;
        if (c0 + 16 <= a.hd) {
          *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          *reinterpret_cast<uint4*>(dst + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        } else {
          for (int j = 0; j < 16 && c0 + j < a.hd; ++j)
            dst[j] = (unsigned short)((j & 1) ? (pk[j >> 1] >> 16) : (pk[j >> 1] & 0xFFFFu));
        }
      }
    }
  }
  tc_fence_before();
  worker_sync(c);
  if (c.tid == 0) {
    mbar_inval(bar_q); mbar_inval(bar_k); mbar_inval(bar_v); mbar_inval(bar_s); mbar_inval(bar_o);
  }
}

}  // namespace vla
