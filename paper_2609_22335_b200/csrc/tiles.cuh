// Tile bodies other than the GEMM (see gemm_tc.cuh): RMSNorm, fused attention, and the
// elementwise / gather tiles, plus the dispatch switch.
#pragma once
#include "attn_tc.cuh"
#include "gemm_tc.cuh"
#include "tiles_common.cuh"

namespace vla {

// ------------------------------------------------------------------ RMSNorm tile (one warp per row, float4 lanes)
// A warp keeps RIF rows in flight (their loads are issued before any arithmetic), each held in registers:
// RIF x NV float4 per lane covers widths up to 128 * NV.
template <int RIF, int NV>
__device__ __forceinline__ void rmsnorm_rows(const NormArgs& a, const float* xbase, const float4* g4, const float4* b4,
                                             const float* mod, unsigned short* out, int r0, int nrows, int lane) {
  const int d4 = a.d >> 2;
  float4 v[RIF][NV];
#pragma unroll
  for (int q = 0; q < RIF; ++q) {
    const float4* x4 = reinterpret_cast<const float4*>(xbase + (size_t)(r0 + q) * a.ldx);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int i = lane + 32 * k;
      v[q][k] = (q < nrows && i < d4) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
#pragma unroll
  for (int q = 0; q < RIF; ++q) {
    if (q >= nrows) break;
    if (a.ln) {                                  // LayerNorm: centre the row first (two passes over registers)
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < NV; ++k) s += (v[q][k].x + v[q][k].y) + (v[q][k].z + v[q][k].w);
      const float mu = warp_sum(s) / (float)a.d;
#pragma unroll
      for (int k = 0; k < NV; ++k)
        if (lane + 32 * k < d4) { v[q][k].x -= mu; v[q][k].y -= mu; v[q][k].z -= mu; v[q][k].w -= mu; }
    }
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      ss = fmaf(v[q][k].x, v[q][k].x, ss); ss = fmaf(v[q][k].y, v[q][k].y, ss);
      ss = fmaf(v[q][k].z, v[q][k].z, ss); ss = fmaf(v[q][k].w, v[q][k].w, ss);
    }
    ss = warp_sum(ss);
    const float inv = 1.0f / sqrtf(ss / (float)a.d + 1e-6f);
    const int r = r0 + q;
    size_t orow = r, ocol0 = 0;
    if (a.shuffle > 1) {
      int y = r / a.grid, xx = r % a.grid, s = a.shuffle;
      orow = (size_t)(y / s) * (a.grid / s) + (xx / s);
      ocol0 = (size_t)((y % s) * s + (xx % s)) * a.d;
    }
    uint2* o2 = reinterpret_cast<uint2*>(out + orow * a.ldo + ocol0);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int i = lane + 32 * k;
      if (i >= d4) continue;
      const float4 t = v[q][k], gg = g4[i];
      float y0 = t.x * inv * gg.x, y1 = t.y * inv * gg.y, y2 = t.z * inv * gg.z, y3 = t.w * inv * gg.w;
      if (b4) {
        const float4 bb = b4[i];
        y0 += bb.x; y1 += bb.y; y2 += bb.z; y3 += bb.w;
      }
      if (mod) {
        float4 ga = reinterpret_cast<const float4*>(mod)[i], be = reinterpret_cast<const float4*>(mod + a.d)[i];
        y0 = y0 * (1.0f + ga.x) + be.x; y1 = y1 * (1.0f + ga.y) + be.y;
        y2 = y2 * (1.0f + ga.z) + be.z; y3 = y3 * (1.0f + ga.w) + be.w;
      }
      __nv_bfloat162 lo = __floats2bfloat162_rn(y0, y1), hi = __floats2bfloat162_rn(y2, y3);
      o2[i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    }
  }
}

__device__ void tile_rmsnorm(const TileCtx& c, const NormArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const float4* g4 = reinterpret_cast<const float4*>(resolve<const float>(c, a.g));
  const float4* b4 = reinterpret_cast<const float4*>(resolve<const float>(c, a.beta));
  const float* mod = resolve<const float>(c, a.mod);
  unsigned short* out = resolve<unsigned short>(c, a.out);
  const float* xbase = resolve<const float>(c, a.x);
  const int d4 = a.d >> 2;                      // widths are multiples of 4
  // this warp's rows: a contiguous share of the tile's rows
  const int per_warp = (a.rows_per_tile + 3) / 4;
  const int row_lo = tile * a.rows_per_tile + warp * per_warp;
  const int row_hi = min(min(row_lo + per_warp, (tile + 1) * a.rows_per_tile), a.M);
  if (d4 <= 128) {
    for (int r = row_lo; r < row_hi; r += 4) rmsnorm_rows<4, 4>(a, xbase, g4, b4, mod, out, r, min(4, row_hi - r), lane);
  } else if (d4 <= 256) {
    for (int r = row_lo; r < row_hi; r += 2) rmsnorm_rows<2, 8>(a, xbase, g4, b4, mod, out, r, min(2, row_hi - r), lane);
  } else if (d4 <= 512) {
    for (int r = row_lo; r < row_hi; ++r) rmsnorm_rows<1, 16>(a, xbase, g4, b4, mod, out, r, 1, lane);
  } else {
    // very wide rows: two passes through L2
    for (int r = row_lo; r < row_hi; ++r) {
      const float4* x4 = reinterpret_cast<const float4*>(xbase + (size_t)r * a.ldx);
      float ss = 0.f;
      for (int i = lane; i < d4; i += 32) {
        float4 t = __ldcg(x4 + i);
        ss = fmaf(t.x, t.x, ss); ss = fmaf(t.y, t.y, ss); ss = fmaf(t.z, t.z, ss); ss = fmaf(t.w, t.w, ss);
      }
      ss = warp_sum(ss);
      const float inv = 1.0f / sqrtf(ss / (float)a.d + 1e-6f);
      uint2* o2 = reinterpret_cast<uint2*>(out + (size_t)r * a.ldo);
      for (int i = lane; i < d4; i += 32) {
        const float4 t = __ldcg(x4 + i), gg = g4[i];
        float y0 = t.x * inv * gg.x, y1 = t.y * inv * gg.y, y2 = t.z * inv * gg.z, y3 = t.w * inv * gg.w;
        if (mod) {
          float4 ga = reinterpret_cast<const float4*>(mod)[i], be = reinterpret_cast<const float4*>(mod + a.d)[i];
          y0 = y0 * (1.0f + ga.x) + be.x; y1 = y1 * (1.0f + ga.y) + be.y;
          y2 = y2 * (1.0f + ga.z) + be.z; y3 = y3 * (1.0f + ga.w) + be.w;
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(y0, y1), hi = __floats2bfloat162_rn(y2, y3);
        o2[i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      }
    }
  }
}

// ------------------------------------------------------------------ elementwise tiles
__device__ void tile_patchify(const TileCtx& c, const PatchArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const float* img = resolve<const float>(c, a.img);
  unsigned short* obase = resolve<unsigned short>(c, a.out);
  const int P = a.patch, pk = 3 * P * P;
  for (int rr = warp; rr < a.rows_per_tile; rr += WORKER_THREADS / 32) {
    const int p = tile * a.rows_per_tile + rr;
    if (p >= a.grid * a.grid) break;
    unsigned short* out = obase + (size_t)p * a.ldo;
    const int py = p / a.grid, px = p % a.grid;
    for (int e = lane; e < pk; e += 32) {
      int ch = e / (P * P), rem = e % (P * P), yy = rem / P, xx = rem % P;
      float v = ld_act(img + ((size_t)ch * a.img_side + (py * P + yy)) * a.img_side + px * P + xx);
      out[e] = f32_to_bf16_bits(v);
    }
  }
}

__device__ void tile_embed(const TileCtx& c, const EmbedArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int* ids = resolve<const int>(c, a.ids);
  const unsigned short* table = resolve<const unsigned short>(c, a.table);
  const float* pos = resolve<const float>(c, a.pos);
  float* obase = resolve<float>(c, a.out);
  unsigned short* o16 = resolve<unsigned short>(c, a.out16);
  float* ss = resolve<float>(c, a.ss_out);
  for (int rr = warp; rr < a.rows_per_tile; rr += WORKER_THREADS / 32) {
    const int r = tile * a.rows_per_tile + rr;
    if (r >= a.n) break;
    int id = ld_act(ids + r);
    id = min(max(id, 0), a.vocab - 1);
    const unsigned short* row = table + (size_t)id * a.ldt;
    float* out = obase + (size_t)r * a.ldo;
    for (int b0 = 0; b0 < a.d; b0 += 128) {            // one 128-column block at a time (4 columns per lane)
      float sq = 0.f;
      for (int i = b0 + lane; i < min(b0 + 128, a.d); i += 32) {
        float v = bf16_bits_to_f32(row[i]);
        if (pos) v += pos[(size_t)r * a.d + i];
        out[i] = v;
        if (o16) o16[(size_t)r * a.ldo16 + i] = f32_to_bf16_bits(v);
        sq = fmaf(v, v, sq);
      }
      sq = warp_sum(sq);
      if (ss && lane == 0) ss[(size_t)r * a.ss_ld + (b0 >> 7)] = sq;
    }
  }
}

__device__ void tile_rope(const TileCtx& c, const RopeArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const float* ibase = resolve<const float>(c, a.in);
  unsigned short* obase = resolve<unsigned short>(c, a.out);
  unsigned short* outT = resolve<unsigned short>(c, a.outT);
  const int half = a.hd / 2;
  const float lnb = 9.210340371976184f;   // ln(10000)
  for (int rr = warp; rr < a.rows_per_tile; rr += WORKER_THREADS / 32) {
    const int r = tile * a.rows_per_tile + rr;
    if (r >= a.M) break;
    const float* in = ibase + (size_t)r * a.ld;
    unsigned short* out = obase + (size_t)r * a.ldo;
    const float pos = (float)(a.pos0 + r);
    for (int i = lane; i < half; i += 32) {
      float inv = expf(-lnb * (2.0f * (float)i) / (float)a.hd);
      float sn, cs;
      sincosf(pos * inv, &sn, &cs);
      for (int hh = 0; hh < a.n_rot_heads; ++hh) {
        float x1 = ld_act(in + hh * a.hd + i), x2 = ld_act(in + hh * a.hd + half + i);
        out[hh * a.hd + i] = f32_to_bf16_bits(x1 * cs - x2 * sn);
        out[hh * a.hd + half + i] = f32_to_bf16_bits(x2 * cs + x1 * sn);
      }
    }
    const int v0 = a.n_rot_heads * a.hd;
    for (int e = v0 + lane; e < a.n_heads * a.hd; e += 32) outT[(size_t)(e - v0) * a.ldoT + r] = f32_to_bf16_bits(ld_act(in + e));
  }
}

__device__ void tile_addrows(const TileCtx& c, const AddRowsArgs& a, int) {
  const float* in = resolve<const float>(c, a.in);
  const float* vec = resolve<const float>(c, a.vec);
  const float* tab = resolve<const float>(c, a.tab);
  float* out = resolve<float>(c, a.out);
  unsigned short* out16 = resolve<unsigned short>(c, a.out16);
  for (int e = c.tid; e < a.M * a.N; e += WORKER_THREADS) {
    int r = e / a.N, col = e % a.N;
    float v = ld_act(in + (size_t)r * a.ldi + col);
    if (vec) v += vec[col];
    if (tab) v += tab[(size_t)r * a.ldt + col];
    if (out) out[(size_t)r * a.ldo + col] = v;
    if (out16) out16[(size_t)r * a.ldo16 + col] = f32_to_bf16_bits(v);
  }
  float* ss = resolve<float>(c, a.ss_out);
  if (ss) {
    // per-row sums of squares of what was just written, one partial per 128 columns (one thread per partial)
    const int nb = (a.N + 127) / 128;
    for (int e = c.tid; e < a.M * nb; e += WORKER_THREADS) {
      const int r = e / nb, b0 = (e % nb) * 128;
      float sq = 0.f;
      for (int col = b0; col < min(b0 + 128, a.N); ++col) {
        float v = ld_act(in + (size_t)r * a.ldi + col);
        if (vec) v += vec[col];
        if (tab) v += tab[(size_t)r * a.ldt + col];
        sq = fmaf(v, v, sq);
      }
      ss[(size_t)r * a.ss_ld + (b0 >> 7)] = sq;
    }
  }
}

__device__ void tile_timeemb(const TileCtx& c, const TimeEmbArgs& a, int) {
  const float* args = resolve<const float>(c, a.args);
  unsigned short* out = resolve<unsigned short>(c, a.out);
  const int half = a.width / 2;
  const float lnb = 9.210340371976184f;
  for (int e = c.tid; e < a.M * half; e += WORKER_THREADS) {
    int m = e / half, i = e % half;
    float om = expf(-lnb * (float)i / (float)half);
    float sn, cs;
    sincosf(args[m] * om, &sn, &cs);
    out[(size_t)m * a.ldo + i] = f32_to_bf16_bits(sn);
    out[(size_t)m * a.ldo + half + i] = f32_to_bf16_bits(cs);
  }
}

// Copies the chunk to the host-visible ring, then publishes the frame id (system-scope fence between).
__device__ void tile_emit(const TileCtx& c, const EmitArgs& a, float* chunk_host, DoneRec* done, uint64_t frame, bool last) {
  const float* x = resolve<const float>(c, a.x);
  chunk_host += a.chunk_off;
  for (int e = c.tid; e < a.H * a.A; e += WORKER_THREADS) {
    int r = e / a.A, col = e % a.A;
    chunk_host[e] = ld_act(x + (size_t)r * a.ldx + col);
  }
  __threadfence_system();
  worker_sync(c);
  if (c.tid == 0 && last) {
    done->frame_plus1 = frame + 1;
    __threadfence_system();
  }
}

__device__ __forceinline__ void run_tile(const DeviceCtx& ctx, const TileCtx& c, const NodeDesc& n, int tile, int inst,
                                         uint64_t frame) {
  switch (n.op) {
    case OP_GEMM: tile_gemm(c, n.u.gemm, tile); break;
    case OP_RMSNORM: tile_rmsnorm(c, n.u.norm, tile); break;
    case OP_ATTN: tile_attention(c, n.u.attn, tile); break;
    case OP_PATCHIFY: tile_patchify(c, n.u.patch, tile); break;
    case OP_EMBED: tile_embed(c, n.u.embed, tile); break;
    case OP_ROPE: tile_rope(c, n.u.rope, tile); break;
    case OP_ADDROWS: tile_addrows(c, n.u.addrows, tile); break;
    case OP_TIMEEMB: tile_timeemb(c, n.u.timeemb, tile); break;
    case OP_EMIT:
    case OP_EMIT_PART:
      tile_emit(c, n.u.emit, ctx.chunk_host + (size_t)inst * ctx.chunk_elems, ctx.done_host + inst, frame, n.op == OP_EMIT);
      break;
    default:
      if (c.tid == 0) atomicCAS(c.error, 0u, (unsigned)DEV_ERR_BAD_OP);
  }
}

}  // namespace vla
