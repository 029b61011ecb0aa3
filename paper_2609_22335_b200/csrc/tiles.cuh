// Tile bodies.  Each body is executed by one worker group of WORKER_THREADS
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
  char* smem;           // this worker's shared-memory slab (16-byte aligned)
  uint32_t tmem;        // this worker's tensor-memory column base
  int tid;              // 0 .. WORKER_THREADS-1
  int bar_id;           // named barrier of this worker
  uint64_t deadline;    // %globaltimer value after which bounded waits give up
  unsigned int* error;  // sticky device error word
};

template <typename T>
__device__ __forceinline__ T* resolve(const TileCtx& c, Ref r) {
  if (r == 0) return nullptr;
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

__device__ __forceinline__ float gelu_tanh_f(float x) {
  const float c = 0.7978845608028654f;
  return 0.5f * x * (1.0f + tanhf(c * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + expf(-x)); }
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
  const float* X; const float* vec; const float* tab; const float* tab2;
  float* out32; unsigned short* out16;
};
__device__ __forceinline__ GemmPtrs gemm_ptrs(const TileCtx& c, const GemmArgs& g) {
  GemmPtrs p;
  p.X = resolve<const float>(c, g.X); p.vec = resolve<const float>(c, g.vec);
  p.tab = resolve<const float>(c, g.tab); p.tab2 = resolve<const float>(c, g.tab2);
  p.out32 = resolve<float>(c, g.out32); p.out16 = resolve<unsigned short>(c, g.out16);
  return p;
}
// out[r][f] = c_x X[r][f] + c_acc * (act(acc) [* acc2]) + vec[f] + tab[r][f] + tab2[r][f]
__device__ __forceinline__ void gemm_store(const GemmArgs& g, const GemmPtrs& p, int r, int f, float acc, float acc2) {
  float v = apply_act(g.act, acc);
  if (g.dual) v *= acc2;
  v *= g.c_acc;
  if (p.X) v += g.c_x * ld_act(p.X + (size_t)r * g.ldx + f);
  if (p.vec) v += p.vec[f];
  if (p.tab) v += p.tab[(size_t)r * g.ldtab + f];
  if (p.tab2) v += p.tab2[(size_t)r * g.ldtab2 + f];
  if (p.out32) p.out32[(size_t)r * g.ldo32 + f] = v;
  if (p.out16) p.out16[(size_t)r * g.ldo16 + f] = f32_to_bf16_bits(v);
}

// ------------------------------------------------------------------ GEMM tile
// Thread t owns output feature f0+t; tokens are the accumulator columns.
__device__ __forceinline__ void gemm_accumulate(const TileCtx& c, const GemmArgs& g, const unsigned short* W,
                                                const unsigned short* A, int f0, int t0, int c0, int nt, float* Ws,
                                                float* As, float (&acc)[GEMM_TOK_CHUNK]) {
  constexpr int WS_LD = GEMM_BK + 4;
  for (int k0 = 0; k0 < g.Kp; k0 += GEMM_BK) {
    worker_sync(c);
    // weights tile: GEMM_BM rows x GEMM_BK, 16-byte vectors, rows beyond N read as zero
    for (int v = c.tid; v < GEMM_BM * (GEMM_BK / 8); v += WORKER_THREADS) {
      int row = v / (GEMM_BK / 8), cv = v % (GEMM_BK / 8);
      float w8[8];
      if (f0 + row < g.N) {
        uint4 raw = *reinterpret_cast<const uint4*>(W + (size_t)(f0 + row) * g.Kp + k0 + cv * 8);
        unpack8(raw, w8);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) w8[i] = 0.f;
      }
      float* dst = Ws + row * WS_LD + cv * 8;
      *reinterpret_cast<float4*>(dst) = make_float4(w8[0], w8[1], w8[2], w8[3]);
      *reinterpret_cast<float4*>(dst + 4) = make_float4(w8[4], w8[5], w8[6], w8[7]);
    }
    for (int v = c.tid; v < GEMM_TOK_CHUNK * (GEMM_BK / 8); v += WORKER_THREADS) {
      int row = v / (GEMM_BK / 8), cv = v % (GEMM_BK / 8);
      float a8[8];
      int r = t0 + c0 + row;
      if (c0 + row < nt) {
        uint4 raw = ld_act(reinterpret_cast<const uint4*>(A + (size_t)r * g.lda + k0 + cv * 8));
        unpack8(raw, a8);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) a8[i] = 0.f;
      }
      float* dst = As + row * GEMM_BK + cv * 8;
      *reinterpret_cast<float4*>(dst) = make_float4(a8[0], a8[1], a8[2], a8[3]);
      *reinterpret_cast<float4*>(dst + 4) = make_float4(a8[4], a8[5], a8[6], a8[7]);
    }
    worker_sync(c);
    const float* wrow = Ws + c.tid * WS_LD;
#pragma unroll 2
    for (int kk = 0; kk < GEMM_BK; kk += 4) {
      float4 w4 = *reinterpret_cast<const float4*>(wrow + kk);
#pragma unroll
      for (int t = 0; t < GEMM_TOK_CHUNK; ++t) {
        float4 a4 = *reinterpret_cast<const float4*>(As + t * GEMM_BK + kk);
        float s = acc[t];
        s = fmaf(w4.x, a4.x, s); s = fmaf(w4.y, a4.y, s); s = fmaf(w4.z, a4.z, s); s = fmaf(w4.w, a4.w, s);
        acc[t] = s;
      }
    }
  }
}

__device__ void tile_gemm(const TileCtx& c, const GemmArgs& g, int tile) {
  const int ft = tile / g.tiles_t, tt = tile % g.tiles_t;
  const int f0 = ft * GEMM_BM, t0 = tt * g.bt;
  const int nt = min(g.bt, g.M - t0);
  const int f = f0 + c.tid;
  const unsigned short* A = resolve<const unsigned short>(c, g.A);
  const unsigned short* W = resolve<const unsigned short>(c, g.W);
  const unsigned short* W2 = resolve<const unsigned short>(c, g.W2);
  GemmPtrs ptrs = gemm_ptrs(c, g);
  float* Ws = reinterpret_cast<float*>(c.smem);                 // [GEMM_BM][GEMM_BK+4]
  float* As = Ws + GEMM_BM * (GEMM_BK + 4);                     // [GEMM_TOK_CHUNK][GEMM_BK]
  for (int c0 = 0; c0 < nt; c0 += GEMM_TOK_CHUNK) {
    float acc[GEMM_TOK_CHUNK], acc2[GEMM_TOK_CHUNK];
#pragma unroll
    for (int i = 0; i < GEMM_TOK_CHUNK; ++i) { acc[i] = 0.f; acc2[i] = 0.f; }
    gemm_accumulate(c, g, W, A, f0, t0, c0, nt, Ws, As, acc);
    if (g.dual) gemm_accumulate(c, g, W2, A, f0, t0, c0, nt, Ws, As, acc2);
    if (f < g.N) {
#pragma unroll
      for (int t = 0; t < GEMM_TOK_CHUNK; ++t)
        if (c0 + t < nt) gemm_store(g, ptrs, t0 + c0 + t, f, acc[t], acc2[t]);
    }
  }
}

// ------------------------------------------------------------------ RMSNorm tile (one warp per row)
__device__ void tile_rmsnorm(const TileCtx& c, const NormArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int r = tile * a.rows_per_tile + warp;
  if (warp >= a.rows_per_tile || r >= a.M) return;
  const float* x = resolve<const float>(c, a.x) + (size_t)r * a.ldx;
  const float* g = resolve<const float>(c, a.g);
  const float* mod = resolve<const float>(c, a.mod);
  unsigned short* out = resolve<unsigned short>(c, a.out);
  float ss = 0.f;
  for (int i = lane; i < a.d; i += 32) { float v = ld_act(x + i); ss = fmaf(v, v, ss); }
  ss = warp_sum(ss);
  const float inv = 1.0f / sqrtf(ss / (float)a.d + 1e-6f);
  size_t orow = r, ocol0 = 0;
  if (a.shuffle > 1) {
    int y = r / a.grid, xx = r % a.grid, s = a.shuffle;
    orow = (size_t)(y / s) * (a.grid / s) + (xx / s);
    ocol0 = (size_t)((y % s) * s + (xx % s)) * a.d;
  }
  unsigned short* o = out + orow * a.ldo + ocol0;
  for (int i = lane; i < a.d; i += 32) {
    float v = ld_act(x + i) * inv * g[i];
    if (mod) v = v * (1.0f + mod[i]) + mod[a.d + i];
    o[i] = f32_to_bf16_bits(v);
  }
}

// ------------------------------------------------------------------ attention tile
// One tile = one query head x bq queries; each warp walks its queries one at a time:
// scores for all keys (lanes over keys), softmax in fp32, then P.V (lanes over head dims).
__device__ void tile_attention(const TileCtx& c, const AttnArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int head = tile / a.q_blocks, qb = tile % a.q_blocks;
  const int g = (head * a.hkv) / a.hq;
  const int tkv = a.t0 + a.t1;
  const unsigned short* Q = resolve<const unsigned short>(c, a.q);
  const unsigned short* K0 = resolve<const unsigned short>(c, a.k0);
  const unsigned short* V0 = resolve<const unsigned short>(c, a.v0);
  const unsigned short* K1 = resolve<const unsigned short>(c, a.k1);
  const unsigned short* V1 = resolve<const unsigned short>(c, a.v1);
  unsigned short* O = resolve<unsigned short>(c, a.out);
  float* qv = reinterpret_cast<float*>(c.smem) + warp * (a.hd + tkv);
  float* sc = qv + a.hd;
  const int per_warp = a.bq / 4;
  for (int qi = 0; qi < per_warp; ++qi) {
    const int q = qb * a.bq + warp * per_warp + qi;
    if (q >= a.tq) break;
    __syncwarp();
    for (int i = lane; i < a.hd; i += 32) qv[i] = bf16_bits_to_f32(ld_act(Q + (size_t)q * a.ldq + head * a.hd + i));
    __syncwarp();
    const int nk = a.causal ? (q + 1) : tkv;
    float mx = -INFINITY;
    for (int j = lane; j < nk; j += 32) {
      const unsigned short* kr = j < a.t0 ? (K0 + (size_t)j * a.ldk0 + g * a.hd) : (K1 + (size_t)(j - a.t0) * a.ldk1 + g * a.hd);
      float s = 0.f;
      for (int d0 = 0; d0 < a.hd; d0 += 8) {
        float k8[8];
        unpack8(ld_act(reinterpret_cast<const uint4*>(kr + d0)), k8);
#pragma unroll
        for (int i = 0; i < 8; ++i) s = fmaf(qv[d0 + i], k8[i], s);
      }
      s *= a.scale;
      sc[j] = s;
      mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < nk; j += 32) {
      float p = expf(sc[j] - mx);
      sc[j] = p;
      sum += p;
    }
    sum = warp_sum(sum);
    __syncwarp();
    const float inv = 1.0f / sum;
    for (int d0 = lane; d0 < a.hd; d0 += 32) {
      float o = 0.f;
      for (int j = 0; j < nk; ++j) {
        const unsigned short* vr = j < a.t0 ? (V0 + (size_t)j * a.ldk0 + g * a.hd) : (V1 + (size_t)(j - a.t0) * a.ldk1 + g * a.hd);
        o = fmaf(sc[j], bf16_bits_to_f32(ld_act(vr + d0)), o);
      }
      O[(size_t)q * a.ldo + head * a.hd + d0] = f32_to_bf16_bits(o * inv);
    }
  }
}

// ------------------------------------------------------------------ elementwise tiles
__device__ void tile_patchify(const TileCtx& c, const PatchArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int p = tile * a.rows_per_tile + warp;
  if (warp >= a.rows_per_tile || p >= a.grid * a.grid) return;
  const float* img = resolve<const float>(c, a.img);
  unsigned short* out = resolve<unsigned short>(c, a.out) + (size_t)p * a.ldo;
  const int py = p / a.grid, px = p % a.grid, P = a.patch, pk = 3 * P * P;
  for (int e = lane; e < pk; e += 32) {
    int ch = e / (P * P), rem = e % (P * P), yy = rem / P, xx = rem % P;
    float v = ld_act(img + ((size_t)ch * a.img_side + (py * P + yy)) * a.img_side + px * P + xx);
    out[e] = f32_to_bf16_bits(v);
  }
}

__device__ void tile_embed(const TileCtx& c, const EmbedArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int r = tile * a.rows_per_tile + warp;
  if (warp >= a.rows_per_tile || r >= a.n) return;
  int id = ld_act(resolve<const int>(c, a.ids) + r);
  id = min(max(id, 0), a.vocab - 1);
  const unsigned short* row = resolve<const unsigned short>(c, a.table) + (size_t)id * a.ldt;
  const float* pos = resolve<const float>(c, a.pos);
  float* out = resolve<float>(c, a.out) + (size_t)r * a.ldo;
  for (int i = lane; i < a.d; i += 32) {
    float v = bf16_bits_to_f32(row[i]);
    if (pos) v += pos[(size_t)r * a.d + i];
    out[i] = v;
  }
}

__device__ void tile_rope(const TileCtx& c, const RopeArgs& a, int tile) {
  const int warp = c.tid >> 5, lane = c.tid & 31;
  const int r = tile * a.rows_per_tile + warp;
  if (warp >= a.rows_per_tile || r >= a.M) return;
  const float* in = resolve<const float>(c, a.in) + (size_t)r * a.ld;
  unsigned short* out = resolve<unsigned short>(c, a.out) + (size_t)r * a.ld;
  const int half = a.hd / 2;
  const float pos = (float)(a.pos0 + r);
  const float lnb = 9.210340371976184f;   // ln(10000)
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
  for (int e = a.n_rot_heads * a.hd + lane; e < a.n_heads * a.hd; e += 32) out[e] = f32_to_bf16_bits(ld_act(in + e));
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
__device__ void tile_emit(const TileCtx& c, const EmitArgs& a, float* chunk_host, DoneRec* done, uint64_t frame) {
  const float* x = resolve<const float>(c, a.x);
  for (int e = c.tid; e < a.H * a.A; e += WORKER_THREADS) {
    int r = e / a.A, col = e % a.A;
    chunk_host[e] = ld_act(x + (size_t)r * a.ldx + col);
  }
  __threadfence_system();
  worker_sync(c);
  if (c.tid == 0) {
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
      tile_emit(c, n.u.emit, ctx.chunk_host + (size_t)inst * ctx.chunk_elems, ctx.done_host + inst, frame);
      break;
    default:
      if (c.tid == 0) atomicCAS(c.error, 0u, (unsigned)DEV_ERR_BAD_OP);
  }
}

}  // namespace vla
