// Shared host/device data structures of the tile program and the dispatcher.
#pragma once
#include <stdint.h>

namespace vla {

// ---- operations a node can be (each node splits into n_tiles independent tiles)
enum Op : int32_t {
  OP_GEMM = 0,      // out = epilogue(A[M,K] * W[N,K]^T), bf16 operands, fp32 accumulate
  OP_RMSNORM = 1,   // bf16 out = rmsnorm(x fp32) * g (optionally * (1+gamma) + beta, optional pixel-shuffle scatter)
  OP_ATTN = 2,      // fused softmax(QK^T/sqrt(hd))V over up to two K/V segments
  OP_PATCHIFY = 3,  // image fp32 -> bf16 patch rows
  OP_EMBED = 4,     // text-embedding gather (+ position table) into the fp32 residual stream
  OP_ROPE = 5,      // fp32 q|k|v rows -> bf16 with rotary embedding on the q and k heads
  OP_ADDROWS = 6,   // out fp32 [M,N] = in fp32 (+ vec) (+ table)
  OP_TIMEEMB = 7,   // sinusoidal timestep embedding rows -> bf16
  OP_EMIT = 8,      // copy the finished chunk to the host-visible ring and publish its frame id
  OP_EMIT_PART = 9, // copy the chunk of one head pass to the host-visible ring (more passes of the frame follow)
  OP_COUNT = 10
};

enum Kind : int32_t { KIND_GEMM = 0, KIND_GEMM2 = 1, KIND_ATTN = 2, KIND_ELEM = 3 };   // GEMM2: two accumulators (gated MLP)
constexpr int N_KINDS = 4;
enum Phase : int32_t { PHASE_VLM = 0, PHASE_ACT = 1 };
constexpr int N_CLASSES = 8;  // phase * N_KINDS + kind: one queue per resource shape and stream

enum Act : int32_t { ACT_NONE = 0, ACT_GELU = 1, ACT_SILU = 2 };

// A device address inside the arena: byte offset, bit 63 set when relative to the
// frame slot (instance) base rather than the arena base.  0 = null.
typedef uint64_t Ref;
constexpr Ref REF_SLOT = 1ull << 63;
// Bit 62: one of the frame's input arrays (index in bits 56..59: 0 image, 1 text ids, 2 state, 3 noise),
// reached through the per-slot input pointer table so resident inputs are read in place.
constexpr Ref REF_INPUT = 1ull << 62;
constexpr int N_FRAME_INPUTS = 4;

constexpr int GEMM_BM = 128;   // output features per GEMM tile (the MMA M dimension)
constexpr int GEMM_BK = 64;    // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int WORKER_THREADS = 128;
constexpr int GEMM_MAX_BT = 128;     // most tokens per GEMM tile (MMA N)
constexpr int GEMM_SMEM_BUDGET = 64 * 1024;  // stage memory a token-rich GEMM tile aims for (at least two stages are always taken)
constexpr int GEMM_SMEM_BUDGET_SMALL = 84 * 1024;  // token-poor tiles (<= 64 tokens) are bound by TMA latency and get deeper
                                                   // pipelines, but must fit the room one finished token-rich tile leaves
                                                   // on an SM that runs three of them (3 x 18 of 55 four-KB units)
// TMA pipeline depth of a GEMM tile with `bt` tokens per tile (a 128-row weight tile plus the activation tile per stage).
inline int gemm_stage_bytes(int bt) { return GEMM_BM * GEMM_BK * 2 + bt * GEMM_BK * 2; }
inline int gemm_stages(int bt, int Kp) {
  const int stage = gemm_stage_bytes(bt);
  int S = (bt <= 64 ? GEMM_SMEM_BUDGET_SMALL : GEMM_SMEM_BUDGET) / stage;
  S = S < 2 ? 2 : (S > 4 ? 4 : S);
  const int nkb = Kp / GEMM_BK;
  return S < nkb ? S : (nkb < 1 ? 1 : nkb);
}
inline int gemm_smem_bytes(int bt, int S) {      // the epilogue parks the tile in the stage memory as fp32
  const int a = S * gemm_stage_bytes(bt), b = bt * GEMM_BM * 4;
  return a > b ? a : b;
}

// Shared memory of one attention tile: Q (128 rows), one K block and one V^T block of 64 keys,
// and the probability tile.  hs = head stride (head dim padded to a multiple of 16).
inline int attn_smem_bytes(int hs) {
  const int nbox = (hs + 63) / 64;
  return nbox * 128 * 128 + nbox * 64 * 128 + hs * 128 + 128 * 128;
}

// Query heads that share a KV head (grouped or multi-query attention) and have few queries are folded into the 128
// rows of one attention tile: the tile streams K and V^T once for all of them.  Returns heads per tile, sets rows per head.
inline int attn_fold(int tq, int hq, int hkv, int* rph) {
  const int group = hkv > 0 ? hq / hkv : 1;
  *rph = (tq + 7) / 8 * 8;
  if (tq > 64 || group < 2) return 1;
  const int fit = 128 / *rph;
  return fit < group ? fit : group;
}

struct GemmArgs {
  Ref A, W, W2;        // A bf16 [M,lda]; W (and W2 when dual) bf16 [N,Kp]
  Ref X;               // optional fp32 addend [M,ldx], scaled by c_x
  Ref vec;             // optional fp32 [N], broadcast over rows
  Ref tab, tab2;       // optional fp32 tables [M,ldtab] added row by row
  Ref out32, out16;    // fp32 and/or bf16 outputs [M,ld]
  Ref outT;            // optional transposed bf16 output: features >= t_col0 go to outT[f - t_col0][token]
  int32_t lda, ldx, ldtab, ldtab2, ldo32, ldo16, ldoT, t_col0;
  int32_t M, N, Kp;    // tokens, output features, padded reduction length (multiple of GEMM_BK)
  int32_t bt, tiles_t; // tokens per tile, number of token tiles
  int32_t act, dual;   // activation; dual (gated): out = act(A W^T) * (A W2^T), 64 output features per tile
  float c_acc, c_x;    // out = c_x * X + c_acc * acc + vec + tab + tab2
  int32_t wmap, w2map, amap;  // tensor-map indices: shared weight maps, activation map relative to the slot's first
  int32_t stages;             // TMA pipeline depth
  int32_t rs_d;               // > 0: A holds the raw residual stream (bf16) and RMSNorm is folded into the GEMM: every
                              // output row is scaled by 1/sqrt(sum_j ss_in[row][j] / rs_d + 1e-6)
  int32_t ss_nft, ss_out_ld, pad_;
  Ref ss_in;                  // fp32 [M, ss_nft]: per-row sums of squares of the stream, one partial per 128 columns
  Ref ss_out;                 // optional fp32 [M, ss_out_ld]: this tile writes the partial of its 128 output features
  Ref bias;                   // optional fp32 [N] added to the accumulator before the activation (not with dual)
};

struct NormArgs {
  Ref x, g, mod, out;  // x fp32 [M,ldx]; g fp32 [d]; mod fp32 [2d] (gamma;beta) or null; out bf16
  Ref beta;            // LayerNorm shift fp32 [d] (ln == 1)
  int32_t ln, pad_;    // 1: LayerNorm (subtract the row mean, biased variance, gain and shift) instead of RMSNorm
  int32_t M, d, ldx, ldo;
  int32_t rows_per_tile;
  int32_t shuffle, grid;   // shuffle s>1: row r=(y,x) of a grid x grid token map goes to row (y/s,x/s), column block (y%s,x%s)
};

struct AttnArgs {
  Ref out;                     // bf16 [tq, ldo], head h at columns h*hd
  int32_t qmap, k0map, v0map, k1map, v1map;   // activation tensor maps: Q and K [tokens, heads*hs], V^T [heads*hs, tokens]
  int32_t ldo;
  int32_t tq, t0, t1;          // queries; keys of segment 0 and segment 1
  int32_t hq, hkv, hd, hs;     // hs = head stride (hd padded to a multiple of 16)
  int32_t causal;
  int32_t bn, q_blocks;        // keys per block; 128-query blocks
  int32_t sfx, pad_;           // blocked suffix mask: queries [0, sfx) see only keys [0, sfx) of segment 1 (0 = no mask)
  int32_t hpt, rph;            // query heads folded into one tile (they share a KV head; 1 = none) and the rows each
                               // takes in the tile (tq rounded up to a multiple of 8); folding needs q_blocks == 1
  float scale_log2e;           // log2(e) / sqrt(hd)
};

struct PatchArgs {
  Ref img, out;        // img fp32 [3,H,W] of one camera; out bf16 [T,ldo]
  int32_t img_side, patch, grid, ldo, rows_per_tile;
};

struct EmbedArgs {
  Ref out16;                  // optional bf16 mirror of the output rows
  Ref ss_out;                 // optional fp32 [n, ss_ld] per-row sums of squares, one partial per 128 columns
  int32_t ldo16, ss_ld;
  Ref ids, table, pos, out;   // ids int32 [n]; table bf16 [vocab,d]; pos fp32 [n,d] or null; out fp32 rows
  int32_t n, d, ldo, vocab, rows_per_tile, ldt;
};

struct RopeArgs {
  Ref in, out, outT;   // in fp32 [M,ld]; out bf16 [M,ldo] (rotated q and k heads); outT bf16 [v features, ldoT] = V^T
  int32_t M, ld, ldo, ldoT, n_rot_heads, n_heads, hd, pos0, rows_per_tile;
};

struct AddRowsArgs {
  Ref in, vec, tab, out, out16;  // fp32; out16 optional bf16 copy
  Ref ss_out;                    // optional fp32 [M, ss_ld] per-row sums of squares, one partial per 128 columns
  int32_t M, N, ldi, ldt, ldo, ldo16, ss_ld, pad_;
};

struct TimeEmbArgs {
  Ref args, out;       // args fp32 [M] time arguments; out bf16 [M,ldo]
  int32_t M, width, ldo;
};

struct EmitArgs {
  Ref x;               // fp32 [H,ldx]
  int32_t H, A, ldx;
  int32_t chunk_off;   // first element of this pass's chunk inside the frame's host-visible chunk block
};

struct NodeDesc {
  int32_t op, cls, n_tiles, n_pred;
  int32_t succ_begin, succ_count;
  int32_t phase, step;
  int32_t smem_bytes, tmem_cols;
  int32_t pad0, pad1;
  union {
    GemmArgs gemm;
    NormArgs norm;
    AttnArgs attn;
    PatchArgs patch;
    EmbedArgs embed;
    RopeArgs rope;
    AddRowsArgs addrows;
    TimeEmbArgs timeemb;
    EmitArgs emit;
  } u;
};

// Per-class static description used by the pick.
struct ClassInfo {
  int32_t tau[3];       // (TC, ALU, MEM) intensity 0..15
  int32_t smem_units;   // largest shared-memory need of the class's tiles, in SMEM_UNIT chunks (a claim must fit this)
  int32_t tmem_units;   // largest tensor-memory need, in TMEM_UNIT column chunks
  int32_t group;        // pick group (the phase: tiles of one stream)
  int32_t pad[2];
};

constexpr int SMEM_UNIT = 4096;
constexpr int TMEM_UNIT = 32;

// A multi-producer multi-consumer ring of tile tickets (one per class).
struct TileQueue {             // one 128-byte line per queue
  unsigned long long head;     // next ticket to hand out
  unsigned long long tail;     // next ticket to reserve for a push
  long long avail;             // committed minus claimed (may dip below zero transiently)
  unsigned long long pad[13];
};

// One queued tile is one 64-bit word, written and read atomically:
//   bits 63..48 generation tag ((ticket / capacity + 1) & 0xFFFF; 0 = never written),
//   bits 47..32 tile index inside the node, bits 31..0 inst << 20 | node.
typedef unsigned long long QueueEntry;

struct AdmitRec {              // written by the host (copy stream), read by the dispatcher
  uint32_t inst;
  uint32_t pad;
  uint64_t frame;
};

struct TraceRec {              // mirrors vla_trace_rec
  uint32_t inst, node, tile;
  uint16_t sm;
  uint8_t worker, cls;
  uint64_t frame, t_start, t_end;
};

// Host-visible completion record per instance (mapped pinned memory).
struct DoneRec {
  volatile uint64_t frame_plus1;   // 0 = nothing yet
  uint64_t pad[7];
};

// Device-resident control block.
struct Control {                 // polled words and hot counters live on separate 128-byte lines
  unsigned int ctrl;             // bit 31 = exiting; low bits = frames in flight
  unsigned int error;            // sticky error code (0 = none)
  unsigned int error_info;
  unsigned int stop;             // host request to exit
  unsigned int pad0[28];
  unsigned long long admit_head; // admission records consumed
  unsigned long long admit_tail; // admission records published (written by host copies)
  unsigned long long pad1[14];
  unsigned long long doorbell;   // bumped whenever tiles are committed to any queue
  unsigned long long pad2[15];
  unsigned long long tiles_done;
  unsigned long long trace_count;
};

enum DevError : uint32_t {
  DEV_OK = 0, DEV_ERR_WAIT_QUEUE = 1, DEV_ERR_QUEUE_FULL = 2, DEV_ERR_WAIT_MBAR = 3, DEV_ERR_IDLE_LIMIT = 4,
  DEV_ERR_BAD_OP = 5
};

// Everything a kernel needs, passed by value.
// One successor edge as the retire path reads it: everything needed to release the node in one 16-byte load.
struct SuccInfo { int32_t node, n_tiles, cls_res, n_pred; };   // cls_res = class | resource units of one tile << 8

struct DeviceCtx {
  char* arena;
  const NodeDesc* nodes;
  const SuccInfo* succ;
  const ClassInfo* classes;
  Control* control;
  TileQueue* queues;             // [N_CLASSES]
  QueueEntry* q_entries;         // [N_CLASSES][q_capacity]
  AdmitRec* admit_ring;
  int32_t* dep_count;            // [n_inst][n_nodes]
  uint64_t* inst_frame;          // [n_inst] frame id currently owning the slot
  const uint64_t* slot_base;     // [n_inst] arena offset of the instance's buffers
  const uint64_t* input_ptrs;    // [n_inst][N_FRAME_INPUTS] device addresses of the frame's input arrays
  const int32_t* roots;          // nodes without predecessors
  TraceRec* trace;
  DoneRec* done_host;            // mapped pinned host memory, [n_inst]
  float* chunk_host;             // mapped pinned host memory, [n_inst][H*A]
  unsigned int* error_host;      // mapped pinned host memory
  const void* tmaps;             // CUtensorMap table (128 B each): weight maps, then n_act_tmaps per frame slot
  int32_t n_weight_tmaps, n_act_tmaps;
  int32_t n_nodes, n_inst, n_roots;
  int32_t q_capacity, q_shift, admit_capacity;   // q_capacity = 1 << q_shift
  uint32_t trace_capacity;
  int32_t policy, workers_per_sm;
  int32_t u_max, pad_u;     // saturation value of the utilisation counters in the pick's score
  uint64_t wait_limit_ns, idle_exit_ns;
  int32_t chunk_elems;
};

}  // namespace vla
