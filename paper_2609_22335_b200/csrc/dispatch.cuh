// Device side of the dispatcher: tile queues, dependency counters, the persistent
// co-scheduling kernel, and the ordinary-kernel wrapper used by the stream modes.
#pragma once
#include "pick.cuh"
#include "tiles.cuh"

namespace vla {

constexpr unsigned CTRL_EXITING = 0x80000000u;
constexpr uint32_t TRACE_ADMIT_NODE = 0xFFFFFFFFu;   // node id of the trace record that marks a frame's admission
constexpr int MAX_WORKERS = 3;
constexpr int SM_CTL_BYTES = 1024;       // per-worker control block (mbarriers, row scales) handed to the tile bodies
constexpr int SM_STATE_BASE = 2048;      // dispatcher state of the SM
constexpr int SM_STATE_BYTES = SM_STATE_BASE + MAX_WORKERS * SM_CTL_BYTES;   // then the tile slab, 1024-byte aligned

__device__ __forceinline__ uint64_t gtimer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned smid() {
  unsigned s;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(s));
  return s;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_volatile_u32(const unsigned* p) { return *reinterpret_cast<const volatile unsigned*>(p); }
__device__ __forceinline__ unsigned long long ld_volatile_u64(const unsigned long long* p) {
  return *reinterpret_cast<const volatile unsigned long long*>(p);
}
__device__ __forceinline__ long long ld_volatile_s64(const long long* p) { return *reinterpret_cast<const volatile long long*>(p); }

__device__ __forceinline__ void set_error(const DeviceCtx& ctx, unsigned code, unsigned info) {
  if (atomicCAS(&ctx.control->error, 0u, code) == 0u) {
    ctx.control->error_info = info;
    *ctx.error_host = code;
    __threadfence_system();
  }
}

// ------------------------------------------------------------------ doorbells inside an SM
// The service warps and idle workers must not spin: every instruction they issue is taken from the worker warps that
// share their scheduler (a claim loop polling flat out cost the tile bodies 10-40 % of their speed).  They wait on
// an mbarrier instead -- suspended by the hardware, no issue slots -- which whoever has news for them rings; the
// wait is bounded by a time hint, so a lost ring (two rings inside one phase look like none) only delays, never hangs.
__device__ __forceinline__ void bell_ring(const void* bell) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bell)) : "memory");
}
// Returns when the bell was rung since the last successful wait or, at the latest, after about `hint_ns`.
__device__ __forceinline__ bool bell_wait(const void* bell, uint32_t& parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bell)), "r"(parity), "r"(hint_ns)
      : "memory");
  if (ok) parity ^= 1u;
  return ok != 0;
}

// ------------------------------------------------------------------ tensor memory (whole-warp calls)
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// ------------------------------------------------------------------ tile queues
// Pushing tiles is split in three so a whole warp can fill the entries in parallel:
// reserve (one thread), fill (any threads, entry i of the range), commit (one thread, after a barrier).
// The ring is sized for every tile of every frame slot, so a reservation can never overrun the head.
// One entry = one 64-bit word: generation (12 bits, never 0 for a written entry of the current lap... the lap count + 1)
// | node (20) | frame slot (9) | tile (12) | and the node's per-tile resource need in units so that a claim needs no
// second load: shared memory (6) and tensor memory (5).
constexpr int QW_NODE_BITS = 20, QW_INST_BITS = 9, QW_TILE_BITS = 12, QW_SMEM_BITS = 6, QW_TMEM_BITS = 5, QW_GEN_BITS = 12;
static_assert(QW_NODE_BITS + QW_INST_BITS + QW_TILE_BITS + QW_SMEM_BITS + QW_TMEM_BITS + QW_GEN_BITS == 64, "queue word layout");
__device__ __forceinline__ unsigned long long queue_gen(const DeviceCtx& ctx, unsigned long long ticket) {
  return ((ticket >> ctx.q_shift) + 1ull) & ((1ull << QW_GEN_BITS) - 1ull);
}
__device__ __forceinline__ unsigned long long queue_word(const DeviceCtx& ctx, unsigned long long ticket, uint32_t inst,
                                                         uint32_t node, uint32_t tile, uint32_t res_units) {
  // res_units = smem units | tmem units << QW_SMEM_BITS
  return (queue_gen(ctx, ticket) << (64 - QW_GEN_BITS)) | ((unsigned long long)res_units << (QW_NODE_BITS + QW_INST_BITS + QW_TILE_BITS)) |
         ((unsigned long long)tile << (QW_NODE_BITS + QW_INST_BITS)) | ((unsigned long long)inst << QW_NODE_BITS) | (unsigned long long)node;
}
__device__ inline unsigned long long queue_reserve(const DeviceCtx& ctx, int cls, int n) {
  return atomicAdd(&ctx.queues[cls].tail, (unsigned long long)n);
}
// Ordering: a consumer may pop a ticket before that ticket's own commit (`avail` counts anybody's commits) and then
// waits for the entry's generation tag with an acquire load.  So the entry store itself must publish everything the
// producer has observed: every filling thread issues a device-scope fence before its (relaxed) entry stores
// -- queue_fill_fence() -- and the thread that watched the dependency counter reach zero fences after that atomic.
// The commit carries no ordering duty of its own.
__device__ __forceinline__ void queue_fill_fence() { __threadfence(); }
__device__ inline void queue_fill(const DeviceCtx& ctx, int cls, unsigned long long base, uint32_t inst, uint32_t node,
                                  uint32_t res_units, int first, int count, int stride) {
  const unsigned long long mask = (unsigned long long)ctx.q_capacity - 1;
  QueueEntry* ent = ctx.q_entries + (size_t)cls * ctx.q_capacity;
  for (int i = first; i < count; i += stride)
    *reinterpret_cast<volatile unsigned long long*>(ent + ((base + i) & mask)) = queue_word(ctx, base + i, inst, node, (uint32_t)i, res_units);
}
__device__ inline void queue_commit(const DeviceCtx& ctx, int cls, int n) {
  atomicAdd(reinterpret_cast<unsigned long long*>(&ctx.queues[cls].avail), (unsigned long long)n);
}
// One thread pushes everything (admission of a frame's root tiles).
__device__ __forceinline__ uint32_t node_res_units(const NodeDesc& nd) {
  return (uint32_t)((__ldg(&nd.smem_bytes) + SMEM_UNIT - 1) / SMEM_UNIT) |
         ((uint32_t)((__ldg(&nd.tmem_cols) + TMEM_UNIT - 1) / TMEM_UNIT) << QW_SMEM_BITS);
}
__device__ inline void queue_push(const DeviceCtx& ctx, int cls, uint32_t inst, uint32_t node, int n) {
  const unsigned long long base = queue_reserve(ctx, cls, n);
  queue_fill_fence();
  queue_fill(ctx, cls, base, inst, node, node_res_units(ctx.nodes[node]), 0, n, 1);
  queue_commit(ctx, cls, n);
}

// Claim one tile if any is committed.  Bounded wait for the claimed ticket's entry to land.
__device__ inline bool queue_try_pop(const DeviceCtx& ctx, int cls, QueueEntry& e, uint64_t deadline) {
  TileQueue* q = ctx.queues + cls;
  long long old = (long long)atomicAdd(reinterpret_cast<unsigned long long*>(&q->avail), (unsigned long long)(-1LL));
  if (old <= 0) {
    atomicAdd(reinterpret_cast<unsigned long long*>(&q->avail), 1ull);
    return false;
  }
  const unsigned long long t = atomicAdd(&q->head, 1ull);
  const unsigned long long mask = (unsigned long long)ctx.q_capacity - 1;
  const unsigned long long want = queue_gen(ctx, t);
  const unsigned long long* slot = ctx.q_entries + (size_t)cls * ctx.q_capacity + (t & mask);
  unsigned spins = 0;
  unsigned long long w;
  while (((w = ld_acquire_u64(slot)) >> (64 - QW_GEN_BITS)) != want) {
    if ((++spins & 63u) == 0 && gtimer() > deadline) {
      set_error(ctx, DEV_ERR_WAIT_QUEUE, cls);
      return false;
    }
  }
  e = w;
  return true;
}

// ------------------------------------------------------------------ per-SM state of the persistent kernel
constexpr int MAX_READY = 6;
constexpr int DISPATCH_THREADS = 64;     // two service warps per SM (claim, retire), after the worker groups
constexpr long long PRIO_WINDOW_NS = 8000;   // an action-head tile may be claimed for a worker this close to the end of its tile
constexpr int PREFETCH_MIN_TOTAL = 600;   // tiles are claimed ahead of need only while this many VLM tiles are queued in all
constexpr int PREFETCH_MIN_AVAIL = 8;     // ... and only from queues at least this deep
constexpr int HELD_DEPTH = 1;            // claimed tiles a worker may have waiting
constexpr unsigned CLAIM_NAP_NS = 60, CLAIM_NAP_MAX_NS = 240;   // claim warp, while a worker of its SM has nothing to run
constexpr unsigned CLAIM_SLEEP_NS = 2000;    // claim warp, every worker busy: longest sleep without a ring
constexpr unsigned RETIRE_SLEEP_NS = 4000;   // retire warp: longest sleep without a ring
constexpr unsigned long long HEAD_WAIT_NS = 1500;   // an action-head tile nobody took for this long may go to a running worker

struct ReadyItem {
  unsigned long long base;   // reserved queue range
  uint32_t node, res_units;
  int n_tiles, cls;
};

struct WorkerTile {
  uint32_t inst, node, tile;
  int cls;
  int smem_unit0, smem_units, tmem_unit0, tmem_units;
  int succ_begin, succ_count, op, pad_;     // of the tile's node, filled in by the worker for the retire warp
  uint64_t t0, t1, frame;
};

// Mailboxes between one worker group and the SM's dispatcher warp (all in shared memory).
struct WorkerSlot {
  volatile unsigned held_tail;   // claimed tiles pushed by the claim warp (single producer)
  volatile unsigned held_head;   // claimed tiles taken by the worker (single consumer)
  volatile int leave;            // claim warp -> worker: go home
  volatile int done_state;       // 0 empty, 1 finished tile posted for the retire warp
  volatile int busy;             // the worker is running a tile (set and cleared by the worker)
  int pad_;
  volatile unsigned prio_tail, prio_head;   // one-deep slot for an action-head tile that goes ahead of the held VLM tiles
  volatile unsigned long long t_busy;       // when the running tile was taken (worker), for the claim warp's estimate of its end
  WorkerTile done, fin, held[HELD_DEPTH], prio;
  int n_ready;
  ReadyItem ready[MAX_READY];
};

struct SmState {
  unsigned long long smem_mask;    // bit i set = shared-memory unit i in use
  unsigned tmem_mask;              // bit i set = tensor-memory unit i in use
  int n_smem_units, n_tmem_units;
  PickState pick;
  unsigned tmem_base;
  volatile int quit;               // claim warp -> retire warp: everyone is leaving
  int smem_promised, tmem_promised;  // units of tiles handed to free workers that have not allocated them yet
  unsigned room_wait;              // a worker waiting for room right now: smem units | tmem units << 8 | (worker + 1) << 16, else 0
                                   // (the latest one when two wait); the claim warp keeps that room out of its offers
  volatile int ema_ns[N_CLASSES];  // running mean of tile durations per class on this SM (retire warp)
  int tau_tab[N_CLASSES * 3];      // the classes' intensity tags (read by the workers when a tile ends)
  unsigned long long bell_claim;   // rung by a worker that took a claimed tile or ran out of work
  unsigned long long bell_retire;  // rung by a worker that posted a finished tile
  unsigned long long bell_worker[MAX_WORKERS];   // rung by the claim warp when it hands worker w a tile or sends it home
  WorkerTile cur[MAX_WORKERS];     // the tile each worker is running (written by its leader)
  WorkerSlot slot[MAX_WORKERS];
};
static_assert(sizeof(SmState) <= SM_STATE_BASE, "SM state too large");

__device__ __forceinline__ unsigned long long unit_bits(int n) { return n >= 64 ? ~0ull : ((1ull << n) - 1ull); }
// Lowest position of `need` consecutive free units among the first `total` (bit set = in use), or -1.
// run keeps the positions where k consecutive free units start; k doubles until it reaches `need`.
__device__ __forceinline__ int find_free(unsigned long long mask, int need, int total) {
  if (need == 0) return 0;
  if (need > total) return -1;
  unsigned long long run = ~mask & unit_bits(total);
  for (int k = 1; k < need;) {
    const int step = min(k, need - k);
    run &= run >> step;
    k += step;
  }
  return run ? __ffsll((long long)run) - 1 : -1;
}

__device__ inline void write_trace(const DeviceCtx& ctx, uint32_t inst, uint32_t node, uint32_t tile, int worker, int cls,
                                   uint64_t frame, uint64_t t0, uint64_t t1) {
  if (ctx.trace_capacity == 0) return;
  unsigned long long idx = atomicAdd(&ctx.control->trace_count, 1ull);
  if (idx >= ctx.trace_capacity) return;
  TraceRec r;
  r.inst = inst; r.node = node; r.tile = tile; r.sm = (uint16_t)smid(); r.worker = (uint8_t)worker; r.cls = (uint8_t)cls;
  r.frame = frame; r.t_start = t0; r.t_end = t1;
  ctx.trace[idx] = r;
}

// A frame became ready (its inputs are in HBM): take its admission record and queue its root tiles.
__device__ inline void try_admit(const DeviceCtx& ctx) {
  Control* ctl = ctx.control;
  const unsigned long long head = ld_volatile_u64(&ctl->admit_head);
  const unsigned long long tail = ld_volatile_u64(&ctl->admit_tail);
  if (head >= tail) return;
  unsigned old = ld_volatile_u32(&ctl->ctrl);
  for (int tries = 0; tries < 8; ++tries) {
    if (old & CTRL_EXITING) return;
    unsigned prev = atomicCAS(&ctl->ctrl, old, old + 1u);
    if (prev == old) { old = 0xffffffffu; break; }
    old = prev;
  }
  if (old != 0xffffffffu) return;
  if (atomicCAS(&ctl->admit_head, head, head + 1ull) != head) {
    atomicSub(&ctl->ctrl, 1u);
    return;
  }
  const volatile AdmitRec* rec = ctx.admit_ring + (head & (unsigned long long)(ctx.admit_capacity - 1));
  const uint32_t inst = rec->inst;
  const uint64_t frame = rec->frame;
  *reinterpret_cast<volatile uint64_t*>(ctx.inst_frame + inst) = frame;
  {   // the frame's admission is a trace record of its own (node = TRACE_ADMIT_NODE): no tile of the frame may start earlier
    const uint64_t now = gtimer();
    write_trace(ctx, inst, TRACE_ADMIT_NODE, 0, 0, 0xFF, frame, now, now);
  }
  __threadfence();
  for (int i = 0; i < ctx.n_roots; ++i) {
    int r = ctx.roots[i];
    queue_push(ctx, ctx.nodes[r].cls, inst, (uint32_t)r, ctx.nodes[r].n_tiles);
  }
}

// Global side of a finished tile: every successor node's counter (which counts its predecessors' tiles)
// goes down by one; a counter reaching zero re-arms itself and releases that node, whose queue range is
// reserved here and returned in `slot` for the warp to fill.
__device__ inline void complete_tile(const DeviceCtx& ctx, const WorkerTile& f, WorkerSlot* slot) {
  const uint32_t inst = f.inst;
  slot->n_ready = 0;
  __threadfence();
  const int n_succ = f.succ_count, succ0 = f.succ_begin;      // carried by the tile's record: no load of its node here
  for (int i0 = 0; i0 < n_succ; i0 += 4) {
    // up to four successors per pass: one 16-byte load each, then their counters are decremented by independent
    // atomics in flight together
    SuccInfo si[4];
    int left[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      si[j].node = -1;
      if (i0 + j < n_succ) {
        const int4 v = __ldg(reinterpret_cast<const int4*>(ctx.succ + succ0 + i0 + j));
        si[j].node = v.x; si[j].n_tiles = v.y; si[j].cls_res = v.z; si[j].n_pred = v.w;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) left[j] = si[j].node >= 0 ? atomicSub(ctx.dep_count + (size_t)inst * ctx.n_nodes + si[j].node, 1) - 1 : 1;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (left[j] != 0) continue;
      ctx.dep_count[(size_t)inst * ctx.n_nodes + si[j].node] = si[j].n_pred;
      const int s_cls = si[j].cls_res & 0xFF;
      const uint32_t s_res = (uint32_t)si[j].cls_res >> 8;
      if (slot->n_ready < MAX_READY) {
        ReadyItem& it = slot->ready[slot->n_ready++];
        it.base = queue_reserve(ctx, s_cls, si[j].n_tiles);
        it.node = (uint32_t)si[j].node; it.n_tiles = si[j].n_tiles; it.cls = s_cls;
        it.res_units = s_res;
      } else {
        queue_push(ctx, s_cls, inst, (uint32_t)si[j].node, si[j].n_tiles);
      }
    }
  }
  if (slot->n_ready > 0) __threadfence();   // acquire side of the counters just read, before the entries are published
  if (f.op == OP_EMIT) atomicSub(&ctx.control->ctrl, 1u);
}

// u[x] += sign * tau[cls][x] on the SM's utilisation counters, with `cls` known only at run time: the class is matched
// against loop-constant positions so that the tag table stays in registers.
__device__ __forceinline__ void tau_add(int* u, const int* tau, int cls, int sign) {
  int t0 = 0, t1 = 0, t2 = 0;
#pragma unroll
  for (int c = 0; c < N_CLASSES; ++c)
    if (c == cls) { t0 = tau[c * 3]; t1 = tau[c * 3 + 1]; t2 = tau[c * 3 + 2]; }
  atomicAdd(u + 0, sign * t0); atomicAdd(u + 1, sign * t1); atomicAdd(u + 2, sign * t2);
}

// ------------------------------------------------------------------ the two service warps of an SM
// Workers never touch global queues or counters.  Two extra warps per SM do it for them, so those
// round trips overlap tile execution instead of sitting between tiles:
//   * the CLAIM warp (lane w serves worker w) claims tiles under the pick policy -- for a busy worker one
//     tile ahead -- and hands a claimed tile over as soon as its worker is free and its exact
//     shared/tensor-memory need fits;
//   * the RETIRE warp (lane w serves worker w) takes a finished tile, frees its memory at once, then does
//     the global bookkeeping (node counter, successors' dependency counters, queue pushes; the whole warp
//     fills the released successors' entries).
// Per-SM state is shared-memory words updated with shared-memory atomics by these two warps only.
__device__ inline void retire_loop(const DeviceCtx& ctx, SmState* sm, int n_workers) {
  const int lane = threadIdx.x & 31;
  const bool serving = lane < n_workers;
  WorkerSlot* slot = sm->slot + (serving ? lane : 0);
  uint32_t bell_parity = 0;
  for (;;) {
    bool have_fin = false;
    if (serving && slot->done_state == 1) {
      slot->fin = slot->done;
      __threadfence_block();
      slot->done_state = 0;
      have_fin = true;
      const WorkerTile& f = slot->fin;
      sm->ema_ns[f.cls] = (3 * sm->ema_ns[f.cls] + (int)(f.t1 - f.t0)) >> 2;
      write_trace(ctx, f.inst, f.node, f.tile, lane, f.cls, f.frame, f.t0, f.t1);
      complete_tile(ctx, f, slot);
    } else if (serving) {
      slot->n_ready = 0;
    }
    __syncwarp();
    const bool any = __any_sync(0xffffffffu, have_fin);
    if (any) {
      bool fenced = false;
      for (int w = 0; w < n_workers; ++w) {
        const int nr = sm->slot[w].n_ready;
        if (nr > 0 && !fenced) { queue_fill_fence(); fenced = true; }
        for (int i = 0; i < nr; ++i) {
          const ReadyItem it = sm->slot[w].ready[i];
          queue_fill(ctx, it.cls, it.base, sm->slot[w].fin.inst, it.node, it.res_units, lane, it.n_tiles, 32);
        }
      }
      __syncwarp();
      if (serving) {
        for (int i = 0; i < slot->n_ready; ++i) queue_commit(ctx, slot->ready[i].cls, slot->ready[i].n_tiles);
        slot->n_ready = 0;
      }
      __syncwarp();
    } else {
      if (sm->quit) break;
      bell_wait(&sm->bell_retire, bell_parity, RETIRE_SLEEP_NS);
    }
  }
}

__device__ inline void claim_loop(const DeviceCtx& ctx, SmState* sm, int n_workers) {
  const int lane = threadIdx.x & 31;
  const bool serving = lane < n_workers;
  Control* ctl = ctx.control;
  WorkerSlot* slot = sm->slot + (serving ? lane : 0);
  // Per-class constants live in registers: the arrays below are only ever read at loop-constant positions, and the
  // shared/tensor-memory needs are packed one byte per class.  (This loop runs on every tile hand-over of the SM;
  // arrays in local memory and global loads here cost 5 % of the whole step's throughput.)
  int tau[N_CLASSES * 3], res_units[N_CLASSES];
  unsigned group_mask[N_CLASSES];
  unsigned long long su_pack = 0ull, tu_pack = 0ull;
  {
    int group[N_CLASSES];
#pragma unroll
    for (int c = 0; c < N_CLASSES; ++c) {
#pragma unroll
      for (int x = 0; x < 3; ++x) tau[c * 3 + x] = ctx.classes[c].tau[x];
      group[c] = ctx.classes[c].group;
      const int su = ctx.classes[c].smem_units, tu = ctx.classes[c].tmem_units;
      res_units[c] = su > 0 ? su : 1;                                                 // R_k of the -R score
      su_pack |= (unsigned long long)(su & 0xFF) << (8 * c);
      tu_pack |= (unsigned long long)(tu & 0xFF) << (8 * c);
    }
#pragma unroll
    for (int c = 0; c < N_CLASSES; ++c) {
      unsigned m = 0;
#pragma unroll
      for (int j = 0; j < N_CLASSES; ++j)
        if (group[j] == group[c]) m |= 1u << j;
      group_mask[c] = m;
    }
  }
  const bool variant = ctx.policy == POLICY_TWO_PHASE_G || ctx.policy == POLICY_TWO_PHASE_R;
  uint64_t idle_start = 0, last_progress = gtimer();
  unsigned iter = 0, nap = CLAIM_NAP_NS, lost = 0;
  uint32_t bell_parity = 0;
  uint64_t pending_since = 0;     // lane c: since when class c has had committed tiles without a break (0: it has none)
  bool leaving = false;

  for (;;) {
    ++iter;
    bool progressed = false;
    long long av = lane < N_CLASSES ? ld_volatile_s64(&ctx.queues[lane].avail) : 0;
    const unsigned pending = __ballot_sync(0xffffffffu, av > 0) & ((1u << N_CLASSES) - 1u);
    // Tiles are claimed ahead of need only while the VLM backlog as a whole exceeds what the GPU's workers can hold
    // (a held tile is a tile no idle worker elsewhere can take), and then from every VLM queue that is not nearly empty.
    long long vlm_total = (lane < N_KINDS && av > 0) ? av : 0;
    vlm_total += __shfl_xor_sync(0xffffffffu, vlm_total, 1);
    vlm_total += __shfl_xor_sync(0xffffffffu, vlm_total, 2);
    vlm_total = __shfl_sync(0xffffffffu, vlm_total, 0);
    const unsigned deep = __ballot_sync(0xffffffffu, vlm_total >= PREFETCH_MIN_TOTAL && av >= PREFETCH_MIN_AVAIL) &
                          ((1u << N_CLASSES) - 1u);
    // classes whose tiles free workers elsewhere did not drain within head_wait_ns (by the clock, not by polling
    // rounds: how fast this loop spins must not change what it decides)
    if (av > 0) { if (pending_since == 0) pending_since = gtimer(); } else pending_since = 0;
    const unsigned waiting = __ballot_sync(0xffffffffu, pending_since != 0 && gtimer() - pending_since >= HEAD_WAIT_NS) &
                             ((1u << N_CLASSES) - 1u);
    int grid[N_CLASSES];                               // G_k of the -G score: the class's tiles still to place
    if (variant) {
      const int depth = (int)(av < 0 ? 0 : (av > (1 << 20) ? (1 << 20) : av));
#pragma unroll
      for (int c = 0; c < N_CLASSES; ++c) grid[c] = __shfl_sync(0xffffffffu, depth, c);
    }
    // ---- choose, lane by lane, which class each worker claims from
    int want = -1, promised_s = 0, promised_t = 0;
    bool to_prio = false;
    const unsigned avoid = lost;      // the class this lane just lost a race for: other SMs drained it
    lost = 0;
    for (int w = 0; w < n_workers; ++w) {
      const unsigned queued = serving ? slot->held_tail - slot->held_head : 0u;
      const unsigned pq = serving ? slot->prio_tail - slot->prio_head : 0u;
      if (lane == w && !leaving && (queued < (unsigned)HELD_DEPTH || pq == 0u)) {
        // A free worker serves the action head first.  A running worker gets VLM tiles claimed ahead of need (from
        // deep queues only), and an action-head tile when that tile has been waiting for more than a round (no
        // free worker anywhere took it) and the running tile is within PRIO_WINDOW_NS of its expected end (this
        // SM's running mean for the class): it goes into the priority slot, ahead of the held VLM tiles, so a
        // short action-head tile is never stuck behind more than the tail of one tile.
        const unsigned act_mask = ((1u << N_KINDS) - 1u) << N_KINDS;
        const bool busy = slot->busy != 0 || queued > 0 || pq > 0;
        const bool head_pending = pick_is_two_phase(ctx.policy) && (pending & act_mask & ~avoid) != 0u;
        unsigned cand;
        if (!busy) cand = head_pending ? (pending & act_mask) : pending;
        else if (pq == 0u && head_pending && (waiting & act_mask & ~avoid) != 0u && slot->busy != 0 &&
                 (long long)(gtimer() - slot->t_busy) + PRIO_WINDOW_NS >= (long long)sm->ema_ns[sm->cur[w].cls]) {
          cand = waiting & act_mask; to_prio = true;
        }
        else if (queued < (unsigned)HELD_DEPTH) cand = deep & ((1u << N_KINDS) - 1u);
        else cand = 0u;
        cand &= ~avoid;
        const unsigned long long smask = *reinterpret_cast<volatile unsigned long long*>(&sm->smem_mask);
        const unsigned tmask = *reinterpret_cast<volatile unsigned*>(&sm->tmem_mask);
        // room: a free run of units now, and enough units left after what was promised to tiles already handed
        // to free workers of this SM (they allocate a moment later)
        int smem_left = sm->n_smem_units - __popcll(smask) - *reinterpret_cast<volatile int*>(&sm->smem_promised);
        int tmem_left = sm->n_tmem_units - __popc(tmask) - *reinterpret_cast<volatile int*>(&sm->tmem_promised);
        {   // a worker of this SM that waits for room is served first: what it needs is not offered to the others
          const unsigned rw = *reinterpret_cast<volatile unsigned*>(&sm->room_wait);
          if (rw != 0u && (int)(rw >> 16) != w + 1) { smem_left -= (int)(rw & 0xFFu); tmem_left -= (int)((rw >> 8) & 0xFFu); }
        }
        unsigned feasible = 0;
        if (busy) feasible = (1u << N_CLASSES) - 1u;   // a tile claimed ahead waits for room when its worker takes it
        else
          for (unsigned m = cand; m != 0u; m &= m - 1u) {                // only the candidate classes are looked at
            const int c = __ffs((int)m) - 1;
            const int su = (int)((su_pack >> (8 * c)) & 0xFFull), tu = (int)((tu_pack >> (8 * c)) & 0xFFull);
            if (su <= smem_left && tu <= tmem_left && find_free(smask, su, sm->n_smem_units) >= 0 &&
                find_free((unsigned long long)tmask, tu, sm->n_tmem_units) >= 0)
              feasible |= 1u << c;
          }
        if ((cand & feasible) != 0u) {
          PickState ps;
#pragma unroll
          for (int c = 0; c < N_CLASSES; ++c) ps.cta_count[c] = *reinterpret_cast<volatile int*>(&sm->pick.cta_count[c]);
#pragma unroll
          for (int x = 0; x < 3; ++x) ps.u[x] = *reinterpret_cast<volatile int*>(&sm->pick.u[x]);
          int phase;
          if (variant)
            want = pick_choose(N_CLASSES, tau, group_mask, cand, feasible, ps, sm->pick.rr, ctx.policy, ctx.u_max, &phase, grid, res_units);
          else
            want = pick_choose(N_CLASSES, tau, group_mask, cand, feasible, ps, sm->pick.rr, ctx.policy, ctx.u_max, &phase);
        }
        if (want >= 0) {
          if (!busy) {                                   // promised until the worker has allocated (or the pop is lost)
            promised_s = (int)((su_pack >> (8 * want)) & 0xFFull); promised_t = (int)((tu_pack >> (8 * want)) & 0xFFull);
            atomicAdd(&sm->smem_promised, promised_s); atomicAdd(&sm->tmem_promised, promised_t);
          }
          atomicAdd(&sm->pick.cta_count[want], 1);     // counted from the claim on, so the next lane sees it
          tau_add(&sm->pick.u[0], tau, want, 1);
          sm->pick.rr = (want + 1) % N_CLASSES;
        }
      }
      __syncwarp();
    }
    // ---- the claims themselves run in parallel across lanes (global atomics)
    if (want >= 0) {
      QueueEntry e;
      if (queue_try_pop(ctx, want, e, gtimer() + ctx.wait_limit_ns)) {
        WorkerTile& h = to_prio ? slot->prio : slot->held[slot->held_tail % HELD_DEPTH];
        h.node = (uint32_t)e & ((1u << QW_NODE_BITS) - 1u);
        h.inst = (uint32_t)(e >> QW_NODE_BITS) & ((1u << QW_INST_BITS) - 1u);
        h.tile = (uint32_t)(e >> (QW_NODE_BITS + QW_INST_BITS)) & ((1u << QW_TILE_BITS) - 1u);
        h.smem_units = (int)((e >> (QW_NODE_BITS + QW_INST_BITS + QW_TILE_BITS)) & ((1u << QW_SMEM_BITS) - 1u));
        h.tmem_units = (int)((e >> (QW_NODE_BITS + QW_INST_BITS + QW_TILE_BITS + QW_SMEM_BITS)) & ((1u << QW_TMEM_BITS) - 1u));
        h.cls = want;
        {   // the worker's first loads are from the node's description: bring its two lines into this SM's L1 now
          const char* ndp = reinterpret_cast<const char*>(ctx.nodes + h.node);
          asm volatile("prefetch.global.L1 [%0];" ::"l"(ndp));
          asm volatile("prefetch.global.L1 [%0];" ::"l"(ndp + 128));
        }
        h.succ_begin = promised_s; h.succ_count = promised_t;   // (fields reused until the worker fills them in) units to un-promise
        __threadfence_block();
        if (to_prio) slot->prio_tail = slot->prio_tail + 1;
        else slot->held_tail = slot->held_tail + 1;      // the worker takes it as soon as it is free
        bell_ring(&sm->bell_worker[lane]);
        progressed = true;
      } else {                                         // lost the race: undo the count
        atomicSub(&sm->pick.cta_count[want], 1);
        tau_add(&sm->pick.u[0], tau, want, -1);
        if (promised_s | promised_t) { atomicSub(&sm->smem_promised, promised_s); atomicSub(&sm->tmem_promised, promised_t); }
        lost = 1u << want;                             // look elsewhere in the next round, which follows at once
      }
    }
    // ---- admission, exit and watchdog (lane 0 decides, every few rounds)
    int verdict = 0;   // 1 = leave
    if (lane == 0 && (iter & 3u) == 0) {              // several dependent round trips: not on every poll
      if (ld_volatile_u32(&ctl->error) != 0u || ld_volatile_u32(&ctl->stop) != 0u) verdict = 1;
      const unsigned cw = ld_volatile_u32(&ctl->ctrl);
      if (cw & CTRL_EXITING) verdict = 1;
      if (!verdict) {
        try_admit(ctx);
        const uint64_t now = gtimer();
        const bool none = cw == 0u && ld_volatile_u64(&ctl->admit_head) >= ld_volatile_u64(&ctl->admit_tail);
        if (none) {
          if (idle_start == 0) idle_start = now;
          else if (now - idle_start > ctx.idle_exit_ns) atomicCAS(&ctl->ctrl, 0u, CTRL_EXITING);
        } else {
          idle_start = 0;
        }
      }
    }
    const bool any_progress = __any_sync(0xffffffffu, progressed || (serving && slot->busy != 0));
    if (any_progress) last_progress = gtimer();
    else if (lane == 0 && !verdict && (iter & 63u) == 0 && gtimer() - last_progress > ctx.wait_limit_ns &&
             ld_volatile_u32(&ctl->ctrl) != 0u) {
      set_error(ctx, DEV_ERR_IDLE_LIMIT, (unsigned)blockIdx.x);   // frames in flight, nothing moved for too long
      verdict = 1;
    }
    verdict = __shfl_sync(0xffffffffu, verdict, 0);
    if (verdict) leaving = true;
    if (leaving) {
      // stop claiming; once every worker is idle and nothing is posted, send them home
      const bool quiet = !serving || (slot->busy == 0 && slot->done_state == 0 && slot->held_tail == slot->held_head &&
                                      slot->prio_tail == slot->prio_head);
      if (__all_sync(0xffffffffu, quiet)) {
        if (serving) { __threadfence_block(); slot->leave = 1; bell_ring(&sm->bell_worker[lane]); }
        __syncwarp();
        if (lane == 0) { __threadfence_block(); sm->quit = 1; bell_ring(&sm->bell_retire); }
        break;
      }
    }
    if (!__any_sync(0xffffffffu, progressed || lost != 0u)) {
      // A free worker with nothing to run: poll the queues at short intervals (its scheduler slots are idle anyway).
      // Every worker busy: sleep until one of them rings (it took its claimed tile, or ran dry) or the hint runs out.
      const bool hungry = serving && slot->busy == 0 && slot->held_tail == slot->held_head && slot->prio_tail == slot->prio_head;
      if (__any_sync(0xffffffffu, hungry)) { __nanosleep(nap); if (nap < CLAIM_NAP_MAX_NS) nap += CLAIM_NAP_NS; }
      else { bell_wait(&sm->bell_claim, bell_parity, CLAIM_SLEEP_NS); nap = CLAIM_NAP_NS; }
    } else nap = CLAIM_NAP_NS;
  }
}

// ------------------------------------------------------------------ the persistent co-scheduling kernel
// One CTA per SM: `workers` worker groups of WORKER_THREADS threads run tiles; one more warp is the
// dispatcher.  Every wait is bounded by ctx.wait_limit_ns.
__global__ void __launch_bounds__(MAX_WORKERS* WORKER_THREADS + DISPATCH_THREADS, 1)
    vla_cosched_kernel(DeviceCtx ctx, int dyn_smem_bytes) {
  extern __shared__ __align__(1024) char smem_raw[];
  SmState* sm = reinterpret_cast<SmState*>(smem_raw);
  char* slab = smem_raw + SM_STATE_BYTES;
  const int n_workers = (blockDim.x - DISPATCH_THREADS) / WORKER_THREADS;
  const bool is_dispatcher = threadIdx.x >= n_workers * WORKER_THREADS;
  const int worker = threadIdx.x / WORKER_THREADS;
  const int wt = threadIdx.x % WORKER_THREADS;
  if (threadIdx.x == 0) {
    sm->smem_mask = 0;
    sm->tmem_mask = 0;
    int units = (dyn_smem_bytes - SM_STATE_BYTES) / SMEM_UNIT;
    sm->n_smem_units = units > 64 ? 64 : units;
    sm->n_tmem_units = 512 / TMEM_UNIT;
    for (int c = 0; c < PICK_MAX_CLASSES; ++c) sm->pick.cta_count[c] = 0;
    sm->pick.u[0] = sm->pick.u[1] = sm->pick.u[2] = 0;
    sm->pick.rr = (int)(blockIdx.x % N_CLASSES);
    sm->tmem_base = 0;
    sm->quit = 0;
    sm->smem_promised = 0; sm->tmem_promised = 0;
    sm->room_wait = 0u;
    mbar_init(smem_u32(&sm->bell_claim), 1); mbar_init(smem_u32(&sm->bell_retire), 1);
    for (int w = 0; w < MAX_WORKERS; ++w) mbar_init(smem_u32(&sm->bell_worker[w]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int c = 0; c < N_CLASSES; ++c) sm->ema_ns[c] = 30000;
    for (int c = 0; c < N_CLASSES; ++c)
      for (int x = 0; x < 3; ++x) sm->tau_tab[c * 3 + x] = ctx.classes[c].tau[x];
    for (int w = 0; w < MAX_WORKERS; ++w) {
      sm->slot[w].held_tail = 0; sm->slot[w].held_head = 0; sm->slot[w].leave = 0; sm->slot[w].done_state = 0;
      sm->slot[w].prio_tail = 0; sm->slot[w].prio_head = 0; sm->slot[w].t_busy = 0;

      sm->slot[w].busy = 0;
      sm->slot[w].n_ready = 0;
    }
  }
  __syncthreads();
  if (threadIdx.x < 32) tmem_alloc(&sm->tmem_base, 512);   // the whole tensor memory of this SM, sub-allocated per tile
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  Control* ctl = ctx.control;

  if (is_dispatcher) {
    if (threadIdx.x < n_workers * WORKER_THREADS + 32) claim_loop(ctx, sm, n_workers);
    else retire_loop(ctx, sm, n_workers);
  } else {
    const int bar_id = worker + 1;
    WorkerSlot* slot = sm->slot + worker;
    unsigned long long tiles = 0;
    uint32_t bell_parity = 0;
    for (;;) {
      if (wt == 0) {
        // take the tile the claim warp holds for this worker, then give it its exact memory need
        int st;
        unsigned naps = 0;
        for (;;) {
          if (slot->prio_tail != slot->prio_head) { st = 3; break; }
          if (slot->held_tail != slot->held_head) { st = 1; break; }
          if (slot->leave) { st = 2; break; }
          if (naps < 8) __nanosleep(20);                               // a claimed tile is usually a moment away
          else bell_wait(&sm->bell_worker[worker], bell_parity, 2000u);
          ++naps;
        }
        WorkerTile& cur = sm->cur[worker];
        if (st == 1 || st == 3) {
          cur = st == 3 ? slot->prio : slot->held[slot->held_head % HELD_DEPTH];
          slot->t_busy = gtimer();
          slot->busy = 1;
          __threadfence_block();
          if (st == 3) slot->prio_head = slot->prio_head + 1;
          else slot->held_head = slot->held_head + 1;   // the claim warp may refill the slot
          bell_ring(&sm->bell_claim);
          const uint64_t lim = gtimer() + ctx.wait_limit_ns;
          bool ok = false;
          for (unsigned spin = 0;; ++spin) {
            const unsigned long long sm_old = *reinterpret_cast<volatile unsigned long long*>(&sm->smem_mask);
            // every worker has a home region (a third of the slab, a third of the columns): a tile that fits it goes
            // there whenever it is free, so tiles of the common shapes never fragment the slab; larger tiles and a
            // home occupied by one of them fall back to the first free run
            const int home_s = worker * (sm->n_smem_units / n_workers), home_t = worker * (sm->n_tmem_units / n_workers);
            int s0 = -1;
            if (cur.smem_units <= sm->n_smem_units / n_workers && ((sm_old >> home_s) & unit_bits(cur.smem_units)) == 0ull) s0 = home_s;
            else s0 = find_free(sm_old, cur.smem_units, sm->n_smem_units);
            if (s0 >= 0) {
              const unsigned long long sbits = unit_bits(cur.smem_units) << s0;
              if (cur.smem_units == 0 || atomicCAS(&sm->smem_mask, sm_old, sm_old | sbits) == sm_old) {
                const unsigned tm_old = *reinterpret_cast<volatile unsigned*>(&sm->tmem_mask);
                int t0 = -1;
                if (cur.tmem_units <= sm->n_tmem_units / n_workers && ((tm_old >> home_t) & (unsigned)unit_bits(cur.tmem_units)) == 0u) t0 = home_t;
                else t0 = find_free((unsigned long long)tm_old, cur.tmem_units, sm->n_tmem_units);
                const unsigned tbits = (unsigned)(unit_bits(cur.tmem_units) << (t0 < 0 ? 0 : t0));
                if (t0 >= 0 && (cur.tmem_units == 0 || atomicCAS(&sm->tmem_mask, tm_old, tm_old | tbits) == tm_old)) {
                  cur.smem_unit0 = s0; cur.tmem_unit0 = t0;
                  ok = true;
                  break;
                }
                if (cur.smem_units) atomicAnd(&sm->smem_mask, ~sbits);   // no tensor memory yet: give the shared memory back
              }
            }
            if (spin == 0)        // waiting for room
              *reinterpret_cast<volatile unsigned*>(&sm->room_wait) =
                  (unsigned)cur.smem_units | ((unsigned)cur.tmem_units << 8) | ((unsigned)(worker + 1) << 16);
            __nanosleep(100);
            if ((spin & 255u) == 255u && (gtimer() > lim || ld_volatile_u32(&ctl->error) != 0u)) break;
          }
          if ((*reinterpret_cast<volatile unsigned*>(&sm->room_wait) >> 16) == (unsigned)(worker + 1))
            *reinterpret_cast<volatile unsigned*>(&sm->room_wait) = 0u;
          if (cur.succ_begin | cur.succ_count) {     // the claim warp's promise of room is settled either way
            atomicSub(&sm->smem_promised, cur.succ_begin); atomicSub(&sm->tmem_promised, cur.succ_count);
          }
          if (!ok) set_error(ctx, DEV_ERR_IDLE_LIMIT, 0x2000u + (unsigned)blockIdx.x);
          cur.t0 = ok ? 1 : 2;              // 1 run, 2 skip (error), 0 leave
        } else {
          cur.t0 = 0;
        }
      }
      asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
      const WorkerTile cmd = sm->cur[worker];
      if (cmd.t0 == 0) break;
      const NodeDesc& n = ctx.nodes[cmd.node];
      TileCtx tc;
      tc.arena = ctx.arena;
      tc.slot_base = ctx.slot_base[cmd.inst];
      tc.smem = slab + (size_t)cmd.smem_unit0 * SMEM_UNIT;
      tc.ctl = smem_raw + SM_STATE_BASE + worker * SM_CTL_BYTES;
      tc.tmem = sm->tmem_base + (unsigned)cmd.tmem_unit0 * TMEM_UNIT;
      tc.tid = wt;
      tc.bar_id = bar_id;
      tc.error = &ctl->error;
      tc.tmaps = ctx.tmaps;
      tc.inputs = ctx.input_ptrs + (size_t)cmd.inst * N_FRAME_INPUTS;
      tc.amap_base = ctx.n_weight_tmaps + (int)cmd.inst * ctx.n_act_tmaps;
      tc.drop_loads = 0;
      const uint64_t t0 = gtimer();
      tc.deadline = t0 + ctx.wait_limit_ns;
      // the frame id is only needed by the emit tile and by the trace
      const int n_op = __ldg(&n.op);
      // the node's successor range travels with the finished tile; read it now, while the description is hot
      const int n_succ_begin = __ldg(&n.succ_begin), n_succ_count = __ldg(&n.succ_count);
      if (wt == 0) {     // the retire warp of this SM will read the successor records when the tile ends
        const char* sp = reinterpret_cast<const char*>(ctx.succ + n_succ_begin);
        asm volatile("prefetch.global.L1 [%0];" ::"l"(sp));
      }
      const uint64_t frame = (ctx.trace_capacity != 0 || n_op == OP_EMIT)
                                 ? *reinterpret_cast<const volatile uint64_t*>(ctx.inst_frame + cmd.inst) : 0ull;
      if (cmd.t0 == 1) run_tile(ctx, tc, n, (int)cmd.tile, (int)cmd.inst, frame);
      // Outputs written here by ordinary stores are read by TMA on other SMs.  The proxy fence that must lie between
      // the two in causality order is the consumer's (first statement of its TMA-issuing thread, after the
      // dependency was observed); a second one here cost 2 % of the throughput and is not needed.
      asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
      // Two lanes share the end of a tile: lane 0 frees the tile's memory and goes straight on to take the next
      // tile, the first lane of warp 1 posts the finished one to the retire warp meanwhile (both meet again at the
      // barrier that opens the next tile).
      if (wt == 0) {
        ++tiles;
        if (cmd.t0 == 1) {
          if (cmd.smem_units) atomicAnd(&sm->smem_mask, ~(unit_bits(cmd.smem_units) << cmd.smem_unit0));
          if (cmd.tmem_units) atomicAnd(&sm->tmem_mask, ~(unsigned)(unit_bits(cmd.tmem_units) << cmd.tmem_unit0));
        }
        slot->busy = 0;
        if (slot->held_tail == slot->held_head && slot->prio_tail == slot->prio_head) bell_ring(&sm->bell_claim);   // out of work
      } else if (wt == 32) {
        const uint64_t t1 = gtimer();
        WorkerTile d = cmd;
        d.t0 = t0; d.t1 = t1; d.frame = frame;
        d.succ_begin = n_succ_begin; d.succ_count = n_succ_count; d.op = n_op;
        unsigned naps = 0;
        while (slot->done_state != 0) {
          __nanosleep(40);
          if ((++naps & 0xFFFFu) == 0 && gtimer() - t0 > 2 * ctx.wait_limit_ns) break;   // retire warp gone: give up posting
        }
        slot->done = d;
        // The tile's writes (all threads, ordered by the barrier above) must be visible device-wide before any
        // successor is released.  That fence is the retire warp's (first statement of complete_tile, after it has
        // read this flag): fences are cumulative, and barrier -> block-scope fence -> flag -> device-scope fence
        // keeps the writes ahead of the counter atomics without a device-scope round trip on the worker's path.
        __threadfence_block();
        slot->done_state = 1;
        bell_ring(&sm->bell_retire);
        atomicSub(&sm->pick.cta_count[cmd.cls], 1);    // the pick's view of this SM, after the completion is on its way
        for (int x = 0; x < 3; ++x) atomicSub(&sm->pick.u[x], sm->tau_tab[cmd.cls * 3 + x]);
      }
    }
    if (wt == 0) atomicAdd(&ctl->tiles_done, tiles);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(sm->tmem_base, 512);
}

// ------------------------------------------------------------------ one node as an ordinary kernel (CTA = tile)
__global__ void __launch_bounds__(WORKER_THREADS) vla_node_kernel(DeviceCtx ctx, const NodeDesc* nodes, int node_idx, int inst) {
  extern __shared__ __align__(1024) char smem_raw[];
  __shared__ uint32_t tmem_base_s;
  __shared__ __align__(16) char ctl_block[1024];
  const NodeDesc& n = nodes[node_idx];
  uint32_t tmem_cols = 0;
  if (n.tmem_cols > 0) {
    tmem_cols = 32;
    while ((int)tmem_cols < n.tmem_cols) tmem_cols <<= 1;
    if (threadIdx.x < 32) tmem_alloc(&tmem_base_s, tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }
  TileCtx tc;
  tc.arena = ctx.arena;
  tc.slot_base = inst >= 0 ? ctx.slot_base[inst] : 0;
  tc.smem = smem_raw;
  tc.ctl = ctl_block;
  tc.tmem = tmem_cols ? tmem_base_s : 0;
  tc.tid = threadIdx.x;
  tc.bar_id = 1;
  tc.error = &ctx.control->error;
  tc.tmaps = ctx.tmaps;
  tc.inputs = ctx.input_ptrs + (size_t)(inst >= 0 ? inst : 0) * N_FRAME_INPUTS;
  tc.amap_base = ctx.n_weight_tmaps + (inst >= 0 ? inst : 0) * ctx.n_act_tmaps;
  tc.drop_loads = 0;
  const uint64_t t0 = gtimer();
  tc.deadline = t0 + ctx.wait_limit_ns;
  const uint64_t frame = inst >= 0 ? ctx.inst_frame[inst] : 0;
  run_tile(ctx, tc, n, (int)blockIdx.x, inst, frame);
  if (inst >= 0 && ctx.trace_capacity) {
    asm volatile("bar.sync 1, %0;" ::"r"(WORKER_THREADS) : "memory");
    if (threadIdx.x == 0) write_trace(ctx, (uint32_t)inst, (uint32_t)node_idx, blockIdx.x, 0, n.cls, frame, t0, gtimer());
  }
  if (tmem_cols) {
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_base_s, tmem_cols);
  }
}

// ------------------------------------------------------------------ pick probe (tests)
__global__ void vla_pick_probe_kernel(int n_cls, const int* tau, unsigned pending, unsigned feasible, PickState* st,
                                      int rr_start, int policy, int u_max, const int* grid, const int* res, int* out) {
  int phase;
  unsigned group_mask[PICK_MAX_CLASSES];
  for (int i = 0; i < PICK_MAX_CLASSES; ++i) group_mask[i] = 1u << i;   // one class per group: the paper's listing
  int k = pick_choose(n_cls, tau, group_mask, pending, feasible, *st, rr_start, policy, u_max, &phase, grid, res);
  if (k >= 0) pick_commit(*st, k, tau);
  out[0] = k;
  out[1] = phase;
}

}  // namespace vla
