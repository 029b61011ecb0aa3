// Device side of the dispatcher: tile queues, dependency counters, the persistent
// co-scheduling kernel, and the ordinary-kernel wrapper used by the stream modes.
#pragma once
#include "pick.cuh"
#include "tiles.cuh"

namespace vla {

constexpr unsigned CTRL_EXITING = 0x80000000u;
constexpr int MAX_WORKERS = 4;
constexpr int SM_STATE_BYTES = 2048;

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

// ------------------------------------------------------------------ tensor memory (whole-warp calls)
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// ------------------------------------------------------------------ tile queues
// Pushing tiles is split in three so a whole worker can fill the entries in parallel:
// reserve (one thread), fill (any threads, entry i of the range), commit (one thread, after a barrier).
__device__ inline unsigned long long queue_reserve(const DeviceCtx& ctx, int cls, int n) {
  TileQueue* q = ctx.queues + cls;
  const unsigned long long base = atomicAdd(&q->tail, (unsigned long long)n);
  const unsigned long long head = ld_volatile_u64(&q->head);
  if (base + n - head > (unsigned long long)ctx.q_capacity) set_error(ctx, DEV_ERR_QUEUE_FULL, cls);
  return base;
}
__device__ inline void queue_fill(const DeviceCtx& ctx, int cls, unsigned long long base, uint32_t inst, uint32_t node, int first,
                                  int count, int stride) {
  const unsigned long long mask = (unsigned long long)ctx.q_capacity - 1;
  QueueEntry* ent = ctx.q_entries + (size_t)cls * ctx.q_capacity;
  unsigned long long* seq = ctx.q_seq + (size_t)cls * ctx.q_capacity;
  for (int i = first; i < count; i += stride) {
    QueueEntry e;
    e.inst_node = (inst << 20) | node;
    e.tile = (uint32_t)i;
    ent[(base + i) & mask] = e;
  }
  __threadfence();   // entries before their sequence words
  for (int i = first; i < count; i += stride)
    *reinterpret_cast<volatile unsigned long long*>(seq + ((base + i) & mask)) = base + i + 1;
}
__device__ inline void queue_commit(const DeviceCtx& ctx, int cls, int n) {
  __threadfence();
  atomicAdd(reinterpret_cast<unsigned long long*>(&ctx.queues[cls].avail), (unsigned long long)n);
  atomicAdd(&ctx.control->doorbell, 1ull);
}
// One thread pushes everything (admission of a frame's root tiles).
__device__ inline void queue_push(const DeviceCtx& ctx, int cls, uint32_t inst, uint32_t node, int n) {
  const unsigned long long base = queue_reserve(ctx, cls, n);
  queue_fill(ctx, cls, base, inst, node, 0, n, 1);
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
  const unsigned long long* seq = ctx.q_seq + (size_t)cls * ctx.q_capacity + (t & mask);
  unsigned spins = 0;
  while (ld_acquire_u64(seq) != t + 1) {
    if ((++spins & 63u) == 0 && gtimer() > deadline) {
      set_error(ctx, DEV_ERR_WAIT_QUEUE, cls);
      return false;
    }
  }
  e = ctx.q_entries[(size_t)cls * ctx.q_capacity + (t & mask)];
  return true;
}

// ------------------------------------------------------------------ per-SM state of the persistent kernel
constexpr int MAX_READY = 6;
struct ReadyItem {
  unsigned long long base;   // reserved queue range
  uint32_t node;
  int n_tiles, cls;
};
struct WorkerCmd {
  int kind;            // 0 run, 1 exit
  uint32_t inst, node, tile;
  int cls;
  int smem_unit0, smem_units, tmem_unit0, tmem_units;
  int n_ready;         // successors released by the tile just finished (filled by the leader)
  ReadyItem ready[MAX_READY];
};

struct SmState {
  unsigned lock;
  unsigned long long smem_mask;    // bit i set = shared-memory unit i in use
  unsigned tmem_mask;              // bit i set = tensor-memory unit i in use
  int n_smem_units, n_tmem_units;
  PickState pick;
  int waiter;                      // worker holding a tile while it waits for room (-1: none)
  unsigned tmem_base;
  unsigned long long tiles;        // tiles this SM ran (added to the global counter at exit)
  WorkerCmd cur[MAX_WORKERS];
};
static_assert(sizeof(SmState) <= SM_STATE_BYTES, "SM state too large");

__device__ __forceinline__ unsigned long long unit_bits(int n) { return n >= 64 ? ~0ull : ((1ull << n) - 1ull); }
__device__ __forceinline__ int find_free(unsigned long long mask, int need, int total) {
  if (need == 0) return 0;
  if (need > total) return -1;
  const unsigned long long want = unit_bits(need);
  for (int i = 0; i + need <= total; ++i)
    if (((mask >> i) & want) == 0) return i;
  return -1;
}

// Tile finished: bump the node's counter; the last tile of a node releases its successors.
// Released successors get their queue range reserved here and are returned in `cmd->ready`
// (the whole worker then fills the entries); without `cmd` they are pushed on the spot.
__device__ inline void complete_tile(const DeviceCtx& ctx, uint32_t inst, uint32_t node_idx, bool persistent, WorkerCmd* cmd) {
  const NodeDesc& n = ctx.nodes[node_idx];
  if (cmd) cmd->n_ready = 0;
  __threadfence();
  int* cnt = ctx.tiles_done + (size_t)inst * ctx.n_nodes + node_idx;
  int done = atomicAdd(cnt, 1) + 1;
  if (done != n.n_tiles) return;
  __threadfence();
  *cnt = 0;
  for (int i = 0; i < n.succ_count; ++i) {
    int s = ctx.succ[n.succ_begin + i];
    int* dep = ctx.dep_count + (size_t)inst * ctx.n_nodes + s;
    int left = atomicSub(dep, 1) - 1;
    if (left == 0) {
      const NodeDesc& sn = ctx.nodes[s];
      *dep = sn.n_pred;
      if (cmd && cmd->n_ready < MAX_READY) {
        ReadyItem& it = cmd->ready[cmd->n_ready++];
        it.base = queue_reserve(ctx, sn.cls, sn.n_tiles);
        it.node = (uint32_t)s; it.n_tiles = sn.n_tiles; it.cls = sn.cls;
      } else {
        queue_push(ctx, sn.cls, inst, (uint32_t)s, sn.n_tiles);
      }
    }
  }
  if (persistent && n.op == OP_EMIT) atomicSub(&ctx.control->ctrl, 1u);
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
  __threadfence();
  for (int i = 0; i < ctx.n_roots; ++i) {
    int r = ctx.roots[i];
    queue_push(ctx, ctx.nodes[r].cls, inst, (uint32_t)r, ctx.nodes[r].n_tiles);
  }
}

// Leader of a worker: find the next tile for this worker under the pick policy.
// Feasibility is tested with each class's smallest footprint; the tile actually claimed is then
// given its exact shared-memory and tensor-memory need.  If that does not fit yet, the worker keeps
// the tile and waits (bounded) for co-resident tiles to finish; meanwhile it is the SM's only
// "waiter" and the other workers admit nothing that needs shared or tensor memory.
__device__ inline bool try_pick(const DeviceCtx& ctx, SmState* sm, int worker, uint64_t deadline) {
  unsigned pending = 0;
  for (int c = 0; c < N_CLASSES; ++c)
    if (ld_volatile_s64(&ctx.queues[c].avail) > 0) pending |= 1u << c;
  if (pending == 0) return false;
  unsigned spins = 0;
  while (atomicCAS(&sm->lock, 0u, 1u) != 0u) {
    __nanosleep(32);
    if ((++spins & 255u) == 0 && gtimer() > deadline) return false;
  }
  bool got = false;
  int tau[N_CLASSES * 3], group[N_CLASSES];
  for (int c = 0; c < N_CLASSES; ++c) {
    for (int x = 0; x < 3; ++x) tau[c * 3 + x] = ctx.classes[c].tau[x];
    group[c] = ctx.classes[c].group;
  }
  const bool blocked = sm->waiter >= 0 && sm->waiter != worker;
  WorkerCmd& cmd = sm->cur[worker];
  for (int attempt = 0; attempt < N_CLASSES && pending; ++attempt) {
    unsigned feasible = 0;
    for (int c = 0; c < N_CLASSES; ++c) {
      const int su = ctx.classes[c].smem_units, tu = ctx.classes[c].tmem_units;
      if (blocked && (su > 0 || tu > 0)) continue;
      if (find_free(sm->smem_mask, su, sm->n_smem_units) >= 0 && find_free(sm->tmem_mask, tu, sm->n_tmem_units) >= 0)
        feasible |= 1u << c;
    }
    int phase;
    int k = pick_choose(N_CLASSES, tau, group, pending, feasible, sm->pick, sm->pick.rr, ctx.policy, &phase);
    if (k < 0) break;
    QueueEntry e;
    if (!queue_try_pop(ctx, k, e, deadline)) {
      pending &= ~(1u << k);
      continue;
    }
    cmd.kind = 0;
    cmd.inst = e.inst_node >> 20;
    cmd.node = e.inst_node & 0xFFFFFu;
    cmd.tile = e.tile;
    cmd.cls = k;
    const NodeDesc& nd = ctx.nodes[cmd.node];
    cmd.smem_units = (nd.smem_bytes + SMEM_UNIT - 1) / SMEM_UNIT;
    cmd.tmem_units = (nd.tmem_cols + TMEM_UNIT - 1) / TMEM_UNIT;
    pick_commit(sm->pick, k, tau);
    sm->pick.rr = (k + 1) % N_CLASSES;
    got = true;
    break;
  }
  if (got) {
    // exact allocation; hold the tile and wait when the SM is too full right now
    for (;;) {
      cmd.smem_unit0 = find_free(sm->smem_mask, cmd.smem_units, sm->n_smem_units);
      cmd.tmem_unit0 = find_free((unsigned long long)sm->tmem_mask, cmd.tmem_units, sm->n_tmem_units);
      if (cmd.smem_unit0 >= 0 && cmd.tmem_unit0 >= 0) break;
      sm->waiter = worker;
      __threadfence_block();
      atomicExch(&sm->lock, 0u);
      __nanosleep(200);
      if (gtimer() > deadline || ld_volatile_u32(&ctx.control->error) != 0u) {
        set_error(ctx, DEV_ERR_IDLE_LIMIT, 0x1000u + (unsigned)blockIdx.x);
        cmd.kind = 1;
        return true;    // leave: kind = exit
      }
      while (atomicCAS(&sm->lock, 0u, 1u) != 0u) __nanosleep(32);
    }
    if (sm->waiter == worker) sm->waiter = -1;
    if (cmd.smem_units) sm->smem_mask |= unit_bits(cmd.smem_units) << cmd.smem_unit0;
    if (cmd.tmem_units) sm->tmem_mask |= (unsigned)(unit_bits(cmd.tmem_units) << cmd.tmem_unit0);
  }
  __threadfence_block();
  atomicExch(&sm->lock, 0u);
  return got;
}

__device__ inline void release_resources(const DeviceCtx& ctx, SmState* sm, const WorkerCmd& cmd) {
  while (atomicCAS(&sm->lock, 0u, 1u) != 0u) __nanosleep(32);
  if (cmd.smem_units) sm->smem_mask &= ~(unit_bits(cmd.smem_units) << cmd.smem_unit0);
  if (cmd.tmem_units) sm->tmem_mask &= ~(unsigned)(unit_bits(cmd.tmem_units) << cmd.tmem_unit0);
  int tau[3] = {ctx.classes[cmd.cls].tau[0], ctx.classes[cmd.cls].tau[1], ctx.classes[cmd.cls].tau[2]};
  sm->pick.cta_count[cmd.cls] -= 1;
  for (int x = 0; x < 3; ++x) sm->pick.u[x] -= tau[x];
  sm->tiles += 1;
  __threadfence_block();
  atomicExch(&sm->lock, 0u);
}

// ------------------------------------------------------------------ the persistent co-scheduling kernel
// One CTA per SM; MAX_WORKERS worker groups of WORKER_THREADS threads.  Each worker's
// first thread is its leader: it admits ready frames, picks a tile, and after the tile
// has run resolves dependencies.  Every wait is bounded by ctx.wait_limit_ns.
__global__ void __launch_bounds__(MAX_WORKERS* WORKER_THREADS, 1) vla_cosched_kernel(DeviceCtx ctx, int dyn_smem_bytes) {
  extern __shared__ __align__(1024) char smem_raw[];
  SmState* sm = reinterpret_cast<SmState*>(smem_raw);
  char* slab = smem_raw + SM_STATE_BYTES;
  const int worker = threadIdx.x / WORKER_THREADS;
  const int wt = threadIdx.x % WORKER_THREADS;
  if (threadIdx.x == 0) {
    sm->lock = 0;
    sm->smem_mask = 0;
    sm->tmem_mask = 0;
    int units = (dyn_smem_bytes - SM_STATE_BYTES) / SMEM_UNIT;
    sm->n_smem_units = units > 64 ? 64 : units;
    sm->n_tmem_units = 512 / TMEM_UNIT;
    for (int c = 0; c < PICK_MAX_CLASSES; ++c) sm->pick.cta_count[c] = 0;
    sm->pick.u[0] = sm->pick.u[1] = sm->pick.u[2] = 0;
    sm->pick.rr = (int)(blockIdx.x % N_CLASSES);
    sm->tmem_base = 0;
    sm->waiter = -1;
    sm->tiles = 0;
  }
  __syncthreads();
  if (threadIdx.x < 32) tmem_alloc(&sm->tmem_base, 512);   // the whole tensor memory of this SM, sub-allocated per tile
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  Control* ctl = ctx.control;
  const int bar_id = worker + 1;

  for (;;) {
    if (wt == 0) {
      WorkerCmd& cmd = sm->cur[worker];
      const uint64_t wait_start = gtimer();
      uint64_t idle_start = 0;
      unsigned backoff = 64, polls = 0;
      unsigned long long bell_seen = ~0ull;
      cmd.kind = 1;
      for (;;) {
        // An idle leader polls one word (the doorbell); the queues are scanned only when it moved.
        const unsigned long long bell = ld_volatile_u64(&ctl->doorbell);
        const bool slow = (polls++ & 15u) == 0;
        if (slow) {
          if (ld_volatile_u32(&ctl->error) != 0u || ld_volatile_u32(&ctl->stop) != 0u) break;
          if (ld_volatile_u32(&ctl->ctrl) & CTRL_EXITING) break;
          try_admit(ctx);
        }
        if (bell != bell_seen || slow) {
          bell_seen = bell;
#ifdef VLA_TILE_TIMING
          const uint64_t tp0 = gtimer();
          const bool hit = try_pick(ctx, sm, worker, wait_start + ctx.wait_limit_ns);
          atomicAdd(ctl->dbg + (hit ? 5 : 7), gtimer() - tp0); atomicAdd(ctl->dbg + (hit ? 6 : 8), 1ull);
          if (hit) break;
#else
          if (try_pick(ctx, sm, worker, wait_start + ctx.wait_limit_ns)) break;   // cmd.kind = 0 now
#endif
        }
        if (slow) {
          const uint64_t now = gtimer();
          const unsigned cw = ld_volatile_u32(&ctl->ctrl);
          if (cw & CTRL_EXITING) break;
          const bool none = cw == 0u && ld_volatile_u64(&ctl->admit_head) >= ld_volatile_u64(&ctl->admit_tail);
          if (none) {
            if (idle_start == 0) idle_start = now;
            else if (now - idle_start > ctx.idle_exit_ns) atomicCAS(&ctl->ctrl, 0u, CTRL_EXITING);
          } else {
            idle_start = 0;
            if (now - wait_start > ctx.wait_limit_ns) {   // frames in flight but nothing runnable for too long
              set_error(ctx, DEV_ERR_IDLE_LIMIT, (unsigned)blockIdx.x);
              break;
            }
          }
        }
        __nanosleep(backoff);
        if (backoff < 2048) backoff <<= 1;
      }
    }
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
    const WorkerCmd cmd = sm->cur[worker];
    if (cmd.kind != 0) break;
    const NodeDesc& n = ctx.nodes[cmd.node];
    TileCtx tc;
    tc.arena = ctx.arena;
    tc.slot_base = ctx.slot_base[cmd.inst];
    tc.smem = slab + (size_t)cmd.smem_unit0 * SMEM_UNIT;
    tc.tmem = sm->tmem_base + (unsigned)cmd.tmem_unit0 * TMEM_UNIT;
    tc.tid = wt;
    tc.bar_id = bar_id;
    tc.error = &ctl->error;
    tc.tmaps = ctx.tmaps;
    tc.dbg = ctl->dbg;
    tc.inputs = ctx.input_ptrs + (size_t)cmd.inst * N_FRAME_INPUTS;
    tc.amap_base = ctx.n_weight_tmaps + (int)cmd.inst * ctx.n_act_tmaps;
    const uint64_t t0 = gtimer();
    tc.deadline = t0 + ctx.wait_limit_ns;
    const uint64_t frame = *reinterpret_cast<const volatile uint64_t*>(ctx.inst_frame + cmd.inst);
    run_tile(ctx, tc, n, (int)cmd.tile, (int)cmd.inst, frame);
    asm volatile("fence.proxy.async;" ::: "memory");   // outputs may be read by TMA on another SM
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
    if (wt == 0) {
      const uint64_t t1 = gtimer();
      write_trace(ctx, cmd.inst, cmd.node, cmd.tile, worker, cmd.cls, frame, t0, t1);
      release_resources(ctx, sm, cmd);
      complete_tile(ctx, cmd.inst, cmd.node, true, &sm->cur[worker]);
#ifdef VLA_TILE_TIMING
      atomicAdd(ctl->dbg + 9, gtimer() - t1); atomicAdd(ctl->dbg + 10, 1ull);
#endif
    }
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
    const int n_ready = sm->cur[worker].n_ready;
    if (n_ready > 0) {
      for (int i = 0; i < n_ready; ++i) {
        const ReadyItem it = sm->cur[worker].ready[i];
        queue_fill(ctx, it.cls, it.base, cmd.inst, it.node, wt, it.n_tiles, WORKER_THREADS);
      }
      asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(WORKER_THREADS) : "memory");
      if (wt == 0)
        for (int i = 0; i < n_ready; ++i) queue_commit(ctx, sm->cur[worker].ready[i].cls, sm->cur[worker].ready[i].n_tiles);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(sm->tmem_base, 512);
  if (threadIdx.x == 0) atomicAdd(&ctl->tiles_done, sm->tiles);
}

// ------------------------------------------------------------------ one node as an ordinary kernel (CTA = tile)
__global__ void __launch_bounds__(WORKER_THREADS) vla_node_kernel(DeviceCtx ctx, const NodeDesc* nodes, int node_idx, int inst) {
  extern __shared__ __align__(1024) char smem_raw[];
  __shared__ uint32_t tmem_base_s;
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
  tc.tmem = tmem_cols ? tmem_base_s : 0;
  tc.tid = threadIdx.x;
  tc.bar_id = 1;
  tc.error = &ctx.control->error;
  tc.tmaps = ctx.tmaps;
  tc.dbg = ctx.control->dbg;
  tc.inputs = ctx.input_ptrs + (size_t)(inst >= 0 ? inst : 0) * N_FRAME_INPUTS;
  tc.amap_base = ctx.n_weight_tmaps + (inst >= 0 ? inst : 0) * ctx.n_act_tmaps;
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
                                      int rr_start, int policy, int* out) {
  int phase;
  int group[PICK_MAX_CLASSES];
  for (int i = 0; i < PICK_MAX_CLASSES; ++i) group[i] = i;   // one class per group: the paper's listing
  int k = pick_choose(n_cls, tau, group, pending, feasible, *st, rr_start, policy, &phase);
  if (k >= 0) pick_commit(*st, k, tau);
  out[0] = k;
  out[1] = phase;
}

}  // namespace vla
