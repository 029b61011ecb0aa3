/*
 * vla.h -- C ABI of the B200 two-phase Vision-Language-Action inference library.
 *
 * The library serves several independent robot request streams.  Every frame of a
 * stream goes through two phases (paper Section 2.1, Figure 1): a VLM prefill
 * (vision patch encoder + decoder layers over image and text tokens) whose
 * output feeds only that frame's action head, which runs a denoising loop and
 * emits one action chunk.  The VLM phase of frame N+1 may run while the action
 * head of frame N is still denoising (Section 2.1, "overlap"); how the two
 * phases share the GPU is the run mode:
 *
 *   VLA_MODE_COSCHED    one persistent kernel, one CTA per SM; worker groups on
 *                       each SM pull tiles from device-resident per-class queues
 *                       under a resource-aware pick (software analogue of the
 *                       paper's Algorithm 1 and Section 3.3 utilisation registers)
 *   VLA_MODE_TWO_STREAM the same tile bodies launched as ordinary kernels, VLM
 *                       nodes on stream_a and action-head nodes on stream_b, as
 *                       CUDA graphs (the paper's "Baseline", Section 4, Fig. 7b)
 *   VLA_MODE_SERIAL     everything on stream_a in program order (Fig. 7a)
 *
 * All three modes run identical tile bodies with identical tile shapes and
 * reduction orders, so their action chunks are bit-identical.
 *
 * Conventions: every function returns an int status (VLA_OK = 0) and never
 * throws or aborts.  "host" / "device" is stated per pointer.  The library owns
 * nothing the caller passes in; it sub-allocates the caller's device arena and
 * owns only a few pinned host buffers, which vla_destroy releases.  Calls on one
 * context must come from one thread at a time.
 */
#ifndef VLA_H_
#define VLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vla_ctx vla_ctx; /* opaque; made by vla_init, freed by vla_destroy */

enum {
  VLA_OK = 0,
  VLA_ERR_INVALID = 1,   /* bad argument; no side effects */
  VLA_ERR_STATE = 2,     /* call not legal now (e.g. submit before weights are loaded) */
  VLA_ERR_BUSY = 3,      /* the stream's frame ring is full: poll first */
  VLA_ERR_NOT_READY = 4, /* no finished chunk for this stream yet */
  VLA_ERR_TIMEOUT = 5,   /* a bounded device-side wait ran out (sticky) */
  VLA_ERR_CUDA = 6,      /* a CUDA call failed (sticky) */
  VLA_ERR_NOMEM = 7      /* arena too small or host allocation failed */
};

enum { VLA_MODE_COSCHED = 0, VLA_MODE_TWO_STREAM = 1, VLA_MODE_SERIAL = 2, VLA_MODE_MULTI_STREAM = 3 };
/* VLA_MODE_MULTI_STREAM: like TWO_STREAM but one (VLM, head) pair of CUDA streams per
 * request stream, created by the library; reported as extra context next to TWO_STREAM. */

/* Pick policies of the persistent kernel.  TWO_PHASE is Algorithm 1; TWO_PHASE_G and TWO_PHASE_R are the two
 * fairness-augmented variants of its Phase-2 score (Section 4, "Implementations"): s * G_k / (c_k + 1) with G_k the
 * class's tiles still queued, and s / (c_k * R_k + 1) with R_k the class's shared-memory units per tile (registers
 * are fixed per worker group here).  CLASS_ORDER and ROUND_ROBIN are resource-blind comparison points. */
enum { VLA_POLICY_TWO_PHASE = 0, VLA_POLICY_CLASS_ORDER = 1, VLA_POLICY_ROUND_ROBIN = 2, VLA_POLICY_TWO_PHASE_G = 3,
       VLA_POLICY_TWO_PHASE_R = 4 };

enum { VLA_MLP_GELU = 0, VLA_MLP_SWIGLU = 1, VLA_MLP_GEGLU = 2 };
enum { VLA_HANDOFF_KV_LAST = 0, VLA_HANDOFF_KV_ALL = 1, VLA_HANDOFF_FEATURES = 2, VLA_HANDOFF_COG = 3 };
enum { VLA_HEAD_A = 0, VLA_HEAD_B = 1, VLA_HEAD_C = 2, VLA_HEAD_D = 3 };
enum { VLA_SOLVER_EULER = 0, VLA_SOLVER_DDIM = 1 };

/* Model description: one "VLM phase feeding an action head" model (Section 2.1).
 * Plain data; every field is a size or a flag.  Head kinds:
 *   A  self-attention + cross-attention straight onto the VLM's last-layer K,V
 *   B  expert whose layer l attends jointly over [VLM layer-l K,V ; its own K,V]
 *   C  DiT alternating self / cross attention (odd layers cross-attend to the
 *      VLM's final features), adaLN time conditioning
 *   D  DiT conditioned in-context on one cognition token (last VLM position) */
typedef struct {
  int32_t n_cam, img, patch;                                   /* cameras, square image side, square patch side */
  int32_t vis_layers, vis_d, vis_heads, vis_hd, vis_mlp;        /* vision encoder (vis_layers = 0: none) */
  int32_t shuffle, connector;                                   /* s x s token pixel-shuffle; linear connector flag */
  int32_t n_text, vocab;
  int32_t llm_layers, d, hq, hkv, hd, mlp, mlp_kind, rope, causal;
  int32_t handoff;
  int32_t head, act_layers, act_d, act_heads, act_mlp, act_mlp_kind;
  int32_t state_dim, horizon, act_dim, n_steps, solver;
  float guidance;           /* head D variant: classifier-free guidance scale s (0 = off).  Every denoising step evaluates the
                             * head twice -- with the condition token of a zero cognition feature, then with the real
                             * one -- and the solver takes eps_u + s (eps_c - eps_u) */
  int32_t suffix_mask;      /* head B variant: 1 = blocked suffix mask (the leading state token attends the prefix and itself,
                             * not the action tokens; the action tokens attend everything); 0 = unmasked joint attention */
  int32_t vis_layernorm;    /* vision encoder variant: 1 = LayerNorm (gain and shift, weights "...n1b", "...n2b", "vis.normb")
                             * in place of RMSNorm, and an fp32 bias vector on every linear layer of the encoder
                             * ("vis.patch.b", "...bq", "...bk", "...bv", "...bo", "...b1", "...b2"); 0 = RMSNorm, no biases */
} vla_model_desc;

typedef struct {
  void* arena;              /* device; caller-owned, >= vla_required_arena_bytes, 256-byte aligned */
  size_t arena_bytes;
  void* stream_a;           /* cudaStream_t, caller-owned: VLM nodes / the persistent kernel */
  void* stream_b;           /* cudaStream_t, caller-owned: action-head nodes (TWO_STREAM) */
  int32_t mode;             /* VLA_MODE_* */
  int32_t n_streams;        /* request streams R */
  int32_t ring_depth;       /* frames in flight per request stream, >= 2 */
  int32_t policy;           /* COSCHED pick: VLA_POLICY_* below */
  uint64_t wait_limit_ns;   /* bound of every device-side wait; 0 = default (5 s) */
  uint32_t trace_capacity;  /* tile records kept by the device trace; 0 = tracing off */
  int32_t workers_per_sm;   /* COSCHED worker groups per SM; 0 = default */
  int32_t u_max;            /* saturation value of the per-SM utilisation counters in the pick's Phase-2 score
                             * (Section 3.3); 0 = default: 15 x worker groups per SM (the hardware proposal's
                             * 8-bit registers would be 255) */
  int32_t head_passes;      /* asynchronous inference (Section 2.1, decoupled update rates of the two phases): the action
                             * head runs this many times per VLM pass, every pass on the same VLM output with its own
                             * robot state and noise sample; 0 or 1 = one pass per frame.  With P passes a frame's
                             * state is [P, state_dim], its noise [P, horizon, act_dim] and its chunk [P, horizon, act_dim] */
  int32_t reserved_;
} vla_runtime_opts;

typedef struct {
  const char* name;         /* e.g. "llm.L3.wq" */
  const void* host_ptr;     /* host; read during the call only */
  int32_t dtype;            /* 0 = fp32 (rounded to bf16 nearest-even where stored as bf16), 1 = bf16 bits */
  int32_t rank;
  int64_t shape[4];
} vla_tensor;

/* One executed tile, as recorded by the device trace (all modes).  In COSCHED mode the admission of a frame into
 * the persistent kernel is recorded too, as a record with node = 0xFFFFFFFF, cls = 0xFF and t_start = t_end. */
typedef struct {
  uint32_t inst;            /* request stream * ring_depth + ring slot */
  uint32_t node;            /* node index in the tile program */
  uint32_t tile;            /* tile index inside the node */
  uint16_t sm;              /* %smid */
  uint8_t worker;           /* worker group on that SM (0 in the ordinary-kernel modes) */
  uint8_t cls;              /* tile class: phase * 4 + kind (GEMM, gated GEMM, attention, elementwise) */
  uint64_t frame;           /* frame id the tile belonged to */
  uint64_t t_start, t_end;  /* %globaltimer, ns */
} vla_trace_rec;

/* Static description of one node of the tile program (for the trace checker). */
typedef struct {
  int32_t op, cls, n_tiles, n_pred;   /* n_pred: tiles of all predecessor nodes (what the node's counter waits for) */
  int32_t phase;            /* 0 VLM, 1 action head */
  int32_t step;             /* denoising step, -1 outside the loop */
  int32_t succ_begin, succ_count; /* range in the successor array */
  int32_t smem_bytes, tmem_cols;  /* shared memory and tensor-memory columns one tile of the node occupies */
  char name[48];
  double flops;             /* algorithmic FLOPs of the node: 2 M N K per matrix product, 4 Tq Tkv Hq hd per attention */
  double weight_bytes;      /* bf16 weight bytes the node's tiles stream (0 for nodes without a weight matrix) */
} vla_node_info;

/* Bytes of device arena a context needs (weights, tile program, queues, per-frame buffers). */
int vla_required_arena_bytes(const vla_model_desc* desc, const vla_runtime_opts* opts, size_t* out_bytes);

/* Builds the tile program for `desc` and lays the arena out.  Problem statement: Section 2.1. */
int vla_init(const vla_model_desc* desc, const vla_runtime_opts* opts, vla_ctx** out_ctx);

/* Copies the named tensors to the device (bf16), then runs the one-off constant
 * precomputation (time-embedding MLP, adaLN modulation vectors) on the GPU.
 * May be called several times; the call that completes the table arms the context.
 * A missing or mis-shaped tensor -> VLA_ERR_INVALID, named in vla_last_error. */
int vla_load_weights(vla_ctx* ctx, const vla_tensor* tensors, size_t n, int32_t final_call);

/* Enqueues one frame of request stream `stream` (Section 2.1: each frame = image(s) +
 * instruction tokens; the head also gets robot state and the initial noise sample).
 * All pointers are HOST memory.  They are copied before the call returns, with one exception:
 * an image of 64 KiB or more in page-locked (pinned) memory is read by an asynchronous copy,
 * so that buffer must stay valid and unmodified until this frame's chunk has been polled:
 * image fp32 [n_cam,3,img,img]; text_ids int32 [n_text]; state fp32 [state_dim] or NULL
 * when the model has none; noise fp32 [horizon,act_dim] (with head_passes = P > 1: state [P,state_dim], noise
 * [P,horizon,act_dim]).  Non-blocking with respect to
 * the GPU.  Ring full -> VLA_ERR_BUSY.  frame_id (optional) gets the per-stream frame number. */
int vla_submit_frame(vla_ctx* ctx, int32_t stream, const float* image, const int32_t* text_ids,
                     const float* state, const float* noise, uint64_t* frame_id);

/* Same as vla_submit_frame but the four inputs are DEVICE pointers (already resident
 * in HBM).  Nothing is copied: the tiles read the arrays in place through the frame
 * slot's pointer table, so the caller must keep them valid and unmodified until this
 * frame's chunk has been returned by vla_poll_actions (or the context is idle). */
int vla_submit_frame_device(vla_ctx* ctx, int32_t stream, const float* image, const int32_t* text_ids,
                            const float* state, const float* noise, uint64_t* frame_id);

/* Fetches the next finished action chunk of `stream`, in frame order (Section 2.1: the
 * head of frame N consumed frame N's VLM output).  chunk: HOST fp32 [horizon,act_dim]
 * ([head_passes,horizon,act_dim] with several head passes per frame: all of a frame's chunks arrive together).
 * Non-blocking; nothing ready -> VLA_ERR_NOT_READY. */
int vla_poll_actions(vla_ctx* ctx, int32_t stream, float* chunk, uint64_t* frame_id);

/* COSCHED mode: while the hold is on, submitted frames are queued for admission but the persistent kernel is not
 * launched; switching it off launches the kernel, which then admits everything queued at once (no counterpart in
 * the paper).  Lets a caller hand over a batch of frames -- up to ring_depth per stream -- as one launch, which is
 * also what a one-pass profiler capture of a whole multi-stream step needs. */
int vla_hold_launches(vla_ctx* ctx, int32_t on);

/* Blocks (host) until every submitted frame has produced its chunk or timeout_ms passed. */
int vla_wait_idle(vla_ctx* ctx, uint32_t timeout_ms);

/* Copies up to `cap` trace records (host memory) and reports how many exist. Call when idle. */
int vla_get_trace(vla_ctx* ctx, vla_trace_rec* recs, size_t cap, size_t* n);
int vla_reset_trace(vla_ctx* ctx);

/* Tile-program introspection for the trace checker: node table and successor array. */
int vla_program_info(vla_ctx* ctx, vla_node_info* nodes, size_t node_cap, size_t* n_nodes,
                     int32_t* succ, size_t succ_cap, size_t* n_succ);

/* Debug fetch of a named per-frame buffer (e.g. "llm.x", "llm.hidden", "act.v") of the ring
 * slot last used by `stream`, widened to fp32 into HOST memory `out` (cap floats). Call when idle. */
int vla_debug_fetch(vla_ctx* ctx, int32_t stream, int32_t slot, const char* buffer, float* out, size_t cap,
                    size_t* n);

/* Counters since init: tiles executed, kernels launched by the library, persistent-kernel launches. */
int vla_get_counters(vla_ctx* ctx, uint64_t* tiles, uint64_t* kernel_launches, uint64_t* persistent_launches);

/* Intensity tags of the eight tile classes (class = phase * 4 + kind, see vla_trace_rec): taus[8][3] =
 * (tau_TC, tau_ALU, tau_MEM), each 0..15 (Section 3.2.1, Table "Intensity Descriptor").  vla_init installs
 * hand-assigned defaults; vla_set_class_tags replaces them, e.g. by tags derived from a profiling pass (Section
 * 3.2.2).  Call while no frame is in flight; the persistent kernel reads the table when it is next launched.  HOST arrays. */
int vla_set_class_tags(vla_ctx* ctx, const int32_t* taus /*[8*3]*/);
int vla_get_class_tags(vla_ctx* ctx, int32_t* taus /*[8*3]*/);

/* Runs the device pick function (the COSCHED policy) once on the GPU for a given per-SM
 * state, so tests can compare it with Algorithm 1.  All arrays HOST, n_cls <= 8.
 * cta_count/u are updated as the admission would; *picked = class or -1; *phase = 1, 2 or 0.
 * u_max: saturation value used by the Phase-2 score (<= 0: the paper's 255). */
int vla_policy_probe(int32_t n_cls, const int32_t* taus /*[n_cls*3]*/, const int32_t* pending, const int32_t* feasible,
                     int32_t* cta_count, int32_t* u /*[3]*/, int32_t rr_start, int32_t u_max, int32_t* picked,
                     int32_t* phase);

/* Same probe for the scoring variants of Section 4: policy = VLA_POLICY_TWO_PHASE, _TWO_PHASE_G (needs grid[n_cls],
 * the G_k) or _TWO_PHASE_R (needs res[n_cls], the R_k); the unused array may be NULL. */
int vla_policy_probe_ex(int32_t n_cls, const int32_t* taus, const int32_t* pending, const int32_t* feasible,
                        int32_t* cta_count, int32_t* u, int32_t rr_start, int32_t u_max, int32_t policy, const int32_t* grid,
                        const int32_t* res, int32_t* picked, int32_t* phase);

/* Test hook for the failure path (no counterpart in the paper; Section 2.1 only states the dependency rule it
 * breaks on purpose): adds `delta` to the dependency counter of `node` in ring slot `slot` of `stream`, with a host
 * copy into the arena, while nothing is in flight.  A positive delta means the node never becomes ready: the next
 * frame through that slot stalls, the idle watchdog runs out after wait_limit_ns, the persistent kernel returns and
 * every later call reports the sticky VLA_ERR_TIMEOUT. */
int vla_debug_bump_dependency(vla_ctx* ctx, int32_t stream, int32_t slot, int32_t node, int32_t delta);

/* Stand-in for a memory checker (no counterpart in the paper): every per-frame and constant buffer of the arena is
 * followed by 64 guard bytes that no tile may write.  fill != 0 writes a pattern into all of them (call when idle,
 * after vla_load_weights); fill == 0 reads them back and reports in *n_bad how many guards were overwritten (the
 * first one is named in vla_last_error).  An out-of-bounds store of a tile body shows up here. */
int vla_debug_guards(vla_ctx* ctx, int32_t fill, size_t* n_bad);

/* ---- stand-alone operators: the engine's tile bodies on caller-owned DEVICE tensors ------------------------
 * Both run asynchronously on `stream` (a cudaStream_t; NULL = default stream). */

/* Fused attention, softmax(Q K^T / sqrt(hd)) V per head with grouped KV heads -- the attention of the VLM
 * decoder layers and of the action head (Section 2.1, Figure 1).  q [tq, hq*hd], k and v [tkv, hkv*hd],
 * out [tq, hq*hd]: bf16, row-major, DEVICE, 16-byte aligned.  hd a multiple of 16, at most 256; hq a
 * multiple of hkv; causal (key j visible to query i iff j <= i) needs tq == tkv.
 * scratch: DEVICE, 256-byte aligned, at least vla_op_attention_scratch_bytes(); the call writes an error
 * word and the transposed copy of v there, so calls sharing a scratch buffer must not overlap on the GPU. */
int vla_op_attention_scratch_bytes(int32_t tkv, int32_t hkv, int32_t hd, size_t* out_bytes);
int vla_op_attention(const void* q, const void* k, const void* v, void* out, int32_t tq, int32_t tkv, int32_t hq,
                     int32_t hkv, int32_t hd, int32_t causal, void* scratch, size_t scratch_bytes, void* stream);

/* Same attention for callers that cannot allocate device memory (no counterpart in the paper: this is a
 * deployment convenience).  Some callers of this library are not allowed to call cudaMalloc or to hand over
 * a scratch buffer: code that runs inside a real-time control loop with a fixed memory budget, a plugin whose
 * host owns every allocation, or a process that must not touch the allocator after start-up.  For them the
 * scratch of vla_op_attention (an error word plus the transposed copy of v) lives in a fixed array in device
 * memory that every GPU loading this library holds until the process exits.  The call allocates nothing:
 * no cudaMalloc, no cudaFree, no allocating library routine; the caller passes only inputs and outputs.
 * Limit: vla_op_attention_scratch_bytes(tkv, hkv, hd) must not exceed vla_op_attention_static_capacity()
 * (256 bytes + 4 MiB for the transposed v, e.g. hkv*hd = 1024 with up to 2048 keys); larger shapes are refused
 * with VLA_ERR_NOMEM and nothing runs.  The first call on each device looks the array's device address up
 * (with that device current); make that first call outside any stream capture.  All calls on a device share
 * the one array, which keeps whatever the previous call left: the call clears what it needs cleared, but two
 * calls that overlap on the GPU (different streams, or the same call from two threads) race on it -- run them
 * one after the other.  Arguments, layouts and results are those of vla_op_attention. */
int vla_op_attention_static_capacity(size_t* out_bytes);
int vla_op_attention_static(const void* q, const void* k, const void* v, void* out, int32_t tq, int32_t tkv, int32_t hq,
                            int32_t hkv, int32_t hd, int32_t causal, void* stream);

/* Linear layer y = act(x W^T) -- the dense contractions of both phases (Section 2.1; Section 2.3 calls them the
 * VLM's "large GEMMs").  a [m,k] and w [n,k] bf16 row-major DEVICE; k a multiple of 8; fp32 accumulation.
 * out32 (fp32 [m,n]) and/or out16 (bf16 [m,n]) DEVICE, either may be NULL.  act: 0 none, 1 GeLU (tanh form), 2 SiLU. */
int vla_op_linear(const void* a, const void* w, float* out32, void* out16, int32_t m, int32_t n, int32_t k, int32_t act,
                  void* stream);

/* Every device-side wait of the operators is bounded (2 s by default); a wait that runs out makes the kernel set
 * the call's error word and return, leaving garbage in the output.  vla_op_status waits for `stream` to drain and
 * reads that word back: VLA_OK, or VLA_ERR_TIMEOUT when a wait ran out.  op selects the word: VLA_OP_LINEAR (one
 * word per device, shared by all vla_op_linear calls on it: query before another call reuses it), VLA_OP_ATTENTION
 * (the word at the start of `scratch`, DEVICE) or VLA_OP_ATTENTION_STATIC (the library's fixed array). */
enum { VLA_OP_LINEAR = 0, VLA_OP_ATTENTION = 1, VLA_OP_ATTENTION_STATIC = 2 };
int vla_op_status(int32_t op, const void* scratch, void* stream);

/* Test hook: while drop_operand_loads is non-zero the operators' TMA producers issue no loads, so their consumers
 * wait for operands that never come and the bounded waits (wait_limit_ns; 0 = the default 2 s) run out.  Process-wide;
 * call with (0, 0) to restore normal operation. */
int vla_debug_op_fault(int32_t drop_operand_loads, uint64_t wait_limit_ns);

const char* vla_last_error(vla_ctx* ctx);
int vla_destroy(vla_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* VLA_H_ */
