// C ABI of the library (see include/vla.h): context set-up, weight upload, frame
// submission / polling, and the three run modes built on the same tile bodies.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <thread>
#include <vector>

#include "../../include/vla.h"
#include "dispatch.cuh"
#include "program.h"

using namespace vla;

struct InstHost {
  int state = 0;            // 0 free, 1 submitted (in flight), chunk not yet polled
  uint64_t frame = 0;
  cudaGraphExec_t g_vlm = nullptr, g_act = nullptr, g_all = nullptr;
  cudaEvent_t ev_in = nullptr, ev_vlm = nullptr;
};

struct vla_ctx {
  Program prog;
  vla_runtime_opts opts;
  DeviceCtx dctx;
  char* arena = nullptr;
  cudaStream_t sa = nullptr, sb = nullptr, scopy = nullptr;
  std::vector<cudaStream_t> multi_a, multi_b;
  bool armed = false;
  std::string err;
  int sticky = VLA_OK;
  // pinned host memory
  char* staging = nullptr;          // [n_inst][staging_bytes] mirror of the slot input region
  size_t staging_bytes = 0;
  uint64_t in_lo = 0;               // slot-relative start of the input region
  DoneRec* done_host = nullptr;
  float* chunk_host = nullptr;
  unsigned* error_host = nullptr;
  AdmitRec* admit_pinned = nullptr; // ring of admission records (source of the device copies)
  unsigned long long* tail_pinned = nullptr;
  unsigned* zero_pinned = nullptr;
  uint64_t* inptr_pinned = nullptr; // [n_inst][N_FRAME_INPUTS] source of the input pointer table copies
  unsigned long long n_admitted = 0;
  std::vector<InstHost> inst;
  std::vector<uint64_t> next_submit, next_poll;   // per request stream frame counters
  // persistent kernel
  cudaEvent_t ev_kernel = nullptr;
  bool kernel_launched = false;
  bool hold_launches = false;       // submits queue their frames but do not launch the persistent kernel
  int sm_count = 0, dyn_smem = 0, workers = MAX_WORKERS;
  uint64_t pending_frames = 0;      // submitted, chunk not yet observed
  uint64_t n_kernel_launches = 0, n_persistent_launches = 0, n_tiles_streams = 0;
  int max_node_smem = 0;
};

namespace {

int fail(vla_ctx* c, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) {
    c->err = buf;
    if (code == VLA_ERR_CUDA || code == VLA_ERR_TIMEOUT) c->sticky = code;
  }
  return code;
}

#define CU(call)                                                                                         \
  do {                                                                                                   \
    cudaError_t e_ = (call);                                                                             \
    if (e_ != cudaSuccess) return fail(c, VLA_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

template <typename T>
T* at(vla_ctx* c, uint64_t off) { return reinterpret_cast<T*>(c->arena + off); }

unsigned short f32_to_bf16_host(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  uint32_t r = ((u >> 16) & 1u) + 0x7FFFu;
  return (unsigned short)((u + r) >> 16);
}

int check_device_error(vla_ctx* c) {
  if (c->sticky != VLA_OK) return c->sticky;
  unsigned code = *reinterpret_cast<volatile unsigned*>(c->error_host);
  if (code != 0) {
    c->sticky = VLA_ERR_TIMEOUT;
    c->err = "device-side wait ran out (code " + std::to_string(code) + ")";
    return c->sticky;
  }
  return VLA_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Encodes every TMA tensor map (2-D bf16, 128-byte swizzle, 64-column boxes, zero fill outside) and uploads the table.
int build_tensor_maps(vla_ctx* c) {
  const Program& p = c->prog;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CU(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(c, VLA_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
  const size_t total = p.wmaps.size() + p.amaps.size() * (size_t)p.n_inst;
  std::vector<CUtensorMap> maps(total + 1);
  auto enc = [&](const TmapSpec& sp, char* base, CUtensorMap* out) -> bool {
    cuuint64_t dims[2] = {(cuuint64_t)sp.cols, (cuuint64_t)sp.rows};
    cuuint64_t strides[1] = {(cuuint64_t)sp.ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)GEMM_BK, (cuuint32_t)sp.box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
  };
  for (size_t i = 0; i < p.wmaps.size(); ++i)
    if (!enc(p.wmaps[i], c->arena + p.wmaps[i].offset, &maps[i])) return fail(c, VLA_ERR_CUDA, "weight tensor map %zu rejected", i);
  for (int inst = 0; inst < p.n_inst; ++inst)
    for (size_t i = 0; i < p.amaps.size(); ++i) {
      const TmapSpec& sp = p.amaps[i];
      char* base = c->arena + sp.offset + (sp.slot ? p.off_slots + (uint64_t)inst * p.slot_bytes : 0);
      if (!enc(sp, base, &maps[p.wmaps.size() + (size_t)inst * p.amaps.size() + i]))
        return fail(c, VLA_ERR_CUDA, "activation tensor map %zu rejected", i);
    }
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  CU(cudaMemcpy(c->arena + p.off_tmaps, maps.data(), total * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
  return VLA_OK;
}

int launch_node(vla_ctx* c, const NodeDesc* dev_nodes, const NodeDesc& n, int idx, int inst, cudaStream_t s) {
  vla_node_kernel<<<n.n_tiles, WORKER_THREADS, n.smem_bytes, s>>>(c->dctx, dev_nodes, idx, inst);
  c->n_kernel_launches++;
  CU(cudaGetLastError());
  return VLA_OK;
}

int capture_graph(vla_ctx* c, int inst, int phase_sel, cudaStream_t s, cudaGraphExec_t* out) {
  const Program& p = c->prog;
  cudaGraph_t g;
  CU(cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal));
  uint64_t launches_before = c->n_kernel_launches;
  for (size_t i = 0; i < p.nodes.size(); ++i) {
    if (phase_sel >= 0 && p.nodes[i].phase != phase_sel) continue;
    int rc = launch_node(c, c->dctx.nodes, p.nodes[i], (int)i, inst, s);
    if (rc != VLA_OK) { cudaStreamEndCapture(s, &g); return rc; }
  }
  c->n_kernel_launches = launches_before;   // captured, not launched
  CU(cudaStreamEndCapture(s, &g));
  CU(cudaGraphInstantiate(out, g, 0));
  CU(cudaGraphDestroy(g));
  return VLA_OK;
}

uint64_t count_phase_nodes(const Program& p, int phase_sel) {
  uint64_t n = 0;
  for (auto& nd : p.nodes) if (phase_sel < 0 || nd.phase == phase_sel) ++n;
  return n;
}

int launch_persistent(vla_ctx* c) {
  // reset the control word in stream order, then launch one CTA per SM
  CU(cudaMemcpyAsync(&c->dctx.control->ctrl, c->zero_pinned, sizeof(unsigned), cudaMemcpyHostToDevice, c->sa));
  vla_cosched_kernel<<<c->sm_count, c->workers * WORKER_THREADS + DISPATCH_THREADS, c->dyn_smem, c->sa>>>(c->dctx, c->dyn_smem);
  CU(cudaGetLastError());
  CU(cudaEventRecord(c->ev_kernel, c->sa));
  c->kernel_launched = true;
  c->n_persistent_launches++;
  c->n_kernel_launches++;
  return VLA_OK;
}

// RMSNorm gains are folded into the matrices that consume the normalised rows: W[n][k] *= g[k] (bf16, nearest even).
__global__ void vla_fold_gain_kernel(unsigned short* w, int64_t rows, int cols, int64_t ld, const float* g) {
  const int64_t total = rows * cols;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = e / cols;
    const int k = (int)(e % cols);
    unsigned short* p = w + r * ld + k;
    *p = f32_to_bf16_bits(bf16_bits_to_f32(*p) * g[k]);
  }
}

// (Re)launch the persistent kernel if it is not running and frames are waiting.
int ensure_persistent(vla_ctx* c) {
  if (c->pending_frames == 0 || c->hold_launches) return VLA_OK;
  if (c->kernel_launched) {
    cudaError_t q = cudaEventQuery(c->ev_kernel);
    if (q == cudaErrorNotReady) return VLA_OK;
    if (q != cudaSuccess) return fail(c, VLA_ERR_CUDA, "persistent kernel failed: %s", cudaGetErrorString(q));
  }
  return launch_persistent(c);
}

int submit_common(vla_ctx* c, int32_t stream, const float* image, const int32_t* text_ids, const float* state,
                  const float* noise, uint64_t* frame_id, bool device_inputs) {
  if (!c) return VLA_ERR_INVALID;
  int rc = check_device_error(c);
  if (rc != VLA_OK) return rc;
  if (!c->armed) return fail(c, VLA_ERR_STATE, "weights are not loaded");
  const Program& p = c->prog;
  const vla_model_desc& d = p.desc;
  if (stream < 0 || stream >= p.n_streams) return fail(c, VLA_ERR_INVALID, "stream %d out of range", stream);
  if (!image || !text_ids || !noise || (d.state_dim > 0 && !state))
    return fail(c, VLA_ERR_INVALID, "a required input pointer is NULL");
  if (!device_inputs)
    for (int i = 0; i < d.n_text; ++i)
      if (text_ids[i] < 0 || text_ids[i] >= d.vocab) return fail(c, VLA_ERR_INVALID, "text id %d out of vocabulary", text_ids[i]);
  const uint64_t f = c->next_submit[stream];
  const int slot = (int)(f % p.ring_depth);
  const int inst = stream * p.ring_depth + slot;
  InstHost& ih = c->inst[inst];
  if (ih.state != 0) return fail(c, VLA_ERR_BUSY, "frame ring of stream %d is full", stream);

  char* slot_dev = c->arena + p.off_slots + (uint64_t)inst * p.slot_bytes;
  uint64_t* ip = c->inptr_pinned + (size_t)inst * N_FRAME_INPUTS;
  if (device_inputs) {
    // resident inputs are read in place: only their addresses travel
    ip[0] = reinterpret_cast<uint64_t>(image); ip[1] = reinterpret_cast<uint64_t>(text_ids);
    ip[2] = reinterpret_cast<uint64_t>(state); ip[3] = reinterpret_cast<uint64_t>(noise);
  } else {
    char* st = c->staging + (size_t)inst * c->staging_bytes;
    // The image is by far the largest input.  From page-locked memory it is copied straight from the caller's
    // buffer (no staging pass on the host, which would keep this thread from polling the other streams);
    // everything else, and images in pageable memory, go through the pinned staging block.
    uint64_t rest_lo = std::min(p.in_text, p.in_noise);
    if (d.state_dim > 0) rest_lo = std::min(rest_lo, p.in_state);
    cudaPointerAttributes pa;
    const bool direct = p.image_bytes >= (64u << 10) && rest_lo >= p.in_image + p.image_bytes &&
                        cudaPointerGetAttributes(&pa, image) == cudaSuccess && pa.type == cudaMemoryTypeHost;
    if (!direct) { cudaGetLastError(); std::memcpy(st + (p.in_image - c->in_lo), image, p.image_bytes); }
    std::memcpy(st + (p.in_text - c->in_lo), text_ids, p.text_bytes);
    if (d.state_dim > 0) std::memcpy(st + (p.in_state - c->in_lo), state, p.state_bytes);
    std::memcpy(st + (p.in_noise - c->in_lo), noise, p.noise_bytes);
    if (direct) {
      CU(cudaMemcpyAsync(slot_dev + p.in_image, image, p.image_bytes, cudaMemcpyHostToDevice, c->scopy));
      CU(cudaMemcpyAsync(slot_dev + rest_lo, st + (rest_lo - c->in_lo), c->in_lo + c->staging_bytes - rest_lo,
                         cudaMemcpyHostToDevice, c->scopy));
    } else {
      CU(cudaMemcpyAsync(slot_dev + c->in_lo, st, c->staging_bytes, cudaMemcpyHostToDevice, c->scopy));
    }
    ip[0] = reinterpret_cast<uint64_t>(slot_dev + p.in_image); ip[1] = reinterpret_cast<uint64_t>(slot_dev + p.in_text);
    ip[2] = reinterpret_cast<uint64_t>(slot_dev + p.in_state); ip[3] = reinterpret_cast<uint64_t>(slot_dev + p.in_noise);
  }
  CU(cudaMemcpyAsync(const_cast<uint64_t*>(c->dctx.input_ptrs) + (size_t)inst * N_FRAME_INPUTS, ip,
                     sizeof(uint64_t) * N_FRAME_INPUTS, cudaMemcpyHostToDevice, c->scopy));
  ih.state = 1;
  ih.frame = f;
  c->done_host[inst].frame_plus1 = 0;
  c->next_submit[stream] = f + 1;
  c->pending_frames++;
  if (frame_id) *frame_id = f;

  // admission record (frame id + slot); in the stream modes only the frame id is used
  const unsigned long long t = c->n_admitted++;
  const size_t ri = (size_t)(t % (unsigned long long)p.admit_capacity);
  c->admit_pinned[ri].inst = (uint32_t)inst;
  c->admit_pinned[ri].pad = 0;
  c->admit_pinned[ri].frame = f;
  c->tail_pinned[ri] = t + 1;

  if (c->opts.mode == VLA_MODE_COSCHED) {
    CU(cudaMemcpyAsync(c->dctx.admit_ring + ri, c->admit_pinned + ri, sizeof(AdmitRec), cudaMemcpyHostToDevice, c->scopy));
    CU(cudaMemcpyAsync(&c->dctx.control->admit_tail, c->tail_pinned + ri, sizeof(unsigned long long),
                       cudaMemcpyHostToDevice, c->scopy));
    return ensure_persistent(c);
  }

  CU(cudaMemcpyAsync(c->dctx.inst_frame + inst, &c->admit_pinned[ri].frame, sizeof(uint64_t), cudaMemcpyHostToDevice, c->scopy));
  CU(cudaEventRecord(ih.ev_in, c->scopy));
  cudaStream_t a = c->sa, b = c->sb;
  if (c->opts.mode == VLA_MODE_MULTI_STREAM) { a = c->multi_a[stream]; b = c->multi_b[stream]; }
  CU(cudaStreamWaitEvent(a, ih.ev_in, 0));
  if (c->opts.mode == VLA_MODE_SERIAL) {
    if (!ih.g_all) { rc = capture_graph(c, inst, -1, a, &ih.g_all); if (rc != VLA_OK) return rc; }
    CU(cudaGraphLaunch(ih.g_all, a));
    c->n_kernel_launches += p.nodes.size();
    return VLA_OK;
  }
  if (!ih.g_vlm) { rc = capture_graph(c, inst, PHASE_VLM, a, &ih.g_vlm); if (rc != VLA_OK) return rc; }
  if (!ih.g_act) { rc = capture_graph(c, inst, PHASE_ACT, b, &ih.g_act); if (rc != VLA_OK) return rc; }
  CU(cudaGraphLaunch(ih.g_vlm, a));
  CU(cudaEventRecord(ih.ev_vlm, a));
  CU(cudaStreamWaitEvent(b, ih.ev_vlm, 0));
  CU(cudaStreamWaitEvent(b, ih.ev_in, 0));
  CU(cudaGraphLaunch(ih.g_act, b));
  c->n_kernel_launches += p.nodes.size();
  return VLA_OK;
}

}  // namespace

extern "C" {

int vla_required_arena_bytes(const vla_model_desc* desc, const vla_runtime_opts* opts, size_t* out_bytes) {
  if (!desc || !opts || !out_bytes) return VLA_ERR_INVALID;
  Program p;
  if (!build_program(*desc, *opts, p)) return VLA_ERR_INVALID;
  *out_bytes = p.arena_bytes;
  return VLA_OK;
}

int vla_init(const vla_model_desc* desc, const vla_runtime_opts* opts, vla_ctx** out_ctx) {
  if (!desc || !opts || !out_ctx) return VLA_ERR_INVALID;
  *out_ctx = nullptr;
  if (opts->mode < 0 || opts->mode > 3 || !opts->arena) return VLA_ERR_INVALID;
  vla_ctx* c = new vla_ctx();
  c->opts = *opts;
  if (!build_program(*desc, *opts, c->prog)) { delete c; return VLA_ERR_INVALID; }
  Program& p = c->prog;
  if (opts->arena_bytes < p.arena_bytes || (reinterpret_cast<uintptr_t>(opts->arena) & 255)) { delete c; return VLA_ERR_NOMEM; }
  c->arena = static_cast<char*>(opts->arena);
  c->sa = static_cast<cudaStream_t>(opts->stream_a);
  c->sb = static_cast<cudaStream_t>(opts->stream_b);
  *out_ctx = c;   // from here on the caller can read vla_last_error and must call vla_destroy

  int dev = 0;
  CU(cudaGetDevice(&dev));
  CU(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
  int max_optin = 0;
  CU(cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  c->dyn_smem = max_optin - 1024;   // leave the static/reserved part alone
  c->workers = opts->workers_per_sm > 0 ? (opts->workers_per_sm > MAX_WORKERS ? MAX_WORKERS : opts->workers_per_sm) : MAX_WORKERS;
  CU(cudaFuncSetAttribute(vla_cosched_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, c->dyn_smem));
  for (auto& n : p.nodes) c->max_node_smem = std::max(c->max_node_smem, n.smem_bytes);
  for (auto& n : p.init_program) c->max_node_smem = std::max(c->max_node_smem, n.smem_bytes);
  if (c->max_node_smem > c->dyn_smem - SM_STATE_BYTES) return fail(c, VLA_ERR_INVALID, "a tile needs more shared memory than an SM has");
  // field widths of a queue entry (one 64-bit word)
  if (p.nodes.size() >= (1u << QW_NODE_BITS) || p.n_inst > (1 << QW_INST_BITS))
    return fail(c, VLA_ERR_INVALID, "tile program too large for the queue entry layout (nodes < 2^20, streams x ring depth <= 512)");
  for (auto& n : p.nodes)
    if (n.n_tiles > (1 << QW_TILE_BITS) || (n.smem_bytes + SMEM_UNIT - 1) / SMEM_UNIT >= (1 << QW_SMEM_BITS) ||
        (n.tmem_cols + TMEM_UNIT - 1) / TMEM_UNIT >= (1 << QW_TMEM_BITS))
      return fail(c, VLA_ERR_INVALID, "a node has more tiles or needs more memory than a queue entry can describe");
  CU(cudaFuncSetAttribute(vla_node_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, std::max(c->max_node_smem, 1024)));
  CU(cudaStreamCreateWithFlags(&c->scopy, cudaStreamNonBlocking));
  CU(cudaEventCreateWithFlags(&c->ev_kernel, cudaEventDisableTiming));

  // zero everything behind the weights, then upload the static tables
  CU(cudaMemsetAsync(c->arena + p.zero_bytes_begin, 0, p.arena_bytes - p.zero_bytes_begin, c->sa));
  CU(cudaStreamSynchronize(c->sa));
  CU(cudaMemcpy(at<char>(c, p.off_nodes), p.nodes.data(), sizeof(NodeDesc) * p.nodes.size(), cudaMemcpyHostToDevice));
  if (!p.init_program.empty())
    CU(cudaMemcpy(at<char>(c, p.off_init_nodes), p.init_program.data(), sizeof(NodeDesc) * p.init_program.size(), cudaMemcpyHostToDevice));
  if (!p.succ.empty()) {
    std::vector<SuccInfo> si(p.succ.size());
    for (size_t i = 0; i < si.size(); ++i) {
      const NodeDesc& sn = p.nodes[p.succ[i]];
      const int res = ((sn.smem_bytes + SMEM_UNIT - 1) / SMEM_UNIT) | (((sn.tmem_cols + TMEM_UNIT - 1) / TMEM_UNIT) << QW_SMEM_BITS);
      si[i] = SuccInfo{p.succ[i], sn.n_tiles, sn.cls | (res << 8), sn.n_pred};
    }
    CU(cudaMemcpy(at<char>(c, p.off_succ), si.data(), sizeof(SuccInfo) * si.size(), cudaMemcpyHostToDevice));
  }
  CU(cudaMemcpy(at<char>(c, p.off_roots), p.roots.data(), 4 * p.roots.size(), cudaMemcpyHostToDevice));
  CU(cudaMemcpy(at<char>(c, p.off_classes), p.classes, sizeof(ClassInfo) * N_CLASSES, cudaMemcpyHostToDevice));
  {
    std::vector<int32_t> dep((size_t)p.n_inst * p.nodes.size());
    for (int i = 0; i < p.n_inst; ++i)
      for (size_t k = 0; k < p.nodes.size(); ++k) dep[(size_t)i * p.nodes.size() + k] = p.nodes[k].n_pred;
    CU(cudaMemcpy(at<char>(c, p.off_dep), dep.data(), 4 * dep.size(), cudaMemcpyHostToDevice));
    std::vector<uint64_t> sb(p.n_inst);
    for (int i = 0; i < p.n_inst; ++i) sb[i] = p.off_slots + (uint64_t)i * p.slot_bytes;
    CU(cudaMemcpy(at<char>(c, p.off_slot_base), sb.data(), 8 * sb.size(), cudaMemcpyHostToDevice));
    int args_buf = p.buf_index.at("const.args");
    CU(cudaMemcpy(c->arena + p.off_consts + p.bufs[args_buf].offset, p.step_args.data(), 4 * p.step_args.size(), cudaMemcpyHostToDevice));
  }

  // pinned host memory
  c->in_lo = p.in_image;
  c->staging_bytes = (size_t)(p.in_noise + p.noise_bytes - c->in_lo);
  CU(cudaHostAlloc(&c->staging, c->staging_bytes * p.n_inst, cudaHostAllocDefault));
  std::memset(c->staging, 0, c->staging_bytes * p.n_inst);
  CU(cudaHostAlloc(&c->done_host, sizeof(DoneRec) * p.n_inst, cudaHostAllocMapped));
  std::memset((void*)c->done_host, 0, sizeof(DoneRec) * p.n_inst);
  const size_t chunk_elems = (size_t)p.head_passes * desc->horizon * desc->act_dim;
  CU(cudaHostAlloc(&c->chunk_host, sizeof(float) * chunk_elems * p.n_inst, cudaHostAllocMapped));
  CU(cudaHostAlloc(&c->error_host, 64, cudaHostAllocMapped));
  *c->error_host = 0;
  CU(cudaHostAlloc(&c->admit_pinned, sizeof(AdmitRec) * p.admit_capacity, cudaHostAllocDefault));
  CU(cudaHostAlloc(&c->tail_pinned, sizeof(unsigned long long) * p.admit_capacity, cudaHostAllocDefault));
  CU(cudaHostAlloc(&c->inptr_pinned, sizeof(uint64_t) * N_FRAME_INPUTS * p.n_inst, cudaHostAllocDefault));
  CU(cudaHostAlloc(&c->zero_pinned, 64, cudaHostAllocDefault));
  std::memset(c->zero_pinned, 0, 64);

  DeviceCtx& x = c->dctx;
  std::memset(&x, 0, sizeof x);
  x.arena = c->arena;
  x.nodes = at<NodeDesc>(c, p.off_nodes);
  x.succ = at<SuccInfo>(c, p.off_succ);
  x.classes = at<ClassInfo>(c, p.off_classes);
  x.control = at<Control>(c, p.off_control);
  x.queues = at<TileQueue>(c, p.off_queues);
  x.q_entries = at<QueueEntry>(c, p.off_q_entries);
  x.admit_ring = at<AdmitRec>(c, p.off_admit);
  x.dep_count = at<int32_t>(c, p.off_dep);
  x.inst_frame = at<uint64_t>(c, p.off_inst_frame);
  x.slot_base = at<uint64_t>(c, p.off_slot_base);
  x.input_ptrs = at<uint64_t>(c, p.off_input_ptrs);
  x.roots = at<int32_t>(c, p.off_roots);
  x.trace = at<TraceRec>(c, p.off_trace);
  void* dp = nullptr;
  CU(cudaHostGetDevicePointer(&dp, (void*)c->done_host, 0)); x.done_host = static_cast<DoneRec*>(dp);
  CU(cudaHostGetDevicePointer(&dp, c->chunk_host, 0)); x.chunk_host = static_cast<float*>(dp);
  CU(cudaHostGetDevicePointer(&dp, c->error_host, 0)); x.error_host = static_cast<unsigned*>(dp);
  x.tmaps = at<char>(c, p.off_tmaps);
  x.n_weight_tmaps = (int)p.wmaps.size();
  x.n_act_tmaps = (int)p.amaps.size();
  {
    int rc = build_tensor_maps(c);
    if (rc != VLA_OK) return rc;
  }
  x.n_nodes = (int)p.nodes.size();
  x.n_inst = p.n_inst;
  x.n_roots = (int)p.roots.size();
  x.q_capacity = p.q_capacity;
  x.q_shift = 0;
  while ((1 << x.q_shift) < p.q_capacity) ++x.q_shift;
  x.admit_capacity = p.admit_capacity;
  x.trace_capacity = p.trace_capacity;
  x.policy = opts->policy;
  x.workers_per_sm = c->workers;
  x.u_max = opts->u_max > 0 ? opts->u_max : 15 * c->workers;
  x.wait_limit_ns = opts->wait_limit_ns ? opts->wait_limit_ns : 5000000000ull;
  x.idle_exit_ns = 200000ull;
  x.chunk_elems = (int)chunk_elems;

  c->inst.resize(p.n_inst);
  for (auto& ih : c->inst) {
    CU(cudaEventCreateWithFlags(&ih.ev_in, cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&ih.ev_vlm, cudaEventDisableTiming));
  }
  c->next_submit.assign(p.n_streams, 0);
  c->next_poll.assign(p.n_streams, 0);
  if (opts->mode == VLA_MODE_MULTI_STREAM) {
    c->multi_a.resize(p.n_streams);
    c->multi_b.resize(p.n_streams);
    for (int r = 0; r < p.n_streams; ++r) {
      CU(cudaStreamCreateWithFlags(&c->multi_a[r], cudaStreamNonBlocking));
      CU(cudaStreamCreateWithFlags(&c->multi_b[r], cudaStreamNonBlocking));
    }
  }
  return VLA_OK;
}

int vla_load_weights(vla_ctx* c, const vla_tensor* tensors, size_t n, int32_t final_call) {
  if (!c || (!tensors && n)) return VLA_ERR_INVALID;
  if (c->sticky != VLA_OK) return c->sticky;
  if (c->armed) return fail(c, VLA_ERR_STATE, "weights already loaded");
  Program& p = c->prog;
  std::vector<unsigned short> tmp;
  for (size_t i = 0; i < n; ++i) {
    const vla_tensor& t = tensors[i];
    if (!t.name || !t.host_ptr) return fail(c, VLA_ERR_INVALID, "tensor %zu has no name or data", i);
    auto it = p.source_index.find(t.name);
    if (it == p.source_index.end()) return fail(c, VLA_ERR_INVALID, "unknown tensor '%s'", t.name);
    SourceTensor& s = p.sources[it->second];
    const DevTensor& dt = p.dev_tensors[s.dev];
    bool shape_ok = s.cols == 0 ? (t.rank == 1 && t.shape[0] == s.rows)
                                : (t.rank == 2 && t.shape[0] == s.rows && t.shape[1] == s.cols);
    if (!shape_ok) return fail(c, VLA_ERR_INVALID, "tensor '%s' has the wrong shape", t.name);
    char* dst = c->arena + p.off_weights + dt.offset;
    if (!dt.is_bf16) {
      if (t.dtype != 0) return fail(c, VLA_ERR_INVALID, "tensor '%s' must be fp32", t.name);
      size_t count = s.cols == 0 ? (size_t)s.rows : (size_t)s.rows * s.cols;
      if (s.cols == 0) dst += (size_t)s.row_offset * 4;        // a vector may be one part of a stacked vector
      if (s.cols == 0 && s.group_rows > 0)                     // per-head parts, each head padded to group_stride
        CU(cudaMemcpy2D(dst, (size_t)s.group_stride * 4, t.host_ptr, (size_t)s.group_rows * 4, (size_t)s.group_rows * 4,
                        (size_t)(s.rows / s.group_rows), cudaMemcpyHostToDevice));
      else
        CU(cudaMemcpy(dst, t.host_ptr, count * 4, cudaMemcpyHostToDevice));
    } else {
      dst += (size_t)s.row_offset * dt.ld * 2;
      const void* src = t.host_ptr;
      if (t.dtype == 0) {
        tmp.resize((size_t)s.rows * s.cols);
        const float* f = static_cast<const float*>(t.host_ptr);
        for (size_t k = 0; k < tmp.size(); ++k) tmp[k] = f32_to_bf16_host(f[k]);
        src = tmp.data();
      } else if (t.dtype != 1) {
        return fail(c, VLA_ERR_INVALID, "tensor '%s': unknown dtype", t.name);
      }
      // padding columns [cols, ld) and padding rows between heads stay zero (the arena was cleared at init)
      if (s.group_rows > 0) {
        for (int64_t g0 = 0, gi = 0; g0 < s.rows; g0 += s.group_rows, ++gi)
          CU(cudaMemcpy2D(dst + (size_t)gi * s.group_stride * dt.ld * 2, (size_t)dt.ld * 2,
                          static_cast<const char*>(src) + (size_t)g0 * s.cols * 2, (size_t)s.cols * 2, (size_t)s.cols * 2,
                          (size_t)s.group_rows, cudaMemcpyHostToDevice));
      } else {
        CU(cudaMemcpy2D(dst, (size_t)dt.ld * 2, src, (size_t)s.cols * 2, (size_t)s.cols * 2, (size_t)s.rows, cudaMemcpyHostToDevice));
      }
    }
    s.loaded = true;
  }
  if (!final_call) return VLA_OK;
  for (auto& s : p.sources)
    if (!s.loaded) return fail(c, VLA_ERR_INVALID, "tensor '%s' was not supplied", s.name.c_str());
  // fold the RMSNorm gains into the weights of the GEMMs that apply those norms (each pair once)
  {
    std::vector<std::pair<int, int>> done;
    for (auto& f : p.folds) {
      if (std::find(done.begin(), done.end(), f) != done.end()) continue;
      done.push_back(f);
      const DevTensor& wt = p.dev_tensors[f.first];
      const DevTensor& gt = p.dev_tensors[f.second];
      vla_fold_gain_kernel<<<592, 256, 0, c->sa>>>(reinterpret_cast<unsigned short*>(c->arena + p.off_weights + wt.offset), wt.rows,
                                                   (int)wt.cols, wt.ld,
                                                   reinterpret_cast<const float*>(c->arena + p.off_weights + gt.offset));
      CU(cudaGetLastError());
    }
  }
  // one-off constants (time-embedding MLP, adaLN modulation) on the GPU, serially
  const NodeDesc* init_dev = at<NodeDesc>(c, p.off_init_nodes);
  for (size_t i = 0; i < p.init_program.size(); ++i) {
    int rc = launch_node(c, init_dev, p.init_program[i], (int)i, -1, c->sa);
    if (rc != VLA_OK) return rc;
  }
  CU(cudaStreamSynchronize(c->sa));
  c->armed = true;
  return VLA_OK;
}

int vla_submit_frame(vla_ctx* c, int32_t stream, const float* image, const int32_t* text_ids, const float* state,
                     const float* noise, uint64_t* frame_id) {
  return submit_common(c, stream, image, text_ids, state, noise, frame_id, false);
}

int vla_submit_frame_device(vla_ctx* c, int32_t stream, const float* image, const int32_t* text_ids, const float* state,
                            const float* noise, uint64_t* frame_id) {
  return submit_common(c, stream, image, text_ids, state, noise, frame_id, true);
}

int vla_poll_actions(vla_ctx* c, int32_t stream, float* chunk, uint64_t* frame_id) {
  if (!c) return VLA_ERR_INVALID;
  int rc = check_device_error(c);
  if (rc != VLA_OK) return rc;
  const Program& p = c->prog;
  if (stream < 0 || stream >= p.n_streams || !chunk) return fail(c, VLA_ERR_INVALID, "bad stream or NULL chunk");
  const uint64_t f = c->next_poll[stream];
  if (f >= c->next_submit[stream]) return VLA_ERR_NOT_READY;
  const int inst = stream * p.ring_depth + (int)(f % p.ring_depth);
  if (c->done_host[inst].frame_plus1 != f + 1) {
    if (c->opts.mode == VLA_MODE_COSCHED) {
      rc = ensure_persistent(c);
      if (rc != VLA_OK) return rc;
    }
    return VLA_ERR_NOT_READY;
  }
  std::atomic_thread_fence(std::memory_order_acquire);
  std::memcpy(chunk, c->chunk_host + (size_t)inst * c->dctx.chunk_elems, sizeof(float) * c->dctx.chunk_elems);
  if (frame_id) *frame_id = f;
  c->inst[inst].state = 0;
  c->next_poll[stream] = f + 1;
  c->pending_frames--;
  return VLA_OK;
}

int vla_hold_launches(vla_ctx* c, int32_t on) {
  if (!c) return VLA_ERR_INVALID;
  c->hold_launches = on != 0;
  if (!c->hold_launches && c->opts.mode == VLA_MODE_COSCHED) {
    CU(cudaStreamSynchronize(c->scopy));      // the queued admission records are in device memory before the launch
    return ensure_persistent(c);
  }
  return VLA_OK;
}

int vla_wait_idle(vla_ctx* c, uint32_t timeout_ms) {
  if (!c) return VLA_ERR_INVALID;
  auto t0 = std::chrono::steady_clock::now();
  const Program& p = c->prog;
  for (;;) {
    int rc = check_device_error(c);
    if (rc != VLA_OK) return rc;
    bool all = true;
    for (int r = 0; r < p.n_streams && all; ++r)
      for (uint64_t f = c->next_poll[r]; f < c->next_submit[r]; ++f) {
        int inst = r * p.ring_depth + (int)(f % p.ring_depth);
        if (c->done_host[inst].frame_plus1 != f + 1) { all = false; break; }
      }
    if (all) break;
    if (c->opts.mode == VLA_MODE_COSCHED) {
      rc = ensure_persistent(c);
      if (rc != VLA_OK) return rc;
    }
    auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
    if (ms > (long long)timeout_ms) return fail(c, VLA_ERR_NOT_READY, "wait_idle timed out");
    std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
  return VLA_OK;
}

int vla_get_trace(vla_ctx* c, vla_trace_rec* recs, size_t cap, size_t* n) {
  if (!c || !n) return VLA_ERR_INVALID;
  CU(cudaDeviceSynchronize());
  Control ctl;
  CU(cudaMemcpy(&ctl, c->dctx.control, sizeof ctl, cudaMemcpyDeviceToHost));
  size_t have = (size_t)std::min<unsigned long long>(ctl.trace_count, c->prog.trace_capacity);
  *n = (size_t)ctl.trace_count;
  size_t take = std::min(have, cap);
  static_assert(sizeof(vla_trace_rec) == sizeof(TraceRec), "trace record layout");
  if (recs && take) CU(cudaMemcpy(recs, c->dctx.trace, take * sizeof(TraceRec), cudaMemcpyDeviceToHost));
  return VLA_OK;
}

int vla_reset_trace(vla_ctx* c) {
  if (!c) return VLA_ERR_INVALID;
  CU(cudaDeviceSynchronize());
  CU(cudaMemset(&c->dctx.control->trace_count, 0, sizeof(unsigned long long)));
  return VLA_OK;
}

int vla_program_info(vla_ctx* c, vla_node_info* nodes, size_t node_cap, size_t* n_nodes, int32_t* succ, size_t succ_cap,
                     size_t* n_succ) {
  if (!c || !n_nodes || !n_succ) return VLA_ERR_INVALID;
  const Program& p = c->prog;
  *n_nodes = p.nodes.size();
  *n_succ = p.succ.size();
  if (nodes)
    for (size_t i = 0; i < std::min(node_cap, p.nodes.size()); ++i) {
      const NodeDesc& n = p.nodes[i];
      vla_node_info& o = nodes[i];
      o.op = n.op; o.cls = n.cls; o.n_tiles = n.n_tiles; o.n_pred = n.n_pred; o.phase = n.phase; o.step = n.step;
      o.succ_begin = n.succ_begin; o.succ_count = n.succ_count;
      o.smem_bytes = n.smem_bytes; o.tmem_cols = n.tmem_cols;
      std::memset(o.name, 0, sizeof o.name);
      std::strncpy(o.name, p.node_names[i].c_str(), sizeof(o.name) - 1);
      o.flops = p.node_flops[i];
      o.weight_bytes = p.node_wbytes[i];
    }
  if (succ)
    for (size_t i = 0; i < std::min(succ_cap, p.succ.size()); ++i) succ[i] = p.succ[i];
  return VLA_OK;
}

int vla_debug_fetch(vla_ctx* c, int32_t stream, int32_t slot, const char* buffer, float* out, size_t cap, size_t* n) {
  if (!c || !buffer || !n) return VLA_ERR_INVALID;
  const Program& p = c->prog;
  auto it = p.buf_index.find(buffer);
  if (it == p.buf_index.end()) return fail(c, VLA_ERR_INVALID, "unknown buffer '%s'", buffer);
  const BufInfo& b = p.bufs[it->second];
  if (b.slot && (stream < 0 || stream >= p.n_streams || slot < 0 || slot >= p.ring_depth)) return VLA_ERR_INVALID;
  size_t count = (size_t)b.rows * b.ld;
  *n = count;
  if (!out) return VLA_OK;
  if (cap < count) return fail(c, VLA_ERR_INVALID, "buffer '%s' needs %zu floats", buffer, count);
  CU(cudaDeviceSynchronize());
  const char* src = c->arena + (b.slot ? p.off_slots + (uint64_t)(stream * p.ring_depth + slot) * p.slot_bytes : p.off_consts) + b.offset;
  if (b.elem == 4) {
    CU(cudaMemcpy(out, src, count * 4, cudaMemcpyDeviceToHost));
  } else {
    std::vector<unsigned short> tmp(count);
    CU(cudaMemcpy(tmp.data(), src, count * 2, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < count; ++i) {
      uint32_t u = (uint32_t)tmp[i] << 16;
      std::memcpy(out + i, &u, 4);
    }
  }
  return VLA_OK;
}

int vla_get_counters(vla_ctx* c, uint64_t* tiles, uint64_t* kernel_launches, uint64_t* persistent_launches) {
  if (!c) return VLA_ERR_INVALID;
  if (tiles) {
    Control ctl;
    CU(cudaMemcpy(&ctl, c->dctx.control, sizeof ctl, cudaMemcpyDeviceToHost));
    *tiles = ctl.tiles_done;
  }
  if (kernel_launches) *kernel_launches = c->n_kernel_launches;
  if (persistent_launches) *persistent_launches = c->n_persistent_launches;
  return VLA_OK;
}

int vla_policy_probe_ex(int32_t n_cls, const int32_t* taus, const int32_t* pending, const int32_t* feasible,
                        int32_t* cta_count, int32_t* u, int32_t rr_start, int32_t u_max, int32_t policy, const int32_t* grid,
                        const int32_t* res, int32_t* picked, int32_t* phase) {
  if (n_cls < 1 || n_cls > PICK_MAX_CLASSES || !taus || !pending || !feasible || !cta_count || !u || !picked || !phase)
    return VLA_ERR_INVALID;
  if (policy < POLICY_TWO_PHASE || policy > POLICY_TWO_PHASE_R) return VLA_ERR_INVALID;
  if ((policy == POLICY_TWO_PHASE_G && !grid) || (policy == POLICY_TWO_PHASE_R && !res)) return VLA_ERR_INVALID;
  // inputs and outputs of the probe in one block: one allocation, one copy each way
  struct Block { PickState st; int tau[PICK_MAX_CLASSES * 3]; int grid[PICK_MAX_CLASSES]; int res[PICK_MAX_CLASSES]; int out[2]; } h;
  std::memset(&h, 0, sizeof h);
  unsigned pm = 0, fm = 0;
  for (int k = 0; k < n_cls; ++k) {
    h.st.cta_count[k] = cta_count[k];
    if (pending[k]) pm |= 1u << k;
    if (feasible[k]) fm |= 1u << k;
    for (int x = 0; x < 3; ++x) h.tau[k * 3 + x] = taus[k * 3 + x];
    h.grid[k] = grid ? grid[k] : 1;
    h.res[k] = res ? res[k] : 1;
  }
  for (int x = 0; x < 3; ++x) h.st.u[x] = u[x];
  h.out[0] = -1;
  Block* d = nullptr;
  if (cudaMalloc(&d, sizeof h) != cudaSuccess) return VLA_ERR_CUDA;
  cudaMemcpy(d, &h, sizeof h, cudaMemcpyHostToDevice);
  vla_pick_probe_kernel<<<1, 1>>>(n_cls, d->tau, pm, fm, &d->st, rr_start, policy, u_max > 0 ? u_max : PICK_U_MAX, d->grid,
                                  d->res, d->out);
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(&h, d, sizeof h, cudaMemcpyDeviceToHost);
  cudaFree(d);
  if (e != cudaSuccess) return VLA_ERR_CUDA;
  for (int k = 0; k < n_cls; ++k) cta_count[k] = h.st.cta_count[k];
  for (int x = 0; x < 3; ++x) u[x] = h.st.u[x];
  *picked = h.out[0];
  *phase = h.out[1];
  return VLA_OK;
}

int vla_policy_probe(int32_t n_cls, const int32_t* taus, const int32_t* pending, const int32_t* feasible, int32_t* cta_count,
                     int32_t* u, int32_t rr_start, int32_t u_max, int32_t* picked, int32_t* phase) {
  return vla_policy_probe_ex(n_cls, taus, pending, feasible, cta_count, u, rr_start, u_max, POLICY_TWO_PHASE, nullptr, nullptr,
                             picked, phase);
}

int vla_set_class_tags(vla_ctx* c, const int32_t* taus) {
  if (!c || !taus) return VLA_ERR_INVALID;
  for (int i = 0; i < N_CLASSES * 3; ++i)
    if (taus[i] < 0 || taus[i] > 15) return fail(c, VLA_ERR_INVALID, "intensity tags are 4-bit values (0..15)");
  if (c->pending_frames != 0) return fail(c, VLA_ERR_STATE, "frames are in flight");
  CU(cudaDeviceSynchronize());          // an idle persistent kernel leaves within its idle limit
  for (int k = 0; k < N_CLASSES; ++k)
    for (int x = 0; x < 3; ++x) c->prog.classes[k].tau[x] = taus[k * 3 + x];
  CU(cudaMemcpy(at<char>(c, c->prog.off_classes), c->prog.classes, sizeof(ClassInfo) * N_CLASSES, cudaMemcpyHostToDevice));
  return VLA_OK;
}

int vla_get_class_tags(vla_ctx* c, int32_t* taus) {
  if (!c || !taus) return VLA_ERR_INVALID;
  for (int k = 0; k < N_CLASSES; ++k)
    for (int x = 0; x < 3; ++x) taus[k * 3 + x] = c->prog.classes[k].tau[x];
  return VLA_OK;
}

int vla_debug_guards(vla_ctx* c, int32_t fill, size_t* n_bad) {
  if (!c || (!fill && !n_bad)) return VLA_ERR_INVALID;
  if (c->pending_frames != 0) return fail(c, VLA_ERR_STATE, "frames are in flight");
  CU(cudaDeviceSynchronize());
  const Program& p = c->prog;
  unsigned char pat[GUARD_BYTES], got[GUARD_BYTES];
  std::memset(pat, 0xC5, sizeof pat);
  size_t bad = 0;
  for (const BufInfo& b : p.bufs) {
    if (b.name.compare(0, 3, "in.") == 0) continue;      // the staged input copy spans the input buffers, guards included
    const int copies = b.slot ? p.n_inst : 1;
    for (int i = 0; i < copies; ++i) {
      char* g = c->arena + (b.slot ? p.off_slots + (uint64_t)i * p.slot_bytes : p.off_consts) + b.offset + b.bytes;
      if (fill) {
        CU(cudaMemcpy(g, pat, GUARD_BYTES, cudaMemcpyHostToDevice));
      } else {
        CU(cudaMemcpy(got, g, GUARD_BYTES, cudaMemcpyDeviceToHost));
        if (std::memcmp(got, pat, GUARD_BYTES) != 0 && bad++ == 0)
          c->err = "guard behind buffer '" + b.name + "' of frame slot " + std::to_string(i) + " was overwritten";
      }
    }
  }
  if (n_bad) *n_bad = bad;
  return VLA_OK;
}

int vla_debug_bump_dependency(vla_ctx* c, int32_t stream, int32_t slot, int32_t node, int32_t delta) {
  if (!c) return VLA_ERR_INVALID;
  const Program& p = c->prog;
  if (stream < 0 || stream >= p.n_streams || slot < 0 || slot >= p.ring_depth || node < 0 || node >= (int)p.nodes.size())
    return fail(c, VLA_ERR_INVALID, "bad stream, slot or node");
  if (c->pending_frames != 0) return fail(c, VLA_ERR_STATE, "frames are in flight");
  CU(cudaDeviceSynchronize());
  int32_t* cnt = c->dctx.dep_count + (size_t)(stream * p.ring_depth + slot) * p.nodes.size() + node;
  int32_t v = 0;
  CU(cudaMemcpy(&v, cnt, sizeof v, cudaMemcpyDeviceToHost));
  v += delta;
  CU(cudaMemcpy(cnt, &v, sizeof v, cudaMemcpyHostToDevice));
  return VLA_OK;
}

const char* vla_last_error(vla_ctx* c) { return c ? c->err.c_str() : "null context"; }

int vla_destroy(vla_ctx* c) {
  if (!c) return VLA_ERR_INVALID;
  if (c->dctx.control && c->kernel_launched) {
    unsigned one = 1;
    cudaMemcpyAsync(&c->dctx.control->stop, &one, sizeof one, cudaMemcpyHostToDevice, c->scopy);
    cudaStreamSynchronize(c->scopy);
  }
  cudaDeviceSynchronize();
  for (auto& ih : c->inst) {
    if (ih.g_vlm) cudaGraphExecDestroy(ih.g_vlm);
    if (ih.g_act) cudaGraphExecDestroy(ih.g_act);
    if (ih.g_all) cudaGraphExecDestroy(ih.g_all);
    if (ih.ev_in) cudaEventDestroy(ih.ev_in);
    if (ih.ev_vlm) cudaEventDestroy(ih.ev_vlm);
  }
  for (auto s : c->multi_a) cudaStreamDestroy(s);
  for (auto s : c->multi_b) cudaStreamDestroy(s);
  if (c->scopy) cudaStreamDestroy(c->scopy);
  if (c->ev_kernel) cudaEventDestroy(c->ev_kernel);
  if (c->staging) cudaFreeHost(c->staging);
  if (c->done_host) cudaFreeHost((void*)c->done_host);
  if (c->chunk_host) cudaFreeHost(c->chunk_host);
  if (c->error_host) cudaFreeHost(c->error_host);
  if (c->admit_pinned) cudaFreeHost(c->admit_pinned);
  if (c->tail_pinned) cudaFreeHost(c->tail_pinned);
  if (c->zero_pinned) cudaFreeHost(c->zero_pinned);
  if (c->inptr_pinned) cudaFreeHost(c->inptr_pinned);
  delete c;
  return VLA_OK;
}

}  // extern "C"

#include "ops_api.cuh"

// ------------------------------------------------------------------------------------------------
// Attention without any allocation: the scratch of vla_op_attention (error word + transposed V)
// lives in a fixed array in device memory that every GPU loading this library holds until exit.
// In host code the array's name is only a handle; the device address is looked up once per device
// with cudaGetSymbolAddress and that pointer is what the kernels receive.
// ------------------------------------------------------------------------------------------------
#define VLA_OP_ATTENTION_STATIC_VT_BYTES (4u << 20)   /* room for the transposed V: 4 MiB */
static __device__ __align__(256) unsigned char g_attention_static_scratch[256 + VLA_OP_ATTENTION_STATIC_VT_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<void*> g_static_scratch_ptr[kMaxDevices];

// Device address of the static scratch on the current device (looked up on the first call per device).
int static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VLA_ERR_CUDA;
  void* p = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_attention_static_scratch) != cudaSuccess || !p) return VLA_ERR_CUDA;
    g_static_scratch_ptr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return VLA_OK;
}
}  // namespace

extern "C" {

int vla_op_attention_static_capacity(size_t* out_bytes) {
  if (!out_bytes) return VLA_ERR_INVALID;
  *out_bytes = sizeof(g_attention_static_scratch);
  return VLA_OK;
}

int vla_op_attention_static(const void* q, const void* k, const void* v, void* out, int32_t tq, int32_t tkv, int32_t hq,
                            int32_t hkv, int32_t hd, int32_t causal, void* stream) {
  if (!q || !k || !v || !out || !vla::op_attention_shape_ok(tq, tkv, hq, hkv, hd)) return VLA_ERR_INVALID;
  if (causal && tq != tkv) return VLA_ERR_INVALID;
  if (vla::op_attention_scratch_bytes(tkv, hkv, hd) > sizeof(g_attention_static_scratch)) return VLA_ERR_NOMEM;
  void* scratch = nullptr;
  int rc = static_scratch_for_current_device(&scratch);
  if (rc != VLA_OK) return rc;
  // op_attention_run clears the error word itself; V^T is fully rewritten for the rows and tokens it reads
  return vla::op_attention_run(q, k, v, out, tq, tkv, hq, hkv, hd, causal, scratch, static_cast<cudaStream_t>(stream));
}

int vla_op_status(int32_t op, const void* scratch, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (op == VLA_OP_LINEAR) {
    unsigned* w = vla::op_linear_error_word();
    return w ? vla::op_status_of(w, s) : VLA_ERR_CUDA;
  }
  if (op == VLA_OP_ATTENTION) {
    if (!scratch) return VLA_ERR_INVALID;
    return vla::op_status_of(static_cast<const unsigned*>(scratch), s);
  }
  if (op == VLA_OP_ATTENTION_STATIC) {
    void* p = nullptr;
    int rc = static_scratch_for_current_device(&p);
    return rc != VLA_OK ? rc : vla::op_status_of(static_cast<const unsigned*>(p), s);
  }
  return VLA_ERR_INVALID;
}

}  // extern "C"
