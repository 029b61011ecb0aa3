// Host-side tile-program compiler: model description -> static DAG of nodes
// (each a set of independent tiles), arena layout, weight table.
#pragma once
#include <map>
#include <string>
#include <vector>

#include "../../include/vla.h"
#include "vla_types.h"

namespace vla {

// One tensor the caller must supply, and where its rows land on the device.
struct SourceTensor {
  std::string name;
  int64_t rows, cols;       // cols == 0: a vector of `rows` elements
  int dev;                  // index into Program::dev_tensors
  int64_t row_offset;       // first row inside the device tensor
  int64_t group_rows = 0;   // > 0: rows arrive in groups of group_rows (one head) placed group_stride rows apart
  int64_t group_stride = 0;
  bool loaded = false;
};

struct DevTensor {
  std::string name;
  int64_t rows, cols, ld;   // ld = padded row length in elements
  bool is_bf16;             // matrices bf16, gains/position tables fp32
  uint64_t offset;          // arena byte offset
  int tmap = -1;            // tensor-map index for GEMM weights
};

struct BufInfo {
  std::string name;
  uint64_t offset;          // slot-relative (or arena-relative for constants)
  uint64_t bytes;
  bool slot;
  int64_t rows, ld;         // logical 2-D view for debug fetch
  int elem;                 // 4 fp32, 2 bf16
};

constexpr uint64_t GUARD_BYTES = 64;   // guard words behind every buffer (see vla_debug_guards)

struct TmapSpec {           // a 2-D bf16 row-major tensor to describe to the TMA unit
  uint64_t offset;          // arena or slot-relative byte offset
  bool slot;
  int64_t rows, cols, ld;   // extents and row pitch in elements
  int box_rows;             // rows per box (box columns = GEMM_BK)
};

struct Program {
  vla_model_desc desc;
  int n_streams = 0, ring_depth = 0, n_inst = 0;
  int head_passes = 1;                  // action-head passes per VLM pass

  std::vector<NodeDesc> nodes;
  std::vector<std::string> node_names;
  std::vector<double> node_flops, node_wbytes;   // algorithmic FLOPs of a node and the weight bytes its tiles stream
  std::vector<int32_t> succ;
  std::vector<int32_t> roots;
  std::vector<int> init_nodes;          // nodes of the one-off constant precomputation (separate program)
  std::vector<NodeDesc> init_program;   // run serially once after the weights are loaded
  ClassInfo classes[N_CLASSES];

  std::vector<SourceTensor> sources;
  std::map<std::string, int> source_index;
  std::vector<DevTensor> dev_tensors;
  std::map<std::string, int> dev_index;
  std::vector<BufInfo> bufs;
  std::map<std::string, int> buf_index;
  std::vector<std::pair<int, int>> folds;  // (weight matrix, gain vector): columns of the matrix get multiplied by the gain at load
  std::vector<TmapSpec> wmaps;          // weight maps (shared by all frame slots)
  std::vector<TmapSpec> amaps;          // activation maps, instantiated once per frame slot

  // time arguments of the denoising steps and solver coefficients
  std::vector<float> step_args, step_c_x, step_c_acc;

  // arena layout (byte offsets)
  uint64_t off_weights = 0, off_consts = 0, off_nodes = 0, off_succ = 0, off_roots = 0, off_classes = 0,
           off_control = 0, off_queues = 0, off_q_entries = 0, off_admit = 0, off_dep = 0,
           off_inst_frame = 0, off_slot_base = 0, off_input_ptrs = 0, off_trace = 0, off_tmaps = 0,
           off_init_nodes = 0, off_slots = 0;
  uint64_t slot_bytes = 0, arena_bytes = 0, zero_bytes_begin = 0;
  int q_capacity = 0, admit_capacity = 0;
  uint32_t trace_capacity = 0;

  // input buffers inside a slot
  uint64_t in_image = 0, in_text = 0, in_state = 0, in_noise = 0;
  uint64_t image_bytes = 0, text_bytes = 0, state_bytes = 0, noise_bytes = 0;

  std::string error;
};

// Builds the program; returns false and sets p.error on an invalid description.
bool build_program(const vla_model_desc& d, const vla_runtime_opts& o, Program& p);

}  // namespace vla
