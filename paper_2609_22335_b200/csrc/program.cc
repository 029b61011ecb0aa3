// Tile-program compiler (host).  Turns a model description into:
//   * the device weight table (fused / padded layouts),
//   * per-frame-slot activation buffers,
//   * a static DAG of nodes in program order, with dependencies derived from the
//     buffers each node reads and writes (RAW, WAW and WAR edges),
//   * the one-off constant precomputation program,
//   * the arena layout.
// The forward pass it encodes is the two-phase VLA model of paper Section 2.1 /
// Figure 1 at the shapes of the five workload descriptions.
#include "program.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>

namespace vla {
namespace {

inline int64_t pad_to(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct View {          // rows [row0, row0+rows) of a buffer, starting at column col0
  int buf = -1;
  int64_t row0 = 0, rows = 0, col0 = 0;
};

struct Access {
  uint64_t lo, hi;
  int node;
  bool write;
};

class Builder {
 public:
  Program& p;
  const vla_model_desc& m;
  std::vector<std::vector<Access>> acc;   // per buffer
  std::vector<std::vector<int>> preds;    // per node
  uint64_t slot_cursor = 0, const_cursor = 0, weight_cursor = 0;
  int phase = PHASE_VLM, step = -1;
  bool init_mode = false;                 // nodes go to the constant-precomputation program
  std::string name_suffix;                // appended to node names (head passes after the first)

  Builder(Program& prog) : p(prog), m(prog.desc) {}

  // ---------------------------------------------------------------- buffers
  int buf(const std::string& name, int64_t rows, int64_t ld, int elem, bool slot = true) {
    BufInfo b;
    b.name = name; b.rows = rows; b.ld = ld; b.elem = elem; b.slot = slot;
    b.bytes = (uint64_t)rows * ld * elem;
    uint64_t& cur = slot ? slot_cursor : const_cursor;
    cur = align_up(cur, 256);
    b.offset = cur;
    cur += b.bytes + GUARD_BYTES;         // guard words behind the buffer: nothing may ever write them
    p.bufs.push_back(b);
    p.buf_index[name] = (int)p.bufs.size() - 1;
    acc.emplace_back();
    return (int)p.bufs.size() - 1;
  }
  std::map<int, int> ss_of;     // bf16 stream mirror -> its per-row partial sums of squares
  // bf16 mirror of a residual stream of width d plus, per row, one sum of squares per 128 columns
  int stream_mirror(const std::string& name, int64_t nrows, int64_t d) {
    int bf = buf(name, nrows, pad_to(d, GEMM_BK), 2);
    int ss = buf(name + ".ss", nrows, (d + GEMM_BM - 1) / GEMM_BM, 4);
    ss_of[bf] = ss;
    return bf;
  }
  View ss_view(const View& v) const {
    auto it = ss_of.find(v.buf);
    if (it == ss_of.end()) return View();
    return View{it->second, v.row0, v.rows, 0};
  }
  static Ref in_ref(int idx, uint64_t byte_off = 0) { return REF_INPUT | ((uint64_t)idx << 56) | byte_off; }
  View all(int b) const { return View{b, 0, p.bufs[b].rows, 0}; }
  View rows(int b, int64_t r0, int64_t n, int64_t c0 = 0) const { return View{b, r0, n, c0}; }
  int64_t ld(const View& v) const { return p.bufs[v.buf].ld; }

  Ref ref(const View& v) const {
    if (v.buf < 0) return 0;
    const BufInfo& b = p.bufs[v.buf];
    uint64_t off = b.offset + (uint64_t)(v.row0 * b.ld + v.col0) * b.elem;
    return b.slot ? (off | REF_SLOT) : (const_base + off);
  }
  static constexpr uint64_t WEIGHT_BASE = 4096;  // arena offset of the weight region (offset 0 stays "null")
  uint64_t const_base = 0;                       // arena offset of the constant region, fixed once all weights are declared

  // ---------------------------------------------------------------- weights
  int dev_tensor(const std::string& name, int64_t rows, int64_t cols, bool is_bf16) {
    DevTensor t;
    t.name = name; t.rows = rows; t.cols = cols; t.is_bf16 = is_bf16;
    t.ld = is_bf16 ? pad_to(cols, GEMM_BK) : cols;
    weight_cursor = align_up(weight_cursor, 256);
    t.offset = weight_cursor;
    weight_cursor += (uint64_t)rows * t.ld * (is_bf16 ? 2 : 4);
    p.dev_tensors.push_back(t);
    p.dev_index[name] = (int)p.dev_tensors.size() - 1;
    return (int)p.dev_tensors.size() - 1;
  }
  void source(const std::string& name, int64_t rows, int64_t cols, int dev, int64_t row_off) {
    SourceTensor s;
    s.name = name; s.rows = rows; s.cols = cols; s.dev = dev; s.row_offset = row_off;
    p.source_index[name] = (int)p.sources.size();
    p.sources.push_back(s);
  }
  // a matrix made of one or more caller tensors stacked by rows
  int matrix(const std::string& dev_name, const std::vector<std::string>& parts, const std::vector<int64_t>& part_rows,
             int64_t cols) {
    int64_t rows = 0;
    for (auto r : part_rows) rows += r;
    int d = dev_tensor(dev_name, rows, cols, true);
    int64_t off = 0;
    for (size_t i = 0; i < parts.size(); ++i) {
      source(parts[i], part_rows[i], cols, d, off);
      off += part_rows[i];
    }
    return d;
  }
  int matrix1(const std::string& name, int64_t rows, int64_t cols) { return matrix(name, {name}, {rows}, cols); }
  // stacked per-head projections whose heads are padded from hd to hs rows (padding rows stay zero)
  int matrix_heads(const std::string& dev_name, const std::vector<std::string>& parts, const std::vector<int64_t>& part_heads,
                   int64_t hd, int64_t hs, int64_t cols) {
    if (hd == hs) {
      std::vector<int64_t> r;
      for (auto h : part_heads) r.push_back(h * hd);
      return matrix(dev_name, parts, r, cols);
    }
    int64_t heads = 0;
    for (auto h : part_heads) heads += h;
    int d = dev_tensor(dev_name, heads * hs, cols, true);
    int64_t off = 0;
    for (size_t i = 0; i < parts.size(); ++i) {
      source(parts[i], part_heads[i] * hd, cols, d, off);
      p.sources.back().group_rows = hd;
      p.sources.back().group_stride = hs;
      off += part_heads[i] * hs;
    }
    return d;
  }
  int table(const std::string& name, int64_t rows, int64_t cols) {   // fp32 position table
    int d = dev_tensor(name, rows, cols, false);
    source(name, rows, cols, d, 0);
    return d;
  }
  int gain(const std::string& name, int64_t n) {
    int d = dev_tensor(name, 1, n, false);
    SourceTensor s;
    s.name = name; s.rows = n; s.cols = 0; s.dev = d; s.row_offset = 0;
    p.source_index[name] = (int)p.sources.size();
    p.sources.push_back(s);
    return d;
  }
  // an fp32 vector made of per-head vectors stacked with each head padded from hd to hs elements (padding stays zero)
  int vector_heads(const std::string& dev_name, const std::vector<std::string>& parts, const std::vector<int64_t>& part_heads,
                   int64_t hd, int64_t hs) {
    int64_t heads = 0;
    for (auto h : part_heads) heads += h;
    int d = dev_tensor(dev_name, 1, heads * hs, false);
    int64_t off = 0;
    for (size_t i = 0; i < parts.size(); ++i) {
      SourceTensor s;
      s.name = parts[i]; s.rows = part_heads[i] * hd; s.cols = 0; s.dev = d; s.row_offset = off;
      if (hd != hs) { s.group_rows = hd; s.group_stride = hs; }
      p.source_index[s.name] = (int)p.sources.size();
      p.sources.push_back(s);
      off += part_heads[i] * hs;
    }
    return d;
  }
  Ref wref(int dev, int64_t row0 = 0) const {
    const DevTensor& t = p.dev_tensors[dev];
    return WEIGHT_BASE + t.offset + (uint64_t)row0 * t.ld * (t.is_bf16 ? 2 : 4);
  }

  // ---------------------------------------------------------------- nodes and dependencies
  void region(const View& v, uint64_t& lo, uint64_t& hi) const {
    const BufInfo& b = p.bufs[v.buf];
    lo = (uint64_t)v.row0 * b.ld * b.elem;
    hi = (uint64_t)(v.row0 + v.rows) * b.ld * b.elem;
  }
  void read(int node, const View& v) {
    if (v.buf < 0 || init_mode) return;
    uint64_t lo, hi;
    region(v, lo, hi);
    for (const Access& a : acc[v.buf])
      if (a.write && a.lo < hi && lo < a.hi && a.node != node) preds[node].push_back(a.node);
    acc[v.buf].push_back(Access{lo, hi, node, false});
  }
  void write(int node, const View& v) {
    if (v.buf < 0 || init_mode) return;
    uint64_t lo, hi;
    region(v, lo, hi);
    auto& list = acc[v.buf];
    for (const Access& a : list)
      if (a.lo < hi && lo < a.hi && a.node != node) preds[node].push_back(a.node);
    // accesses fully covered by this write are superseded: later nodes reach them through this one
    list.erase(std::remove_if(list.begin(), list.end(),
                              [&](const Access& a) { return a.lo >= lo && a.hi <= hi && a.node != node; }),
               list.end());
    list.push_back(Access{lo, hi, node, true});
  }

  int add(NodeDesc n, const std::string& name, int kind) {
    n.phase = phase;
    n.step = step;
    n.cls = phase * N_KINDS + kind;
    n.n_pred = 0;
    n.succ_begin = n.succ_count = 0;
    if (init_mode) {
      p.init_program.push_back(n);
      return (int)p.init_program.size() - 1;
    }
    p.nodes.push_back(n);
    p.node_names.push_back(name + name_suffix);
    p.node_flops.push_back(0.0);
    p.node_wbytes.push_back(0.0);
    preds.emplace_back();
    return (int)p.nodes.size() - 1;
  }
  NodeDesc& node(int i) { return init_mode ? p.init_program[i] : p.nodes[i]; }

  // ---------------------------------------------------------------- op builders
  struct GemmOpt {
    View X; float c_x = 1.f, c_acc = 1.f;
    Ref vec = 0;
    Ref tab = 0; int ldtab = 0;
    Ref tab2 = 0; int ldtab2 = 0;
    View out32, out16, outT;
    View tabv;               // an fp32 [M, ld] addend that is one of the frame's buffers (read dependency tracked)
    int t_col0 = 0;
    int act = ACT_NONE;
    int W2 = -1;
    int bias = -1;           // >= 0: an fp32 [N] device tensor added to the accumulator before the activation
    int64_t w_row0 = 0;
    int norm_gain = -1;      // >= 0: A is the raw residual stream; RMSNorm with this gain is folded into the GEMM
    int norm_d = 0;
  };
  int gemm(const std::string& name, const View& A, int W, int64_t N, const GemmOpt& o) {
    const DevTensor& wt = p.dev_tensors[W];
    NodeDesc n;
    std::memset(&n, 0, sizeof(n));
    n.op = OP_GEMM;
    GemmArgs& g = n.u.gemm;
    g.A = ref(A); g.lda = (int)ld(A);
    g.W = wref(W, o.w_row0);
    g.W2 = o.W2 >= 0 ? wref(o.W2, o.w_row0) : 0;
    g.dual = o.W2 >= 0;
    g.M = (int)A.rows; g.N = (int)N; g.Kp = (int)wt.ld;
    g.X = ref(o.X); g.ldx = o.X.buf >= 0 ? (int)ld(o.X) : 0;
    g.c_x = o.c_x; g.c_acc = o.c_acc;
    g.bias = o.bias >= 0 ? wref(o.bias) : 0;
    g.vec = o.vec; g.tab = o.tab; g.ldtab = o.ldtab; g.tab2 = o.tab2; g.ldtab2 = o.ldtab2;
    if (o.tabv.buf >= 0) { g.tab = ref(o.tabv); g.ldtab = (int)ld(o.tabv); }
    g.out32 = ref(o.out32); g.ldo32 = o.out32.buf >= 0 ? (int)ld(o.out32) : 0;
    g.out16 = ref(o.out16); g.ldo16 = o.out16.buf >= 0 ? (int)ld(o.out16) : 0;
    g.outT = ref(o.outT); g.ldoT = o.outT.buf >= 0 ? (int)ld(o.outT) : 0; g.t_col0 = o.t_col0;
    g.act = o.act;
    g.rs_d = 0; g.ss_nft = 0; g.ss_out_ld = 0; g.ss_in = 0; g.ss_out = 0;
    const View ss_in = o.norm_gain >= 0 ? ss_view(A) : View();
    const View ss_out = ss_view(o.out16);
    if (ss_in.buf >= 0) { g.ss_in = ref(ss_in); g.ss_nft = (int)ld(ss_in); }
    if (ss_out.buf >= 0) { g.ss_out = ref(ss_out); g.ss_out_ld = (int)ld(ss_out); }
    if (o.norm_gain >= 0) {
      if (ss_in.buf < 0) p.error = "internal: folded norm needs a stream mirror as operand (" + name + ")";
      g.rs_d = o.norm_d;
      p.folds.push_back({W, o.norm_gain});
      if (o.W2 >= 0) p.folds.push_back({o.W2, o.norm_gain});
    }
    int tiles_t = (int)((g.M + GEMM_MAX_BT - 1) / GEMM_MAX_BT);
    int bt = (int)pad_to((g.M + tiles_t - 1) / tiles_t, 16);
    g.bt = bt; g.tiles_t = tiles_t;
    {
      // pipeline depth from the stage size; tensor maps for the operands
      // A gated tile covers 64 output features: rows 0..63 of its 128-row weight tile come from the gate matrix,
      // rows 64..127 from the up matrix (two 64-row TMA boxes), so it is one accumulator and has the shared and
      // tensor-memory shape of a plain tile.
      const int S = gemm_stages(bt, g.Kp);
      g.stages = S;
      n.smem_bytes = gemm_smem_bytes(bt, S);
      n.tmem_cols = (int)pad_to((int64_t)bt, TMEM_UNIT);
      g.wmap = weight_map(W, N, g.dual ? GEMM_BM / 2 : GEMM_BM);
      g.w2map = o.W2 >= 0 ? weight_map(o.W2, N, GEMM_BM / 2) : 0;
      if (g.dual && o.bias >= 0) p.error = "a gated GEMM takes no bias";
      if (g.dual && (N % 4 != 0 || o.X.buf >= 0 || o.outT.buf >= 0 || o.out32.buf >= 0 || o.tab || o.tab2 || o.vec))
        p.error = "internal: a gated GEMM writes bf16 only, width a multiple of 4 (" + name + ")";
      g.amap = act_map(A, g.Kp, bt);
    }
    const int feat_per_tile = g.dual ? GEMM_BM / 2 : GEMM_BM;
    n.n_tiles = (int)((g.N + feat_per_tile - 1) / feat_per_tile) * tiles_t;
    int id = add(n, name, g.dual ? KIND_GEMM2 : KIND_GEMM);
    if (!init_mode) {
      const double mats = g.dual ? 2.0 : 1.0;
      p.node_flops[id] = mats * 2.0 * (double)g.M * (double)g.N * (double)wt.cols;
      p.node_wbytes[id] = mats * 2.0 * (double)g.N * (double)wt.cols;
    }
    read(id, A);
    if (o.X.buf >= 0) read(id, o.X);
    if (o.tabv.buf >= 0) read(id, o.tabv);
    if (o.out32.buf >= 0) write(id, o.out32);
    if (o.out16.buf >= 0) write(id, o.out16);
    if (o.outT.buf >= 0) write(id, o.outT);
    if (ss_in.buf >= 0) read(id, ss_in);
    if (ss_out.buf >= 0) write(id, ss_out);
    if (A.rows * 1 > 0 && p.bufs[A.buf].ld < wt.ld && !init_mode) {
      p.error = "internal: activation row pitch shorter than padded K in " + name;
    }
    return id;
  }

  int weight_map(int W, int64_t N, int box_rows = GEMM_BM) {
    const DevTensor& t = p.dev_tensors[W];
    TmapSpec sp{WEIGHT_BASE + t.offset, false, N, t.ld, t.ld, box_rows};
    for (size_t i = 0; i < p.wmaps.size(); ++i)
      if (p.wmaps[i].offset == sp.offset && p.wmaps[i].rows == sp.rows && p.wmaps[i].box_rows == sp.box_rows) return (int)i;
    p.wmaps.push_back(sp);
    return (int)p.wmaps.size() - 1;
  }
  int act_map(const View& A, int64_t cols, int box_rows) {
    const BufInfo& bi = p.bufs[A.buf];
    uint64_t off = bi.offset + (uint64_t)(A.row0 * bi.ld + A.col0) * bi.elem;
    if (!bi.slot) off += const_base;
    TmapSpec sp{off, bi.slot, A.rows, cols, bi.ld, box_rows};
    if ((A.col0 * 2) % 16 != 0 || bi.elem != 2) p.error = "internal: TMA view must be bf16 and start on a 16-byte boundary";
    for (size_t i = 0; i < p.amaps.size(); ++i) {
      const TmapSpec& q = p.amaps[i];
      if (q.offset == sp.offset && q.slot == sp.slot && q.rows == sp.rows && q.cols == sp.cols && q.ld == sp.ld &&
          q.box_rows == sp.box_rows)
        return (int)i;
    }
    p.amaps.push_back(sp);
    return (int)p.amaps.size() - 1;
  }

  int rmsnorm(const std::string& name, const View& x, int g_dev, const View& out, Ref mod = 0, int shuffle = 1,
              int grid = 0, int beta_dev = -1) {
    NodeDesc n;
    std::memset(&n, 0, sizeof(n));
    n.op = OP_RMSNORM;
    NormArgs& a = n.u.norm;
    a.x = ref(x); a.g = wref(g_dev); a.mod = mod; a.out = ref(out);
    a.M = (int)x.rows; a.d = (int)p.dev_tensors[g_dev].cols; a.ldx = (int)ld(x); a.ldo = (int)ld(out);
    a.rows_per_tile = 16; a.shuffle = shuffle; a.grid = grid;
    if (beta_dev >= 0) { a.ln = 1; a.beta = wref(beta_dev); }
    if (a.d % 4) p.error = "model widths must be multiples of 4";
    if (a.ln && a.d > 2048) p.error = "LayerNorm rows wider than 2048 are not supported";
    n.n_tiles = (a.M + a.rows_per_tile - 1) / a.rows_per_tile;
    int id = add(n, name, KIND_ELEM);
    read(id, x);
    write(id, out);
    return id;
  }

  // A projected q|k buffer plus the transposed V buffer of one attention input.
  struct QKV {
    int qk = -1, vt = -1;      // qk bf16 [T, (hq+hkv)*hs]; vt bf16 [hkv*hs, pad64(T)]
    int T = 0, hq = 0, hkv = 0, hs = 0;
  };
  QKV make_qkv(const std::string& name, int T, int hq, int hkv, int hs) {
    QKV q;
    q.T = T; q.hq = hq; q.hkv = hkv; q.hs = hs;
    q.qk = buf(name + ".qk", T, (int64_t)(hq + hkv) * hs, 2);
    q.vt = buf(name + ".vt", (int64_t)hkv * hs, pad_to(T, 64), 2);
    return q;
  }

  // Fused attention of the queries in `q` (rows [0,tq), head h at column h*hs) over the keys/values of
  // kv0 (all its T tokens) and then, optionally, kv1.
  int attention(const std::string& name, const View& q, int tq, const QKV& kv0, const QKV* kv1, const View& out, int hq,
                int hkv, int hd, int hs, bool causal, int sfx = 0) {
    NodeDesc n;
    std::memset(&n, 0, sizeof(n));
    n.op = OP_ATTN;
    AttnArgs& a = n.u.attn;
    a.out = ref(out); a.ldo = (int)ld(out);
    a.tq = tq; a.t0 = kv0.T; a.t1 = kv1 ? kv1->T : 0;
    a.hq = hq; a.hkv = hkv; a.hd = hd; a.hs = hs; a.causal = causal; a.sfx = sfx;
    a.bn = 64;
    a.q_blocks = (tq + 127) / 128;
    a.scale_log2e = 1.4426950408889634f / std::sqrt((float)hd);
    n.smem_bytes = attn_smem_bytes(hs);
    n.tmem_cols = (int)pad_to(a.bn + hs, TMEM_UNIT);
    n.n_tiles = hq * a.q_blocks;
    a.hpt = attn_fold(tq, hq, hkv, &a.rph);
    if (a.hpt > 1) n.n_tiles = hkv * (((hq / hkv) + a.hpt - 1) / a.hpt);
    // tensor maps: Q rows in 128-row boxes (rph-row boxes when heads are folded), K rows in bn-row boxes, V^T in
    // hs-row boxes of 64 tokens
    const int64_t qcols = ld(q) - q.col0;
    a.qmap = act_map(q, qcols, a.hpt > 1 ? a.rph : 128);
    auto kview = [&](const QKV& s_) { return rows(s_.qk, 0, s_.T, (int64_t)s_.hq * s_.hs); };
    a.k0map = act_map(kview(kv0), (int64_t)kv0.hkv * kv0.hs, a.bn);
    a.v0map = act_map(all(kv0.vt), kv0.T, hs);
    if (kv1) {
      a.k1map = act_map(kview(*kv1), (int64_t)kv1->hkv * kv1->hs, a.bn);
      a.v1map = act_map(all(kv1->vt), kv1->T, hs);
    }
    int id = add(n, name, KIND_ATTN);
    if (!init_mode) p.node_flops[id] = 4.0 * (double)tq * (double)(a.t0 + a.t1) * (double)hq * (double)hd;
    read(id, q);
    read(id, all(kv0.qk)); read(id, all(kv0.vt));
    if (kv1) { read(id, all(kv1->qk)); read(id, all(kv1->vt)); }
    write(id, out);
    return id;
  }

  // q|k|v projection of `A` into `dst`: one GEMM whose V columns are written transposed; with RoPE the
  // GEMM writes fp32 and a rotary tile produces the bf16 q|k and V^T.
  void qkv_project(const std::string& name, const View& A, int W, const QKV& dst, int hd, int scratch32, int pos0,
                   int norm_gain = -1, int norm_d = 0, int bias = -1) {
    const int64_t nqk = (int64_t)(dst.hq + dst.hkv) * dst.hs, nall = nqk + (int64_t)dst.hkv * dst.hs;
    if (scratch32 >= 0) {
      GemmOpt gq; gq.out32 = all(scratch32); gq.norm_gain = norm_gain; gq.norm_d = norm_d;
      gemm(name + "qkv", A, W, nall, gq);
      NodeDesc n;
      std::memset(&n, 0, sizeof n);
      n.op = OP_ROPE;
      RopeArgs& r = n.u.rope;
      r.in = ref(all(scratch32)); r.out = ref(all(dst.qk)); r.outT = ref(all(dst.vt));
      r.M = dst.T; r.ld = (int)nall; r.ldo = (int)nqk; r.ldoT = (int)p.bufs[dst.vt].ld;
      r.n_rot_heads = dst.hq + dst.hkv; r.n_heads = dst.hq + 2 * dst.hkv; r.hd = hd; r.pos0 = pos0;
      r.rows_per_tile = 16;
      n.n_tiles = (dst.T + 15) / 16;
      int id = add(n, name + "rope", KIND_ELEM);
      read(id, all(scratch32));
      write(id, all(dst.qk));
      write(id, all(dst.vt));
    } else {
      GemmOpt gq; gq.out16 = all(dst.qk); gq.outT = all(dst.vt); gq.t_col0 = (int)nqk; gq.bias = bias;
      gq.norm_gain = norm_gain; gq.norm_d = norm_d;
      gemm(name + "qkv", A, W, nall, gq);
    }
  }

  int elem_node(NodeDesc& n, const std::string& name) { return add(n, name, KIND_ELEM); }

  int addrows(const std::string& name, const View& in, Ref in_raw, int ldi, int M, int N, Ref vec, Ref tab, int ldt,
              const View& out, const View& out16) {
    NodeDesc n;
    std::memset(&n, 0, sizeof(n));
    n.op = OP_ADDROWS;
    AddRowsArgs& a = n.u.addrows;
    a.in = in.buf >= 0 ? ref(in) : in_raw;
    a.ldi = in.buf >= 0 ? (int)ld(in) : ldi;
    a.vec = vec; a.tab = tab; a.ldt = ldt;
    a.out = ref(out); a.ldo = out.buf >= 0 ? (int)ld(out) : 0;
    a.out16 = ref(out16); a.ldo16 = out16.buf >= 0 ? (int)ld(out16) : 0;
    const View ssv = ss_view(out16);
    a.ss_out = ref(ssv); a.ss_ld = ssv.buf >= 0 ? (int)ld(ssv) : 0;
    a.M = M; a.N = N;
    n.n_tiles = 1;
    int id = add(n, name, KIND_ELEM);
    if (in.buf >= 0) read(id, in);
    if (out.buf >= 0) write(id, out);
    if (out16.buf >= 0) write(id, out16);
    if (ssv.buf >= 0) write(id, ssv);
    return id;
  }
};

constexpr uint64_t Builder::WEIGHT_BASE;

void set_err(Program& p, const char* msg) { p.error = msg; }

bool validate(const vla_model_desc& d, Program& p) {
  auto bad = [&](const char* s) { set_err(p, s); return false; };
  if (d.n_cam < 1 || d.img < 1 || d.patch < 1 || d.img % d.patch) return bad("image side must be a positive multiple of the patch side");
  int grid = d.img / d.patch;
  if (d.shuffle < 1 || grid % d.shuffle) return bad("token grid must be a multiple of the shuffle factor");
  if (d.vis_layers < 0 || d.llm_layers < 1 || d.act_layers < 1) return bad("layer counts out of range");
  if (d.vis_layers > 0 && (d.vis_heads < 1 || d.vis_hd < 1 || d.vis_mlp < 1)) return bad("vision encoder sizes missing");
  if (d.vis_layers > 0 && !d.connector) return bad("a vision encoder needs the linear connector");
  if (!d.connector && (d.shuffle != 1 || d.vis_d != d.d)) return bad("without a connector the patch width must equal the LLM width and shuffle must be 1");
  if (d.vis_layers == 0 && d.shuffle != 1) return bad("pixel-shuffle needs a vision encoder");
  if (d.vis_d < 1 || d.d < 1 || d.hq < 1 || d.hkv < 1 || d.hd < 2 || d.hq % d.hkv) return bad("LLM head geometry invalid");
  if (d.hd % 2) return bad("head dimension must be even");
  if (d.mlp < 1 || d.mlp_kind < 0 || d.mlp_kind > 2 || d.act_mlp < 1 || d.act_mlp_kind < 0 || d.act_mlp_kind > 2) return bad("MLP description invalid");
  if (d.n_text < 1 || d.vocab < 1) return bad("text description invalid");
  if (d.head < 0 || d.head > 3) return bad("unknown head kind");
  if (d.act_d < 2 || d.act_d % 2) return bad("head width must be even");
  if (d.head != VLA_HEAD_B && (d.act_heads < 1 || d.act_d % d.act_heads)) return bad("head width must be a multiple of its head count");
  if (d.horizon < 1 || d.act_dim < 1 || d.n_steps < 1 || d.state_dim < 0) return bad("chunk description invalid");
  if (d.solver < 0 || d.solver > 1) return bad("unknown solver");
  if (d.solver == VLA_SOLVER_DDIM && (100 % d.n_steps)) return bad("DDIM step count must divide 100");
  if (d.head == VLA_HEAD_A && d.handoff != VLA_HANDOFF_KV_LAST) return bad("head A needs the kv_last handoff");
  if (d.head == VLA_HEAD_B && (d.handoff != VLA_HANDOFF_KV_ALL || d.act_layers != d.llm_layers)) return bad("head B needs kv_all and as many layers as the LLM");
  if (d.head == VLA_HEAD_C && d.handoff != VLA_HANDOFF_FEATURES) return bad("head C needs the features handoff");
  if (d.head == VLA_HEAD_D && (d.handoff != VLA_HANDOFF_COG || d.state_dim != 0)) return bad("head D needs the cog handoff and no state");
  if (d.head == VLA_HEAD_A && d.state_dim == 0) return bad("head A needs a state token");
  if (d.guidance != 0.0f && (d.head != VLA_HEAD_D || d.solver != VLA_SOLVER_DDIM))
    return bad("classifier-free guidance needs head D with the DDIM solver");
  if (d.vis_layernorm != 0 && d.vis_layernorm != 1) return bad("vis_layernorm must be 0 or 1");
  if (d.suffix_mask != 0 && (d.suffix_mask != 1 || d.head != VLA_HEAD_B || d.state_dim == 0))
    return bad("the blocked suffix mask needs head B with a state token");
  return true;
}

std::vector<double> ddim_alpha_bar(int T) {
  auto c = [](double u) { double x = std::cos((u + 0.008) / 1.008 * M_PI / 2); return x * x; };
  std::vector<double> ab;
  double prod = 1.0;
  for (int s = 0; s < T; ++s) {
    double beta = std::min(1.0 - c((s + 1.0) / T) / c((double)s / T), 0.999);
    prod *= 1.0 - beta;
    ab.push_back(prod);
  }
  return ab;
}

}  // namespace

bool build_program(const vla_model_desc& d, const vla_runtime_opts& o, Program& p) {
  p = Program();
  p.desc = d;
  if (!validate(d, p)) return false;
  if (o.n_streams < 1 || o.n_streams > 1024 || o.ring_depth < 2 || o.ring_depth > 64) {
    set_err(p, "n_streams must be 1..1024 and ring_depth 2..64");
    return false;
  }
  p.n_streams = o.n_streams;
  p.ring_depth = o.ring_depth;
  p.n_inst = o.n_streams * o.ring_depth;
  p.head_passes = o.head_passes > 1 ? o.head_passes : 1;
  if (p.head_passes > 64) { set_err(p, "head_passes must be at most 64"); return false; }
  const int P = p.head_passes;
  if (p.n_inst >= 4096) { set_err(p, "too many frame slots"); return false; }

  Builder b(p);
  const int grid = d.img / d.patch;
  const int T = grid * grid;                                   // tokens per camera in the encoder
  const int tpc = T / (d.shuffle * d.shuffle);                 // tokens per camera entering the LLM
  const int n_img = d.n_cam * tpc;
  const int S = n_img + d.n_text;
  const int patch_k = 3 * d.patch * d.patch;
  const int dv = d.vis_d, D = d.d, da = d.act_d;
  const bool has_state = d.state_dim > 0;
  const int first = (has_state || d.head == VLA_HEAD_D) ? 1 : 0;
  const int Ta = d.horizon + first;
  const bool head_pos = !(d.head == VLA_HEAD_B && d.rope);
  const bool gated = d.mlp_kind != VLA_MLP_GELU, agated = d.act_mlp_kind != VLA_MLP_GELU;
  const int hvd = d.vis_heads * d.vis_hd;
  const int vhs = (int)pad_to(std::max(d.vis_hd, 1), 16);          // vision head stride (72 -> 80)
  const int lhs = (int)pad_to(d.hd, 16);                            // LLM head stride
  const int nq = d.hq * d.hd, nkv = d.hkv * d.hd, nqkv = (d.hq + 2 * d.hkv) * lhs;
  if (lhs != d.hd) { set_err(p, "LLM head dimension must be a multiple of 16"); return false; }
  auto P64 = [](int64_t x) { return pad_to(x, GEMM_BK); };
  char nm[96];
  auto N_ = [&](const char* fmt, int a = 0, int c = 0) { std::snprintf(nm, sizeof nm, fmt, a, c); return std::string(nm); };

  // ================================================================== weights
  const bool vln = d.vis_layernorm != 0;     // LayerNorm-and-bias variant of the vision encoder
  int w_patch = b.matrix1("vis.patch.w", dv, patch_k);
  int w_patch_b = vln ? b.gain("vis.patch.b", dv) : -1;
  int w_vpos = b.table("vis.pos", T, dv);
  struct EncW { int n1, wqkv, wo, n2, w1, w2, n1b = -1, bqkv = -1, bo = -1, n2b = -1, b1 = -1, b2 = -1; };
  std::vector<EncW> venc(d.vis_layers);
  for (int i = 0; i < d.vis_layers; ++i) {
    std::string pre = N_("vis.L%d.", i);
    venc[i].n1 = b.gain(pre + "n1", dv);
    venc[i].wqkv = b.matrix_heads(pre + "wqkv", {pre + "wq", pre + "wk", pre + "wv"},
                                  {d.vis_heads, d.vis_heads, d.vis_heads}, d.vis_hd, vhs, dv);
    venc[i].wo = b.matrix1(pre + "wo", dv, hvd);
    venc[i].n2 = b.gain(pre + "n2", dv);
    venc[i].w1 = b.matrix1(pre + "w1", d.vis_mlp, dv);
    venc[i].w2 = b.matrix1(pre + "w2", dv, d.vis_mlp);
    if (vln) {
      venc[i].n1b = b.gain(pre + "n1b", dv);
      venc[i].bqkv = b.vector_heads(pre + "bqkv", {pre + "bq", pre + "bk", pre + "bv"},
                                    {d.vis_heads, d.vis_heads, d.vis_heads}, d.vis_hd, vhs);
      venc[i].bo = b.gain(pre + "bo", dv);
      venc[i].n2b = b.gain(pre + "n2b", dv);
      venc[i].b1 = b.gain(pre + "b1", d.vis_mlp);
      venc[i].b2 = b.gain(pre + "b2", dv);
    }
  }
  int w_vnorm = d.vis_layers > 0 ? b.gain("vis.norm", dv) : -1;
  int w_vnorm_b = (vln && d.vis_layers > 0) ? b.gain("vis.normb", dv) : -1;
  int w_conn = d.connector ? b.matrix1("conn.w", D, (int64_t)d.shuffle * d.shuffle * dv) : -1;
  int w_emb = b.matrix1("txt.emb", d.vocab, D);
  int w_lpos = d.rope ? -1 : b.table("llm.pos", S, D);
  struct LlmW { int n1, wqkv, wo, n2, w1, w2, wg, wu, wd; };
  std::vector<LlmW> lw(d.llm_layers);
  for (int i = 0; i < d.llm_layers; ++i) {
    std::string pre = N_("llm.L%d.", i);
    lw[i].n1 = b.gain(pre + "n1", D);
    lw[i].wqkv = b.matrix(pre + "wqkv", {pre + "wq", pre + "wk", pre + "wv"}, {nq, nkv, nkv}, D);
    lw[i].wo = b.matrix1(pre + "wo", D, nq);
    lw[i].n2 = b.gain(pre + "n2", D);
    if (gated) {
      lw[i].wg = b.matrix1(pre + "wg", d.mlp, D);
      lw[i].wu = b.matrix1(pre + "wu", d.mlp, D);
      lw[i].wd = b.matrix1(pre + "wd", D, d.mlp);
    } else {
      lw[i].w1 = b.matrix1(pre + "w1", d.mlp, D);
      lw[i].w2 = b.matrix1(pre + "w2", D, d.mlp);
    }
  }
  int w_lnorm = b.gain("llm.norm", D);

  int w_ain = b.matrix1("act.in", da, d.act_dim);
  int w_astate = has_state ? b.matrix1("act.state", da, d.state_dim) : -1;
  int w_acond = d.head == VLA_HEAD_D ? b.matrix1("act.cond", da, D) : -1;
  int w_apos = head_pos ? b.table("act.pos", Ta, da) : -1;
  int w_t1 = b.matrix1("act.t1", da, da);
  int w_t2 = b.matrix1("act.t2", da, da);
  struct ActW { int n1, n2, n3, wqkv, wo, cq, ckv, co, ada1, ada2, w1, w2, wg, wu, wd; };
  std::vector<ActW> aw(d.act_layers);
  for (int i = 0; i < d.act_layers; ++i) {
    std::string pre = N_("act.L%d.", i);
    ActW& a = aw[i];
    a.n1 = b.gain(pre + "n1", da);
    if (d.head == VLA_HEAD_B) {
      a.wqkv = b.matrix(pre + "wqkv", {pre + "wq", pre + "wk", pre + "wv"}, {nq, nkv, nkv}, da);
      a.wo = b.matrix1(pre + "wo", da, nq);
    } else if (d.head == VLA_HEAD_C && (i % 2 == 1)) {
      a.cq = b.matrix1(pre + "cq", da, da);
      a.ckv = b.matrix(pre + "ckv", {pre + "ck", pre + "cv"}, {da, da}, D);
      a.co = b.matrix1(pre + "co", da, da);
    } else {
      a.wqkv = b.matrix(pre + "wqkv", {pre + "wq", pre + "wk", pre + "wv"}, {da, da, da}, da);
      a.wo = b.matrix1(pre + "wo", da, da);
    }
    a.n2 = b.gain(pre + "n2", da);
    if (d.head == VLA_HEAD_A) {
      a.cq = b.matrix1(pre + "cq", nq, da);
      a.co = b.matrix1(pre + "co", da, nq);
      a.n3 = b.gain(pre + "n3", da);
    }
    if (d.head == VLA_HEAD_C) {
      a.ada1 = b.matrix1(pre + "ada1", 2 * da, da);
      a.ada2 = b.matrix1(pre + "ada2", 2 * da, da);
    }
    if (agated) {
      a.wg = b.matrix1(pre + "wg", d.act_mlp, da);
      a.wu = b.matrix1(pre + "wu", d.act_mlp, da);
      a.wd = b.matrix1(pre + "wd", da, d.act_mlp);
    } else {
      a.w1 = b.matrix1(pre + "w1", d.act_mlp, da);
      a.w2 = b.matrix1(pre + "w2", da, d.act_mlp);
    }
  }
  int w_anorm = b.gain("act.norm", da);
  int w_aout = b.matrix1("act.out", d.act_dim, da);

  // ================================================================== solver constants
  const int ns = d.n_steps;
  p.step_args.resize(ns); p.step_c_x.resize(ns); p.step_c_acc.resize(ns);
  if (d.solver == VLA_SOLVER_EULER) {
    for (int k = 0; k < ns; ++k) {
      p.step_args[k] = 1000.0f * (float)k / (float)ns;
      p.step_c_x[k] = 1.0f;
      p.step_c_acc[k] = 1.0f / (float)ns;
    }
  } else {
    // deterministic DDIM: x' = sqrt(a_prev) (x - sqrt(1-a_t) e)/sqrt(a_t) + sqrt(1-a_prev) e, folded to c_x x + c_acc e
    std::vector<double> ab = ddim_alpha_bar(100);
    int stride = 100 / ns;
    for (int k = 0; k < ns; ++k) {
      int tau = (ns - 1 - k) * stride;
      double a_t = ab[tau], a_prev = tau - stride >= 0 ? ab[tau - stride] : 1.0;
      p.step_args[k] = (float)tau;
      p.step_c_x[k] = (float)(std::sqrt(a_prev) / std::sqrt(a_t));
      p.step_c_acc[k] = (float)(std::sqrt(1.0 - a_prev) - std::sqrt(a_prev) * std::sqrt(1.0 - a_t) / std::sqrt(a_t));
    }
  }

  // ================================================================== constant buffers + their precomputation
  b.const_base = align_up(Builder::WEIGHT_BASE + b.weight_cursor, 4096);
  int c_args = b.buf("const.args", 1, pad_to(ns, 4), 4, false);
  int c_temb = b.buf("const.temb", ns, P64(da), 2, false);
  int c_th = b.buf("const.th", ns, P64(da), 2, false);
  int c_ct = b.buf("const.ct", ns, da, 4, false);
  int c_sct = d.head == VLA_HEAD_C ? b.buf("const.sct", ns, P64(da), 2, false) : -1;
  std::vector<int> c_mod1(d.act_layers, -1), c_mod2(d.act_layers, -1);
  if (d.head == VLA_HEAD_C)
    for (int i = 0; i < d.act_layers; ++i) {
      c_mod1[i] = b.buf(N_("const.mod1.%d", i), ns, 2 * da, 4, false);
      c_mod2[i] = b.buf(N_("const.mod2.%d", i), ns, 2 * da, 4, false);
    }
  b.init_mode = true;
  b.phase = PHASE_ACT;
  {
    NodeDesc n;
    std::memset(&n, 0, sizeof n);
    n.op = OP_TIMEEMB;
    n.u.timeemb.args = b.ref(b.all(c_args));
    n.u.timeemb.out = b.ref(b.all(c_temb));
    n.u.timeemb.M = ns; n.u.timeemb.width = da; n.u.timeemb.ldo = (int)P64(da);
    n.n_tiles = 1;
    b.add(n, "init.temb", KIND_ELEM);
    Builder::GemmOpt g1; g1.act = ACT_SILU; g1.out16 = b.all(c_th);
    b.gemm("init.t1", b.all(c_temb), w_t1, da, g1);
    Builder::GemmOpt g2; g2.out32 = b.all(c_ct);
    b.gemm("init.t2", b.all(c_th), w_t2, da, g2);
    if (d.head == VLA_HEAD_C) {
      Builder::GemmOpt g3; g3.act = ACT_SILU; g3.out16 = b.all(c_sct);
      b.gemm("init.t2s", b.all(c_th), w_t2, da, g3);
      for (int i = 0; i < d.act_layers; ++i) {
        Builder::GemmOpt ga; ga.out32 = b.all(c_mod1[i]);
        b.gemm("init.ada1", b.all(c_sct), aw[i].ada1, 2 * da, ga);
        Builder::GemmOpt gb; gb.out32 = b.all(c_mod2[i]);
        b.gemm("init.ada2", b.all(c_sct), aw[i].ada2, 2 * da, gb);
      }
    }
  }
  b.init_mode = false;

  // ================================================================== frame-slot buffers
  // inputs
  int in_img = b.buf("in.image", d.n_cam, (int64_t)3 * d.img * d.img, 4);
  int in_txt = b.buf("in.text", 1, pad_to(d.n_text, 4), 4);
  int in_state = has_state ? b.buf("in.state", P, d.state_dim, 4) : -1;
  int in_noise = b.buf("in.noise", (int64_t)P * d.horizon, d.act_dim, 4);
  p.in_image = p.bufs[in_img].offset; p.image_bytes = p.bufs[in_img].bytes;
  p.in_text = p.bufs[in_txt].offset; p.text_bytes = (uint64_t)d.n_text * 4;
  if (has_state) { p.in_state = p.bufs[in_state].offset; p.state_bytes = (uint64_t)P * d.state_dim * 4; }
  p.in_noise = p.bufs[in_noise].offset; p.noise_bytes = p.bufs[in_noise].bytes;

  // LLM
  int x = b.buf("llm.x", S, D, 4);
  int xb = b.stream_mirror("llm.xb", S, D);                // bf16 mirror of the residual stream (GEMM operand)
  int qkv32 = d.rope ? b.buf("llm.qkv32", S, nqkv, 4) : -1;
  std::vector<Builder::QKV> lq(d.llm_layers);
  {
    bool have_shared = false;
    Builder::QKV shared;
    for (int i = 0; i < d.llm_layers; ++i) {
      bool own = d.handoff == VLA_HANDOFF_KV_ALL || (d.handoff == VLA_HANDOFF_KV_LAST && i == d.llm_layers - 1);
      if (own) lq[i] = b.make_qkv(N_("llm.qkv.%d", i), S, d.hq, d.hkv, lhs);
      else {
        if (!have_shared) { shared = b.make_qkv("llm.qkv", S, d.hq, d.hkv, lhs); have_shared = true; }
        lq[i] = shared;
      }
    }
  }
  int att = b.buf("llm.att", S, P64(nq), 2);
  int mid = b.buf("llm.mid", S, P64(d.mlp), 2);
  int hidden = b.buf("llm.hidden", S, P64(D), 2);

  // ================================================================== VLM phase
  b.phase = PHASE_VLM;
  b.step = -1;
  for (int c = 0; c < d.n_cam; ++c) {
    int patches = b.buf(N_("vis%d.patches", c), T, P64(patch_k), 2);
    {
      NodeDesc n;
      std::memset(&n, 0, sizeof n);
      n.op = OP_PATCHIFY;
      PatchArgs& a = n.u.patch;
      a.img = Builder::in_ref(0, (uint64_t)c * 3 * d.img * d.img * 4);
      a.out = b.ref(b.all(patches));
      a.img_side = d.img; a.patch = d.patch; a.grid = grid; a.ldo = (int)P64(patch_k); a.rows_per_tile = 16;
      n.n_tiles = (T + 15) / 16;
      int id = b.add(n, N_("vis%d.patchify", c), KIND_ELEM);
      b.write(id, b.all(patches));
    }
    if (d.vis_layers == 0 && !d.connector) {
      // patch embedding feeds the LLM residual stream directly
      Builder::GemmOpt g;
      g.tab = b.wref(w_vpos); g.ldtab = dv;
      if (w_lpos >= 0) { g.tab2 = b.wref(w_lpos, (int64_t)c * tpc); g.ldtab2 = D; }
      g.out32 = b.rows(x, (int64_t)c * tpc, tpc);
      g.out16 = b.rows(xb, (int64_t)c * tpc, tpc);
      g.bias = w_patch_b;
      b.gemm(N_("vis%d.patch", c), b.all(patches), w_patch, dv, g);
      continue;
    }
    int xv = b.buf(N_("vis%d.x", c), T, dv, 4);
    // GEMM operand of the layers: the bf16 mirror of the residual stream (RMSNorm folded into the GEMMs), or, in the
    // LayerNorm variant, the normalised rows written by a norm node of their own
    int xvb = vln ? -1 : b.stream_mirror(N_("vis%d.xb", c), T, dv);
    int hv = (vln && d.vis_layers > 0) ? b.buf(N_("vis%d.h", c), T, P64(dv), 2) : -1;
    Builder::QKV vq;
    if (d.vis_layers > 0) vq = b.make_qkv(N_("vis%d.qkv", c), T, d.vis_heads, d.vis_heads, vhs);
    int vatt = d.vis_layers > 0 ? b.buf(N_("vis%d.att", c), T, P64(hvd), 2) : -1;
    int vmid = d.vis_layers > 0 ? b.buf(N_("vis%d.mid", c), T, P64(d.vis_mlp), 2) : -1;
    int shuf = b.buf(N_("vis%d.shuf", c), tpc, P64((int64_t)d.shuffle * d.shuffle * dv), 2);
    {
      Builder::GemmOpt g;
      g.tab = b.wref(w_vpos); g.ldtab = dv;
      if (d.vis_layers > 0) { g.out32 = b.all(xv); if (!vln) g.out16 = b.all(xvb); } else g.out16 = b.all(shuf);
      g.bias = w_patch_b;
      b.gemm(N_("vis%d.patch", c), b.all(patches), w_patch, dv, g);
    }
    for (int i = 0; vln && i < d.vis_layers; ++i) {
      const EncW& e = venc[i];
      b.rmsnorm(N_("vis%d.L%d.n1", c, i), b.all(xv), e.n1, b.all(hv), 0, 1, 0, e.n1b);
      b.qkv_project(N_("vis%d.L%d.", c, i), b.all(hv), e.wqkv, vq, d.vis_hd, -1, 0, -1, 0, e.bqkv);
      b.attention(N_("vis%d.L%d.attn", c, i), b.rows(vq.qk, 0, T, 0), T, vq, nullptr, b.all(vatt), d.vis_heads, d.vis_heads,
                  d.vis_hd, vhs, false);
      Builder::GemmOpt go; go.X = b.all(xv); go.out32 = b.all(xv); go.bias = e.bo;
      b.gemm(N_("vis%d.L%d.wo", c, i), b.all(vatt), e.wo, dv, go);
      b.rmsnorm(N_("vis%d.L%d.n2", c, i), b.all(xv), e.n2, b.all(hv), 0, 1, 0, e.n2b);
      Builder::GemmOpt g1; g1.act = ACT_GELU; g1.out16 = b.all(vmid); g1.bias = e.b1;
      b.gemm(N_("vis%d.L%d.w1", c, i), b.all(hv), e.w1, d.vis_mlp, g1);
      Builder::GemmOpt g2; g2.X = b.all(xv); g2.out32 = b.all(xv); g2.bias = e.b2;
      b.gemm(N_("vis%d.L%d.w2", c, i), b.all(vmid), e.w2, dv, g2);
    }
    for (int i = 0; !vln && i < d.vis_layers; ++i) {
      // the two RMSNorms of a layer are folded into the GEMMs that consume them (A = bf16 mirror of the stream)
      b.qkv_project(N_("vis%d.L%d.", c, i), b.all(xvb), venc[i].wqkv, vq, d.vis_hd, -1, 0, venc[i].n1, dv);
      b.attention(N_("vis%d.L%d.attn", c, i), b.rows(vq.qk, 0, T, 0), T, vq, nullptr, b.all(vatt), d.vis_heads, d.vis_heads,
                  d.vis_hd, vhs, false);
      Builder::GemmOpt go; go.X = b.all(xv); go.out32 = b.all(xv); go.out16 = b.all(xvb);
      b.gemm(N_("vis%d.L%d.wo", c, i), b.all(vatt), venc[i].wo, dv, go);
      Builder::GemmOpt g1; g1.act = ACT_GELU; g1.out16 = b.all(vmid); g1.norm_gain = venc[i].n2; g1.norm_d = dv;
      b.gemm(N_("vis%d.L%d.w1", c, i), b.all(xvb), venc[i].w1, d.vis_mlp, g1);
      Builder::GemmOpt g2; g2.X = b.all(xv); g2.out32 = b.all(xv); g2.out16 = b.all(xvb);
      b.gemm(N_("vis%d.L%d.w2", c, i), b.all(vmid), venc[i].w2, dv, g2);
    }
    if (d.vis_layers > 0)
      b.rmsnorm(N_("vis%d.norm", c), b.all(xv), w_vnorm, b.all(shuf), 0, d.shuffle, grid, w_vnorm_b);
    {
      Builder::GemmOpt g;
      if (w_lpos >= 0) { g.tab = b.wref(w_lpos, (int64_t)c * tpc); g.ldtab = D; }
      g.out32 = b.rows(x, (int64_t)c * tpc, tpc);
      g.out16 = b.rows(xb, (int64_t)c * tpc, tpc);
      b.gemm(N_("vis%d.conn", c), b.all(shuf), w_conn, D, g);
    }
  }
  {
    NodeDesc n;
    std::memset(&n, 0, sizeof n);
    n.op = OP_EMBED;
    EmbedArgs& a = n.u.embed;
    a.ids = Builder::in_ref(1);
    a.table = b.wref(w_emb);
    a.pos = w_lpos >= 0 ? b.wref(w_lpos, n_img) : 0;
    a.out = b.ref(b.rows(x, n_img, d.n_text));
    a.n = d.n_text; a.d = D; a.ldo = D; a.vocab = d.vocab; a.rows_per_tile = 16; a.ldt = (int)P64(D);
    a.out16 = b.ref(b.rows(xb, n_img, d.n_text)); a.ldo16 = (int)P64(D);
    {
      View sv = b.ss_view(b.rows(xb, n_img, d.n_text));
      a.ss_out = b.ref(sv); a.ss_ld = (int)b.ld(sv);
    }
    n.n_tiles = (d.n_text + 15) / 16;
    int id = b.add(n, "llm.embed", KIND_ELEM);
    b.write(id, b.rows(x, n_img, d.n_text));
    b.write(id, b.rows(xb, n_img, d.n_text));
    b.write(id, b.ss_view(b.rows(xb, n_img, d.n_text)));
  }
  for (int i = 0; i < d.llm_layers; ++i) {
    b.qkv_project(N_("llm.L%d.", i), b.all(xb), lw[i].wqkv, lq[i], d.hd, qkv32, 0, lw[i].n1, D);
    b.attention(N_("llm.L%d.attn", i), b.rows(lq[i].qk, 0, S, 0), S, lq[i], nullptr, b.all(att), d.hq, d.hkv, d.hd, lhs,
                d.causal != 0);
    Builder::GemmOpt go; go.X = b.all(x); go.out32 = b.all(x); go.out16 = b.all(xb);
    b.gemm(N_("llm.L%d.wo", i), b.all(att), lw[i].wo, D, go);
    Builder::GemmOpt g1; g1.out16 = b.all(mid); g1.norm_gain = lw[i].n2; g1.norm_d = D;
    if (gated) {
      g1.W2 = lw[i].wu;
      g1.act = d.mlp_kind == VLA_MLP_SWIGLU ? ACT_SILU : ACT_GELU;
      b.gemm(N_("llm.L%d.gu", i), b.all(xb), lw[i].wg, d.mlp, g1);
    } else {
      g1.act = ACT_GELU;
      b.gemm(N_("llm.L%d.w1", i), b.all(xb), lw[i].w1, d.mlp, g1);
    }
    Builder::GemmOpt g2; g2.X = b.all(x); g2.out32 = b.all(x); g2.out16 = b.all(xb);
    b.gemm(N_("llm.L%d.w2", i), b.all(mid), gated ? lw[i].wd : lw[i].w2, D, g2);
  }
  b.rmsnorm("llm.norm", b.all(x), w_lnorm, b.all(hidden));
  const int ahd = d.head == VLA_HEAD_B ? d.hd : da / d.act_heads;
  const int ahs = (int)pad_to(ahd, 16);
  if (ahs != ahd) { set_err(p, "action-head head dimension must be a multiple of 16"); return false; }
  std::vector<Builder::QKV> ckv(d.act_layers);
  if (d.head == VLA_HEAD_C)
    for (int i = 1; i < d.act_layers; i += 2) {
      ckv[i] = b.make_qkv(N_("act.ckv.%d", i), S, 0, d.act_heads, ahs);
      b.qkv_project(N_("act.L%d.c", i), b.all(hidden), aw[i].ckv, ckv[i], ahd, -1, 0);
    }

  // ================================================================== action-head phase
  b.phase = PHASE_ACT;
  b.step = -1;
  const int a_hq = d.head == VLA_HEAD_B ? d.hq : d.act_heads, a_hkv = d.head == VLA_HEAD_B ? d.hkv : d.act_heads;
  const int a_nq = a_hq * ahs, a_nqkv = (a_hq + 2 * a_hkv) * ahs;
  int xs = b.buf("act.x", d.horizon, d.act_dim, 4);
  int xbf = b.buf("act.xbf", d.horizon, P64(d.act_dim), 2);
  int z = b.buf("act.z", Ta, da, 4);
  int zb = b.stream_mirror("act.zb", Ta, da);              // bf16 mirror of the head's residual stream (GEMM operand)
  int hz = d.head == VLA_HEAD_C ? b.buf("act.h", Ta, P64(da), 2) : -1;   // adaLN-modulated norms are separate tiles
  Builder::QKV aq = b.make_qkv("act.qkv", Ta, a_hq, a_hkv, ahs);
  int aqkv32 = (d.head == VLA_HEAD_B && d.rope) ? b.buf("act.qkv32", Ta, a_nqkv, 4) : -1;
  int aatt = b.buf("act.att", Ta, P64(std::max(a_nq, nq)), 2);
  int aqc = (d.head == VLA_HEAD_A || d.head == VLA_HEAD_C) ? b.buf("act.qc", Ta, d.head == VLA_HEAD_A ? nq : da, 2) : -1;
  int amid = b.buf("act.mid", Ta, P64(d.act_mlp), 2);
  int tok0 = first ? b.buf("act.tok0", 1, da, 4) : -1;
  const bool guided = d.guidance != 0.0f;
  int vu = guided ? b.buf("act.vu", d.horizon, d.act_dim, 4) : -1;   // the unconditional branch's share of the update
  int state_bf = has_state ? b.buf("act.state_bf", 1, P64(d.state_dim), 2) : -1;

  // Asynchronous inference: the head runs P times on the same VLM output, pass by pass on the same buffers (the
  // buffer accesses order the passes), every pass with its own robot state and noise sample and its own chunk.
  for (int pass = 0; pass < P; ++pass) {
  if (pass > 0) { std::snprintf(nm, sizeof nm, ".p%d", pass); b.name_suffix = nm; }
  b.step = -1;
  if (has_state) {
    b.addrows("act.state_cvt", View(), Builder::in_ref(2, (uint64_t)pass * d.state_dim * 4), d.state_dim, 1, d.state_dim, 0, 0, 0,
              View(), b.all(state_bf));
    Builder::GemmOpt g;
    if (head_pos) { g.tab = b.wref(w_apos, 0); g.ldtab = da; }
    g.out32 = b.all(tok0);
    b.gemm("act.state_tok", b.all(state_bf), w_astate, da, g);
  } else if (d.head == VLA_HEAD_D) {
    Builder::GemmOpt g;
    if (head_pos) { g.tab = b.wref(w_apos, 0); g.ldtab = da; }
    g.out32 = b.all(tok0);
    b.gemm("act.cond_tok", b.rows(hidden, S - 1, 1), w_acond, da, g);
  }
  b.addrows("act.x_init", View(), Builder::in_ref(3, (uint64_t)pass * d.horizon * d.act_dim * 4), d.act_dim, d.horizon, d.act_dim,
            0, 0, 0, b.all(xs), b.all(xbf));

  for (int k = 0; k < ns; ++k) {
    b.step = k;
    Ref ct_k = b.ref(b.rows(c_ct, k, 1));
    // classifier-free guidance: the head runs twice per step on the same buffers, first with the condition token of a
    // zero cognition feature (its epsilon, scaled, parked in act.vu), then with the real one
    for (int branch = guided ? 0 : 1; branch < 2; ++branch) {
    const bool uncond = branch == 0;
    const std::string saved_suffix = b.name_suffix;
    if (uncond) b.name_suffix += ".u";
    if (first) {
      if (uncond)     // W_c . 0 + pos_0 + c_t
        b.addrows(N_("act.s%d.tok0", k), View(), b.wref(w_apos, 0), da, 1, da, ct_k, 0, 0, b.rows(z, 0, 1), b.rows(zb, 0, 1));
      else
        b.addrows(N_("act.s%d.tok0", k), b.all(tok0), 0, 0, 1, da, d.head == VLA_HEAD_D ? ct_k : 0, 0, 0, b.rows(z, 0, 1),
                  b.rows(zb, 0, 1));
    }
    {
      Builder::GemmOpt g;
      if (d.head == VLA_HEAD_A || d.head == VLA_HEAD_B) g.vec = ct_k;
      if (head_pos) { g.tab = b.wref(w_apos, first); g.ldtab = da; }
      g.out32 = b.rows(z, first, d.horizon);
      g.out16 = b.rows(zb, first, d.horizon);
      b.gemm(N_("act.s%d.in", k), b.all(xbf), w_ain, da, g);
    }
    for (int i = 0; i < d.act_layers; ++i) {
      const ActW& a = aw[i];
      auto NN = [&](const char* leaf) { std::snprintf(nm, sizeof nm, "act.s%d.L%d.%s", k, i, leaf); return std::string(nm); };
      Ref mod1 = d.head == VLA_HEAD_C ? b.ref(b.rows(c_mod1[i], k, 1)) : 0;
      Ref mod2 = d.head == VLA_HEAD_C ? b.ref(b.rows(c_mod2[i], k, 1)) : 0;
      // Without adaLN the RMSNorms are folded into the GEMMs that consume them (A = bf16 mirror zb);
      // with adaLN (head C) the modulated norm stays a tile of its own writing hz.
      const bool fold = d.head != VLA_HEAD_C;
      View nin = fold ? b.all(zb) : b.all(hz);
      if (!fold) b.rmsnorm(NN("n1"), b.all(z), a.n1, b.all(hz), mod1);
      bool cross_only = d.head == VLA_HEAD_C && (i % 2 == 1);
      auto resid = [&]() { Builder::GemmOpt go; go.X = b.all(z); go.out32 = b.all(z); go.out16 = b.all(zb); return go; };
      if (!cross_only) {
        b.qkv_project(NN(""), nin, a.wqkv, aq, ahd, aqkv32, S, fold ? a.n1 : -1, da);
        View att_out = b.rows(aatt, 0, Ta);
        if (d.head == VLA_HEAD_B)
          b.attention(NN("attn"), b.rows(aq.qk, 0, Ta, 0), Ta, lq[i], &aq, att_out, d.hq, d.hkv, d.hd, lhs, false,
                      d.suffix_mask ? first : 0);
        else
          b.attention(NN("attn"), b.rows(aq.qk, 0, Ta, 0), Ta, aq, nullptr, att_out, d.act_heads, d.act_heads, ahd, ahs, false);
        b.gemm(NN("wo"), b.all(aatt), a.wo, da, resid());
      }
      int mlp_gain = a.n2;
      if (d.head == VLA_HEAD_A) {
        Builder::GemmOpt gq; gq.out16 = b.all(aqc); gq.norm_gain = a.n2; gq.norm_d = da;
        b.gemm(NN("cq"), b.all(zb), a.cq, nq, gq);
        b.attention(NN("xattn"), b.all(aqc), Ta, lq[d.llm_layers - 1], nullptr, b.all(aatt), d.hq, d.hkv, d.hd, lhs, false);
        b.gemm(NN("co"), b.all(aatt), a.co, da, resid());
        mlp_gain = a.n3;
      } else if (cross_only) {
        Builder::GemmOpt gq; gq.out16 = b.all(aqc);
        b.gemm(NN("cq"), b.all(hz), a.cq, da, gq);
        b.attention(NN("xattn"), b.all(aqc), Ta, ckv[i], nullptr, b.all(aatt), d.act_heads, d.act_heads, ahd, ahs, false);
        b.gemm(NN("co"), b.all(aatt), a.co, da, resid());
        b.rmsnorm(NN("n2"), b.all(z), a.n2, b.all(hz), mod2);
      } else if (!fold) {
        b.rmsnorm(NN("n2"), b.all(z), a.n2, b.all(hz), mod2);
      }
      Builder::GemmOpt g1; g1.out16 = b.all(amid);
      if (fold) { g1.norm_gain = mlp_gain; g1.norm_d = da; }
      if (agated) {
        g1.W2 = a.wu;
        g1.act = d.act_mlp_kind == VLA_MLP_SWIGLU ? ACT_SILU : ACT_GELU;
        b.gemm(NN("gu"), nin, a.wg, d.act_mlp, g1);
      } else {
        g1.act = ACT_GELU;
        b.gemm(NN("w1"), nin, a.w1, d.act_mlp, g1);
      }
      b.gemm(NN("w2"), b.all(amid), agated ? a.wd : a.w2, da, resid());
    }
    {
      // final RMSNorm folded into the output projection; the solver update is its epilogue
      Builder::GemmOpt g;
      g.norm_gain = w_anorm; g.norm_d = da;
      if (uncond) {          // vu = c_acc (1 - s) eps_u
        g.c_acc = p.step_c_acc[k] * (1.0f - d.guidance);
        g.out32 = b.all(vu);
      } else {               // x <- c_x x + c_acc s eps_c + vu   (s = 1 and vu = 0 without guidance)
        g.X = b.all(xs); g.c_x = p.step_c_x[k]; g.c_acc = guided ? p.step_c_acc[k] * d.guidance : p.step_c_acc[k];
        if (guided) g.tabv = b.all(vu);
        g.out32 = b.all(xs); g.out16 = b.all(xbf);
      }
      b.gemm(N_("act.s%d.out", k), b.rows(zb, first, d.horizon), w_aout, d.act_dim, g);
    }
    b.name_suffix = saved_suffix;
    }   // guidance branches
  }
  b.step = -1;
  {
    NodeDesc n;
    std::memset(&n, 0, sizeof n);
    n.op = pass == P - 1 ? OP_EMIT : OP_EMIT_PART;        // the last pass's emit publishes the frame
    n.u.emit.x = b.ref(b.all(xs));
    n.u.emit.H = d.horizon; n.u.emit.A = d.act_dim; n.u.emit.ldx = d.act_dim;
    n.u.emit.chunk_off = pass * d.horizon * d.act_dim;
    n.n_tiles = 1;
    int id = b.add(n, "act.emit", KIND_ELEM);
    b.read(id, b.all(xs));
  }
  }   // head passes
  b.name_suffix.clear();
  if (!p.error.empty()) return false;

  // ================================================================== successors, roots
  const int nn = (int)p.nodes.size();
  if (nn >= (1 << 20)) { set_err(p, "tile program too large"); return false; }
  {
    // the emit node closes the frame: it also waits for every node nothing else consumes,
    // so a frame slot is never handed back while one of its tiles is still pending
    std::vector<char> has_succ(nn, 0);
    for (int i = 0; i < nn; ++i)
      for (int q : b.preds[i]) has_succ[q] = 1;
    for (int i = 0; i < nn - 1; ++i)
      if (!has_succ[i]) b.preds[nn - 1].push_back(i);
  }
  std::vector<std::vector<int>> succ(nn);
  for (int i = 0; i < nn; ++i) {
    auto& pr = b.preds[i];
    std::sort(pr.begin(), pr.end());
    pr.erase(std::unique(pr.begin(), pr.end()), pr.end());
    int pred_tiles = 0;                     // the counter a node waits on counts its predecessors' tiles
    for (int q : pr) pred_tiles += p.nodes[q].n_tiles;
    p.nodes[i].n_pred = pred_tiles;
    for (int q : pr) succ[q].push_back(i);
    if (pr.empty()) p.roots.push_back(i);
  }
  for (int i = 0; i < nn; ++i) {
    p.nodes[i].succ_begin = (int)p.succ.size();
    p.nodes[i].succ_count = (int)succ[i].size();
    for (int s : succ[i]) p.succ.push_back(s);
  }

  // ================================================================== per-class tags and resources
  // (tau_TC, tau_ALU, tau_MEM): hand-assigned intensities per tile class (Section 3.2 of the paper
  // derives them by profiling; the values below follow the per-class roofline of the tile bodies).
  const int taus[N_CLASSES][3] = {{15, 2, 3}, {15, 4, 3}, {8, 8, 2}, {0, 4, 10}, {2, 3, 12}, {2, 4, 12}, {1, 8, 4}, {0, 3, 6}};
  for (int c = 0; c < N_CLASSES; ++c) {
    for (int x_ = 0; x_ < 3; ++x_) p.classes[c].tau[x_] = taus[c][x_];
    p.classes[c].smem_units = 0;
    p.classes[c].tmem_units = 0;
    p.classes[c].group = c / N_KINDS;
    p.classes[c].pad[0] = p.classes[c].pad[1] = 0;
  }
  for (const NodeDesc& n : p.nodes) {
    if (n.smem_bytes > 54 * SMEM_UNIT) { set_err(p, "a tile needs more shared memory than one SM offers"); return false; }
    if (n.n_tiles >= 65536) { set_err(p, "a node has too many tiles"); return false; }
    ClassInfo& ci = p.classes[n.cls];
    ci.smem_units = std::max(ci.smem_units, (n.smem_bytes + SMEM_UNIT - 1) / SMEM_UNIT);
    ci.tmem_units = std::max(ci.tmem_units, (n.tmem_cols + TMEM_UNIT - 1) / TMEM_UNIT);
  }

  // ================================================================== arena layout
  uint64_t cur = b.const_base + b.const_cursor;
  auto place = [&](uint64_t bytes, uint64_t align = 256) {
    cur = align_up(cur, align);
    uint64_t o_ = cur;
    cur += bytes;
    return o_;
  };
  p.off_weights = Builder::WEIGHT_BASE;
  p.off_consts = b.const_base;
  p.zero_bytes_begin = 0;   // the whole arena starts zeroed: weight padding rows and columns rely on it
  p.off_nodes = place(sizeof(NodeDesc) * p.nodes.size());
  p.off_init_nodes = place(sizeof(NodeDesc) * p.init_program.size());
  p.off_succ = place(sizeof(SuccInfo) * std::max<size_t>(p.succ.size(), 1));
  p.off_roots = place(sizeof(int32_t) * std::max<size_t>(p.roots.size(), 1));
  p.off_classes = place(sizeof(ClassInfo) * N_CLASSES);
  p.off_control = place(sizeof(Control));
  p.off_queues = place(sizeof(TileQueue) * N_CLASSES);
  // queue capacity: every tile of every in-flight frame could be queued at once in the worst case
  uint64_t tiles_per_frame = 0;
  for (const NodeDesc& n : p.nodes) tiles_per_frame += n.n_tiles;
  uint64_t want = tiles_per_frame * (uint64_t)p.n_inst + 1024;
  int cap = 1 << 12;
  while ((uint64_t)cap < want && cap < (1 << 24)) cap <<= 1;
  if ((uint64_t)cap < want) { set_err(p, "tile program x frame slots needs a queue of more than 2^24 entries per class"); return false; }
  p.q_capacity = cap;
  p.off_q_entries = place(sizeof(QueueEntry) * (uint64_t)cap * N_CLASSES);
  p.admit_capacity = 1;
  while (p.admit_capacity < 2 * p.n_inst) p.admit_capacity <<= 1;
  p.off_admit = place(sizeof(AdmitRec) * p.admit_capacity);
  p.off_dep = place(sizeof(int32_t) * (uint64_t)nn * p.n_inst);
  p.off_inst_frame = place(sizeof(uint64_t) * p.n_inst);
  p.off_slot_base = place(sizeof(uint64_t) * p.n_inst);
  p.off_input_ptrs = place(sizeof(uint64_t) * N_FRAME_INPUTS * p.n_inst);
  p.trace_capacity = o.trace_capacity;
  p.off_trace = place(sizeof(TraceRec) * (uint64_t)std::max<uint32_t>(o.trace_capacity, 1));
  p.off_tmaps = place(128ull * (p.wmaps.size() + p.amaps.size() * (size_t)p.n_inst + 1), 128);
  p.slot_bytes = align_up(b.slot_cursor, 4096);
  p.off_slots = place(p.slot_bytes * p.n_inst, 4096);
  p.arena_bytes = align_up(cur, 4096);
  return true;
}

}  // namespace vla
