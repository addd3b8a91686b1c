// Host side of the ERASE step library: model layout, the per-block operation lists, the two
// schedules (serial, and early backward on side streams released by per-block events), whole-step
// CUDA-graph replay, and the C ABI declared in include/erase.h.
#include "../../include/erase.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "gemm_tc.cuh"
#include "nccl_dyn.cuh"
#include "kernels.cuh"

using namespace erase;

namespace {

thread_local std::string g_create_error;

struct Op {
  std::function<cudaError_t(cudaStream_t)> fn;
  int launches;
  const char* name = "op";  // kernel class, for the per-operation profile
  double flops = 0;         // algorithmic floating-point operations of one run
  double bytes = 0;         // algorithmic bytes (each operand read once, each result written once)
  bool leaf = false;        // backward op that only produces parameter gradients: nothing in B_b reads its output
  // What the persistent schedule needs to run this operation inside the dual-list kernel instead:
  std::vector<GemmArgs> pg;                              // the tensor-core GEMMs it consists of ...
  std::function<cudaError_t(cudaStream_t)> post;         // ... and what follows them (split-K reduction), if anything
  int post_launches = 0;
  int pew = 0;                                           // 1: ew_dst = gelu(ew_src), 2: ew_dst *= gelu'(ew_src)  (bf16)
  const void* ew_src = nullptr;
  void* ew_dst = nullptr;
  long long ew_n = 0;
};
typedef std::vector<Op> OpList;

struct Tensor {
  int block;
  std::string name;
  int rank;
  int64_t shape[2];
  bool trainable;
  size_t n;    // elements
  size_t off;  // element offset inside the frozen or the trainable arena
  bool set;
  int table = -1;   // index of the CTR input table this tensor is (trained by the main network with train_input), else -1
};

struct GraphKey {
  const void* x;
  const void* ids;
  const void* y;
  int n_streams;
  unsigned flags;
  bool operator<(const GraphKey& o) const {
    return std::tie(x, ids, y, n_streams, flags) < std::tie(o.x, o.ids, o.y, o.n_streams, o.flags);
  }
};

}  // namespace

struct erase_model {
  erase_model_spec spec;
  std::vector<erase_block_spec> blocks;
  bool bf16 = false;
  bool dry = false;  // sizing pass: no device memory is touched
  int rows = 0;      // samples, or tokens = batch*seq
  int B = 0;
  size_t esz = 4;    // bytes per activation element

  std::vector<Tensor> tensors;
  size_t frozen_n = 0, train_n = 0;
  float* frozen = nullptr;
  float* theta = nullptr;
  float* grad = nullptr;
  float* mom1 = nullptr;
  float* mom2 = nullptr;
  void* shadow = nullptr;  // bf16 copy of theta (operands of the bf16 GEMMs)
  double* tick = nullptr;  // {t, 1-beta1^t, 1-beta2^t}
  int* status = nullptr;   // device word: non-zero once a bounded device-side wait has expired
  float* losses = nullptr;

  // device memory
  char* arena = nullptr;
  size_t arena_bytes = 0, arena_used = 0;
  std::vector<void*> owned;

  cudaStream_t main = nullptr;
  std::vector<cudaStream_t> side;
  std::vector<cudaEvent_t> ev_f, ev_b;
  unsigned long long* stamps = nullptr;            // device clock stamps of the phase boundaries (ERASE_STAMPS)
  bool timeline_stamps = false;
  std::vector<cudaStream_t> leaf;                 // second side stream per block (ERASE_SPLIT_BWD)
  std::vector<std::vector<cudaEvent_t>> ev_leaf;  // per block: one event per chain->leaf hand-over, plus the join
  cudaEvent_t ev_opt = nullptr;
  std::vector<cudaEvent_t> ev_time;  // 2*(2B+1) timing events + 1 step start
  std::vector<cudaEvent_t> ev_prof;  // pairs around every operation of a profiled step
  bool timeline_valid = false;

  OpList stage, opt;
  OpList opt_tick_op;            // advances the Adam step counter (per-block optimizer mode)
  OpList opt_tables;             // the input tables' sparse update (per-block optimizer mode: behind the main block's backward)
  std::vector<OpList> opt_blk;   // the optimizer restricted to block b's slice of the parameter arena
  std::vector<OpList> fwd, hfwd, bwd;  // per block: body forward, local head + loss, backward
  erase_batch cur = {nullptr, nullptr, nullptr};
  std::map<GraphKey, std::pair<cudaGraphExec_t, int64_t>> graphs;   // executable graph and the kernels it launches

  // The main network's gradient into the input tables (train_input): sparse result of the last step.
  bool train_input = false;
  int* emb_sorted = nullptr; int* emb_seg = nullptr; int* emb_uniq = nullptr; int* emb_nuniq = nullptr;
  float* emb_grow = nullptr;
  float* mom1_in = nullptr; float* mom2_in = nullptr;   // Adam moments of the tables (frozen-arena offsets)
  long long table_stride = 0;

  // Persistent schedule (ERASE_PERSISTENT): stage s runs F_s and B_{s-1} in one dual-list kernel.
  struct PStage {
    std::vector<Op*> pre;        // operations of B_{s-1} in front of its first tensor-core GEMM (head dz, its reductions)
    TcDualPlan* plan = nullptr;
    std::vector<Op*> covered;    // operations whose GEMMs / elementwise passes run inside the kernel (their `post` follows it)
    std::vector<Op*> after;      // parameter-gradient leaves of B_{s-1} that stay ordinary launches
  };
  std::vector<PStage> pstage;
  int* pdone = nullptr;          // device counters of the dual-list kernels, tc_dual_max() per stage
  bool persistent_ok = false;
  std::string persistent_why;

  // Data-parallel replicas: every replica steps on its own rows; block b's slice of the gradient arena is
  // summed over the replicas right behind B_b, on the stream B_b ran on.
  int replicas = 1;                                  // the losses are means over replicas * rows rows
  NcclComm comm = nullptr;
  int comm_rank = 0, comm_world = 1;
  bool exchange_on = false;                          // this step sums gradients and losses over the replicas
  std::vector<std::pair<size_t, size_t>> blk_seg;    // per block: offset and length of its slice of the trainable arena
  std::vector<int> exch_order;                       // block index of every exchange the last step enqueued, in order (-1: the losses)

  int sm_budget = 0;   // CTA cap for persistent GEMMs enqueued next (0 = all SMs); set per stream by the scheduler
  int64_t launches = 0;
  bool stepped = false;
  std::string err;
  erase_status fail(erase_status st, const std::string& msg) {
    err = msg;
    return st;
  }
};

namespace {

#define CK(call)                                                                     \
  do {                                                                               \
    cudaError_t e_ = (call);                                                         \
    if (e_ != cudaSuccess)                                                           \
      return m->fail(ERASE_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
  } while (0)

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Host<->device copies are ordered on the model's main stream (a non-blocking stream does not
// synchronise with the legacy default stream that a plain cudaMemcpy uses) and waited for.
cudaError_t copy_sync(erase_model* m, void* dst, const void* src, size_t bytes, cudaMemcpyKind kind) {
  cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, m->main);
  if (e != cudaSuccess) return e;
  return cudaStreamSynchronize(m->main);
}

// ---- device memory: bump allocation from the caller's arena, else cudaMalloc ---------------
void* dev_alloc(erase_model* m, size_t bytes, bool* ok) {
  bytes = round_up(bytes ? bytes : 1, 256);
  if (m->dry) {
    m->arena_used += bytes;
    return (void*)(uintptr_t)(4096 + m->arena_used);  // never dereferenced
  }
  if (m->arena) {
    if (m->arena_used + bytes > m->arena_bytes) { *ok = false; return nullptr; }
    void* p = m->arena + m->arena_used;
    m->arena_used += bytes;
    if (cudaMemset(p, 0, bytes) != cudaSuccess) *ok = false;
    return p;
  }
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) { *ok = false; cudaGetLastError(); return nullptr; }
  m->owned.push_back(p);
  if (cudaMemset(p, 0, bytes) != cudaSuccess) *ok = false;
  return p;
}

// ---- spec validation ------------------------------------------------------------------------
bool validate(const erase_model_spec* s, std::string* why) {
  auto bad = [&](const char* w) { *why = w; return false; };
  if (!s) return bad("spec is NULL");
  if (s->dtype != ERASE_F32 && s->dtype != ERASE_BF16) return bad("dtype");
  if (s->input < 0 || s->input > ERASE_IN_CTR) return bad("input kind");
  if (s->topo != ERASE_TOPO_CHAIN && s->topo != ERASE_TOPO_PARALLEL) return bad("topology");
  if (s->batch < 1 || s->width < 1) return bad("batch/width must be positive");
  if (s->n_blocks < 1 || s->n_blocks > 4096 || !s->blocks) return bad("n_blocks/blocks");
  if (s->opt < 0 || s->opt > ERASE_OPT_ADAMW) return bad("optimizer kind");
  if (!(s->lr >= 0.f)) return bad("lr");
  if (s->opt != ERASE_OPT_SGD && (!(s->beta1 >= 0.f && s->beta1 < 1.f) || !(s->beta2 >= 0.f && s->beta2 < 1.f) || !(s->eps > 0.f)))
    return bad("Adam constants");
  if (s->input == ERASE_IN_TOKENS && (s->seq < 1 || s->vocab < 1)) return bad("seq/vocab");
  if ((long long)s->batch * (s->input == ERASE_IN_TOKENS ? s->seq : 1) > (1LL << 30)) return bad("too many rows");
  if (s->input == ERASE_IN_CTR) {
    if (s->n_dense < 0 || s->n_sparse < 1 || s->table_rows < 1 || s->emb_dim < 1) return bad("CTR sizes");
    if (s->width < s->n_sparse * s->emb_dim + s->n_dense) return bad("CTR width too small for x0");
  }
  if (s->arena && ((uintptr_t)s->arena & 255)) return bad("arena must be 256-byte aligned");
  int prev = s->width;
  for (int b = 0; b < s->n_blocks; b++) {
    const erase_block_spec& k = s->blocks[b];
    int in = s->topo == ERASE_TOPO_PARALLEL ? s->width : prev;
    if (k.n_dims < 1 || k.n_dims > ERASE_MAX_DIMS) return bad("block n_dims");
    for (int i = 0; i < k.n_dims; i++)
      if (k.dims[i] < 1) return bad("block dims must be positive");
    if (k.act < 0 || k.act > ERASE_ACT_GELU) return bad("block act");
    if (k.head == ERASE_HEAD_BCE) {
      if (k.head_out != 1) return bad("BCE head_out must be 1");
      if (s->input == ERASE_IN_TOKENS) return bad("BCE head needs labels (dense or CTR input)");
    } else if (k.head == ERASE_HEAD_SOFTMAX_CE) {
      if (s->input != ERASE_IN_TOKENS) return bad("softmax-CE head needs token input");
      if (k.head_out != s->vocab) return bad("softmax-CE head_out must equal vocab");
    } else if (k.head == ERASE_HEAD_GOODNESS) {
      if (k.head_out != 1) return bad("goodness head_out must be 1");
      if (s->input == ERASE_IN_TOKENS) return bad("goodness head needs labels (dense or CTR input)");
    } else return bad("head kind");
    int out = 0;
    switch (k.kind) {
      case ERASE_BLK_MLP:
      case ERASE_BLK_TOWER:
        if (k.n_dims < 2) return bad("MLP/TOWER need at least two dims");
        if (k.dims[0] != in) return bad("block input width does not match its producer");
        out = k.dims[k.n_dims - 1];
        break;
      case ERASE_BLK_TRANSFORMER:
        if (s->input != ERASE_IN_TOKENS) return bad("transformer block needs token input");
        if (k.n_dims != 2 || k.dims[0] != in) return bad("transformer dims = {d_model, d_ff}");
        if (k.n_heads < 1 || k.dims[0] % k.n_heads || k.dims[0] / k.n_heads > 128) return bad("n_heads");
        out = k.dims[0];
        break;
      case ERASE_BLK_CROSS:
        if (k.n_dims != 1 || k.dims[0] != in || k.n_cross < 0 || k.n_cross > 64) return bad("cross dims/n_cross");
        out = in;
        break;
      case ERASE_BLK_DOT: {
        if (s->input != ERASE_IN_CTR || s->topo != ERASE_TOPO_PARALLEL) return bad("dot block needs CTR input, parallel topology");
        if (k.n_dims < 2) return bad("dot block needs a tower");
        int nv = s->n_sparse + 1;
        if (k.dims[0] < nv * (nv - 1) / 2 + s->emb_dim) return bad("dot feature width too small");
        if (s->width - s->n_sparse * s->emb_dim < 1) return bad("dot block needs dense columns");
        out = k.dims[k.n_dims - 1];
        break;
      }
      case ERASE_BLK_MAIN: {
        if (b != s->n_blocks - 1 || s->n_blocks < 2) return bad("a MAIN block must be the last of at least two blocks");
        if (s->input == ERASE_IN_TOKENS || k.head != ERASE_HEAD_BCE) return bad("MAIN block needs labels (dense or CTR input) and a BCE head");
        if (k.n_dims < 2) return bad("MAIN block needs a tower");
        long long w = (k.flags & ERASE_MAIN_READS_INPUT) ? s->width : 0;
        int pw = s->width;
        for (int i = 0; i < b; i++) {
          const erase_block_spec& q = s->blocks[i];
          const int o = (q.kind == ERASE_BLK_CROSS || q.kind == ERASE_BLK_TRANSFORMER) ? q.dims[0] : q.dims[q.n_dims - 1];
          w += o;
          pw = o;
        }
        (void)pw;
        if (k.dims[0] != w) return bad("MAIN dims[0] must be the width of [z_0 | z_1 | .. | z_B]");
        if (b + 1 > CONCAT_MAX) return bad("too many blocks in front of a MAIN block");
        out = k.dims[k.n_dims - 1];
        break;
      }
      default:
        return bad("block kind");
    }
    prev = out;
  }
  if (s->replicas < 0 || s->replicas > 65536) return bad("replicas out of range");
  if (s->train_input) {
    const erase_block_spec& last = s->blocks[s->n_blocks - 1];
    if (s->input != ERASE_IN_CTR || last.kind != ERASE_BLK_MAIN || !(last.flags & ERASE_MAIN_READS_INPUT))
      return bad("train_input needs CTR input and a MAIN block that reads z_0");
    if (s->batch > embed_max_batch()) return bad("train_input: batch too large for the embedding backward");
  }
  return true;
}

// ---- tensor table ---------------------------------------------------------------------------
void add_tensor(erase_model* m, int block, const std::string& name, int64_t d0, int64_t d1, bool trainable) {
  Tensor t;
  t.block = block;
  t.name = name;
  t.rank = d1 > 0 ? 2 : 1;
  t.shape[0] = d0;
  t.shape[1] = d1 > 0 ? d1 : 0;
  t.trainable = trainable;
  t.n = (size_t)d0 * (size_t)(d1 > 0 ? d1 : 1);
  size_t& top = trainable ? m->train_n : m->frozen_n;
  t.off = top;
  top += round_up(t.n, 64);
  t.set = false;
  m->tensors.push_back(t);
}

void build_tensor_table(erase_model* m) {
  const erase_model_spec& s = m->spec;
  if (s.input == ERASE_IN_TOKENS) {
    add_tensor(m, -1, "tok_emb", s.vocab, s.width, false);
    add_tensor(m, -1, "pos_emb", s.seq, s.width, false);
  } else if (s.input == ERASE_IN_CTR) {
    for (int t = 0; t < s.n_sparse; t++) {
      add_tensor(m, -1, "table" + std::to_string(t), s.table_rows, s.emb_dim, false);
      if (s.train_input) m->tensors.back().table = t;
    }
  }
  for (int b = 0; b < m->B; b++) {
    const erase_block_spec& k = m->blocks[b];
    int out = 0;
    auto linears = [&](int first) {
      for (int i = first; i + 1 < k.n_dims; i++) {
        add_tensor(m, b, "W" + std::to_string(i - first), k.dims[i + 1], k.dims[i], true);
        add_tensor(m, b, "b" + std::to_string(i - first), k.dims[i + 1], 0, true);
      }
      out = k.dims[k.n_dims - 1];
    };
    switch (k.kind) {
      case ERASE_BLK_MLP:
      case ERASE_BLK_TOWER:
      case ERASE_BLK_MAIN:
        linears(0);
        break;
      case ERASE_BLK_TRANSFORMER: {
        int d = k.dims[0], ff = k.dims[1];
        add_tensor(m, b, "ln1_g", d, 0, true);
        add_tensor(m, b, "ln1_b", d, 0, true);
        add_tensor(m, b, "Wqkv", 3 * d, d, true);
        add_tensor(m, b, "bqkv", 3 * d, 0, true);
        add_tensor(m, b, "Wproj", d, d, true);
        add_tensor(m, b, "bproj", d, 0, true);
        add_tensor(m, b, "ln2_g", d, 0, true);
        add_tensor(m, b, "ln2_b", d, 0, true);
        add_tensor(m, b, "W1", ff, d, true);
        add_tensor(m, b, "b1", ff, 0, true);
        add_tensor(m, b, "W2", d, ff, true);
        add_tensor(m, b, "b2", d, 0, true);
        out = d;
        break;
      }
      case ERASE_BLK_CROSS:
        for (int i = 0; i < k.n_cross; i++) {
          add_tensor(m, b, "Wc" + std::to_string(i), k.dims[0], k.dims[0], true);
          add_tensor(m, b, "bc" + std::to_string(i), k.dims[0], 0, true);
        }
        out = k.dims[0];
        break;
      case ERASE_BLK_DOT:
        add_tensor(m, b, "Wd", m->spec.emb_dim, m->spec.width - m->spec.n_sparse * m->spec.emb_dim, true);
        add_tensor(m, b, "bd", m->spec.emb_dim, 0, true);
        linears(0);
        break;
    }
    if (k.head != ERASE_HEAD_GOODNESS) add_tensor(m, b, "Wh", k.head_out, out, true);   // the goodness head has only its threshold
    add_tensor(m, b, "bh", k.head_out, 0, true);
  }
}

// ---- plan builder ---------------------------------------------------------------------------
struct Builder {
  erase_model* m;
  bool ok = true;
  int cursor = 0;  // next tensor index of the block being built

  void* act_buf(size_t elems) { return dev_alloc(m, elems * m->esz, &ok); }
  float* f32_buf(size_t elems) { return (float*)dev_alloc(m, elems * sizeof(float), &ok); }
  int* tickets(int cols) { return (int*)dev_alloc(m, (size_t)((cols + 63) / 64) * sizeof(int), &ok); }  // zero-initialised

  const Tensor& T(int idx) const { return m->tensors[idx]; }
  const void* Wop(int idx) const {  // GEMM operand copy of a weight matrix
    return m->bf16 ? (const void*)((const __nv_bfloat16*)m->shadow + T(idx).off) : (const void*)(m->theta + T(idx).off);
  }
  const float* Wf(int idx) const { return m->theta + T(idx).off; }
  float* G(int idx) const { return m->grad + T(idx).off; }

  static void note(OpList& ops, const char* name, double flops = 0, double bytes = 0) {
    ops.back().name = name;
    ops.back().flops = flops;
    ops.back().bytes = bytes;
  }
  const char* gemm_tag = "gemm";

  // Small column reductions of the block being built (bias gradients, LayerNorm gain/shift
  // gradients, the BCE head's own gradients): collected here and run as ONE launch at the end of
  // the block's backward.  Their inputs are written once per step and nothing in B_b reads their
  // outputs, so deferring them changes no value.
  std::vector<ReduceJob> jobs;
  double jobs_flops = 0, jobs_bytes = 0;
  // When the collected jobs run: always at the end of B_b; the BCE head's own reductions also right
  // behind the head (measured: C5 w512/b4096 0.825 ms against 0.861 ms), a transformer block's
  // first three not separately (C2 1.054 ms against 1.065 ms with a launch half-way).
  int flush_mode = getenv("ERASE_REDUCE_FLUSH") ? atoi(getenv("ERASE_REDUCE_FLUSH")) : 1;   // 0 end only, 1 + after a BCE head, 2 every job, 3 + half-way in a transformer block
  void add_job(OpList& ops, ReduceJob j, double flops, double bytes) {
    j.strips = reduce_job_strips(j);
    jobs.push_back(j);
    jobs_flops += flops;
    jobs_bytes += bytes;
    if (flush_mode == 2) flush_jobs(ops);
  }
  void head_flush(OpList& ops) { if (flush_mode == 1 || flush_mode == 3) flush_jobs(ops); }
  void mid_flush(OpList& ops) { if (flush_mode == 3) flush_jobs(ops); }
  void colsum_job(OpList& ops, const void* X, bool x_bf16, long long ldx, int rows, int cols, const float* scale, float* out,
                  int dact, const float* colscale, double flops, double bytes) {
    ReduceJob j;
    j.kind = 0; j.x_f32 = x_bf16 ? 0 : 1; j.dact = dact;
    j.rows = rows; j.cols = cols; j.ldx = ldx;      // chunks and workspace are set when the batch is flushed
    j.X = X; j.a = scale; j.b = colscale;
    j.out0 = out; j.tickets = tickets(cols);
    add_job(ops, j, flops, bytes);
  }
  void flush_jobs(OpList& bw) {
    if (jobs.empty()) return;
    // Row partition: the launch as a whole gets about two CTAs per SM, shared out over the jobs'
    // column strips, so that a CTA has a few hundred rows to stream instead of 64.
    int all_strips = 0;
    for (const ReduceJob& j : jobs) all_strips += j.strips;
    static const int batch_ctas = getenv("ERASE_REDUCE_CTAS") ? atoi(getenv("ERASE_REDUCE_CTAS")) : 296;
    int total = 0;
    for (ReduceJob& j : jobs) {
      int chunks = std::max(1, batch_ctas / std::max(1, all_strips));
      static const int rows_per_cta = getenv("ERASE_REDUCE_ROWS") ? atoi(getenv("ERASE_REDUCE_ROWS")) : 256;
      chunks = std::max(chunks, (j.rows + rows_per_cta - 1) / rows_per_cta);   // a CTA streams at most about that many rows
      chunks = std::min(chunks, std::max(1, j.rows / 64));
      j.chunks = chunks;
      j.ws = chunks > 1 ? f32_buf((size_t)(j.kind == 1 ? 2 : 1) * chunks * j.cols) : nullptr;
      j.cta_begin = total;
      total += j.strips * j.chunks;
    }
    const int n = (int)jobs.size();
    ReduceJob* dev = (ReduceJob*)dev_alloc(m, sizeof(ReduceJob) * jobs.size(), &ok);
    if (ok && dev && !m->dry && cudaMemcpy(dev, jobs.data(), sizeof(ReduceJob) * jobs.size(), cudaMemcpyHostToDevice) != cudaSuccess) ok = false;
    bw.push_back({[=](cudaStream_t s) { return reduce_batch(dev, n, total, s); }, 1});
    note(bw, "reduce_batch", jobs_flops, jobs_bytes);
    bw.back().leaf = true;
    jobs.clear();
    jobs_flops = jobs_bytes = 0;
  }

  void gemm(OpList& ops, GemmArgs g, bool* xcol_used = nullptr) {
    size_t before = ops.size();
    gemm_inner(ops, g, xcol_used);
    double fl = 2.0 * g.M * g.N * g.K;
    double by = ((double)g.M * g.K + (double)g.N * g.K) * m->esz + (double)g.M * g.N * (g.c_f32 ? 4 : m->esz);
    if (ops.size() > before) note(ops, gemm_tag, fl, by);
  }
  void gemm_inner(OpList& ops, GemmArgs g, bool* xcol_used = nullptr) {
    if (xcol_used) *xcol_used = false;
    const bool bf = m->bf16;
    const bool tc_ok = bf && tc_gemm_supported(g);
    void* out = g.C;
    const long long ldo = g.ldc;
    const bool out_bf = bf && !g.c_f32;   // split-K partials are summed in fp32 and rounded once
    if (g.splits > 1) g.ws = f32_buf((size_t)g.splits * g.M * g.N);
    TcPlan plan;
    int* sched = tc_ok ? (int*)dev_alloc(m, 2 * sizeof(int), &ok) : nullptr;   // dynamic tile scheduler words (zeroed)
    const bool use_tc = tc_ok && !m->dry && tc_gemm_plan(g, m->status, &plan);
    plan.sched = sched;
    if (use_tc && xcol_used) *xcol_used = plan.xcol != 0;
    if (use_tc) {
      if (g.splits > 1) {
        ops.push_back({[g, plan, out, ldo, out_bf, mm = m](cudaStream_t s) {
                         cudaError_t e = tc_gemm_launch(g, plan, s, mm->sm_budget);
                         if (e != cudaSuccess) return e;
                         return splitk_reduce(g.ws, g.splits, (long long)g.M * g.N, g.N, out, ldo, s, out_bf);
                       }, 2});
        ops.back().post = [g, out, ldo, out_bf](cudaStream_t s) { return splitk_reduce(g.ws, g.splits, (long long)g.M * g.N, g.N, out, ldo, s, out_bf); };
        ops.back().post_launches = 1;
      } else {
        ops.push_back({[g, plan, mm = m](cudaStream_t s) { return tc_gemm_launch(g, plan, s, mm->sm_budget); }, 1});
      }
      ops.back().pg = {g};
      return;
    }
    if (g.splits > 1) {
      ops.push_back({[g, bf, out, ldo, out_bf](cudaStream_t s) {
                       cudaError_t e = gemm_simt(g, bf, s);
                       if (e != cudaSuccess) return e;
                       return splitk_reduce(g.ws, g.splits, (long long)g.M * g.N, g.N, out, ldo, s, out_bf);
                     }, 2});
    } else {
      ops.push_back({[g, bf](cudaStream_t s) { return gemm_simt(g, bf, s); }, 1});
    }
  }

  // GELU is NOT fused into the GEMM epilogues: its erf/exp chain on the few epilogue warps made
  // those GEMMs 2-3x slower than the GEMM plus a separate, fully occupied elementwise pass
  // (which moves 4-6 bytes per element at HBM speed).  ReLU (a compare) stays fused.
  void act_op(OpList& ops, const void* u, void* y, int act, long long n) {
    bool bf = m->bf16;
    ops.push_back({[=](cudaStream_t s) { return ew_act(u, y, act, n, bf, s); }, 1});
    note(ops, "ew_act", 10.0 * n, 2.0 * n * m->esz);
    if (bf && act == ACT_GELU) { ops.back().pew = 1; ops.back().ew_src = u; ops.back().ew_dst = y; ops.back().ew_n = n; }
  }
  void dact_op(OpList& ops, void* d, const void* src, int act, long long n) {
    bool bf = m->bf16;
    ops.push_back({[=](cudaStream_t s) { return ew_dact(d, src, act, n, bf, s); }, 1});
    note(ops, "ew_dact", 10.0 * n, 3.0 * n * m->esz);
    if (bf && act == ACT_GELU) { ops.back().pew = 2; ops.back().ew_src = src; ops.back().ew_dst = d; ops.back().ew_n = n; }
  }

  // Split count for a GEMM of `tiles` 256 x 256 CTA-pair tiles over a contraction of length `kdim`, written
  // as fp32 partials: few tiles -> fill one wave of the 74 pairs; a little more than a whole number of
  // waves (96 tiles: two waves, the second 30 % full) -> the split that fills its last wave best, as long
  // as every split keeps at least 4096 of the contraction (C4's head dgrad, K = 32768: 393 -> 296 us).
  static int pair_wave_splits(long long tiles, int kdim) {
    const int smax = std::min(8, kdim / 1024);
    if (smax < 2 || tiles < 1) return 1;
    if (tiles <= 37) return (int)std::min<long long>(74 / tiles, smax);
    auto eff = [&](int s) { const long long t = tiles * s; return (double)t / (74.0 * ((t + 73) / 74)); };
    int best = 1;
    for (int s = 2; s <= smax && kdim / s >= 4096; s++)     // (a split of a 3072-long contraction cost more in partials than it won: 47 -> 56 us)
      if (eff(s) > eff(best) + 0.04) best = s;
    return eff(best) >= eff(1) + 0.15 ? best : 1;
  }

  // Y[M,N] = epi(X[M,K] W[N,K]^T)
  void lin_fwd(OpList& ops, const void* X, long long ldx, int widx, int bidx, void* Y, int M, int N, int K, Epilogue e) {
    GemmArgs g;
    g.M = M; g.N = N; g.K = K;
    g.A = X; g.sa_m = ldx; g.sa_k = 1;
    g.B = Wop(widx); g.sb_n = K; g.sb_k = 1;
    g.C = Y; g.ldc = N;
    e.bias = bidx >= 0 ? Wf(bidx) : nullptr;
    if (e.ld_aux == 0) e.ld_aux = N;
    g.epi = e;
    gemm_tag = "gemm_fwd";
    gemm(ops, g);
  }
  // dX[M,K] = epi(dY[M,N] W[N,K])
  void lin_dgrad(OpList& ops, const void* dY, int widx, void* dX, int M, int N, int K, Epilogue e) {
    GemmArgs g;
    g.M = M; g.N = K; g.K = N;
    g.A = dY; g.sa_m = N; g.sa_k = 1;
    g.B = Wop(widx); g.sb_n = 1; g.sb_k = K;
    g.C = dX; g.ldc = K;
    if (e.ld_aux == 0) e.ld_aux = K;
    g.epi = e;
    // A narrow dX (few output tiles) with a long contraction leaves most SMs idle and each busy one
    // bound by what a single SM can pull from L2: split the contraction over CTA pairs instead
    // (fp32 partials, summed in a fixed order and rounded once).
    const bool plain = !e.bias && e.act == ACT_NONE && !e.mul && !e.res && e.dact == ACT_NONE && !e.pre_out && e.alpha == 1.f;
    if (m->bf16 && plain && M >= 256 && K >= 256 && N >= 2048) {
      const int splits = pair_wave_splits((long long)((M + 255) / 256) * ((K + 255) / 256), N);
      if (splits > 1) g.splits = splits;
    }
    gemm_tag = "gemm_dgrad";
    gemm(ops, g);
  }
  // dW[N,K] = dY[M,N]^T X[M,K]  (fp32, deterministic split over M), db[N] = column sums of dY
  // xcol_out (with xcol_used): X has 16 more columns behind its K; ask the GEMM for dY^T times the first of them as
  // well (GemmArgs::xcol_out).  *xcol_used says whether the plan took it; if not, the caller forms that product itself.
  void lin_wgrad(OpList& ops, const void* dY, const void* X, long long ldx, int widx, int bidx, int M, int N, int K,
                 bool skip_bias = false, bool bias_now = false, float* xcol_out = nullptr, bool* xcol_used = nullptr) {
    GemmArgs g;
    g.M = N; g.N = K; g.K = M;
    g.A = dY; g.sa_m = 1; g.sa_k = N;
    g.B = X; g.sb_n = 1; g.sb_k = ldx;
    g.C = G(widx); g.ldc = K; g.c_f32 = 1;
    g.xcol_out = xcol_out;
    if (xcol_used) *xcol_used = false;
    if (groupable(g)) {   // a small weight gradient: runs with the block's other small ones in one launch
      g.xcol_out = nullptr;
      group.push_back(g);
      if (bidx >= 0 && !skip_bias) {
        if (bias_now || (double)M * N * m->esz > 16.0e6) { bias_grad(ops, dY, N, M, N, bidx); ops.back().leaf = true; }
        else colsum_job(ops, dY, m->bf16, N, M, N, nullptr, G(bidx), ACT_NONE, nullptr, (double)M * N, (double)M * N * m->esz);
      }
      if ((int)group.size() == 4) flush_group(ops);
      return;
    }
    long long tiles = (long long)((N + 63) / 64) * ((K + 63) / 64);
    int splits = (int)((296 + tiles - 1) / tiles);
    int maxs = M / 64 > 0 ? M / 64 : 1;
    if (splits > maxs) splits = maxs;
    if (splits > 64) splits = 64;
    // wide enough for 256 x 256 tiles over CTA pairs: split so that one wave of the 74 pairs is nearly full
    if (m->bf16 && N >= 256 && K > 128) {
      const long long pt = (long long)((N + 255) / 256) * ((K + 255) / 256);
      const int s_lo = (int)(74 / pt);
      static const int pair_min = getenv("ERASE_WGRAD_PAIR_MIN") ? atoi(getenv("ERASE_WGRAD_PAIR_MIN")) : 66;
      if (s_lo >= 1 && pt * s_lo >= pair_min && s_lo <= M / 512 && s_lo <= 16) splits = s_lo;
    }
    g.splits = splits < 1 ? 1 : splits;
    gemm_tag = "gemm_wgrad";
    const size_t before = ops.size();
    if (g.splits > 1) g.xcol_out = nullptr;
    gemm(ops, g, xcol_used);
    if (bidx >= 0 && !skip_bias) {
      // a large dY (the logits) is summed right behind its wgrad, while it is still in L2
      if (bias_now || (double)M * N * m->esz > 16.0e6) bias_grad(ops, dY, N, M, N, bidx);
      else colsum_job(ops, dY, m->bf16, N, M, N, nullptr, G(bidx), ACT_NONE, nullptr, (double)M * N, (double)M * N * m->esz);
    }
    for (size_t i = before; i < ops.size(); i++) ops[i].leaf = true;
  }
  // ---- small weight gradients of a block, grouped into one launch --------------------------------
  std::vector<GemmArgs> group;
  int group_mode = getenv("ERASE_WGRAD_GROUP") ? atoi(getenv("ERASE_WGRAD_GROUP")) : 1;
  bool groupable(const GemmArgs& g) const {
    if (!group_mode || !m->bf16 || !tc_gemm_supported(g)) return false;
    const long long tiles = (long long)((g.M + 127) / 128) * ((g.N + 127) / 128);
    return tiles <= 32 && g.K >= 512 && g.N % 4 == 0 && g.ldc % 4 == 0 && (reinterpret_cast<uintptr_t>(g.C) & 15) == 0;
  }
  void flush_group(OpList& ops) {
    const int n = (int)group.size();
    if (n == 0) return;
    long long tiles = 0;
    int kmin = 1 << 30;
    for (const GemmArgs& g : group) {
      tiles += (long long)((g.M + 127) / 128) * ((g.N + 127) / 128);
      kmin = std::min(kmin, g.K);
    }
    // CTAs of the launch: a full wave (148) is fastest alone (C2 serial 1.41 ms against 1.51 ms
    // ungrouped) but its persistent CTAs then hold every SM while the other streams' kernels wait
    // (C2 ERASE 1.120 ms against 1.088 ms); about 64 keeps most of the serial gain (1.44 ms) at no
    // cost under ERASE (1.087 ms; C3 1.196 ms against 1.285 ms ungrouped at any setting).
    static const int group_ctas = getenv("ERASE_GROUP_CTAS") ? atoi(getenv("ERASE_GROUP_CTAS")) : 64;
    int splits = (int)(group_ctas / tiles);
    splits = std::max(1, std::min(std::min(splits, kmin / 128), 16));
    double flops = 0, bytes = 0;
    std::vector<ReduceJob> rj;
    int total = 0;
    for (GemmArgs& g : group) {
      g.splits = splits;
      g.ws = f32_buf((size_t)splits * g.M * g.N);
      ReduceJob j;
      j.kind = 2; j.x_f32 = 1; j.rows = splits; j.cols = g.N; j.chunks = 1; j.ldx = g.ldc; j.mn = (long long)g.M * g.N;
      j.X = g.ws; j.out0 = (float*)g.C;
      j.strips = reduce_job_strips(j);
      j.cta_begin = total;
      total += j.strips;
      rj.push_back(j);
      flops += 2.0 * g.M * g.N * g.K;
      bytes += ((double)g.M * g.K + (double)g.N * g.K) * m->esz + 4.0 * g.M * g.N;
    }
    ReduceJob* dev = (ReduceJob*)dev_alloc(m, sizeof(ReduceJob) * rj.size(), &ok);
    if (ok && dev && !m->dry && cudaMemcpy(dev, rj.data(), sizeof(ReduceJob) * rj.size(), cudaMemcpyHostToDevice) != cudaSuccess) ok = false;
    TcGroupPlan plan;
    const bool planned = !m->dry && tc_wgrad_group_plan(group.data(), n, m->status, &plan);
    std::vector<GemmArgs> gs = group;
    erase_model* mm = m;
    if (planned)
      ops.push_back({[plan, dev, n, total, mm](cudaStream_t s) {
                       cudaError_t e = tc_wgrad_group_launch(plan, s, mm->sm_budget);
                       if (e != cudaSuccess) return e;
                       return reduce_batch(dev, n, total, s);
                     }, 2});
    else   // descriptors could not be encoded (never expected): the same partials from the SIMT kernel
      ops.push_back({[gs, dev, n, total](cudaStream_t s) {
                       for (const GemmArgs& g : gs) {
                         cudaError_t e = gemm_simt(g, true, s);
                         if (e != cudaSuccess) return e;
                       }
                       return reduce_batch(dev, n, total, s);
                     }, n + 1});
    note(ops, "gemm_wgrad", flops, bytes);
    ops.back().leaf = true;
    if (planned) {
      ops.back().pg = gs;
      ops.back().post = [dev, n, total](cudaStream_t s) { return reduce_batch(dev, n, total, s); };
      ops.back().post_launches = 1;
    }
    group.clear();
  }

  void bias_grad(OpList& ops, const void* dY, long long ld, int M, int N, int bidx) {
    int chunks = colsum_chunks(M, N);
    float* ws = chunks > 1 ? f32_buf((size_t)chunks * N) : nullptr;
    float* out = G(bidx);
    bool bf = m->bf16;
    int* tk = tickets(N);
    ops.push_back({[=](cudaStream_t s) { return colsum(dY, bf, ld, M, N, nullptr, ws, chunks, tk, out, s); }, 1});
    note(ops, "colsum", (double)M * N, (double)M * N * m->esz);
  }

  // ---- heads: forward computes the local loss and the loss gradient, backward the head's own
  // gradients and dz (times act'(src) when the block ends in an activation) ------------------
  // last_bias >= 0 (BCE head only): also emit the gradient of the bias of the Linear that produced z,
  // db[c] = w[c] * sum_r ds[r] * act'(src[r,c]), from the fp32 loss gradient rather than from the
  // bf16-rounded dz (the sum over r cancels heavily when the labels are balanced).  Returns true
  // if it did, so that the caller skips the ordinary column sum for that bias.
  bool head(int b, const erase_block_spec& k, const void* z, int d, int wh, int bh, OpList& /*body forward*/, OpList& bw, void* dz,
            int dact, const void* dact_src, int last_bias = -1) {
    erase_model* mm = m;
    OpList& f = m->hfwd[b];   // the head and its loss form their own list: only the backward consumes them
    bool bf = m->bf16;
    int rows = m->rows;
    float* rowloss = f32_buf(rows);
    float* loss_out = m->losses + b;
    float inv = 1.f / ((float)rows * (float)m->replicas);   // mean over every replica's rows: the replicas' gradients then simply add
    if (k.head == ERASE_HEAD_GOODNESS) {
      // Section 2.1: BCE on the goodness score G = sum_j z_j^2 with the logit G + bh.  The head has
      // no weight tensor, so its threshold sits where Wh would (index wh).
      const int bh_idx = wh;
      float* ds = f32_buf(rows);
      const float* bb = Wf(bh_idx);
      f.push_back({[=](cudaStream_t s) { return goodness_head_fwd(z, d, bb, mm->cur.y, rowloss, ds, rows, d, inv, bf, s); }, 1});
      note(f, "goodness_head_fwd", 2.0 * rows * d, (double)rows * d * m->esz);
      f.push_back({[=](cudaStream_t s) { return reduce_sum(rowloss, rows, inv, loss_out, s); }, 1});
      note(f, "loss_reduce", rows, 4.0 * rows);
      bw.push_back({[=](cudaStream_t s) { return goodness_head_dz(ds, z, dz, dact, dact_src, rows, d, bf, s); }, 1});
      note(bw, "goodness_head_dz", 2.0 * rows * d, 2.0 * rows * d * m->esz);
      colsum_job(bw, ds, false, 1, rows, 1, nullptr, G(bh_idx), ACT_NONE, nullptr, rows, 4.0 * rows);
      head_flush(bw);
      return false;
    }
    if (k.head == ERASE_HEAD_BCE) {
      float* ds = f32_buf(rows);
      const float* w = Wf(wh);
      const float* bb = Wf(bh);
      f.push_back({[=](cudaStream_t s) { return bce_head_fwd(z, d, w, bb, mm->cur.y, rowloss, ds, rows, d, inv, bf, s); }, 1});
      note(f, "bce_head_fwd", 2.0 * rows * d, (double)rows * d * m->esz);
      f.push_back({[=](cudaStream_t s) { return reduce_sum(rowloss, rows, inv, loss_out, s); }, 1});
      note(f, "loss_reduce", rows, 4.0 * rows);
      bw.push_back({[=](cudaStream_t s) { return bce_head_dz(ds, w, dz, dact, dact_src, rows, d, bf, s); }, 1});
      note(bw, "bce_head_dz", (double)rows * d, (double)rows * d * m->esz);
      colsum_job(bw, z, bf, d, rows, d, ds, G(wh), ACT_NONE, nullptr, 2.0 * rows * d, (double)rows * d * m->esz);
      colsum_job(bw, ds, false, 1, rows, 1, nullptr, G(bh), ACT_NONE, nullptr, rows, 4.0 * rows);
      if (last_bias >= 0) {
        const void* src = dact != ACT_NONE ? dact_src : nullptr;
        colsum_job(bw, src, bf, d, rows, d, ds, G(last_bias), src ? dact : ACT_NONE, w, 2.0 * rows * d,
                   src ? (double)rows * d * m->esz : 4.0 * rows);
        head_flush(bw);   // the head's own reductions read what the forward left: run them at the start of B_b
        return true;
      }
      head_flush(bw);
      return false;
    } else {
      int V = k.head_out, T_ = m->spec.seq;
      void* logits = act_buf((size_t)rows * V);
      if (head_ce_exp(b, z, d, wh, bh, logits, V, T_, rowloss, loss_out, inv, f, bw, dz)) {
        if (dact != ACT_NONE) {
          long long n = (long long)rows * d;
          bw.push_back({[=](cudaStream_t s) { return ew_dact(dz, dact_src, dact, n, bf, s); }, 1});
          note(bw, "ew_dact", (double)n, 3.0 * n * m->esz);
        }
        return false;
      }
      lin_fwd(f, z, d, wh, bh, logits, rows, V, d, Epilogue());
      const int ce_fused = getenv("ERASE_CE_FUSED") ? atoi(getenv("ERASE_CE_FUSED")) : 1;   // 0 never, 1 by size, 2 whenever supported
      // worth it when the gradient matrix is far larger than L2 (C4: 1 GB; 346 + 27 us against 322 + 97 us);
      // a 64 MB one (C2) is re-read from L2 by the plain column sum faster than the per-CTA partials cost
      const bool fused = ce_fused && softmax_ce_fused_supported(V, bf, logits) && (ce_fused == 2 || (double)rows * V * 2 > 256.0e6);
      if (fused) {
        // the loss pass also leaves per-CTA column sums of dlogits: the bias gradient needs no second read of them
        const int ctas = softmax_ce_fused_ctas(rows);
        float* colpart = f32_buf((size_t)ctas * V);
        f.push_back({[=](cudaStream_t s) { return softmax_ce_fused(logits, mm->cur.ids, T_, rowloss, colpart, rows, V, inv, s); }, 1});
        note(f, "softmax_ce", 4.0 * rows * V, 2.0 * rows * V * m->esz);
        colsum_job(bw, colpart, false, V, ctas, V, nullptr, G(bh), ACT_NONE, nullptr, (double)ctas * V, 4.0 * ctas * V);
      } else {
        f.push_back({[=](cudaStream_t s) { return softmax_ce_inplace(logits, mm->cur.ids, T_, rowloss, rows, V, inv, bf, s); }, 1});
        note(f, "softmax_ce", 4.0 * rows * V, 2.0 * rows * V * m->esz);
      }
      f.push_back({[=](cudaStream_t s) { return reduce_sum(rowloss, rows, inv, loss_out, s); }, 1});
      note(f, "loss_reduce", rows, 4.0 * rows);
      lin_wgrad(bw, logits, z, d, wh, bh, rows, V, d, fused, true);
      lin_dgrad(bw, logits, wh, dz, rows, V, d, Epilogue());
      if (dact != ACT_NONE) {
        long long n = (long long)rows * d;
        bw.push_back({[=](cudaStream_t s) { return ew_dact(dz, dact_src, dact, n, bf, s); }, 1});
        note(bw, "ew_dact", (double)n, 3.0 * n * m->esz);
      }
      return false;
    }
  }

  // ---- softmax cross-entropy head whose loss and gradient never read the logits back ------------
  // (bf16 models whose head GEMM runs on the tensor cores; the kernels are described in kernels.cu).
  // Forward: target logit -> head GEMM with the exp epilogue (P and partial sums) -> finalize (loss,
  // row scales, one patched element of P per row) -> exact recomputation of unsafe rows (normally
  // none) -> mean loss.  Backward: the gradient of the logits is (row scale) (.) P, so dW_h comes from P
  // and the scaled copy of z, db_h from a weighted column sum of P, dz from P W_h.
  // Returns false (nothing enqueued) when the head does not qualify: the caller then takes the
  // path with a separate softmax pass.
  bool head_ce_exp(int /*b*/, const void* z, int d, int wh, int bh, void* logits, int V, int T_, float* rowloss, float* loss_out,
                   float inv, OpList& f, OpList& bw, void* dz) {
    const int ce_mode = getenv("ERASE_CE_MODE") ? atoi(getenv("ERASE_CE_MODE")) : 1;   // 0: separate softmax pass
    erase_model* mm = m;
    const int rows = m->rows;
    if (!ce_mode || !m->bf16 || V % 8 || d % 8 || V < 16 || d < 64) return false;
    GemmArgs g;
    g.M = rows; g.N = V; g.K = d;
    g.A = z; g.sa_m = d; g.sa_k = 1;
    g.B = Wop(wh); g.sb_n = d; g.sb_k = 1;
    g.C = logits; g.ldc = V;
    g.epi.bias = Wf(bh);
    g.epi.ld_aux = V;
    if (!tc_gemm_supported(g)) return false;
    // partial sums: one per row and group of columns; the group width (64..128) follows the tile
    // choice, which is only known with real pointers, so the buffer is sized for the narrowest
    const int max_groups = (V + 63) / 64;
    float* psum = f32_buf((size_t)rows * max_groups);
    float* ref = f32_buf(rows);
    float* lt = f32_buf(rows);
    float* rowscale = f32_buf(rows);
    int* tgt = (int*)dev_alloc(m, (size_t)rows * sizeof(int), &ok);
    int* bad = (int*)dev_alloc(m, (size_t)(rows + 1) * sizeof(int), &ok);
    // r (.) z for the weight-gradient GEMM, each row followed by [r_n, 0 x 15]: with those the same GEMM also
    // forms the bias gradient sum_n r_n P[n,:] (GemmArgs::xcol_out) where its plan allows
    const int ldzs = d + 16;
    void* zs = act_buf((size_t)rows * ldzs);
    g.epi.ce_ref = ref;
    g.epi.ce_psum = psum;
    TcPlan plan;
    int* sched = (int*)dev_alloc(m, 2 * sizeof(int), &ok);
    int groups = max_groups;
    if (!m->dry) {
      if (!tc_gemm_plan(g, m->status, &plan)) { ok = false; return true; }
      plan.sched = sched;
      if (!plan.tma_c) { ok = false; return true; }
      const int gc = tc_ce_group_cols(plan);
      groups = (V + gc - 1) / gc;
      g.epi.ce_groups = groups;
    }
    const void* Wb = Wop(wh);
    const float* bias = Wf(bh);
    f.push_back({[=](cudaStream_t s) { return ce_target_logit(z, Wb, bias, mm->cur.ids, T_, rows, d, V, tgt, ref, lt, bad, s); }, 1});
    note(f, "ce_target_logit", 2.0 * rows * d, 4.0 * rows * d);
    f.push_back({[g, plan, mm](cudaStream_t s) { return tc_gemm_launch(g, plan, s, mm->sm_budget); }, 1});
    note(f, "gemm_fwd", 2.0 * rows * V * d, ((double)rows * d + (double)V * d) * 2 + 2.0 * rows * V);
    f.push_back({[=](cudaStream_t s) { return ce_finalize(psum, groups, ref, lt, tgt, logits, V, z, zs, ldzs, rowloss, rowscale, bad, rows, d, inv, s); }, 1});
    note(f, "ce_finalize", (double)rows * groups, 4.0 * rows * groups + 4.0 * rows * d);
    f.push_back({[=](cudaStream_t s) { return ce_fixup(bad, mm->status, tgt, z, Wb, bias, logits, ref, lt, zs, ldzs, rowloss, rowscale, rows, d, V, inv, s); }, 1});
    note(f, "ce_fixup", 0, 0);
    f.push_back({[=](cudaStream_t s) { return reduce_sum(rowloss, rows, inv, loss_out, s); }, 1});
    note(f, "loss_reduce", rows, 4.0 * rows);
    // backward: parameter gradients (leaves) ...
    const size_t before = bw.size();
    const int env_xcol = getenv("ERASE_HEAD_XCOL") ? atoi(getenv("ERASE_HEAD_XCOL")) : 1;   // 0: separate weighted column sum of P
    bool db_in_wgrad = false;
    lin_wgrad(bw, logits, zs, ldzs, wh, -1, rows, V, d, true, false, env_xcol ? G(bh) : nullptr, &db_in_wgrad);
    {
      // (the scratch of the separate pass is laid out either way: the sizing pass cannot know the GEMM's plan)
      const int chunks = colsum_chunks(rows, V);
      float* ws = chunks > 1 ? f32_buf((size_t)chunks * V) : nullptr;
      float* out = G(bh);
      int* tk = tickets(V);
      if (!db_in_wgrad) {
        bw.push_back({[=](cudaStream_t s) { return colsum(logits, true, V, rows, V, rowscale, ws, chunks, tk, out, s); }, 1});
        note(bw, "colsum", 2.0 * rows * V, 2.0 * rows * V);
      }
    }
    for (size_t i = before; i < bw.size(); i++) bw[i].leaf = true;
    // ... and the gradient chain: dz = r (.) (P W_h) from fp32 partials of the GEMM
    GemmArgs q;
    q.M = rows; q.N = d; q.K = V;
    q.A = logits; q.sa_m = V; q.sa_k = 1;
    q.B = Wop(wh); q.sb_n = 1; q.sb_k = d;
    q.c_f32 = 1;
    q.epi.ld_aux = d;
    int splits = 1;
    if (rows >= 256 && d >= 256 && V >= 2048)     // few output tiles (or a badly filled last wave), long contraction: split it over the CTA pairs
      splits = pair_wave_splits((long long)((rows + 255) / 256) * ((d + 255) / 256), V);
    float* part = f32_buf((size_t)splits * rows * d);
    q.splits = splits;
    if (splits > 1) { q.ws = part; q.C = part; q.ldc = d; }
    else { q.C = part; q.ldc = d; }
    TcPlan qplan;
    int* qsched = (int*)dev_alloc(m, 2 * sizeof(int), &ok);
    const bool q_tc = !m->dry && tc_gemm_supported(q) && tc_gemm_plan(q, m->status, &qplan);
    qplan.sched = qsched;
    bw.push_back({[=](cudaStream_t s) {
                    cudaError_t e = q_tc ? tc_gemm_launch(q, qplan, s, mm->sm_budget) : gemm_simt(q, true, s);
                    if (e != cudaSuccess) return e;
                    return ce_dz_finish(part, splits, rows, d, rowscale, dz, s);
                  }, 2});
    note(bw, "gemm_dgrad", 2.0 * rows * V * d, ((double)rows * V + (double)V * d) * 2 + 2.0 * rows * d);
    return true;
  }

  // ---- Linear stack (MLP / TOWER / tower of the DOT block) ---------------------------------
  // returns the output buffer; fills last-activation info for the head backward
  struct Stack {
    std::vector<const void*> in;   // input of layer i
    std::vector<const void*> src;  // activation-derivative source of layer i (pre-act for GELU, output for ReLU)
    std::vector<int> act;          // activation after layer i
    void* out = nullptr;
  };
  Stack stack_fwd(OpList& f, const erase_block_spec& k, const void* zin, long long ldin, bool act_last, int first_tensor) {
    Stack st;
    int L = k.n_dims - 1;
    const void* h = zin;
    long long ldh = ldin;
    for (int i = 0; i < L; i++) {
      int K = k.dims[i], N = k.dims[i + 1];
      bool use = act_last || i < L - 1;
      int a = use ? k.act : ACT_NONE;
      void* y = act_buf((size_t)m->rows * N);
      Epilogue e;
      const void* src = y;
      if (a == ACT_GELU) {
        void* u = act_buf((size_t)m->rows * N);
        lin_fwd(f, h, ldh, first_tensor + 2 * i, first_tensor + 2 * i + 1, u, m->rows, N, K, e);
        act_op(f, u, y, a, (long long)m->rows * N);
        src = u;
      } else {
        e.act = a;
        lin_fwd(f, h, ldh, first_tensor + 2 * i, first_tensor + 2 * i + 1, y, m->rows, N, K, e);
      }
      st.in.push_back(h);
      st.src.push_back(src);
      st.act.push_back(a);
      h = y;
      ldh = N;
      st.out = y;
    }
    return st;
  }
  // d = gradient w.r.t. the stack output already multiplied by the last activation's derivative.
  // Returns the gradient w.r.t. the stack input when need_dx.
  void* stack_bwd(OpList& bw, const erase_block_spec& k, const Stack& st, long long ldin, void* d, int first_tensor, bool need_dx,
                  bool last_bias_done) {
    int L = k.n_dims - 1;
    for (int i = L - 1; i >= 0; i--) {
      int K = k.dims[i], N = k.dims[i + 1];
      lin_wgrad(bw, d, st.in[i], i == 0 ? ldin : K, first_tensor + 2 * i, first_tensor + 2 * i + 1, m->rows, N, K,
                last_bias_done && i == L - 1);
      if (i > 0 || need_dx) {
        void* dx = act_buf((size_t)m->rows * K);
        Epilogue e;
        const int da = i > 0 ? st.act[i - 1] : ACT_NONE;
        if (da == ACT_RELU) {
          e.dact = da;
          e.dact_src = st.src[i - 1];
        }
        lin_dgrad(bw, d, first_tensor + 2 * i, dx, m->rows, N, K, e);
        if (da == ACT_GELU) dact_op(bw, dx, st.src[i - 1], da, (long long)m->rows * K);
        d = dx;
      }
    }
    return d;
  }

  // ---- blocks ----------------------------------------------------------------------------------
  // Each returns z_b (output buffer).  `first` is the tensor index of the block's first tensor.
  void* block_mlp(int b, const erase_block_spec& k, const void* zin, int first, OpList& f, OpList& bw) {
    bool tower = k.kind == ERASE_BLK_TOWER;
    int L = k.n_dims - 1;
    Stack st = stack_fwd(f, k, zin, k.dims[0], tower, first);
    int dout = k.dims[L];
    void* dz = act_buf((size_t)m->rows * dout);
    bool lb = head(b, k, st.out, dout, first + 2 * L, first + 2 * L + 1, f, bw, dz, st.act[L - 1], st.src[L - 1],
                   first + 2 * (L - 1) + 1);
    stack_bwd(bw, k, st, k.dims[0], dz, first, false, lb);
    return st.out;
  }

  void* block_transformer(int b, const erase_block_spec& k, const void* z, int first, OpList& f, OpList& bw) {
    const int d = k.dims[0], ff = k.dims[1], H = k.n_heads, dh = d / H;
    const int rows = m->rows, batch = m->spec.batch, T_ = m->spec.seq;
    const bool bf = m->bf16;
    erase_model* mm = m;
    enum { LN1G = 0, LN1B, WQKV, BQKV, WPROJ, BPROJ, LN2G, LN2B, W1, B1, W2, B2, WH, BH };
    auto t = [&](int i) { return first + i; };
    // forward
    void* a = act_buf((size_t)rows * d);
    float* mean1 = f32_buf(rows); float* rstd1 = f32_buf(rows);
    void* qkv = act_buf((size_t)rows * 3 * d);
    void* o = act_buf((size_t)rows * d);
    float* lse = f32_buf((size_t)batch * H * T_);
    void* h = act_buf((size_t)rows * d);
    void* mm2 = act_buf((size_t)rows * d);
    float* mean2 = f32_buf(rows); float* rstd2 = f32_buf(rows);
    void* u = act_buf((size_t)rows * ff);
    void* g = act_buf((size_t)rows * ff);
    void* zout = act_buf((size_t)rows * d);
    {
      const float* g1 = Wf(t(LN1G)); const float* b1 = Wf(t(LN1B));
      f.push_back({[=](cudaStream_t s) { return layernorm_fwd(z, g1, b1, a, mean1, rstd1, rows, d, bf, s); }, 1});
      note(f, "layernorm_fwd", 8.0 * rows * d, 2.0 * rows * d * m->esz);
      lin_fwd(f, a, d, t(WQKV), t(BQKV), qkv, rows, 3 * d, d, Epilogue());
      f.push_back({[=](cudaStream_t s) { return attention_fwd(qkv, o, lse, batch, T_, H, dh, bf, s, mm->status); }, 1});
      note(f, "attention_fwd", 4.0 * batch * H * ((double)T_ * (T_ + 1) / 2) * dh, 4.0 * rows * d * m->esz);
      Epilogue e1; e1.res = z;
      lin_fwd(f, o, d, t(WPROJ), t(BPROJ), h, rows, d, d, e1);
      const float* g2 = Wf(t(LN2G)); const float* b2 = Wf(t(LN2B));
      f.push_back({[=](cudaStream_t s) { return layernorm_fwd(h, g2, b2, mm2, mean2, rstd2, rows, d, bf, s); }, 1});
      note(f, "layernorm_fwd", 8.0 * rows * d, 2.0 * rows * d * m->esz);
      lin_fwd(f, mm2, d, t(W1), t(B1), u, rows, ff, d, Epilogue());
      act_op(f, u, g, ACT_GELU, (long long)rows * ff);
      Epilogue e3; e3.res = h;
      lin_fwd(f, g, ff, t(W2), t(B2), zout, rows, d, ff, e3);
    }
    // head + backward
    void* dz = act_buf((size_t)rows * d);
    head(b, k, zout, d, t(WH), t(BH), f, bw, dz, ACT_NONE, nullptr);
    void* du = act_buf((size_t)rows * ff);
    void* dm = act_buf((size_t)rows * d);
    void* dhb = act_buf((size_t)rows * d);
    void* dO = act_buf((size_t)rows * d);
    void* dqkv = act_buf((size_t)rows * 3 * d);
    float* delta = f32_buf((size_t)batch * H * T_);
    void* da = act_buf((size_t)rows * d);
    {
      lin_wgrad(bw, dz, g, ff, t(W2), t(B2), rows, d, ff);
      lin_dgrad(bw, dz, t(W2), du, rows, d, ff, Epilogue());
      dact_op(bw, du, u, ACT_GELU, (long long)rows * ff);
      lin_wgrad(bw, du, mm2, d, t(W1), t(B1), rows, ff, d);
      lin_dgrad(bw, du, t(W1), dm, rows, ff, d, Epilogue());
      ln_bwd(bw, dm, h, mean2, rstd2, t(LN2G), t(LN2B), dz, dhb, d);
      flush_group(bw);  // dW2 and dW1 in one launch; dWproj and dWqkv at the end of B_b
      mid_flush(bw);   // (off by default) b2, b1, LN2 half-way; the rest (bproj, bqkv, LN1) at the end of B_b
      lin_wgrad(bw, dhb, o, d, t(WPROJ), t(BPROJ), rows, d, d);
      lin_dgrad(bw, dhb, t(WPROJ), dO, rows, d, d, Epilogue());
      bw.push_back({[=](cudaStream_t s) { return attention_bwd(qkv, o, dO, lse, delta, dqkv, batch, T_, H, dh, bf, s, mm->status); }, 3});
      note(bw, "attention_bwd", 8.0 * batch * H * ((double)T_ * (T_ + 1) / 2) * dh, 8.0 * rows * d * m->esz);
      lin_wgrad(bw, dqkv, a, d, t(WQKV), t(BQKV), rows, 3 * d, d);
      lin_dgrad(bw, dqkv, t(WQKV), da, rows, 3 * d, d, Epilogue());
      // LN1: only its gain/shift gradients; dx would flow into the detached z_{b-1}
      ln_bwd(bw, da, z, mean1, rstd1, t(LN1G), t(LN1B), nullptr, nullptr, d);
    }
    return zout;
  }
  // dx = LNbwd(dy) + add (skipped when dx == nullptr); gain/shift gradients always
  void ln_bwd(OpList& bw, const void* dy, const void* x, const float* mean, const float* rstd, int gidx, int bidx,
              const void* add, void* dx, int d) {
    int rows = m->rows;
    bool bf = m->bf16;
    const float* gain = Wf(gidx);
    if (dx) bw.push_back({[=](cudaStream_t s) { return layernorm_bwd_dx(dy, x, gain, mean, rstd, add, dx, rows, d, bf, s); }, 1});
    if (dx) note(bw, "layernorm_bwd", 12.0 * rows * d, 4.0 * rows * d * m->esz);
    ReduceJob j;
    j.kind = 1; j.x_f32 = bf ? 0 : 1;
    j.rows = rows; j.cols = d; j.ldx = d;
    j.X = dy; j.X2 = x; j.a = mean; j.b = rstd;
    j.out0 = G(gidx); j.out1 = G(bidx); j.tickets = tickets(d);
    add_job(bw, j, 4.0 * rows * d, 2.0 * rows * d * m->esz);
  }

  void* block_cross(int b, const erase_block_spec& k, const void* x0, int first, OpList& f, OpList& bw) {
    const int w = k.dims[0], L = k.n_cross, rows = m->rows;
    const bool bf = m->bf16;
    std::vector<const void*> xs;
    const void* xl = x0;
    for (int l = 0; l < L; l++) {
      void* y = act_buf((size_t)rows * w);
      Epilogue e; e.mul = x0; e.res = xl;
      lin_fwd(f, xl, w, first + 2 * l, first + 2 * l + 1, y, rows, w, w, e);
      xs.push_back(xl);
      xl = y;
    }
    void* dz = act_buf((size_t)rows * w);
    head(b, k, xl, w, first + 2 * L, first + 2 * L + 1, f, bw, dz, ACT_NONE, nullptr);
    void* d = dz;
    for (int l = L - 1; l >= 0; l--) {
      void* tt = act_buf((size_t)rows * w);
      long long n = (long long)rows * w;
      const void* dc = d;
      bw.push_back({[=](cudaStream_t s) { return ew_mul(dc, x0, tt, n, bf, s); }, 1});
      note(bw, "ew_mul", (double)n, 3.0 * n * m->esz);
      lin_wgrad(bw, tt, xs[l], w, first + 2 * l, first + 2 * l + 1, rows, w, w);
      if (l > 0) {
        void* dn = act_buf((size_t)rows * w);
        Epilogue e; e.res = d;
        lin_dgrad(bw, tt, first + 2 * l, dn, rows, w, w, e);
        d = dn;
      }
    }
    return const_cast<void*>(xl);
  }

  void* block_dot(int b, const erase_block_spec& k, const void* x0, int first, OpList& f, OpList& bw) {
    const erase_model_spec& s = m->spec;
    const int rows = m->rows, e_ = s.emb_dim, ns = s.n_sparse, w0 = s.width;
    const int dp = w0 - ns * e_;  // padded dense columns
    const int fw = k.dims[0];
    const bool bf = m->bf16;
    const char* dense_cols = (const char*)x0 + (size_t)ns * e_ * m->esz;
    void* proj = act_buf((size_t)rows * e_);
    lin_fwd(f, dense_cols, w0, first, first + 1, proj, rows, e_, dp, Epilogue());
    void* feats = act_buf((size_t)rows * fw);
    f.push_back({[=](cudaStream_t st) { return dot_fwd(proj, x0, w0, feats, rows, ns, e_, fw, bf, st); }, 1});
    note(f, "dot_fwd", (double)rows * (ns + 1) * ns * e_, (double)rows * (w0 + fw) * m->esz);
    int L = k.n_dims - 1;
    Stack st = stack_fwd(f, k, feats, fw, true, first + 2);
    int dout = k.dims[L];
    void* dz = act_buf((size_t)rows * dout);
    bool lb = head(b, k, st.out, dout, first + 2 + 2 * L, first + 2 + 2 * L + 1, f, bw, dz, st.act[L - 1], st.src[L - 1],
                   first + 2 + 2 * (L - 1) + 1);
    void* dfeat = stack_bwd(bw, k, st, fw, dz, first + 2, true, lb);
    void* dproj = act_buf((size_t)rows * e_);
    bw.push_back({[=](cudaStream_t s2) { return dot_bwd(dfeat, x0, w0, dproj, rows, ns, e_, fw, bf, s2); }, 1});
    note(bw, "dot_bwd", 2.0 * rows * ns * e_, (double)rows * (w0 + fw) * m->esz);
    lin_wgrad(bw, dproj, dense_cols, w0, first, first + 1, rows, e_, dp);
    return st.out;
  }

  // ---- the undetached remainder (Eq. 2): main network over u = [z_0 | sg z_1 | .. | sg z_B] --------------
  std::vector<const void*> outs;      // z_1 .. z_B as the blocks are built
  std::vector<int> out_w;
  void* block_main(int b, const erase_block_spec& k, const void* z0, int first, OpList& f, OpList& bw) {
    erase_model* mm = m;
    const erase_model_spec& s = m->spec;
    const int rows = m->rows, win = k.dims[0];
    const bool bf = m->bf16, reads = (k.flags & ERASE_MAIN_READS_INPUT) != 0;
    void* u = act_buf((size_t)rows * win);
    ConcatArgs ca;
    int off = 0;
    auto src = [&](const void* p, int w) {
      ca.src[ca.n] = p; ca.width[ca.n] = w; ca.offset[ca.n] = off; ca.ld[ca.n] = w;
      ca.n++; off += w;
    };
    if (reads) src(z0, s.width);
    for (size_t i = 0; i < outs.size(); i++) src(outs[i], out_w[i]);
    ca.total = win;
    f.push_back({[=](cudaStream_t st) { return concat_cols(ca, u, rows, bf, st); }, 1});
    note(f, "concat", 0, 2.0 * rows * win * m->esz);
    const int L = k.n_dims - 1;
    Stack st = stack_fwd(f, k, u, win, true, first);
    const int dout = k.dims[L];
    void* dz = act_buf((size_t)rows * dout);
    bool lb = head(b, k, st.out, dout, first + 2 * L, first + 2 * L + 1, f, bw, dz, st.act[L - 1], st.src[L - 1], first + 2 * (L - 1) + 1);
    const bool need_du = reads && s.train_input;
    void* du = stack_bwd(bw, k, st, win, dz, first, need_du, lb);
    if (need_du) {
      // only the z_0 columns of du carry on: the sg z_b columns pass nothing back (Eq. 1)
      const int ns = s.n_sparse, e_ = s.emb_dim, trows = s.table_rows, batch = s.batch;
      m->emb_sorted = (int*)dev_alloc(m, (size_t)ns * batch * sizeof(int), &ok);
      m->emb_seg = (int*)dev_alloc(m, (size_t)ns * (batch + 1) * sizeof(int), &ok);
      m->emb_uniq = (int*)dev_alloc(m, (size_t)ns * batch * sizeof(int), &ok);
      m->emb_nuniq = (int*)dev_alloc(m, (size_t)ns * sizeof(int), &ok);
      m->emb_grow = f32_buf((size_t)ns * batch * e_);
      int* so = m->emb_sorted; int* sg_ = m->emb_seg; int* un = m->emb_uniq; int* nu = m->emb_nuniq;
      float* gr = m->emb_grow;
      bw.push_back({[=](cudaStream_t s2) { return embed_backward(du, win, mm->cur.ids, batch, ns, e_, trows, so, sg_, un, nu, gr, bf, s2); }, 2});
      note(bw, "embed_backward", (double)batch * ns * e_, (double)batch * ns * e_ * (m->esz + 4));
    }
    return st.out;
  }

  bool build() {
    erase_model* mm = m;
    const erase_model_spec& s = m->spec;
    const bool bf = m->bf16;
    // arenas
    m->frozen = m->frozen_n ? f32_buf(m->frozen_n) : nullptr;
    m->theta = f32_buf(m->train_n);
    m->grad = f32_buf(m->train_n);
    if (s.opt != ERASE_OPT_SGD) { m->mom1 = f32_buf(m->train_n); m->mom2 = f32_buf(m->train_n); }
    if (bf) m->shadow = dev_alloc(m, m->train_n * 2, &ok);
    m->train_input = s.train_input != 0;
    if (m->train_input && s.opt != ERASE_OPT_SGD) { m->mom1_in = f32_buf(m->frozen_n); m->mom2_in = f32_buf(m->frozen_n); }
    m->table_stride = s.input == ERASE_IN_CTR && s.n_sparse > 1 ? (long long)(m->tensors[1].off - m->tensors[0].off) : 0;
    m->tick = (double*)dev_alloc(m, 3 * sizeof(double), &ok);
    m->status = (int*)dev_alloc(m, sizeof(int), &ok);
    m->losses = f32_buf(m->B);
    m->stamps = (unsigned long long*)dev_alloc(m, (size_t)(2 * (2 * m->B + 1) + 1) * sizeof(unsigned long long), &ok);
    m->pdone = (int*)dev_alloc(m, (size_t)(m->B + 1) * tc_dual_max() * sizeof(int), &ok);
    // z_0
    // z_0: dense batches are copied into a model-owned buffer (so every block reads memory whose
    // address is fixed at build time); token and CTR batches are gathered from the frozen tables.
    const void* z0 = nullptr;
    {
      void* buf = act_buf((size_t)m->rows * s.width);
      z0 = buf;
      if (s.input == ERASE_IN_DENSE) {
        size_t bytes = (size_t)m->rows * s.width * m->esz;
        m->stage.push_back({[=](cudaStream_t st) { return cudaMemcpyAsync(buf, mm->cur.x, bytes, cudaMemcpyDeviceToDevice, st); }, 0});
        note(m->stage, "copy_input", 0, 2.0 * bytes);
      } else if (s.input == ERASE_IN_TOKENS) {
        const float* tok = m->frozen + m->tensors[0].off;
        const float* pos = m->frozen + m->tensors[1].off;
        int batch = s.batch, T_ = s.seq, d = s.width;
        const int vocab = s.vocab;
        m->stage.push_back({[=](cudaStream_t st) { return gather_tokens(tok, pos, mm->cur.ids, buf, batch, T_, d, vocab, mm->status, bf, st); }, 1});
        note(m->stage, "gather_tokens", (double)m->rows * d, (double)m->rows * d * (4 + m->esz));
      } else {
        const float* tables = m->frozen;
        long long stride = s.n_sparse > 1 ? (long long)(m->tensors[1].off - m->tensors[0].off) : 0;
        int batch = s.batch, ns = s.n_sparse, e_ = s.emb_dim, nd = s.n_dense, w0 = s.width, trows = s.table_rows;
        m->stage.push_back({[=](cudaStream_t st) {
                              return gather_ctr(tables, stride, mm->cur.ids, (const float*)mm->cur.x, buf, batch, ns, e_, nd, w0, trows, mm->status, bf, st);
                            }, 1});
        note(m->stage, "gather_ctr", 0, (double)m->rows * w0 * (4 + m->esz));
      }
    }
    int first = 0;
    while (first < (int)m->tensors.size() && m->tensors[first].block < 0) first++;
    m->fwd.resize(m->B);
    m->hfwd.resize(m->B);
    m->bwd.resize(m->B);
    const void* z = z0;
    for (int b = 0; b < m->B; b++) {
      const erase_block_spec& k = m->blocks[b];
      const void* zin = s.topo == ERASE_TOPO_PARALLEL ? z0 : z;
      void* zout = nullptr;
      switch (k.kind) {
        case ERASE_BLK_MLP:
        case ERASE_BLK_TOWER: zout = block_mlp(b, k, zin, first, m->fwd[b], m->bwd[b]); break;
        case ERASE_BLK_TRANSFORMER: zout = block_transformer(b, k, zin, first, m->fwd[b], m->bwd[b]); break;
        case ERASE_BLK_CROSS: zout = block_cross(b, k, zin, first, m->fwd[b], m->bwd[b]); break;
        case ERASE_BLK_DOT: zout = block_dot(b, k, zin, first, m->fwd[b], m->bwd[b]); break;
        case ERASE_BLK_MAIN: zout = block_main(b, k, z0, first, m->fwd[b], m->bwd[b]); break;
      }
      outs.push_back(zout);
      out_w.push_back((k.kind == ERASE_BLK_CROSS || k.kind == ERASE_BLK_TRANSFORMER) ? k.dims[0] : k.dims[k.n_dims - 1]);
      flush_group(m->bwd[b]);
      flush_jobs(m->bwd[b]);
      z = zout;
      while (first < (int)m->tensors.size() && m->tensors[first].block == b) first++;
    }
    // optimizer: one sweep over the flat parameter arena
    {
      float* th = m->theta; float* gr = m->grad; float* m1 = m->mom1; float* m2 = m->mom2;
      void* sh = m->shadow; double* tick = m->tick;
      long long n = (long long)m->train_n;
      int kind = s.opt;
      float lr = s.lr, b1 = s.beta1, b2 = s.beta2, eps = s.eps, wd = s.weight_decay;
      m->opt.push_back({[=](cudaStream_t st) { return opt_tick(tick, b1, b2, st); }, 1});
      note(m->opt, "opt_tick");
      m->opt.push_back({[=](cudaStream_t st) { return opt_update(th, gr, m1, m2, sh, n, kind, lr, b1, b2, eps, wd, tick, st); }, 1});
      note(m->opt, "opt_update", 10.0 * n, (double)n * (kind == ERASE_OPT_SGD ? 12 : 28) + (sh ? 2.0 * n : 0));
      if (m->train_input) {      // the input tables: only the rows this batch read (follows the embedding backward of the main block)
        float* tb = m->frozen; float* mi = m->mom1_in; float* vi = m->mom2_in;
        const long long tstride = m->table_stride;
        const int batch = s.batch, ns = s.n_sparse, e_ = s.emb_dim;
        int* un = m->emb_uniq; int* nu = m->emb_nuniq; float* gr = m->emb_grow;
        Op top{[=](cudaStream_t st) { return embed_update(tb, tstride, mi, vi, batch, ns, e_, un, nu, gr, kind, lr, b1, b2, eps, wd, tick, st); }, 1};
        top.name = "embed_update";
        top.bytes = (double)batch * ns * e_ * (kind == ERASE_OPT_SGD ? 12 : 28);
        m->opt.push_back(top);
        m->opt_tables.push_back(top);
      }
      // per-block variant: the same update on block b's contiguous slice, runnable as soon as B_b is done
      m->opt_tick_op.push_back({[=](cudaStream_t st) { return opt_tick(tick, b1, b2, st); }, 1});
      note(m->opt_tick_op, "opt_tick");
      m->opt_blk.resize(m->B);
      m->blk_seg.assign(m->B, std::make_pair((size_t)0, (size_t)0));
      for (int b = 0; b < m->B; b++) {
        size_t lo = (size_t)-1, hi = 0;
        for (const Tensor& t : m->tensors)
          if (t.trainable && t.block == b) {
            if (t.off < lo) lo = t.off;
            size_t end = t.off + round_up(t.n, 64);
            if (end > hi) hi = end;
          }
        if (hi <= lo) continue;
        long long nb = (long long)(hi - lo);
        m->blk_seg[b] = std::make_pair(lo, hi - lo);
        float* thb = th + lo; float* grb = gr + lo;
        float* m1b = m1 ? m1 + lo : nullptr; float* m2b = m2 ? m2 + lo : nullptr;
        void* shb = sh ? (void*)((__nv_bfloat16*)sh + lo) : nullptr;
        m->opt_blk[b].push_back({[=](cudaStream_t st) { return opt_update(thb, grb, m1b, m2b, shb, nb, kind, lr, b1, b2, eps, wd, tick, st); }, 1});
        note(m->opt_blk[b], "opt_update", 10.0 * nb, (double)nb * (kind == ERASE_OPT_SGD ? 12 : 28) + (sh ? 2.0 * nb : 0));
      }
    }
    return ok;
  }
};

erase_status init_model(erase_model* m, const erase_model_spec* spec, bool dry) {
  m->spec = *spec;
  m->blocks.assign(spec->blocks, spec->blocks + spec->n_blocks);
  m->spec.blocks = m->blocks.data();
  m->B = spec->n_blocks;
  m->bf16 = spec->dtype == ERASE_BF16;
  m->esz = m->bf16 ? 2 : 4;
  m->rows = spec->batch * (spec->input == ERASE_IN_TOKENS ? spec->seq : 1);
  m->replicas = spec->replicas > 1 ? spec->replicas : 1;
  m->dry = dry;
  if (!dry && spec->arena) {
    m->arena = (char*)spec->arena;
    m->arena_bytes = spec->arena_bytes;
  }
  build_tensor_table(m);
  Builder bld;
  bld.m = m;
  if (!bld.build()) return m->fail(ERASE_ENOMEM, m->arena ? "arena too small" : "device allocation failed");
  return ERASE_OK;
}

int tensor_check(erase_model* m, int32_t idx, size_t n) {
  return m && idx >= 0 && idx < (int)m->tensors.size() && m->tensors[idx].n == n;
}

cudaError_t run_ops(erase_model* m, OpList& ops, cudaStream_t s) {
  for (Op& op : ops) {
    cudaError_t e = op.fn(s);
    if (e != cudaSuccess) return e;
    m->launches += op.launches;
  }
  return cudaSuccess;
}

// Data-parallel exchange of block b (b = -1: the B local losses): an in-place sum over the replicas,
// enqueued on the stream that just produced the values.  Every replica enqueues its exchanges in the
// same order because the order is a function of (n_streams, flags) alone and the host enqueues in program order.
erase_status exchange(erase_model* m, int b, cudaStream_t st) {
  if (!m->exchange_on) return ERASE_OK;
  float* buf = b < 0 ? m->losses : m->grad + m->blk_seg[b].first;
  const size_t n = b < 0 ? (size_t)m->B : m->blk_seg[b].second;
  m->exch_order.push_back(b);
  if (n == 0) return ERASE_OK;
  std::string why;
  const NcclApi* api = nccl_api(&why);
  if (!api) return m->fail(ERASE_ECOMM, why);
  const int r = api->all_reduce(buf, buf, n, NCCL_FLOAT32, NCCL_SUM, m->comm, st);
  if (r != 0) return m->fail(ERASE_ECOMM, std::string("ncclAllReduce: ") + api->error_string(r));
  return ERASE_OK;
}
#define CKX(call)                          \
  do {                                     \
    erase_status x_ = (call);              \
    if (x_ != ERASE_OK) return x_;         \
  } while (0)

// Persistent schedule: which operations of F_s and B_{s-1} go into stage s's dual-list kernel.
// Qualifies: bf16 chains whose block bodies consist of tensor-core GEMMs and GELU passes (MLP and
// tower blocks); anything else leaves persistent_ok false with the reason in persistent_why.
void plan_persistent(erase_model* m) {
  m->persistent_ok = false;
  if (!m->bf16) { m->persistent_why = "the persistent schedule needs a bf16 model"; return; }
  if (m->spec.topo != ERASE_TOPO_CHAIN) { m->persistent_why = "the persistent schedule needs a chain of blocks"; return; }
  const int B = m->B;
  m->pstage.assign(B + 1, erase_model::PStage());
  auto capable = [](const Op& op) { return !op.pg.empty() || op.pew != 0; };
  for (int s = 0; s <= B; s++) {
    erase_model::PStage& st = m->pstage[s];
    std::vector<DualItem> items;
    auto add = [&](Op& op, int list) {
      if (op.pew) {
        DualItem it;
        it.kind = op.pew; it.ew_src = op.ew_src; it.ew_dst = op.ew_dst; it.ew_n = op.ew_n; it.list = list; it.leaf = op.leaf ? 1 : 0;
        items.push_back(it);
      } else {
        for (const GemmArgs& g : op.pg) {
          DualItem it;
          it.kind = 0; it.g = g; it.list = list; it.leaf = op.leaf ? 1 : 0;
          items.push_back(it);
        }
      }
      st.covered.push_back(&op);
    };
    if (s < B)
      for (Op& op : m->fwd[s]) {
        if (!capable(op)) { m->persistent_why = std::string("block forward holds an operation the dual-list kernel does not cover: ") + op.name; return; }
        add(op, 0);
      }
    if (s >= 1) {
      bool started = false;
      for (Op& op : m->bwd[s - 1]) {
        if (capable(op)) { started = true; add(op, 1); }
        else if (!started) st.pre.push_back(&op);
        else if (op.leaf) st.after.push_back(&op);
        else { m->persistent_why = std::string("block backward holds an operation the dual-list kernel does not cover: ") + op.name; return; }
      }
    }
    if (items.empty()) continue;
    if ((int)items.size() > tc_dual_max()) { m->persistent_why = "a stage has more problems than the dual-list kernel takes"; return; }
    st.plan = tc_dual_plan(items.data(), (int)items.size(), m->pdone + (size_t)s * tc_dual_max(), m->status);
    if (!st.plan) { m->persistent_why = "a GEMM of the model does not fit the dual-list kernel (shape, alignment or epilogue)"; return; }
  }
  m->persistent_ok = true;
}

// One step in the persistent schedule, all on the main stream: stage s = [front of B_{s-1}] ->
// dual-list kernel {F_s || B_{s-1}} -> split-K reductions and parameter-gradient leaves -> local head of block s.
erase_status enqueue_persistent(erase_model* m, unsigned flags) {
  const int B = m->B;
  cudaStream_t st = m->main;
  CK(run_ops(m, m->stage, st));
  for (int s = 0; s <= B; s++) {
    erase_model::PStage& ps = m->pstage[s];
    for (Op* op : ps.pre) { CK(op->fn(st)); m->launches += op->launches; }
    if (ps.plan) { CK(tc_dual_launch(ps.plan, st)); m->launches += 1; }
    for (Op* op : ps.covered)
      if (op->post) { CK(op->post(st)); m->launches += op->post_launches; }
    for (Op* op : ps.after) { CK(op->fn(st)); m->launches += op->launches; }
    if (s >= 1) CKX(exchange(m, s - 1, st));                 // B_{s-1} is complete
    if (s < B) CK(run_ops(m, m->hfwd[s], st));
  }
  CKX(exchange(m, -1, st));
  if (!(flags & ERASE_NO_OPT)) CK(run_ops(m, m->opt, st));
  return ERASE_OK;
}

// timed: 0 no timeline, 1 CUDA events (never while capturing), 2 device clock stamps written by
// one-thread kernels (these can be captured, so the timeline of a graph replay can be read).
erase_status enqueue_step(erase_model* m, int n_streams, unsigned flags, int timed) {
  const int B = m->B;
  const bool do_opt = !(flags & ERASE_NO_OPT);
  auto mark = [&](int i, cudaStream_t st) -> cudaError_t {
    if (timed == 1) return cudaEventRecord(m->ev_time[i], st);
    if (timed == 2) { m->launches += 1; return stamp_time(m->stamps + i, st); }
    return cudaSuccess;
  };
  CK(mark(2 * (2 * B + 1), m->main));
  CK(run_ops(m, m->stage, m->main));
  const bool early_head = (flags & ERASE_EARLY_HEAD) != 0;
  // per-block optimizer: theta_b is read by F_b and B_b only, so it can be updated right behind B_b
  const bool block_opt = do_opt && n_streams > 1 && (flags & ERASE_BLOCK_OPT) != 0;
  const bool split_bwd = n_streams > 1 && (flags & ERASE_SPLIT_BWD) != 0;
  if (block_opt) CK(run_ops(m, m->opt_tick_op, m->main));
  if (n_streams <= 1) {
    for (int b = 0; b < B; b++) {
      CK(mark(2 * b, m->main));
      CK(run_ops(m, m->fwd[b], m->main));
      CK(run_ops(m, m->hfwd[b], m->main));
      CK(mark(2 * b + 1, m->main));
    }
    for (int b = B - 1; b >= 0; b--) {
      CK(mark(2 * (B + b), m->main));
      CK(run_ops(m, m->bwd[b], m->main));
      CK(mark(2 * (B + b) + 1, m->main));
      CKX(exchange(m, b, m->main));
    }
  } else {
    const int ns = n_streams - 1;
    // SM budget: persistent GEMMs of the main stream and of the side streams each leave SMs free
    // for the other, so that B_b really runs beside F_{b+1} instead of queueing behind it.
    static const int env_main = getenv("ERASE_SM_MAIN") ? atoi(getenv("ERASE_SM_MAIN")) : 0;
    static const int env_side = getenv("ERASE_SM_SIDE") ? atoi(getenv("ERASE_SM_SIDE")) : 0;
    const int budget_main = env_main, budget_side = env_side;
    // Parallel topology (every block reads z_0): the forwards are independent of one another too, so
    // with ERASE_PAR_FWD block b's whole chain F_b, l_b, B_b (and its optimizer) runs on its side
    // stream, released by ONE event behind the input staging.
    // (a main network reads every block's output: its forward stays behind all the others on the main stream)
    const bool par_fwd = (flags & ERASE_PAR_FWD) != 0 && m->spec.topo == ERASE_TOPO_PARALLEL && m->blocks[B - 1].kind != ERASE_BLK_MAIN;
    if (par_fwd) CK(cudaEventRecord(m->ev_opt, m->main));
    for (int b = 0; b < B; b++) {
      cudaStream_t sd = m->side[b % ns];
      cudaStream_t fs = par_fwd ? sd : m->main;          // the stream F_b runs on
      if (par_fwd) CK(cudaStreamWaitEvent(sd, m->ev_opt, 0));
      m->sm_budget = budget_main;
      CK(mark(2 * b, fs));
      CK(run_ops(m, m->fwd[b], fs));
      if (!early_head) CK(run_ops(m, m->hfwd[b], fs));
      CK(mark(2 * b + 1, fs));
      if (!par_fwd) {
        CK(cudaEventRecord(m->ev_f[b], m->main));          // F_b (and l_b) are enqueued: release B_b
        CK(cudaStreamWaitEvent(sd, m->ev_f[b], 0));
      }
      CK(mark(2 * (B + b), sd));
      m->sm_budget = budget_side;
      if (early_head) CK(run_ops(m, m->hfwd[b], sd));    // z_b's only other consumer is F_{b+1}, which does not wait
      if (!split_bwd) {
        CK(run_ops(m, m->bwd[b], sd));
      } else {
        // The gradient chain (dgrads, attention, LayerNorm dx, ...) stays on sd; every operation
        // that only produces a parameter gradient goes to a second stream behind the chain op
        // whose output it reads.  Every backward buffer is written once per step, so a leaf never
        // races with a later chain op; the two streams join before the block's optimizer.
        cudaStream_t lf = m->leaf[b % ns];
        size_t ne = 0;
        bool handed = false;   // has lf already been made to wait for everything enqueued on sd so far?
        for (Op& op : m->bwd[b]) {
          if (op.leaf) {
            if (!handed) {
              cudaEvent_t e = m->ev_leaf[b][ne++];
              CK(cudaEventRecord(e, sd));
              CK(cudaStreamWaitEvent(lf, e, 0));
              handed = true;
            }
            CK(op.fn(lf));
          } else {
            CK(op.fn(sd));
            handed = false;
          }
          m->launches += op.launches;
        }
        cudaEvent_t e = m->ev_leaf[b][ne++];
        CK(cudaEventRecord(e, lf));
        CK(cudaStreamWaitEvent(sd, e, 0));
      }
      CK(mark(2 * (B + b) + 1, sd));
      CKX(exchange(m, b, sd));     // overlaps the later blocks' forwards like B_b itself; the optimizer waits for it
      if (block_opt) CK(run_ops(m, m->opt_blk[b], sd));
      if (block_opt && b == B - 1) CK(run_ops(m, m->opt_tables, sd));
      CK(cudaEventRecord(m->ev_b[b], sd));
    }
    for (int b = 0; b < B; b++) CK(cudaStreamWaitEvent(m->main, m->ev_b[b], 0));  // join
    m->sm_budget = 0;
  }
  CKX(exchange(m, -1, m->main));
  CK(mark(4 * B, m->main));
  if (do_opt && !block_opt) CK(run_ops(m, m->opt, m->main));
  CK(mark(4 * B + 1, m->main));
  return ERASE_OK;
}

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================
extern "C" {

size_t erase_arena_bytes(const erase_model_spec* spec) {
  std::string why;
  if (!validate(spec, &why)) return 0;
  erase_model tmp;
  if (init_model(&tmp, spec, true) != ERASE_OK) return 0;
  return tmp.arena_used + 4096;
}

erase_status erase_create(const erase_model_spec* spec, erase_model** out) {
  if (!out) { g_create_error = "out is NULL"; return ERASE_EINVAL; }
  std::string why;
  if (!validate(spec, &why)) { g_create_error = "invalid spec: " + why; return ERASE_EINVAL; }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    g_create_error = "no CUDA device";
    return ERASE_ECUDA;
  }
  erase_model* m = new (std::nothrow) erase_model();
  if (!m) { g_create_error = "host allocation failed"; return ERASE_ENOMEM; }
  erase_status st = init_model(m, spec, false);
  auto bail = [&](erase_status s, const std::string& msg) {
    g_create_error = msg;
    erase_destroy(m);
    return s;
  };
  if (st != ERASE_OK) return bail(st, m->err);
  if (cudaStreamCreateWithFlags(&m->main, cudaStreamNonBlocking) != cudaSuccess) return bail(ERASE_ECUDA, "stream creation failed");
  m->side.resize(m->B);
  for (int i = 0; i < m->B; i++)
    if (cudaStreamCreateWithFlags(&m->side[i], cudaStreamNonBlocking) != cudaSuccess) { m->side.resize(i); return bail(ERASE_ECUDA, "stream creation failed"); }
  m->leaf.resize(m->B);
  for (int i = 0; i < m->B; i++)
    if (cudaStreamCreateWithFlags(&m->leaf[i], cudaStreamNonBlocking) != cudaSuccess) { m->leaf.resize(i); return bail(ERASE_ECUDA, "stream creation failed"); }
  auto mk = [&](cudaEvent_t* e, unsigned fl) { return cudaEventCreateWithFlags(e, fl) == cudaSuccess; };
  m->ev_leaf.resize(m->B);
  for (int b = 0; b < m->B; b++) {
    size_t n = 1;   // the join
    bool prev_leaf = false;
    for (const Op& op : m->bwd[b]) { if (op.leaf && !prev_leaf) n++; prev_leaf = op.leaf; }
    m->ev_leaf[b].assign(n, nullptr);
    for (auto& e : m->ev_leaf[b])
      if (!mk(&e, cudaEventDisableTiming)) return bail(ERASE_ECUDA, "event creation failed");
  }
  m->ev_f.assign(m->B, nullptr);
  m->ev_b.assign(m->B, nullptr);
  for (int i = 0; i < m->B; i++)
    if (!mk(&m->ev_f[i], cudaEventDisableTiming) || !mk(&m->ev_b[i], cudaEventDisableTiming)) return bail(ERASE_ECUDA, "event creation failed");
  if (!mk(&m->ev_opt, cudaEventDisableTiming)) return bail(ERASE_ECUDA, "event creation failed");
  m->ev_time.assign(2 * (2 * m->B + 1) + 1, nullptr);
  for (auto& e : m->ev_time)
    if (!mk(&e, cudaEventDefault)) return bail(ERASE_ECUDA, "event creation failed");
  plan_persistent(m);
  if (cudaDeviceSynchronize() != cudaSuccess) return bail(ERASE_ECUDA, "device error after model set-up");
  *out = m;
  return ERASE_OK;
}

void erase_destroy(erase_model* m) {
  if (!m) return;
  if (m->main) cudaStreamSynchronize(m->main);
  for (auto s : m->side) if (s) cudaStreamSynchronize(s);
  for (auto s : m->leaf) if (s) cudaStreamSynchronize(s);
  if (m->comm) {
    if (const NcclApi* api = nccl_api(nullptr)) api->comm_destroy(m->comm);
    m->comm = nullptr;
  }
  for (auto& kv : m->graphs) cudaGraphExecDestroy(kv.second.first);
  for (auto e : m->ev_f) if (e) cudaEventDestroy(e);
  for (auto e : m->ev_b) if (e) cudaEventDestroy(e);
  for (auto e : m->ev_time) if (e) cudaEventDestroy(e);
  for (auto e : m->ev_prof) if (e) cudaEventDestroy(e);
  if (m->ev_opt) cudaEventDestroy(m->ev_opt);
  for (auto& v : m->ev_leaf) for (auto e : v) if (e) cudaEventDestroy(e);
  for (auto s : m->side) if (s) cudaStreamDestroy(s);
  for (auto s : m->leaf) if (s) cudaStreamDestroy(s);
  if (m->main) cudaStreamDestroy(m->main);
  for (auto& ps : m->pstage) if (ps.plan) tc_dual_free(ps.plan);
  for (void* p : m->owned) cudaFree(p);
  cudaGetLastError();
  delete m;
}

int32_t erase_num_tensors(const erase_model* m) { return m ? (int32_t)m->tensors.size() : 0; }

erase_status erase_tensor_info(const erase_model* m, int32_t idx, int32_t* block, char name[32], int32_t* rank,
                               int64_t shape[4], int32_t* trainable) {
  if (!m || idx < 0 || idx >= (int)m->tensors.size()) return ERASE_EINVAL;
  const Tensor& t = m->tensors[idx];
  if (block) *block = t.block;
  if (name) { std::strncpy(name, t.name.c_str(), 31); name[31] = 0; }
  if (rank) *rank = t.rank;
  if (shape) { shape[0] = t.shape[0]; shape[1] = t.rank > 1 ? t.shape[1] : 0; shape[2] = shape[3] = 0; }
  if (trainable) *trainable = (t.trainable || t.table >= 0) ? 1 : 0;
  return ERASE_OK;
}

erase_status erase_sync(erase_model* m) {
  if (!m) return ERASE_EINVAL;
  CK(cudaStreamSynchronize(m->main));
  for (auto s : m->side) CK(cudaStreamSynchronize(s));
  if (m->status) {
    int st = 0;
    CK(copy_sync(m, &st, m->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (st != 0) {
      int zero = 0;
      CK(copy_sync(m, m->status, &zero, sizeof(int), cudaMemcpyHostToDevice));
      if (st == STATUS_BAD_ID)
        return m->fail(ERASE_EINVAL, "a token or sparse id of the batch lies outside its table; it was not used as an index, and the results of the step are void");
      return m->fail(ERASE_ETIMEOUT, "a bounded device-side wait expired (code " + std::to_string(st) + "); results of the step are void");
    }
  }
  return ERASE_OK;
}

erase_status erase_set_params(erase_model* m, int32_t idx, const float* src, size_t n) {
  if (!m) return ERASE_EINVAL;
  if (!src || !tensor_check(m, idx, n)) return m->fail(ERASE_EINVAL, "erase_set_params: bad index, size or pointer");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  Tensor& t = m->tensors[idx];
  float* dst = (t.trainable ? m->theta : m->frozen) + t.off;
  CK(copy_sync(m, dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
  if (t.trainable && m->shadow) {
    CK(to_bf16(dst, (__nv_bfloat16*)m->shadow + t.off, (long long)n, m->main));
    m->launches++;
    CK(cudaStreamSynchronize(m->main));
  }
  t.set = true;
  return ERASE_OK;
}

static erase_status copy_out(erase_model* m, int32_t idx, float* dst, size_t n, const float* base_train, const float* base_frozen, const char* who) {
  if (!m) return ERASE_EINVAL;
  if (!dst || !tensor_check(m, idx, n)) return m->fail(ERASE_EINVAL, std::string(who) + ": bad index, size or pointer");
  const Tensor& t = m->tensors[idx];
  const float* base = t.trainable ? base_train : base_frozen;
  if (!base) return m->fail(ERASE_EINVAL, std::string(who) + ": tensor has no such data");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  CK(copy_sync(m, dst, base + t.off, n * sizeof(float), cudaMemcpyDeviceToHost));
  return ERASE_OK;
}

erase_status erase_params(erase_model* m, int32_t idx, float* dst, size_t n) {
  return copy_out(m, idx, dst, n, m ? m->theta : nullptr, m ? m->frozen : nullptr, "erase_params");
}
erase_status erase_grads(erase_model* m, int32_t idx, float* dst, size_t n) {
  if (m && dst && tensor_check(m, idx, n) && m->tensors[idx].table >= 0) {
    // an input table trained by the main network: the step left its gradient as (distinct row, summed slice)
    // pairs; the dense gradient is assembled here on the host (rows nobody read are exactly zero)
    if (!m->stepped) return m->fail(ERASE_ESTATE, "erase_grads: no step has run");
    erase_status st = erase_sync(m);
    if (st != ERASE_OK) return st;
    const int t = m->tensors[idx].table, batch = m->spec.batch, e = m->spec.emb_dim;
    int nu = 0;
    CK(copy_sync(m, &nu, m->emb_nuniq + t, sizeof(int), cudaMemcpyDeviceToHost));
    if (nu < 0 || nu > batch) return m->fail(ERASE_ESTATE, "erase_grads: no table gradient has been computed");
    std::vector<int> rows((size_t)nu);
    std::vector<float> vals((size_t)nu * e);
    if (nu) {
      CK(copy_sync(m, rows.data(), m->emb_uniq + (size_t)t * batch, (size_t)nu * sizeof(int), cudaMemcpyDeviceToHost));
      CK(copy_sync(m, vals.data(), m->emb_grow + (size_t)t * batch * e, (size_t)nu * e * sizeof(float), cudaMemcpyDeviceToHost));
    }
    std::memset(dst, 0, n * sizeof(float));
    for (int i = 0; i < nu; i++) std::memcpy(dst + (size_t)rows[i] * e, vals.data() + (size_t)i * e, (size_t)e * sizeof(float));
    return ERASE_OK;
  }
  return copy_out(m, idx, dst, n, m ? m->grad : nullptr, nullptr, "erase_grads");
}

erase_status erase_opt_state(erase_model* m, int32_t idx, float* mom1, float* mom2, size_t n, int64_t* t) {
  if (!m) return ERASE_EINVAL;
  if (!tensor_check(m, idx, n) || !(m->tensors[idx].trainable || m->tensors[idx].table >= 0)) return m->fail(ERASE_EINVAL, "erase_opt_state: bad index or size");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  const Tensor& tt = m->tensors[idx];
  if (tt.table >= 0) {      // an input table: its moments live beside the frozen arena
    if (mom1) { if (m->mom1_in) CK(copy_sync(m, mom1, m->mom1_in + tt.off, n * 4, cudaMemcpyDeviceToHost)); else std::memset(mom1, 0, n * 4); }
    if (mom2) { if (m->mom2_in) CK(copy_sync(m, mom2, m->mom2_in + tt.off, n * 4, cudaMemcpyDeviceToHost)); else std::memset(mom2, 0, n * 4); }
    mom1 = mom2 = nullptr;
  }
  if (mom1) { if (m->mom1) CK(copy_sync(m, mom1, m->mom1 + tt.off, n * 4, cudaMemcpyDeviceToHost)); else std::memset(mom1, 0, n * 4); }
  if (mom2) { if (m->mom2) CK(copy_sync(m, mom2, m->mom2 + tt.off, n * 4, cudaMemcpyDeviceToHost)); else std::memset(mom2, 0, n * 4); }
  if (t) {
    double tk[3];
    CK(copy_sync(m, tk, m->tick, sizeof(tk), cudaMemcpyDeviceToHost));
    *t = (int64_t)tk[0];
  }
  return ERASE_OK;
}

erase_status erase_set_opt_state(erase_model* m, int32_t idx, const float* mom1, const float* mom2, size_t n, int64_t t) {
  if (!m) return ERASE_EINVAL;
  if (!tensor_check(m, idx, n) || !(m->tensors[idx].trainable || m->tensors[idx].table >= 0) || t < 0) return m->fail(ERASE_EINVAL, "erase_set_opt_state: bad index, size or t");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  const Tensor& tt = m->tensors[idx];
  if (tt.table >= 0) {
    if (mom1 && m->mom1_in) CK(copy_sync(m, m->mom1_in + tt.off, mom1, n * 4, cudaMemcpyHostToDevice));
    if (mom2 && m->mom2_in) CK(copy_sync(m, m->mom2_in + tt.off, mom2, n * 4, cudaMemcpyHostToDevice));
    mom1 = mom2 = nullptr;
  }
  if (mom1 && m->mom1) CK(copy_sync(m, m->mom1 + tt.off, mom1, n * 4, cudaMemcpyHostToDevice));
  if (mom2 && m->mom2) CK(copy_sync(m, m->mom2 + tt.off, mom2, n * 4, cudaMemcpyHostToDevice));
  double tk[3] = {(double)t, 1.0 - std::pow((double)m->spec.beta1, (double)t), 1.0 - std::pow((double)m->spec.beta2, (double)t)};
  CK(copy_sync(m, m->tick, tk, sizeof(tk), cudaMemcpyHostToDevice));
  return ERASE_OK;
}

static erase_status check_step_args(erase_model* m, const erase_batch* batch);

erase_status erase_step_ex(erase_model* m, const erase_batch* batch, int32_t n_streams, uint32_t flags) {
  if (!m) return ERASE_EINVAL;
  if (n_streams < 1) return m->fail(ERASE_EINVAL, "erase_step: n_streams must be >= 1");
  if (flags & ~(ERASE_GRAPH | ERASE_NO_OPT | ERASE_EARLY_HEAD | ERASE_BLOCK_OPT | ERASE_SPLIT_BWD | ERASE_STAMPS | ERASE_PAR_FWD | ERASE_PERSISTENT |
                ERASE_LOCAL_GRADS))
    return m->fail(ERASE_EINVAL, "erase_step: unknown flag");
  m->exchange_on = m->comm != nullptr && !(flags & ERASE_LOCAL_GRADS);
  if (m->replicas > 1 && !m->comm && !(flags & ERASE_LOCAL_GRADS))
    return m->fail(ERASE_ESTATE, "erase_step: the model was built for several replicas: attach a communicator (erase_comm_init) or pass ERASE_LOCAL_GRADS");
  if (m->exchange_on && (flags & ERASE_GRAPH))
    return m->fail(ERASE_EUNSUPPORTED, "erase_step: ERASE_GRAPH is not offered while a communicator is attached (pass ERASE_LOCAL_GRADS to step without the exchange)");
  flags &= ~ERASE_LOCAL_GRADS;   // not a property of the enqueued work: keeps graph keys and schedules as they were
  const bool persistent = (flags & ERASE_PERSISTENT) != 0;
  if (persistent) {
    if (!m->persistent_ok) return m->fail(ERASE_EUNSUPPORTED, "erase_step: ERASE_PERSISTENT: " + m->persistent_why);
    if (flags & ERASE_STAMPS) return m->fail(ERASE_EINVAL, "erase_step: ERASE_PERSISTENT records no timeline");
    flags &= ~(ERASE_EARLY_HEAD | ERASE_BLOCK_OPT | ERASE_SPLIT_BWD | ERASE_PAR_FWD);   // stream placements: meaningless on one stream
  }
  const int stamp_mode = (flags & ERASE_STAMPS) ? 2 : 0;
  erase_status cst = check_step_args(m, batch);
  if (cst != ERASE_OK) return cst;
  if (n_streams > m->B + 1) n_streams = m->B + 1;
  m->cur = *batch;
  m->exch_order.clear();
  if (flags & ERASE_GRAPH) {
    GraphKey key{batch->x, batch->ids, batch->y, n_streams, flags};
    auto it = m->graphs.find(key);
    if (it == m->graphs.end()) {
      int64_t before = m->launches;
      CK(cudaStreamBeginCapture(m->main, cudaStreamCaptureModeThreadLocal));
      erase_status st = persistent ? enqueue_persistent(m, flags) : enqueue_step(m, n_streams, flags, stamp_mode);
      cudaGraph_t graph = nullptr;
      cudaError_t e = cudaStreamEndCapture(m->main, &graph);
      const int64_t captured = m->launches - before;
      m->launches = before;
      if (st != ERASE_OK) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return st; }
      if (e != cudaSuccess) return m->fail(ERASE_ECUDA, std::string("graph capture: ") + cudaGetErrorString(e));
      cudaGraphExec_t exec = nullptr;
      e = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      if (e != cudaSuccess) return m->fail(ERASE_ECUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
      it = m->graphs.emplace(key, std::make_pair(exec, captured)).first;
    }
    CK(cudaGraphLaunch(it->second.first, m->main));
    m->launches += it->second.second;
    m->timeline_valid = stamp_mode != 0;
    m->timeline_stamps = true;
  } else {
    erase_status st = persistent ? enqueue_persistent(m, flags) : enqueue_step(m, n_streams, flags, stamp_mode ? 2 : 1);
    if (st != ERASE_OK) return st;
    m->timeline_valid = !persistent;
    m->timeline_stamps = stamp_mode != 0;
  }
  m->stepped = true;
  return ERASE_OK;
}

static erase_status check_step_args(erase_model* m, const erase_batch* batch) {
  if (!batch) return m->fail(ERASE_EINVAL, "erase_step: batch is NULL");
  const erase_model_spec& s = m->spec;
  bool need_x = s.input != ERASE_IN_TOKENS, need_ids = s.input != ERASE_IN_DENSE, need_y = s.input != ERASE_IN_TOKENS;
  if ((need_x && !batch->x) || (need_ids && !batch->ids) || (need_y && !batch->y))
    return m->fail(ERASE_EINVAL, "erase_step: a batch pointer this input kind needs is NULL");
  for (const Tensor& t : m->tensors)
    if (!t.set) return m->fail(ERASE_ESTATE, "erase_step: tensor '" + t.name + "' was never set");
  return ERASE_OK;
}

erase_status erase_profile_step(erase_model* m, const erase_batch* batch, erase_op_record* out, int32_t cap, int32_t* n) {
  if (!m) return ERASE_EINVAL;
  if (!out || !n || cap < 0) return m->fail(ERASE_EINVAL, "erase_profile_step: out or n is NULL");
  erase_status st = check_step_args(m, batch);
  if (st != ERASE_OK) return st;
  m->cur = *batch;
  struct Ref { Op* op; int block, phase; };
  std::vector<Ref> refs;
  for (auto& op : m->stage) refs.push_back({&op, -1, 0});
  for (int b = 0; b < m->B; b++) {
    for (auto& op : m->fwd[b]) refs.push_back({&op, b, 1});
    for (auto& op : m->hfwd[b]) refs.push_back({&op, b, 1});
  }
  for (int b = m->B - 1; b >= 0; b--) for (auto& op : m->bwd[b]) refs.push_back({&op, b, 2});
  for (auto& op : m->opt) refs.push_back({&op, -1, 3});
  while (m->ev_prof.size() < 2 * refs.size()) {
    cudaEvent_t e;
    CK(cudaEventCreate(&e));
    m->ev_prof.push_back(e);
  }
  for (size_t i = 0; i < refs.size(); i++) {
    CK(cudaEventRecord(m->ev_prof[2 * i], m->main));
    CK(refs[i].op->fn(m->main));
    m->launches += refs[i].op->launches;
    CK(cudaEventRecord(m->ev_prof[2 * i + 1], m->main));
  }
  CK(cudaStreamSynchronize(m->main));
  m->stepped = true;
  m->timeline_valid = false;
  *n = (int32_t)refs.size();
  for (size_t i = 0; i < refs.size() && (int32_t)i < cap; i++) {
    erase_op_record& r = out[i];
    std::memset(&r, 0, sizeof(r));
    std::strncpy(r.name, refs[i].op->name, 31);
    r.block = refs[i].block;
    r.phase = refs[i].phase;
    r.launches = refs[i].op->launches;
    r.flops = refs[i].op->flops;
    r.bytes = refs[i].op->bytes;
    CK(cudaEventElapsedTime(&r.ms, m->ev_prof[2 * i], m->ev_prof[2 * i + 1]));
  }
  return ERASE_OK;
}

erase_status erase_step(erase_model* m, const erase_batch* batch, int32_t n_streams) {
  return erase_step_ex(m, batch, n_streams, 0);
}

erase_status erase_losses(erase_model* m, float* dst, int32_t n_blocks) {
  if (!m) return ERASE_EINVAL;
  if (!dst || n_blocks != m->B) return m->fail(ERASE_EINVAL, "erase_losses: dst is NULL or n_blocks differs from the model's");
  if (!m->stepped) return m->fail(ERASE_ESTATE, "erase_losses: no step has run");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  CK(copy_sync(m, dst, m->losses, m->B * sizeof(float), cudaMemcpyDeviceToHost));
  return ERASE_OK;
}

erase_status erase_selftest_timeout(erase_model* m, int32_t limit_us) {
  if (!m) return ERASE_EINVAL;
  if (limit_us < 1 || limit_us > 100000) return m->fail(ERASE_EINVAL, "erase_selftest_timeout: limit_us must be in [1, 100000]");
  CK(tc_wait_selftest(m->status, (long long)limit_us * 2000LL, m->main));   // SM clock <= 2 GHz: at least limit_us
  m->launches++;
  return ERASE_OK;
}

void* erase_main_stream(erase_model* m) { return m ? (void*)m->main : nullptr; }

int64_t erase_launch_count(const erase_model* m) { return m ? m->launches : 0; }

erase_status erase_timeline(erase_model* m, float* out, int32_t n) {
  if (!m) return ERASE_EINVAL;
  const int need = 2 * (2 * m->B + 1);
  if (!out || n != need) return m->fail(ERASE_EINVAL, "erase_timeline: out is NULL or n != 2*(2*n_blocks+1)");
  if (!m->timeline_valid) return m->fail(ERASE_ESTATE, "erase_timeline: the last step recorded no timeline");
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  if (m->timeline_stamps) {
    std::vector<unsigned long long> h(need + 1);
    CK(copy_sync(m, h.data(), m->stamps, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    for (int i = 0; i < need; i++) out[i] = (float)((double)((long long)h[i] - (long long)h[need]) * 1e-6);   // ns -> ms
    return ERASE_OK;
  }
  for (int i = 0; i < need; i++) CK(cudaEventElapsedTime(&out[i], m->ev_time[need], m->ev_time[i]));
  return ERASE_OK;
}

erase_status erase_gemm(int32_t dtype, int32_t M, int32_t N, int32_t K, const void* A, int64_t sa_m, int64_t sa_k,
                        const void* B, int64_t sb_n, int64_t sb_k, void* C, int64_t ldc, int32_t c_f32, int32_t splits,
                        int32_t engine, void* stream) {
  if ((dtype != ERASE_F32 && dtype != ERASE_BF16) || M < 1 || N < 1 || K < 1 || !A || !B || !C || splits < 1 ||
      splits > 1024 || (engine != 0 && engine != 1) || ldc < N || (sa_m != 1 && sa_k != 1) || (sb_n != 1 && sb_k != 1)) {
    g_create_error = "erase_gemm: bad argument";
    return ERASE_EINVAL;
  }
  cudaStream_t st = (cudaStream_t)stream;
  GemmArgs g;
  g.M = M; g.N = N; g.K = K;
  g.A = A; g.sa_m = sa_m; g.sa_k = sa_k;
  g.B = B; g.sb_n = sb_n; g.sb_k = sb_k;
  g.C = C; g.ldc = ldc; g.c_f32 = (c_f32 || dtype == ERASE_F32) ? 1 : 0;
  g.splits = splits;
  g.epi.ld_aux = N;
  const bool bf = dtype == ERASE_BF16;
  if (engine == 1 && (!bf || !tc_gemm_supported(g))) {
    g_create_error = "erase_gemm: the tensor-core kernel does not take this shape/alignment/dtype";
    return ERASE_EUNSUPPORTED;
  }
  if (splits > 1 && !g.c_f32) {
    g_create_error = "erase_gemm: split-K needs a float result (c_f32)";
    return ERASE_EINVAL;
  }
  float* ws = nullptr;
  int* status = nullptr;
  auto cleanup = [&]() { if (ws) cudaFree(ws); if (status) cudaFree(status); cudaGetLastError(); };
  auto cuda_fail = [&](cudaError_t e, const char* what) {
    g_create_error = std::string("erase_gemm: ") + what + ": " + cudaGetErrorString(e);
    cleanup();
    return ERASE_ECUDA;
  };
  if (splits > 1 && cudaMalloc(&ws, (size_t)splits * M * N * sizeof(float)) != cudaSuccess) { cleanup(); g_create_error = "erase_gemm: workspace allocation failed"; return ERASE_ENOMEM; }
  if (cudaMalloc(&status, 4 * sizeof(int)) != cudaSuccess) { cleanup(); g_create_error = "erase_gemm: allocation failed"; return ERASE_ENOMEM; }
  cudaError_t e = cudaMemsetAsync(status, 0, 4 * sizeof(int), st);   // status word + two scheduler words
  if (e != cudaSuccess) return cuda_fail(e, "memset");
  g.ws = ws;
#ifdef ERASE_DEV_AIDS
  long long* dbg = nullptr;
#endif
  if (engine == 1) {
    TcPlan plan;
    if (!tc_gemm_plan(g, status, &plan)) { cleanup(); g_create_error = "erase_gemm: TMA descriptor encoding failed"; return ERASE_EUNSUPPORTED; }
    plan.sched = status + 1;
#ifdef ERASE_DEV_AIDS
    if (getenv("ERASE_TC_TIMELINE")) {   // development aid: print CTA 0's clock stamps for its first tile
      if (cudaMalloc(&dbg, 16 * sizeof(long long)) == cudaSuccess) {
        long long h[16] = {0};
        h[15] = atoll(getenv("ERASE_TC_TIMELINE"));   // bit 0: skip the stores, bit 1: skip the TMEM loads
        cudaMemcpyAsync(dbg, h, sizeof(h), cudaMemcpyHostToDevice, st);
        cudaStreamSynchronize(st);
      }
      plan.dbg = dbg;
    }
#endif
    e = tc_gemm_launch(g, plan, st);
  } else {
    e = gemm_simt(g, bf, st);
  }
  if (e != cudaSuccess) return cuda_fail(e, "launch");
  if (splits > 1) {
    e = splitk_reduce(ws, splits, (long long)M * N, N, (float*)C, ldc, st);
    if (e != cudaSuccess) return cuda_fail(e, "reduce launch");
  }
  int hst = 0;
  e = cudaMemcpyAsync(&hst, status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "execution");
#ifdef ERASE_DEV_AIDS
  if (dbg) {
    long long h[16];
    if (cudaMemcpy(h, dbg, sizeof(h), cudaMemcpyDeviceToHost) == cudaSuccess)
      fprintf(stderr, "tc timeline (cycles from CTA start): setup %lld | first TMA issued %lld | 4th TMA issued %lld | first stage landed %lld | 4th stage landed %lld | "
              "tile MMAs issued %lld | epilogue starts %lld | epilogue done %lld | CTA end %lld\n",
              h[1] - h[0], h[2] - h[0], h[8] - h[0], h[3] - h[0], h[9] - h[0], h[4] - h[0], h[5] - h[0], h[6] - h[0], h[7] - h[0]);
    fprintf(stderr, "   epilogue detail: staged %lld | store issued %lld | loop done %lld | fenced %lld | arrived %lld\n",
            h[10] - h[0], h[11] - h[0], h[12] - h[0], h[13] - h[0], h[6] - h[0]);
    if (getenv("ERASE_TC_PAIR")) fprintf(stderr, "   pair kernel: TMEM base of the leader %lld, of the peer %lld\n", h[8], h[9]);
    if (getenv("ERASE_TC_WAITS"))
      fprintf(stderr, "   pair kernel, CTA 0 (cycles): MMA thread first tile -> last operand wait %lld over %lld tiles | waiting for a drained accumulator %lld | "
              "for operands %lld || epilogue warp 0: waiting for an accumulator %lld | draining %lld || producer waiting for a free stage %lld\n",
              h[3] - h[0], h[10], h[1], h[2], h[4], h[5], h[7]);
    cudaFree(dbg);
  }
#endif
  cleanup();
  if (hst != 0) { g_create_error = "erase_gemm: a bounded device-side wait expired (code " + std::to_string(hst) + ")"; return ERASE_ETIMEOUT; }
  return ERASE_OK;
}

erase_status erase_comm_unique_id(void* id_out) {
  if (!id_out) { g_create_error = "erase_comm_unique_id: id_out is NULL"; return ERASE_EINVAL; }
  std::string why;
  const NcclApi* api = nccl_api(&why);
  if (!api) { g_create_error = "erase_comm_unique_id: " + why; return ERASE_ECOMM; }
  NcclId id;
  const int r = api->get_unique_id(&id);
  if (r != 0) { g_create_error = std::string("ncclGetUniqueId: ") + api->error_string(r); return ERASE_ECOMM; }
  std::memcpy(id_out, id.bytes, NCCL_ID_BYTES);
  return ERASE_OK;
}

erase_status erase_comm_init(erase_model* m, int32_t rank, int32_t world, const void* id) {
  if (!m) return ERASE_EINVAL;
  if (!id || world < 1 || rank < 0 || rank >= world) return m->fail(ERASE_EINVAL, "erase_comm_init: id is NULL or rank/world out of range");
  if (world != m->replicas) return m->fail(ERASE_EINVAL, "erase_comm_init: world differs from the spec's replicas");
  if (m->comm) return m->fail(ERASE_ESTATE, "erase_comm_init: a communicator is already attached");
  if (world > 1 && m->train_input)
    return m->fail(ERASE_EUNSUPPORTED, "erase_comm_init: the sparse table gradients of train_input are not exchanged between replicas");
  std::string why;
  const NcclApi* api = nccl_api(&why);
  if (!api) return m->fail(ERASE_ECOMM, "erase_comm_init: " + why);
  erase_status st = erase_sync(m);
  if (st != ERASE_OK) return st;
  NcclId nid;
  std::memcpy(nid.bytes, id, NCCL_ID_BYTES);
  NcclComm c = nullptr;
  const int r = api->comm_init_rank(&c, world, nid, rank);
  if (r != 0) return m->fail(ERASE_ECOMM, std::string("ncclCommInitRank: ") + api->error_string(r));
  m->comm = c;
  m->comm_rank = rank;
  m->comm_world = world;
  return ERASE_OK;
}

erase_status erase_comm_order(erase_model* m, int32_t* blocks_out, int32_t cap, int32_t* n_out) {
  if (!m) return ERASE_EINVAL;
  if (!n_out || cap < 0 || (cap > 0 && !blocks_out)) return m->fail(ERASE_EINVAL, "erase_comm_order: bad argument");
  *n_out = (int32_t)m->exch_order.size();
  for (int32_t i = 0; i < cap && i < *n_out; i++) blocks_out[i] = m->exch_order[i];
  return ERASE_OK;
}

const char* erase_last_error(const erase_model* m) { return m ? m->err.c_str() : g_create_error.c_str(); }

}  // extern "C"
