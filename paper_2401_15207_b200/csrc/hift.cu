// Engine and C entry points of the hierarchical fine-tuning step (see include/hift.h).
//
// One hift_step = one iteration of the paper's Algorithm 1:
//   select group (c-g)  ->  forward (h)  ->  state to GPU (i)  ->  backward truncated at the
//   group + update + clear gradients  ->  state to host (k)  ->  delayed learning rate.
// Activations below the group's lowest unit are not kept (two ping-pong buffers); above it only
// what activation gradients need is kept; inside it the GEMM inputs are kept too.
#include "hift.h"

#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <string>
#include <vector>

#include "gemm_tc.h"
#include "grad_chunks.h"
#include "kernels_adafactor.cuh"
#include "launchers.cuh"

using namespace hift;

namespace {

constexpr size_t kAlignElems = 128;   // every tensor starts on a multiple of 128 elements
constexpr size_t kGuardBytes = 256;   // checked mode: guard region behind every arena slice
constexpr unsigned char kGuardByte = 0xC5;
int g_checked_arena = 0;              // hift_test_switch 5: contexts created while set carry guard regions
int g_fail_pinned_in = -1;            // hift_test_switch 4: the n-th pinned allocation from now fails (-1: off)
constexpr int kScalWords = 8;         // the step's scalar words: loss, valid count, bad input, (time-out flag), gate

// Per-block activation slots.  Residual-stream tensors are fp32 in every configuration;
// GEMM operands have the parameter type (bf16 or fp32).
//   pre-norm blocks:  XIN x (stream) | H1 norm1(x) | QKV | O | LSE | X2 x + attn (stream) |
//                     H2 norm2(x2) | A pre-activation | U activation output
//   post-LN blocks:   XIN x (stream) + XINA operand copy | QKV | O | LSE | X2 y = x + attn (stream) |
//                     H2 x1 = LN1(y) operand copy + H2R stream copy | A | U | Z z = x1 + ffn (stream)
enum Slot { S_XIN = 0, S_XINA, S_H1, S_QKV, S_O, S_LSE, S_X2, S_ST1, S_H2, S_H2R, S_A, S_U, S_Z, S_ST2, S_NUM };

struct TensorRec {
  char name[64];
  int unit;
  int64_t rows, cols;
  size_t numel, off;
  int init_kind;   // 0 normal, 1 ones, 2 zeros
  size_t af_off;   // Adafactor: offset of this tensor's factored state inside its group's compact state
};
struct GroupRec {
  int unit_lo, unit_hi;
  size_t off, numel;      // span in the flat parameter buffer (padded)
  size_t own_lo, own_n;   // the part of the span whose master / state this rank holds (all of it unless sharded)
  int64_t tau;            // updates so far
  char* blob;             // pinned host: [master][state]; compact master: [state][low halves u16][carry bits]
  size_t blob_bytes;
  size_t state_floats;    // floats of optimizer state (n_state * numel, or the compact Adafactor state)
  size_t af_base;         // Adafactor, state resident: offset of the group's compact state in af_all
};
struct BlockIdx {          // tensor indices of one block, -1 if absent
  int n1_g, n1_b, w_qkv, b_qkv, w_o, b_o, n2_g, n2_b, w_fc1, b_fc1, w_fc2, b_fc2;
};
struct ProfRec { int cls; cudaEvent_t e0, e1; double work; };
// What one step trains: one state group (the fixed partition), or, with the literal queue of Algorithm 1
// when m does not divide n, the m units popped from the queue's head, whose membership drifts from cycle to
// cycle; then every unit is a state group of its own and a set is a list of them.
struct ActiveSet {
  int id = -1;                         // set id: group index, or position in the queue walk's period
  std::vector<int> groups;             // state groups trained, ascending units
  std::vector<size_t> grad_base;       // element offset of each group's span in the gradient buffer
  std::vector<size_t> slot_base;       // byte offset of each group's planes in a state slot
  size_t grad_numel = 0, slot_bytes = 0;
  int lo_unit = 0;
};
// One device staging slot of the paged optimizer state, laid out like a group's blob.
constexpr int kMaxSlots = 4;
struct SlotRec {
  char* mem = nullptr;
  int group = -1;            // group whose latest master / state the slot holds (-1: nothing valid)
  int64_t step = -1;         // step the slot is reserved for (< current step: free to evict)
  bool d2h_pending = false;  // a write-back from this slot has been enqueued (ev_d2h recorded)
  int64_t h2d_for_step = -1; // the step whose request started the upload that filled the slot
  cudaEvent_t ev_h2d, ev_opt, ev_d2h;   // ordering only
  cudaEvent_t tl_h2d0, tl_h2d1;         // timed: begin / end of the upload
};

}  // namespace

struct hift_ctx {
  hift_model_cfg m;
  hift_group_cfg gc;
  hift_opt_cfg oc;
  cudaStream_t st = nullptr, st_h2d = nullptr, st_d2h = nullptr;   // compute and copy streams (owned, non-blocking)
  cudaStream_t caller = nullptr;    // the stream given to hift_create: inputs are ordered after it
  cudaEvent_t ev_in;
  int es = 2;                       // bytes per parameter / GEMM-operand element
  int L = 0, d = 0, f = 0, fa = 0, H = 0, dh = 0, T = 0, B = 0, S = 0, V = 0, Vp = 0;
  int n_state = 2;
  bool mixed = true, offload = false;
  int shard_rank = 0, shard_world = 1;   // optimizer state sharded over data-parallel ranks (ZeRO stage 1)
  bool drop_on = false;             // dropout at the residual-branch outputs and the embedding output
  uint32_t drop_thr = 0; float drop_scale = 1.f;
  uint32_t adrop_thr = 0; float adrop_scale = 1.f;   // dropout on attention probabilities (site 1000 + block)
  bool recompute = false;           // frozen blocks above the group keep only their input; see plan_slots
  bool keep_all = false;            // set while such a block is recomputed: its forward must store what the backward reads
  bool compact = false;             // paged master = low halves + carry bits beside the bf16 copy (see blob layout)
  std::vector<TensorRec> tens;
  std::vector<std::vector<int>> unit_tens;
  std::vector<GroupRec> groups;
  std::vector<int> group_sizes;     // caller-chosen chunk lengths (empty = the uniform rule)
  std::vector<int> order;
  std::vector<BlockIdx> bidx;
  int t_tok = -1, t_pos = -1, t_eg = -1, t_eb = -1, t_fg = -1, t_fb = -1, t_wh = -1, t_wc = -1, t_bc = -1;
  size_t total = 0, max_group = 0;
  int64_t t = 0;
  int forced = -1, last_group = -1;     // last_group: id of the set trained by the step in flight / the last one
  bool queue = false;                   // literal queue (group membership drifts); see ActiveSet
  std::vector<int> queue_units;         // the queue's initial order of unit ids
  int n_sets = 0;                       // distinct sets in one period of the schedule
  int k_cycle = 1;                      // steps per learning-rate cycle: the paper's k
  ActiveSet act;
  std::vector<size_t> grad_off;         // per tensor: element offset in the gradient buffer, SIZE_MAX if not trained now
  std::vector<char> unit_on;            // per unit: trained by the step in flight
  std::vector<int> forced_seq;      // hift_force_sequence: groups of the coming steps, cyclic from step forced_seq_t0
  int64_t forced_seq_t0 = 0;
  int cur_sl = 0; double cur_lr = 0.0;   // slot and learning rate of the step in flight
  bool pending_update = false;           // between hift_step_begin and hift_step_end
  // chunks of the active group's gradient in completion order (data-parallel overlap)
  struct ChunkRec { size_t off, n; cudaEvent_t ev; };
  GradChunkPlanner planner;
  std::vector<int> planner_idx;          // tensor -> index in the planner (-1: not in the active group)
  std::vector<ChunkRec> chunks;
  std::vector<cudaEvent_t> chunk_events; // pool, grown on demand
  size_t chunk_min_elems = (size_t)8 << 20;   // 32 MB of fp32 gradient
  cudaEvent_t ev_bwd;                    // forward + backward (and the gate word) complete

  // device memory
  std::vector<void*> dev_allocs;
  size_t dev_bytes = 0, pinned_bytes = 0;
  char* params = nullptr;           // [total] of element type
  float* master_all = nullptr;      // non-offload mixed mode
  float* s0_all = nullptr; float* s1_all = nullptr;
  float* af_all = nullptr;          // Adafactor, state resident: compact state of every group
  float* af_scratch = nullptr;      // Adafactor work space, sized for the largest tensor
  bool af = false;
  SlotRec slot[kMaxSlots];          // offload staging ring
  int n_slots = 1;
  int lookahead = 0;                // steps ahead of the current one whose state is uploaded early
  int* gate = nullptr;              // device word: non-zero = the step failed, the optimizer must not write
  float* grad = nullptr;            // gradient buffer of the largest set: fp32 elements, or bf16 ones (gbf)
  bool gbf = false; int ges = 4;    // gradients kept in bf16; bytes per gradient element
  float* stage = nullptr;           // set-up only, with bf16 gradients: fp32 staging that the gradient buffer is too small for
  char* arena = nullptr; size_t arena_cap = 0, arena_off = 0, arena_fixed = 0;
  bool checked = false;             // guard regions behind every arena slice, verified by hift_check_arena
  bool record_guards = false;
  std::vector<size_t> guards;       // offsets of the guard regions of the current plan
  size_t n_fixed_guards = 0;        // the first of them belong to the fixed work buffers
  cudaEvent_t ev_fwd;
  cudaEvent_t tl[7];                // timeline of the last step: start, (unused x2), optimizer wait begin/end, d2h begin/end
  bool tl_valid = false;
  bool events_made = false;
  // fixed work buffers
  int32_t *tok_dev = nullptr, *lab_dev = nullptr;
  int32_t* lens_dev = nullptr;      // [B] valid keys per batch entry (key padding), used while use_lens
  bool use_lens = false;
  float *dxa = nullptr, *dxb = nullptr;             // residual-stream gradients (fp32)
  char *dxa_a = nullptr, *dxb_a = nullptr;          // the same, rounded once to the operand type
  char *dt1 = nullptr, *dqkv = nullptr, *dbig = nullptr, *dsw = nullptr;
  float *x_final = nullptr, *emb_e = nullptr, *pp[2] = {nullptr, nullptr};
  char *x_final_a = nullptr, *ppa[2] = {nullptr, nullptr};
  char *xf = nullptr, *logits = nullptr;
  float *stf = nullptr, *st_e = nullptr, *dsum = nullptr, *partial = nullptr, *rowloss = nullptr, *rope_cs = nullptr;
  float* scal = nullptr;            // device: [0] loss, [1] nvalid(int), [2] bad(int)
  float* scal_host = nullptr;       // pinned, mapped mirror
  float* scal_host_dev = nullptr;   // its device-side address
  std::vector<std::vector<char*>> slots;   // [block][slot]; entry L holds the scratch copies
  // instrumentation
  bool prof_on = false;
  std::vector<cudaEvent_t> ev_pool; size_t ev_used = 0;
  std::vector<ProfRec> prof_recs;
  int64_t prof_launches[HIFT_K_NUM]; double prof_ms[HIFT_K_NUM], prof_work[HIFT_K_NUM];
  int64_t step_launches = 0;
  size_t step_h2d = 0, step_d2h = 0;
  cudaError_t first_err = cudaSuccess;

  // ---- helpers
  void note(cudaError_t e) { if (e != cudaSuccess && first_err == cudaSuccess) first_err = e; }
  void* P(int ti) const { return params + tens[ti].off * es; }
  void* Pn(int ti) const { return ti < 0 ? nullptr : P(ti); }
  void* G(int ti) const { return (char*)grad + grad_off[ti] * ges; }
  void pre(int cls, double work) {
    ++step_launches;
    if (!prof_on) return;
    if (ev_used + 2 > ev_pool.size()) {
      for (int i = 0; i < 256; ++i) { cudaEvent_t e; note(cudaEventCreate(&e)); ev_pool.push_back(e); }
    }
    ProfRec r{cls, ev_pool[ev_used], ev_pool[ev_used + 1], work};
    ev_used += 2;
    note(cudaEventRecord(r.e0, st));
    prof_recs.push_back(r);
  }
  void post() {
    note(cudaGetLastError());
    if (prof_on) note(cudaEventRecord(prof_recs.back().e1, st));
  }
  void prof_collect() {
    for (auto& r : prof_recs) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess) {
        prof_launches[r.cls]++; prof_ms[r.cls] += ms; prof_work[r.cls] += r.work;
      }
    }
    prof_recs.clear();
    ev_used = 0;
  }
};

#define LAUNCH(cls, work, ...) do { c->pre(cls, work); __VA_ARGS__; c->post(); } while (0)

namespace {
void emit_chunk(hift_ctx* c, size_t off, size_t n) {
  if (c->chunks.size() == c->chunk_events.size()) {
    cudaEvent_t e;
    c->note(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    c->chunk_events.push_back(e);
  }
  cudaEvent_t ev = c->chunk_events[c->chunks.size()];
  c->note(cudaEventRecord(ev, c->st));
  c->chunks.push_back(hift_ctx::ChunkRec{off, n, ev});
}
// The gradient of tensor ti has had its last contribution enqueued.
void grad_done(hift_ctx* c, int ti) {
  if (ti < 0 || c->planner_idx[ti] < 0) return;
  size_t off, n;
  if (c->planner.complete(c->planner_idx[ti], &off, &n)) emit_chunk(c, off, n);
}
}  // namespace

namespace {

// ------------------------------------------------------------------ schedule (host, integers)
// SplitMix64 (Steele, Lea, Flood 2014): the one-time shuffle of the "random" strategy.
uint64_t splitmix64_next(uint64_t& s) {
  s += 0x9E3779B97F4A7C15ull;
  uint64_t z = s;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
std::vector<int> make_order(int k, int order, uint64_t seed) {
  std::vector<int> o(k);
  for (int i = 0; i < k; ++i) o[i] = i;
  if (order == 1) std::reverse(o.begin(), o.end());
  if (order == 2) {
    uint64_t s = seed;
    for (int i = k - 1; i > 0; --i) {
      const int j = (int)(splitmix64_next(s) % (uint64_t)(i + 1));
      std::swap(o[i], o[j]);
    }
  }
  return o;
}
double lr_for_cycle(const hift_opt_cfg& oc, int64_t cycle) {
  if (oc.sched == 0) return oc.lr;
  const int64_t W = oc.warmup_cycles, C = oc.total_cycles;
  if (cycle < W) return oc.lr * (double)cycle / (double)W;
  const double fct = (double)(C - cycle) / (double)(C - W > 1 ? C - W : 1);
  return oc.lr * (fct > 0.0 ? fct : 0.0);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int add_tensor(hift_ctx* c, int unit, const std::string& name, int64_t rows, int64_t cols, int kind) {
  TensorRec r;
  memset(&r, 0, sizeof(r));
  snprintf(r.name, sizeof(r.name), "%s", name.c_str());
  r.unit = unit; r.rows = rows; r.cols = cols; r.numel = (size_t)rows * cols; r.init_kind = kind;
  r.off = c->total;
  c->total = align_up(c->total + r.numel, kAlignElems);
  c->tens.push_back(r);
  c->unit_tens[unit].push_back((int)c->tens.size() - 1);
  return (int)c->tens.size() - 1;
}

void build_layout(hift_ctx* c) {
  const hift_model_cfg& m = c->m;
  const int L = m.n_blocks, d = m.d_model, f = m.d_ffn, V = m.vocab;
  c->unit_tens.assign(L + 2, {});
  c->t_tok = add_tensor(c, 0, "tok_emb", V, d, 0);
  if (m.arch != 2) c->t_pos = add_tensor(c, 0, "pos_emb", m.max_pos, d, 0);
  if (m.arch == 1) {
    c->t_eg = add_tensor(c, 0, "emb_ln_g", 1, d, 1);
    c->t_eb = add_tensor(c, 0, "emb_ln_b", 1, d, 2);
  }
  c->bidx.resize(L);
  for (int i = 0; i < L; ++i) {
    const std::string p = "b" + std::to_string(i) + ".";
    BlockIdx& b = c->bidx[i];
    const int u = i + 1;
    if (m.arch == 2) {
      b.n1_g = add_tensor(c, u, p + "rms1_g", 1, d, 1); b.n1_b = -1;
      b.w_qkv = add_tensor(c, u, p + "w_qkv", 3 * d, d, 0); b.b_qkv = -1;
      b.w_o = add_tensor(c, u, p + "w_o", d, d, 0); b.b_o = -1;
      b.n2_g = add_tensor(c, u, p + "rms2_g", 1, d, 1); b.n2_b = -1;
      b.w_fc1 = add_tensor(c, u, p + "w_gu", 2 * f, d, 0); b.b_fc1 = -1;
      b.w_fc2 = add_tensor(c, u, p + "w_down", d, f, 0); b.b_fc2 = -1;
    } else {
      b.n1_g = add_tensor(c, u, p + "ln1_g", 1, d, 1); b.n1_b = add_tensor(c, u, p + "ln1_b", 1, d, 2);
      b.w_qkv = add_tensor(c, u, p + "w_qkv", 3 * d, d, 0); b.b_qkv = add_tensor(c, u, p + "b_qkv", 1, 3 * d, 2);
      b.w_o = add_tensor(c, u, p + "w_o", d, d, 0); b.b_o = add_tensor(c, u, p + "b_o", 1, d, 2);
      b.n2_g = add_tensor(c, u, p + "ln2_g", 1, d, 1); b.n2_b = add_tensor(c, u, p + "ln2_b", 1, d, 2);
      b.w_fc1 = add_tensor(c, u, p + "w_fc1", f, d, 0); b.b_fc1 = add_tensor(c, u, p + "b_fc1", 1, f, 2);
      b.w_fc2 = add_tensor(c, u, p + "w_fc2", d, f, 0); b.b_fc2 = add_tensor(c, u, p + "b_fc2", 1, d, 2);
    }
  }
  const int hu = L + 1;
  if (m.arch == 1) {
    c->t_wc = add_tensor(c, hu, "w_cls", m.n_classes, d, 0);
    c->t_bc = add_tensor(c, hu, "b_cls", 1, m.n_classes, 2);
  } else {
    if (m.arch == 2) c->t_fg = add_tensor(c, hu, "rmsf_g", 1, d, 1);
    else { c->t_fg = add_tensor(c, hu, "lnf_g", 1, d, 1); c->t_fb = add_tensor(c, hu, "lnf_b", 1, d, 2); }
    if (!m.tie_head) c->t_wh = add_tensor(c, hu, "w_head", V, d, 0);
  }
  // groups: consecutive chunks of m units (paper, Notation), or embedding | chunks | head
  const int n = L + 2, mm = c->gc.layers_per_group;
  std::vector<std::pair<int, int>> spans;
  if (c->queue) {
    for (int u = 0; u < n; ++u) spans.push_back({u, u});       // every unit keeps its own state
  } else if (!c->group_sizes.empty()) {
    int u = 0;
    for (int sz : c->group_sizes) { spans.push_back({u, u + sz - 1}); u += sz; }
  } else if (c->gc.split_emb_head) {
    spans.push_back({0, 0});
    for (int u = 1; u <= L; u += mm) spans.push_back({u, std::min(u + mm - 1, L)});
    spans.push_back({n - 1, n - 1});
  } else {
    for (int u = 0; u < n; u += mm) spans.push_back({u, std::min(u + mm - 1, n - 1)});
  }
  for (auto& sp : spans) {
    GroupRec g;
    memset(&g, 0, sizeof(g));
    g.unit_lo = sp.first; g.unit_hi = sp.second;
    const int t_first = c->unit_tens[sp.first].front();
    const int t_last = c->unit_tens[sp.second].back();
    g.off = c->tens[t_first].off;
    g.numel = align_up(c->tens[t_last].off + c->tens[t_last].numel, kAlignElems) - g.off;
    c->max_group = std::max(c->max_group, g.numel);
    c->groups.push_back(g);
  }
  if (c->queue) {
    // Algorithm 1, c-d: the queue holds the units in the strategy's order; each step pops m from the head and
    // appends them to the tail, so step t trains queue positions t m .. t m + m - 1 (mod n)
    c->queue_units = make_order(n, c->gc.order, c->gc.order_seed);
    int a = n, b = mm;
    while (b) { const int r = a % b; a = b; b = r; }
    c->n_sets = n / a;
    c->k_cycle = (n + mm - 1) / mm;
    c->order.clear();
  } else {
    c->order = make_order((int)c->groups.size(), c->gc.order, c->gc.order_seed);
    c->n_sets = c->k_cycle = (int)c->groups.size();
  }
}

// The state groups of set `id`, with their places in the gradient buffer and in a state slot.
void fill_set(const hift_ctx* c, int id, ActiveSet* a) {
  a->id = id;
  a->groups.clear(); a->grad_base.clear(); a->slot_base.clear();
  if (c->queue) {
    const int n = (int)c->groups.size(), mm = c->gc.layers_per_group;
    for (int j = 0; j < mm && j < n; ++j) a->groups.push_back(c->queue_units[(size_t)(((int64_t)id * mm + j) % n)]);
    std::sort(a->groups.begin(), a->groups.end());
  } else {
    a->groups.push_back(id);
  }
  size_t go = 0, so = 0;
  for (int g : a->groups) {
    a->grad_base.push_back(go); a->slot_base.push_back(so);
    go += c->groups[g].numel;
    so += align_up(c->groups[g].blob_bytes, 256);
  }
  a->grad_numel = go; a->slot_bytes = so;
  a->lo_unit = c->groups[a->groups.front()].unit_lo;
}
bool unit_in_set(const hift_ctx* c, const ActiveSet& a, int u) {
  for (int g : a.groups) if (u >= c->groups[g].unit_lo && u <= c->groups[g].unit_hi) return true;
  return false;
}

hift_status dev_alloc(hift_ctx* c, void** p, size_t bytes) {
  *p = nullptr;
  if (bytes == 0) bytes = 256;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) { cudaGetLastError(); return HIFT_ERR_OOM_DEVICE; }
  c->dev_allocs.push_back(*p);
  c->dev_bytes += bytes;
  return HIFT_OK;
}

char* arena_take(hift_ctx* c, size_t bytes) {
  const size_t o = c->arena_off;
  c->arena_off = align_up(o + bytes, 256);
  if (c->checked) {
    if (c->record_guards) c->guards.push_back(c->arena_off);
    c->arena_off += kGuardBytes;
  }
  return c->arena ? c->arena + o : (char*)(uintptr_t)o;
}
// pinned host memory through one door, so that a test can make the n-th request fail
cudaError_t pinned_alloc(void** p, size_t bytes, unsigned flags) {
  if (g_fail_pinned_in >= 0 && g_fail_pinned_in-- == 0) { *p = nullptr; return cudaErrorMemoryAllocation; }
  return cudaHostAlloc(p, bytes, flags);
}

// Lowest level at which a slot must outlive the forward pass: 1 = activation gradients need
// it, 2 = only weight gradients need it, 3 = never (forward scratch), 99 = unused by the arch.
int slot_min_level(int arch, int s) {
  if (arch == 1) {
    switch (s) {
      case S_XIN: return 3; case S_XINA: return 2; case S_H1: return 99; case S_QKV: return 1;
      case S_O: return 1; case S_LSE: return 1; case S_X2: return 1; case S_ST1: return 1;
      case S_H2: return 2; case S_H2R: return 3; case S_A: return 1; case S_U: return 2;
      case S_Z: return 1; case S_ST2: return 1;
    }
  } else {
    switch (s) {
      case S_XIN: return 1; case S_XINA: return 99; case S_H1: return 2; case S_QKV: return 1;
      case S_O: return 1; case S_LSE: return 1; case S_X2: return 1; case S_ST1: return 1;
      case S_H2: return 2; case S_H2R: return 99; case S_A: return 1; case S_U: return 2;
      case S_Z: return 99; case S_ST2: return 1;
    }
  }
  return 99;
}
size_t slot_bytes(const hift_ctx* c, int s) {
  const size_t T = c->T, d = c->d, es = c->es;
  switch (s) {
    case S_XIN: case S_X2: case S_Z: case S_H2R: return T * d * sizeof(float);
    case S_XINA: case S_H1: case S_O: case S_H2: return T * d * es;
    case S_QKV: return T * 3 * d * es;
    case S_A: return T * (size_t)c->fa * es;
    case S_U: return T * (size_t)c->f * es;
    case S_LSE: return (size_t)c->B * c->H * c->S * sizeof(float);
    case S_ST1: case S_ST2: return 2 * T * sizeof(float);
  }
  return 0;
}
int level_of_block(const hift_ctx* c, const ActiveSet& a, int i) {
  const int u = i + 1;
  if (u < a.lo_unit) return 0;
  return unit_in_set(c, a, u) ? 2 : 1;
}
// Assign the per-block activation slots for a step that trains group g.  Returns the arena
// bytes used.  With assign == false only sizes are computed.
size_t plan_slots(hift_ctx* c, const ActiveSet& g, bool assign) {
  c->arena_off = c->arena_fixed;
  if (c->checked && assign) { c->guards.resize(c->n_fixed_guards); c->record_guards = true; }
  for (int i = 0; i < c->L; ++i) {
    const int lvl = level_of_block(c, g, i);
    for (int s = 0; s < S_NUM; ++s) {
      const int need = slot_min_level(c->m.arch, s);
      if (need == 99) { if (assign) c->slots[i][s] = nullptr; continue; }
      // recompute: a frozen block above the group keeps its input only (stream, and operand copy where the
      // architecture has one); everything else lives in the shared scratch copy until the backward pass redoes it
      const bool keep = (c->recompute && lvl == 1) ? (s == S_XIN || s == S_XINA) : lvl >= need;
      if (keep) {
        char* p = arena_take(c, slot_bytes(c, s));
        if (assign) c->slots[i][s] = p;
      } else if (assign) {
        c->slots[i][s] = (s == S_XIN) ? (char*)c->pp[i & 1] : (s == S_XINA) ? c->ppa[i & 1] : c->slots[c->L][s];
      }
    }
  }
  c->record_guards = false;
  return c->arena_off;
}

// ------------------------------------------------------------------ thin launch helpers
void gemm(hift_ctx* c, int cls, int M, int N, int K, const void* a, int64_t sam, int64_t sak,
          const void* b, int64_t sbk, int64_t sbn, void* out, int64_t ldc, const void* bias,
          const float* residual, int64_t ldr, bool out_f32) {
  GemmArgs g{M, N, K, a, sam, sak, b, sbk, sbn, out, ldc, bias, residual, ldr, out_f32};
  const double work = 2.0 * M * (double)N * K;
  if (c->mixed && gemm_tc_eligible(g)) {
    LAUNCH(cls, work, c->note(gemm_tc_launch(c->st, g)));
    return;
  }
  LAUNCH(cls, work, launch_gemm_simt(c->st, c->mixed ? 1 : 0, g));
}
// y[M,N] = x[M,K] w[N,K]^T + bias (+ residual).  to_stream: the output (and the residual) is
// the fp32 residual stream.
void linear_fwd(hift_ctx* c, int M, int N, int K, const void* x, int64_t ldx, const void* w,
                void* y, int64_t ldy, const void* bias, const float* res, int64_t ldr, bool to_stream) {
  gemm(c, HIFT_K_GEMM_FWD, M, N, K, x, ldx, 1, w, 1, K, y, ldy, bias, res, ldr, to_stream);
}
// dx[M,K] = dy[M,N] w[N,K] (+ residual)
void linear_dx(hift_ctx* c, int M, int N, int K, const void* dy, int64_t ldy, const void* w,
               void* dx, int64_t ldx, const float* res, int64_t ldr, bool to_stream) {
  gemm(c, HIFT_K_GEMM_DX, M, K, N, dy, ldy, 1, w, K, 1, dx, ldx, nullptr, res, ldr, to_stream);
}
// dw[N,K] = dy[M,N]^T x[M,K]   (fp32 out)
void linear_dw(hift_ctx* c, int M, int N, int K, const void* dy, int64_t ldy, const void* x,
               int64_t ldx, void* dw) {
  gemm(c, HIFT_K_GEMM_DW, N, K, M, dy, 1, ldy, x, ldx, 1, dw, K, nullptr, nullptr, 0, !c->gbf);
}
void norm_fwd(hift_ctx* c, const float* x, int tg, int tb, void* y_a, float* y_r, float* stats) {
  const int kind = c->m.arch == 2 ? 1 : 0;
  LAUNCH(HIFT_K_NORM, (double)c->T * c->d * (4 + c->es + (y_r ? 4 : 0)),
         launch_norm_fwd(c->st, c->mixed, kind, c->T, c->d, (float)c->m.norm_eps, x, c->P(tg),
                         c->Pn(tb), y_a, y_r, stats));
}
void norm_bwd_dx(hift_ctx* c, const void* dy, bool dy_f32, const float* x, const float* stats, int tg,
                 const float* add, float* dx_r, void* dx_a) {
  const int kind = c->m.arch == 2 ? 1 : 0;
  const double bytes = (double)c->T * c->d * ((dy_f32 ? 4 : c->es) + 4 + (add ? 4 : 0) + 4 + (dx_a ? c->es : 0));
  LAUNCH(HIFT_K_NORM, bytes,
         launch_norm_bwd_dx(c->st, c->mixed, kind, dy_f32, c->T, c->d, dy, x, stats, c->P(tg), add, dx_r, dx_a));
}
void norm_bwd_params(hift_ctx* c, const void* dy, bool dy_f32, const float* x, const float* stats, int tg, int tb) {
  const int mode = c->m.arch == 2 ? 2 : 1;
  LAUNCH(HIFT_K_REDUCE, (double)c->T * c->d * ((dy_f32 ? 4 : c->es) + 4),
         launch_colreduce(c->st, c->mixed && !dy_f32, mode, c->T, c->d, dy, c->d, x, stats, c->partial,
                          c->G(tg), tb >= 0 ? c->G(tb) : nullptr, c->gbf));
  ++c->step_launches;   // two kernels per call
}
void bias_grad(hift_ctx* c, const void* dy, bool dy_f32, int64_t rows, int cols, int64_t ld, int tb) {
  if (tb < 0) return;
  LAUNCH(HIFT_K_REDUCE, (double)rows * cols * (dy_f32 ? 4 : c->es),
         launch_colreduce(c->st, c->mixed && !dy_f32, 0, rows, cols, dy, ld, nullptr, nullptr, c->partial,
                          c->G(tb), nullptr, c->gbf));
  ++c->step_launches;
}
// dropout on the attention probabilities of block `blk`: thr = 0 when the rate is 0
DropArgs attn_drop_args(const hift_ctx* c, int blk) {
  DropArgs a;
  a.k0 = (uint32_t)c->m.dropout_seed; a.k1 = (uint32_t)(c->m.dropout_seed >> 32);
  a.site = (uint32_t)(1000 + blk); a.step = (uint32_t)c->t; a.thr = c->adrop_thr; a.scale = c->adrop_scale;
  return a;
}
void attn_fwd(hift_ctx* c, int blk, const void* qkv, void* o, float* lse) {
  const double work = 4.0 * c->B * c->H * (double)c->S * c->S * c->dh * (c->m.causal ? 0.5 : 1.0);
  LAUNCH(HIFT_K_ATTN_FWD, work,
         launch_attention_fwd(c->st, c->mixed, c->B, c->S, c->H, c->dh, c->m.causal, qkv, o, lse,
                              c->use_lens ? c->lens_dev : nullptr, attn_drop_args(c, blk)));
}
void attn_bwd(hift_ctx* c, int blk, const void* qkv, const void* o, const float* lse, const void* dout, void* dqkv) {
  const double work = 10.0 * c->B * c->H * (double)c->S * c->S * c->dh * (c->m.causal ? 0.5 : 1.0);
  LAUNCH(HIFT_K_ATTN_BWD, work,
         launch_attention_bwd(c->st, c->mixed, c->B, c->S, c->H, c->dh, c->m.causal, qkv, o, lse,
                              dout, dqkv, c->dsum, c->use_lens ? c->lens_dev : nullptr, attn_drop_args(c, blk)));
  c->step_launches += (attention_use_mma(c->mixed, c->dh) && !c->adrop_thr) ? 2 : 1;   // dsum, dq, dkv or dq, dkv
}
// qkv projection of a rotary model: on the tensor-core path the rotation of the q and k column blocks
// happens in the GEMM's epilogue (head size 128); otherwise the projection is followed by the
// in-place kernel below.
void rope(hift_ctx* c, void* qkv, float sign);
void linear_fwd_qkv_rope(hift_ctx* c, int M, int d, const void* x, const void* w, void* qkv, const void* bias) {
  GemmArgs g{M, 3 * d, d, x, d, 1, w, 1, d, qkv, 3 * d, bias, nullptr, 0, false};
  g.rope_cs = c->rope_cs; g.rope_seq = c->S; g.rope_dh = c->dh; g.rope_cols = 2 * (int64_t)d;
  if (c->mixed && gemm_tc_eligible(g)) {
    LAUNCH(HIFT_K_GEMM_FWD, 2.0 * M * 3.0 * d * d, c->note(gemm_tc_launch(c->st, g)));
    return;
  }
  linear_fwd(c, M, 3 * d, d, x, d, w, qkv, 3 * d, bias, nullptr, 0, false);
  rope(c, qkv, 1.0f);
}
void rope(hift_ctx* c, void* qkv, float sign) {
  const size_t n = (size_t)c->T * c->H * (c->dh / 16);      // one thread per 8 pairs
  LAUNCH(HIFT_K_ELEMWISE, 64.0 * n * c->es,
         if (c->mixed) launch_pdl(rope_kernel<bf16>, dim3(grid_for(n, 256)), dim3(256), 0, c->st, (bf16*)qkv, c->rope_cs, (int64_t)c->T, c->S, c->H, c->dh, sign);
         else launch_pdl(rope_kernel<float>, dim3(grid_for(n, 256)), dim3(256), 0, c->st, (float*)qkv, c->rope_cs, (int64_t)c->T, c->S, c->H, c->dh, sign));
}
void act_fwd(hift_ctx* c, const void* a, void* u) {
  const size_t n = (size_t)c->T * c->f;
  if (c->m.arch == 2) {
    LAUNCH(HIFT_K_ELEMWISE, 3.0 * n * c->es,
           if (c->mixed) swiglu_fwd_kernel<bf16><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const bf16*)a, (bf16*)u, c->T, c->f);
           else swiglu_fwd_kernel<float><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const float*)a, (float*)u, c->T, c->f));
  } else {
    LAUNCH(HIFT_K_ELEMWISE, 2.0 * n * c->es,
           if (c->mixed) gelu_fwd_kernel<bf16><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const bf16*)a, (bf16*)u, n / 8);
           else gelu_fwd_kernel<float><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const float*)a, (float*)u, n / 8));
  }
}
// Gate | up projection of a SwiGLU block followed by the activation: on the tensor-core path one GEMM
// whose epilogue stores silu(gate) * up, and the pre-activations only if the backward pass will read
// them (`keep`); otherwise the projection and the activation kernel.
void linear_fwd_swiglu(hift_ctx* c, int M, int f, int K, const void* x, const void* w, void* gu, void* sact,
                       const void* bias, bool keep) {
  GemmArgs g{M, 2 * f, K, x, K, 1, w, 1, K, keep ? gu : nullptr, 2 * (int64_t)f, bias, nullptr, 0, false};
  g.swiglu_out = sact;
  if (c->mixed && gemm_tc_eligible(g)) {
    LAUNCH(HIFT_K_GEMM_FWD, 2.0 * M * 2.0 * f * K, c->note(gemm_tc_launch(c->st, g)));
    return;
  }
  linear_fwd(c, M, 2 * f, K, x, K, w, gu, 2 * f, bias, nullptr, 0, false);
  act_fwd(c, gu, sact);
}
// Up projection of a GELU block followed by the activation, and the down projection's dX product followed by
// the activation's backward: one GEMM each on the tensor-core path (the activation runs in the epilogue),
// else the GEMM and the activation kernel.
void linear_fwd_gelu(hift_ctx* c, int M, int f, int K, const void* x, const void* w, void* a, void* u, const void* bias, bool keep) {
  GemmArgs g{M, f, K, x, K, 1, w, 1, K, keep ? a : nullptr, (int64_t)f, bias, nullptr, 0, false};
  g.gelu_out = u;
  if (c->mixed && gemm_tc_eligible(g)) {
    LAUNCH(HIFT_K_GEMM_FWD, 2.0 * M * (double)f * K, c->note(gemm_tc_launch(c->st, g)));
    return;
  }
  linear_fwd(c, M, f, K, x, K, w, a, f, bias, nullptr, 0, false);
  act_fwd(c, a, u);
}
void act_bwd(hift_ctx* c, const void* a);
void linear_dx_gelu_bwd(hift_ctx* c, int M, int N, int f, const void* dy, const void* w, const void* a) {
  GemmArgs g{M, f, N, dy, N, 1, w, f, 1, c->dbig, (int64_t)f, nullptr, nullptr, 0, false};
  g.gelu_bwd_a = a;
  if (c->mixed && gemm_tc_eligible(g)) {
    LAUNCH(HIFT_K_GEMM_DX, 2.0 * M * (double)f * N, c->note(gemm_tc_launch(c->st, g)));
    return;
  }
  linear_dx(c, M, N, f, dy, N, w, c->dbig, f, nullptr, 0, false);
  act_bwd(c, a);
}
// GELU: du (in c->dbig, [T,f]) *= gelu'(a) in place.
// SwiGLU: ds (in c->dsw, [T,f]) -> dgu in c->dbig [T,2f].
void act_bwd(hift_ctx* c, const void* a) {
  const size_t n = (size_t)c->T * c->f;
  if (c->m.arch == 2) {
    LAUNCH(HIFT_K_ELEMWISE, 5.0 * n * c->es,
           if (c->mixed) swiglu_bwd_kernel<bf16><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const bf16*)c->dsw, (const bf16*)a, (bf16*)c->dbig, c->T, c->f);
           else swiglu_bwd_kernel<float><<<grid_for(n / 8, 256), 256, 0, c->st>>>((const float*)c->dsw, (const float*)a, (float*)c->dbig, c->T, c->f));
  } else {
    LAUNCH(HIFT_K_ELEMWISE, 3.0 * n * c->es,
           if (c->mixed) gelu_bwd_kernel<bf16><<<grid_for(n / 8, 256), 256, 0, c->st>>>((bf16*)c->dbig, (const bf16*)a, n / 8);
           else gelu_bwd_kernel<float><<<grid_for(n / 8, 256), 256, 0, c->st>>>((float*)c->dbig, (const float*)a, n / 8));
  }
}

// ------------------------------------------------------------------ dropout sites
DropArgs drop_args(const hift_ctx* c, int site) {
  DropArgs a;
  a.k0 = (uint32_t)c->m.dropout_seed; a.k1 = (uint32_t)(c->m.dropout_seed >> 32);
  a.site = (uint32_t)site; a.step = (uint32_t)c->t; a.thr = c->drop_thr; a.scale = c->drop_scale;
  return a;
}
// out = res + mask * t over the [T, d] stream
void drop_add(hift_ctx* c, int site, const float* t, const float* res, float* out) {
  const size_t n4 = (size_t)c->T * c->d / 4;
  LAUNCH(HIFT_K_ELEMWISE, 48.0 * n4, dropout_add_kernel<<<grid_for(n4, 256), 256, 0, c->st>>>(t, res, out, n4, drop_args(c, site)));
}
void drop_inplace(hift_ctx* c, int site, float* x, void* x_a) {
  const size_t n4 = (size_t)c->T * c->d / 4;
  LAUNCH(HIFT_K_ELEMWISE, (32.0 + (x_a ? 4.0 * c->es : 0.0)) * n4,
         if (c->mixed) dropout_inplace_kernel<bf16><<<grid_for(n4, 256), 256, 0, c->st>>>(x, (bf16*)x_a, n4, drop_args(c, site));
         else dropout_inplace_kernel<float><<<grid_for(n4, 256), 256, 0, c->st>>>(x, (float*)x_a, n4, drop_args(c, site)));
}
// masked copies of the stream gradient dx: fp32 into the (idle in the backward pass) ping-pong buffer, operand into mop
const float* drop_bwd(hift_ctx* c, int site, const float* dx, void* mop) {
  const size_t n4 = (size_t)c->T * c->d / 4;
  float* mf = c->pp[1];
  LAUNCH(HIFT_K_ELEMWISE, (32.0 + 4.0 * c->es) * n4,
         if (c->mixed) dropout_bwd_kernel<bf16><<<grid_for(n4, 256), 256, 0, c->st>>>(dx, mf, (bf16*)mop, n4, drop_args(c, site));
         else dropout_bwd_kernel<float><<<grid_for(n4, 256), 256, 0, c->st>>>(dx, mf, (float*)mop, n4, drop_args(c, site)));
  return mf;
}
// y = (x w^T + bias) [dropped] + res into the residual stream
void linear_fwd_to_stream(hift_ctx* c, int site, int M, int N, int K, const void* x, const void* w, float* y, const void* bias,
                          const float* res) {
  if (!c->drop_on) { linear_fwd(c, M, N, K, x, K, w, y, N, bias, res, N, true); return; }
  // the branch output in fp32 (dxb is idle in the forward pass), then the masked addition
  linear_fwd(c, M, N, K, x, K, w, c->dxb, N, bias, nullptr, 0, true);
  drop_add(c, site, c->dxb, res, y);
}

// ------------------------------------------------------------------ forward
// x_r / x_a: the block input on the residual stream and (post-LN only) its operand copy.
void forward_block(hift_ctx* c, int i, const float* x_r, const char* x_a, float* xo_r, char* xo_a) {
  const BlockIdx& b = c->bidx[i];
  std::vector<char*>& s = c->slots[i];
  const int T = c->T, d = c->d, f = c->f, fa = c->fa;
  float* x2 = (float*)s[S_X2];
  if (c->m.arch == 1) {
    float* x1r = (float*)s[S_H2R];
    float* z = (float*)s[S_Z];
    linear_fwd(c, T, 3 * d, d, x_a, d, c->P(b.w_qkv), s[S_QKV], 3 * d, c->Pn(b.b_qkv), nullptr, 0, false);
    attn_fwd(c, i, s[S_QKV], s[S_O], (float*)s[S_LSE]);
    linear_fwd_to_stream(c, 1 + 2 * i, T, d, d, s[S_O], c->P(b.w_o), x2, c->Pn(b.b_o), x_r);       // y
    norm_fwd(c, x2, b.n1_g, b.n1_b, s[S_H2], x1r, (float*)s[S_ST1]);                                 // x1
    linear_fwd_gelu(c, T, f, d, s[S_H2], c->P(b.w_fc1), s[S_A], s[S_U], c->Pn(b.b_fc1), c->keep_all || s[S_A] != c->slots[c->L][S_A]);
    linear_fwd_to_stream(c, 2 + 2 * i, T, d, f, s[S_U], c->P(b.w_fc2), z, c->Pn(b.b_fc2), x1r);     // z
    norm_fwd(c, z, b.n2_g, b.n2_b, xo_a, xo_r, (float*)s[S_ST2]);
    return;
  }
  norm_fwd(c, x_r, b.n1_g, b.n1_b, s[S_H1], nullptr, (float*)s[S_ST1]);
  if (c->m.arch == 2) linear_fwd_qkv_rope(c, T, d, s[S_H1], c->P(b.w_qkv), s[S_QKV], c->Pn(b.b_qkv));
  else linear_fwd(c, T, 3 * d, d, s[S_H1], d, c->P(b.w_qkv), s[S_QKV], 3 * d, c->Pn(b.b_qkv), nullptr, 0, false);
  attn_fwd(c, i, s[S_QKV], s[S_O], (float*)s[S_LSE]);
  linear_fwd_to_stream(c, 1 + 2 * i, T, d, d, s[S_O], c->P(b.w_o), x2, c->Pn(b.b_o), x_r);
  norm_fwd(c, x2, b.n2_g, b.n2_b, s[S_H2], nullptr, (float*)s[S_ST2]);
  if (c->m.arch == 2) {
    // blocks below the active group keep nothing: their pre-activations live in the scratch slot and are never read
    linear_fwd_swiglu(c, T, f, d, s[S_H2], c->P(b.w_fc1), s[S_A], s[S_U], c->Pn(b.b_fc1), c->keep_all || s[S_A] != c->slots[c->L][S_A]);
  } else {
    linear_fwd_gelu(c, T, f, d, s[S_H2], c->P(b.w_fc1), s[S_A], s[S_U], c->Pn(b.b_fc1), c->keep_all || s[S_A] != c->slots[c->L][S_A]);
  }
  // a block that is only being recomputed for its backward needs everything above, not its output
  if (!c->keep_all) linear_fwd_to_stream(c, 2 + 2 * i, T, d, f, s[S_U], c->P(b.w_fc2), xo_r, c->Pn(b.b_fc2), x2);
}

// ------------------------------------------------------------------ backward
// On entry c->dxa (fp32; pre-norm blocks also c->dxa_a) holds the gradient of the block output;
// on exit (need_dx) the gradient of the block input, in the same buffers.
void backward_block(hift_ctx* c, int i, const float* x_r, const char* x_a, bool on, bool need_dx) {
  const BlockIdx& b = c->bidx[i];
  std::vector<char*>& s = c->slots[i];
  const int T = c->T, d = c->d, f = c->f, fa = c->fa;
  char* dact_in = c->m.arch == 2 ? c->dsw : c->dbig;    // gradient w.r.t. the activation output
  float* x2 = (float*)s[S_X2];
  if (c->m.arch == 1) {
    float* z = (float*)s[S_Z];
    if (on) { norm_bwd_params(c, c->dxa, true, z, (float*)s[S_ST2], b.n2_g, b.n2_b); grad_done(c, b.n2_b); grad_done(c, b.n2_g); }
    norm_bwd_dx(c, c->dxa, true, z, (float*)s[S_ST2], b.n2_g, nullptr, c->dxb, c->dxb_a);          // dz
    // through the dropout of the feed-forward output: the branch sees the masked gradient, the residual path dz itself
    const float* gf = c->drop_on ? drop_bwd(c, 2 + 2 * i, c->dxb, c->dxb_a) : c->dxb;
    linear_dx_gelu_bwd(c, T, d, f, c->dxb_a, c->P(b.w_fc2), s[S_A]);                                // du -> da
    if (on) { linear_dw(c, T, d, f, c->dxb_a, d, s[S_U], f, c->G(b.w_fc2)); bias_grad(c, gf, true, T, d, d, b.b_fc2); grad_done(c, b.b_fc2); grad_done(c, b.w_fc2); }
    linear_dx(c, T, f, d, c->dbig, f, c->P(b.w_fc1), c->dxa, d, c->dxb, d, true);                   // dx1
    if (on) { linear_dw(c, T, f, d, c->dbig, f, s[S_H2], d, c->G(b.w_fc1)); bias_grad(c, c->dbig, false, T, f, f, b.b_fc1); grad_done(c, b.b_fc1); grad_done(c, b.w_fc1); }
    if (on) { norm_bwd_params(c, c->dxa, true, x2, (float*)s[S_ST1], b.n1_g, b.n1_b); grad_done(c, b.n1_b); grad_done(c, b.n1_g); }
    norm_bwd_dx(c, c->dxa, true, x2, (float*)s[S_ST1], b.n1_g, nullptr, c->dxb, c->dxb_a);         // dy
    const float* ga = c->drop_on ? drop_bwd(c, 1 + 2 * i, c->dxb, c->dxb_a) : c->dxb;
    linear_dx(c, T, d, d, c->dxb_a, d, c->P(b.w_o), c->dt1, d, nullptr, 0, false);                  // do
    if (on) { linear_dw(c, T, d, d, c->dxb_a, d, s[S_O], d, c->G(b.w_o)); bias_grad(c, ga, true, T, d, d, b.b_o); grad_done(c, b.b_o); grad_done(c, b.w_o); }
    attn_bwd(c, i, s[S_QKV], s[S_O], (float*)s[S_LSE], c->dt1, c->dqkv);
    if (on) { linear_dw(c, T, 3 * d, d, c->dqkv, 3 * d, x_a, d, c->G(b.w_qkv)); bias_grad(c, c->dqkv, false, T, 3 * d, 3 * d, b.b_qkv); grad_done(c, b.b_qkv); grad_done(c, b.w_qkv); }
    if (need_dx) linear_dx(c, T, 3 * d, d, c->dqkv, 3 * d, c->P(b.w_qkv), c->dxa, d, c->dxb, d, true);
    return;
  }
  // through the dropout of the feed-forward output: the branch's GEMMs read the masked operand copy (dxa_a is not
  // needed unmasked again: the residual path goes on in fp32), the bias gradient the masked fp32 copy
  const float* gf = c->drop_on ? drop_bwd(c, 2 + 2 * i, c->dxa, c->dxa_a) : c->dxa;
  // SwiGLU on the tensor-core path: the dX product of the down projection stores d gate | d up directly
  bool act_done = false;
  if (c->m.arch == 2 && c->mixed) {
    GemmArgs g{T, f, d, c->dxa_a, d, 1, c->P(b.w_fc2), f, 1, c->dbig, 2 * (int64_t)f, nullptr, nullptr, 0, false};
    g.swiglu_bwd_gu = s[S_A];
    if (gemm_tc_eligible(g)) {
      LAUNCH(HIFT_K_GEMM_DX, 2.0 * T * (double)f * d, c->note(gemm_tc_launch(c->st, g)));
      act_done = true;
    }
  }
  if (!act_done && c->m.arch != 2) { linear_dx_gelu_bwd(c, T, d, f, c->dxa_a, c->P(b.w_fc2), s[S_A]); act_done = true; }
  if (!act_done) linear_dx(c, T, d, f, c->dxa_a, d, c->P(b.w_fc2), dact_in, f, nullptr, 0, false);  // ds
  if (on) { linear_dw(c, T, d, f, c->dxa_a, d, s[S_U], f, c->G(b.w_fc2)); bias_grad(c, gf, true, T, d, d, b.b_fc2); grad_done(c, b.b_fc2); grad_done(c, b.w_fc2); }
  if (!act_done) act_bwd(c, s[S_A]);                                                                // da in dbig [T,fa]
  linear_dx(c, T, fa, d, c->dbig, fa, c->P(b.w_fc1), c->dt1, d, nullptr, 0, false);                 // dh2
  if (on) { linear_dw(c, T, fa, d, c->dbig, fa, s[S_H2], d, c->G(b.w_fc1)); bias_grad(c, c->dbig, false, T, fa, fa, b.b_fc1); grad_done(c, b.b_fc1); grad_done(c, b.w_fc1); }
  if (on) { norm_bwd_params(c, c->dt1, false, x2, (float*)s[S_ST2], b.n2_g, b.n2_b); grad_done(c, b.n2_b); grad_done(c, b.n2_g); }
  norm_bwd_dx(c, c->dt1, false, x2, (float*)s[S_ST2], b.n2_g, c->dxa, c->dxb, c->dxb_a);            // dx2
  const float* ga = c->drop_on ? drop_bwd(c, 1 + 2 * i, c->dxb, c->dxb_a) : c->dxb;
  linear_dx(c, T, d, d, c->dxb_a, d, c->P(b.w_o), c->dt1, d, nullptr, 0, false);                    // do
  if (on) { linear_dw(c, T, d, d, c->dxb_a, d, s[S_O], d, c->G(b.w_o)); bias_grad(c, ga, true, T, d, d, b.b_o); grad_done(c, b.b_o); grad_done(c, b.w_o); }
  attn_bwd(c, i, s[S_QKV], s[S_O], (float*)s[S_LSE], c->dt1, c->dqkv);
  if (c->m.arch == 2) rope(c, c->dqkv, -1.0f);
  linear_dx(c, T, 3 * d, d, c->dqkv, 3 * d, c->P(b.w_qkv), c->dt1, d, nullptr, 0, false);           // dh1
  if (on) { linear_dw(c, T, 3 * d, d, c->dqkv, 3 * d, s[S_H1], d, c->G(b.w_qkv)); bias_grad(c, c->dqkv, false, T, 3 * d, 3 * d, b.b_qkv); grad_done(c, b.b_qkv); grad_done(c, b.w_qkv); }
  if (on) { norm_bwd_params(c, c->dt1, false, x_r, (float*)s[S_ST1], b.n1_g, b.n1_b); grad_done(c, b.n1_b); grad_done(c, b.n1_g); }
  if (need_dx) norm_bwd_dx(c, c->dt1, false, x_r, (float*)s[S_ST1], b.n1_g, c->dxb, c->dxa, c->dxa_a);
}

// ------------------------------------------------------------------ state paging (Algorithm 1, steps i and k)
// The group order is known ahead, so the uploads need not wait for their own step: a ring of
// slots holds the group being trained, the groups of the next `lookahead` steps (upload in flight
// or landed) and groups whose write-back is still draining.  Only two orderings are enforced: an
// upload into a slot waits for that slot's last write-back, and the optimizer waits for its own
// slot's upload (and, when the group was still resident from an earlier step, for that slot's
// write-back, which reads what the optimizer is about to overwrite).  A group is in at most one
// slot, and a slot that holds a group holds its latest values: they change only by the optimizer
// running in that slot, followed by the write-back from it.
int group_at(const hift_ctx* c, int64_t step) {
  if (c->forced >= 0) return c->forced;
  if (!c->forced_seq.empty()) {
    const int64_t n = (int64_t)c->forced_seq.size();
    return c->forced_seq[(size_t)((((step - c->forced_seq_t0) % n) + n) % n)];
  }
  if (c->queue) return (int)(step % (int64_t)c->n_sets);
  return c->order[step % (int64_t)c->groups.size()];
}
void drop_reservations(hift_ctx* c) { for (int i = 0; i < c->n_slots; ++i) c->slot[i].step = -1; }
// after the host has rewritten blobs (every stream idle): nothing on the device is current any more
void invalidate_slots(hift_ctx* c) {
  for (int i = 0; i < c->n_slots; ++i) { c->slot[i].group = -1; c->slot[i].step = -1; c->slot[i].d2h_pending = false; }
}
// Makes group g resident for step s (>= the current step c->t).  Returns its slot, or -1 when every
// slot is reserved (only possible for look-ahead requests).
int acquire_slot(hift_ctx* c, int g, int64_t s, bool after_forward) {
  for (int i = 0; i < c->n_slots; ++i)
    if (c->slot[i].group == g) {                      // still (or already) resident: no transfer
      if (c->slot[i].step < s) c->slot[i].step = s;
      return i;
    }
  int v = -1;
  for (int i = 0; i < c->n_slots; ++i) {
    if (c->slot[i].step >= c->t) continue;            // reserved for the current or a coming step
    if (v < 0 || (c->slot[i].group < 0 && c->slot[v].group >= 0) ||
        ((c->slot[i].group < 0) == (c->slot[v].group < 0) && c->slot[i].step < c->slot[v].step))
      v = i;
  }
  if (v < 0) return -1;
  SlotRec& sr = c->slot[v];
  ActiveSet a;
  fill_set(c, g, &a);
  if (after_forward) c->note(cudaStreamWaitEvent(c->st_h2d, c->ev_fwd, 0));
  if (sr.d2h_pending) c->note(cudaStreamWaitEvent(c->st_h2d, sr.ev_d2h, 0));
  c->note(cudaEventRecord(sr.tl_h2d0, c->st_h2d));
  for (size_t i = 0; i < a.groups.size(); ++i) {
    const GroupRec& gr = c->groups[a.groups[i]];
    if (gr.blob_bytes) c->note(cudaMemcpyAsync(sr.mem + a.slot_base[i], gr.blob, gr.blob_bytes, cudaMemcpyHostToDevice, c->st_h2d));
    c->step_h2d += gr.blob_bytes;
  }
  c->note(cudaEventRecord(sr.tl_h2d1, c->st_h2d));
  c->note(cudaEventRecord(sr.ev_h2d, c->st_h2d));
  sr.group = g; sr.step = s; sr.d2h_pending = false; sr.h2d_for_step = s;
  return v;
}
// Step start (overlapped modes): the current group, then the groups of the next steps.
void page_in_ahead(hift_ctx* c) {
  c->cur_sl = acquire_slot(c, group_at(c, c->t), c->t, false);
  for (int j = 1; j <= c->lookahead; ++j) {
    const int gj = group_at(c, c->t + j);
    bool earlier = false;                              // trained before step t + j: its blob is not final yet
    for (int i = 0; i < j; ++i) earlier = earlier || group_at(c, c->t + i) == gj;
    if (!earlier) acquire_slot(c, gj, c->t + j, false);
  }
}

// Forward and truncated backward of one step, enqueued on the context's stream; the active group's
// gradient is left in c->grad.
hift_status enqueue_forward_backward(hift_ctx* c, const int32_t* tok, const int32_t* lab) {
  const hift_model_cfg& m = c->m;
  const int L = c->L, T = c->T, d = c->d, V = c->V, Vp = c->Vp, B = c->B, S = c->S;
  if (c->stage) { cudaStreamSynchronize(c->st); cudaFree(c->stage); c->stage = nullptr; }     // set-up is over
  const int g = group_at(c, c->t);
  fill_set(c, g, &c->act);
  const ActiveSet& act = c->act;
  const int lo = act.lo_unit;                                  // the backward pass stops below this unit
  const double lr = lr_for_cycle(c->oc, c->t / c->k_cycle);
  c->last_group = g;
  c->step_launches = 0; c->step_h2d = 0; c->step_d2h = 0;
  c->first_err = cudaSuccess;
  c->cur_sl = 0; c->cur_lr = lr;
  // where each trained tensor's gradient lives: the set's groups side by side, ascending units
  c->unit_on.assign(L + 2, 0);
  c->grad_off.assign(c->tens.size(), SIZE_MAX);
  for (size_t i = 0; i < act.groups.size(); ++i) {
    const GroupRec& gi = c->groups[act.groups[i]];
    for (int u = gi.unit_lo; u <= gi.unit_hi; ++u) {
      c->unit_on[u] = 1;
      for (int ti : c->unit_tens[u]) c->grad_off[ti] = act.grad_base[i] + (c->tens[ti].off - gi.off);
    }
  }
  auto active = [&](int u) { return c->unit_on[u] != 0; };

  plan_slots(c, act, true);
  if (c->arena_off > c->arena_cap) return HIFT_ERR_CFG;
  if (c->checked)      // the plan moves with the group: paint this step's guard regions before anything runs
    for (size_t o : c->guards) c->note(cudaMemsetAsync(c->arena + o, kGuardByte, kGuardBytes, c->st));
  // the group's tensors, for the completion-ordered chunks of its gradient
  c->planner.reset(act.grad_numel, c->chunk_min_elems);
  c->planner_idx.assign(c->tens.size(), -1);
  c->chunks.clear();
  for (int gi : act.groups)
    for (int u = c->groups[gi].unit_lo; u <= c->groups[gi].unit_hi; ++u)
      for (int ti : c->unit_tens[u]) c->planner_idx[ti] = c->planner.add(c->grad_off[ti], c->tens[ti].numel);
  // inputs produced on the caller's stream are visible to the step
  c->note(cudaEventRecord(c->ev_in, c->caller));
  c->note(cudaStreamWaitEvent(c->st, c->ev_in, 0));
  c->note(cudaEventRecord(c->tl[0], c->st));

  if (c->offload && c->oc.prefetch_groups) page_in_ahead(c);

  // "Clear gradients": the group's span of the gradient buffer starts at zero
  c->note(cudaMemsetAsync(c->grad, 0, act.grad_numel * c->ges, c->st));
  c->note(cudaMemsetAsync(c->scal, 0, kScalWords * sizeof(float), c->st));
  int* bad = (int*)(c->scal + 2);
  int* nvalid = (int*)(c->scal + 1);

  // ---------------- forward (Algorithm 1, step h)
  std::vector<float*> chain_r(L + 1);
  std::vector<char*> chain_a(L + 1, nullptr);
  for (int i = 0; i < L; ++i) { chain_r[i] = (float*)c->slots[i][S_XIN]; chain_a[i] = c->slots[i][S_XINA]; }
  chain_r[L] = c->x_final; chain_a[L] = c->x_final_a;
  {
    float* x0 = m.arch == 1 ? c->emb_e : chain_r[0];
    LAUNCH(HIFT_K_EMBED, (double)T * d * (c->es * (c->t_pos >= 0 ? 2 : 1) + 4),
           if (c->mixed) embed_fwd_kernel<bf16><<<T, norm_threads(d), 0, c->st>>>(tok, (const bf16*)c->P(c->t_tok), (const bf16*)c->Pn(c->t_pos), x0, S, d, V, bad);
           else embed_fwd_kernel<float><<<T, norm_threads(d), 0, c->st>>>(tok, (const float*)c->P(c->t_tok), (const float*)c->Pn(c->t_pos), x0, S, d, V, bad));
    if (m.arch == 1) norm_fwd(c, c->emb_e, c->t_eg, c->t_eb, chain_a[0], chain_r[0], c->st_e);
    if (c->drop_on) drop_inplace(c, 0, chain_r[0], m.arch == 1 ? chain_a[0] : nullptr);
  }
  for (int i = 0; i < L; ++i) forward_block(c, i, chain_r[i], chain_a[i], chain_r[i + 1], chain_a[i + 1]);
  if (m.arch == 1) {
    const int C = m.n_classes;
    // pooled = first token of every sequence: rows of the last block's output with stride S*d
    linear_fwd(c, B, C, d, c->x_final_a, (int64_t)S * d, c->P(c->t_wc), c->logits, C, c->P(c->t_bc), nullptr, 0, false);
    LAUNCH(HIFT_K_CE, 2.0 * B * C * c->es,
           launch_cross_entropy(c->st, c->mixed, B, C, C, c->logits, lab, c->rowloss, nvalid, bad, c->scal));
    c->step_launches += 2;
  } else {
    norm_fwd(c, c->x_final, c->t_fg, c->t_fb, c->xf, nullptr, c->stf);
    const int tw = m.tie_head ? c->t_tok : c->t_wh;
    linear_fwd(c, T, V, d, c->xf, d, c->P(tw), c->logits, Vp, nullptr, nullptr, 0, false);
    LAUNCH(HIFT_K_CE, 2.0 * T * (double)Vp * c->es,       // one read of the logits, one write of their gradient
           launch_cross_entropy(c->st, c->mixed, T, V, Vp, c->logits, lab, c->rowloss, nvalid, bad, c->scal));
    c->step_launches += 2;
  }
  if (c->offload && !c->oc.prefetch_groups) {
    // the paper's order: optimizer state moves to the GPU after the forward pass (step i)
    c->note(cudaEventRecord(c->ev_fwd, c->st));
    c->cur_sl = acquire_slot(c, g, c->t, true);
  }

  // ---------------- backward, truncated at the group ("Backpropagation")
  const bool head_on = active(L + 1);
  bool done = false;
  if (m.arch == 1) {
    const int C = m.n_classes;
    if (head_on) {
      // dWc[C,d] = dlogits^T pooled ; pooled rows have stride S*d
      gemm(c, HIFT_K_GEMM_DW, C, d, B, c->logits, 1, C, c->x_final_a, (int64_t)S * d, 1, c->G(c->t_wc), d, nullptr, nullptr, 0, !c->gbf);
      bias_grad(c, c->logits, false, B, C, C, c->t_bc);
      grad_done(c, c->t_bc); grad_done(c, c->t_wc);
    }
    if (lo == L + 1) done = true;
    else {
      c->note(cudaMemsetAsync(c->dxa, 0, (size_t)T * d * sizeof(float), c->st));
      // dx[b*S,:] = dlogits[b,:] Wc
      gemm(c, HIFT_K_GEMM_DX, B, d, C, c->logits, C, 1, c->P(c->t_wc), d, 1, c->dxa, (int64_t)S * d, nullptr, nullptr, 0, true);
    }
  } else {
    const int tw = m.tie_head ? c->t_tok : c->t_wh;
    const bool w_on = m.tie_head ? active(0) : head_on;
    if (w_on) linear_dw(c, T, V, d, c->logits, Vp, c->xf, d, c->G(tw));
    if (w_on && !m.tie_head) grad_done(c, tw);          // a tied matrix still gets the embedding's share
    linear_dx(c, T, V, d, c->logits, Vp, c->P(tw), c->dt1, d, nullptr, 0, false);
    if (head_on) { norm_bwd_params(c, c->dt1, false, c->x_final, c->stf, c->t_fg, c->t_fb); grad_done(c, c->t_fb); grad_done(c, c->t_fg); }
    if (lo == L + 1) done = true;
    else norm_bwd_dx(c, c->dt1, false, c->x_final, c->stf, c->t_fg, nullptr, c->dxa, c->dxa_a);
  }
  if (!done) {
    for (int i = L - 1; i >= 0; --i) {
      const int u = i + 1;
      if (u < lo) break;
      if (c->recompute && !active(u)) {
        // redo this frozen block's forward from its kept input into the scratch slots (its output goes nowhere)
        c->keep_all = true;
        forward_block(c, i, chain_r[i], chain_a[i], c->pp[0], c->ppa[0]);
        c->keep_all = false;
      }
      backward_block(c, i, chain_r[i], chain_a[i], active(u), u > lo);
      if (u == lo) break;
    }
  }
  if (active(0)) {
    const float* src = c->dxa;
    if (c->drop_on) drop_inplace(c, 0, c->dxa, nullptr);      // back through the dropout of the embedding output
    if (m.arch == 1) {
      norm_bwd_params(c, c->dxa, true, c->emb_e, c->st_e, c->t_eg, c->t_eb);
      grad_done(c, c->t_eb); grad_done(c, c->t_eg);
      norm_bwd_dx(c, c->dxa, true, c->emb_e, c->st_e, c->t_eg, nullptr, c->dxb, nullptr);
      src = c->dxb;
    }
    LAUNCH(HIFT_K_EMBED, (double)T * d * 12,
           embed_bwd_tok_kernel<<<T, 128, 0, c->st>>>(tok, src, c->G(c->t_tok), c->gbf, T, d, V));
    if (c->t_pos >= 0) {
      LAUNCH(HIFT_K_EMBED, (double)T * d * 4 + (double)S * d * 4,
             embed_bwd_pos_kernel<<<S, 128, 0, c->st>>>(src, c->G(c->t_pos), c->gbf, B, S, d));
      grad_done(c, c->t_pos);
    }
    grad_done(c, c->t_tok);
  }
  {
    size_t off, n;
    if (c->planner.flush(&off, &n)) emit_chunk(c, off, n);
  }
  // the gate word of this step's update: set once the whole pass is behind it, before the last chunk is released
  step_gate_kernel<<<1, 32, 0, c->st>>>(c->scal, c->mixed ? gemm_tc_error_device_ptr() : nullptr, c->gate);
  c->note(cudaGetLastError());
  c->note(cudaEventRecord(c->ev_bwd, c->st));
  return HIFT_OK;
}

// Optimizer on the active group and write-back of its state, enqueued after the backward pass.
// The optimizer kernels read the step's gate word and leave every buffer as it is when the step
// failed (a bounded wait gave up, a token or label was out of range, the loss is not finite).
void enqueue_update(hift_ctx* c) {
  const ActiveSet& act = c->act;
  const int sl = c->cur_sl;
  SlotRec* sr = c->offload ? &c->slot[sl] : nullptr;
  const double lr = c->cur_lr;
  if (c->offload) {
    c->note(cudaEventRecord(c->tl[3], c->st));
    c->note(cudaStreamWaitEvent(c->st, sr->ev_h2d, 0));
    // a group still resident from an earlier step: its write-back reads what is about to change
    if (sr->d2h_pending) c->note(cudaStreamWaitEvent(c->st, sr->ev_d2h, 0));
    c->note(cudaEventRecord(c->tl[4], c->st));
  }
  // ---------------- group-local optimizer (Algorithm 1: P now points at theta_s only); one pass per state group
  for (size_t gi = 0; gi < act.groups.size(); ++gi) {
    GroupRec& gr = c->groups[act.groups[gi]];
    char* slot_mem = c->offload ? sr->mem + act.slot_base[gi] : nullptr;      // this group's planes in the slot
    const char* grad_g = (const char*)c->grad + act.grad_base[gi] * c->ges;  // and its span of the gradient buffer
    gr.tau += 1;
    if (c->af) {
      // Adafactor works tensor by tensor (its statistics are per row and column of each matrix)
      float* base = (float*)slot_mem;
      for (int u = gr.unit_lo; u <= gr.unit_hi; ++u)
        for (int ti : c->unit_tens[u]) {
          const TensorRec& r = c->tens[ti];
          float* mst_t;
          if (!c->mixed) mst_t = (float*)c->params + r.off;
          else mst_t = c->offload ? base + (r.off - gr.off) : c->master_all + r.off;
          float* st_t = c->offload ? base + (c->mixed ? gr.numel : 0) + r.af_off : c->af_all + gr.af_base + r.af_off;
          c->pre(HIFT_K_OPT, (double)r.numel * (20.0 + (c->mixed ? 2.0 : 0.0)));
          const int nk = launch_adafactor_tensor(c->st, r.rows, r.cols, c->mixed ? c->P(ti) : nullptr, mst_t, (const float*)c->G(ti), st_t,
                                                 c->af_scratch, lr, c->oc.eps, c->oc.weight_decay, gr.tau, c->gate);
          c->post();
          c->step_launches += nk - 1;
        }
      continue;
    }
    float *mst, *s0, *s1;
    void* pbf = nullptr;
    // the range of the group whose master / state this rank holds and updates (all of it unless sharded)
    const size_t o0 = gr.off + gr.own_lo, on = gr.own_n;
    const void* gsrc = grad_g + gr.own_lo * c->ges;
    if (c->offload) {
      float* base = (float*)slot_mem;
      if (c->compact) { mst = nullptr; s0 = base; s1 = base + on; pbf = c->params + o0 * c->es; }
      else if (c->mixed) { mst = base; s0 = base + on; s1 = base + 2 * on; pbf = c->params + o0 * c->es; }
      else { mst = (float*)c->params + o0; s0 = base; s1 = base + on; }
    } else {
      if (c->mixed) { mst = c->master_all + o0; pbf = c->params + o0 * c->es; }
      else mst = (float*)c->params + o0;
      s0 = c->s0_all ? c->s0_all + o0 : nullptr;
      s1 = c->s1_all ? c->s1_all + o0 : nullptr;
    }
    const OptScalars hs = make_opt_scalars(c->oc.kind, lr, c->oc.beta1, c->oc.beta2, c->oc.eps,
                                           c->oc.weight_decay, c->oc.momentum, gr.tau);
    if (c->compact) {
      // read p, lo, carry, gradient, state; write p, lo, carry, state
      const double opt_bytes = (double)on * (8.25 + c->ges + 8.0 * c->n_state);
      uint16_t* lo16 = (uint16_t*)((float*)slot_mem + gr.state_floats);
      uint8_t* carry8 = (uint8_t*)(lo16 + on);
      LAUNCH(HIFT_K_OPT, opt_bytes, launch_fused_opt_compact(c->st, c->oc.kind, on, pbf, lo16, carry8, gsrc, s0, s1, hs, c->gate, c->gbf));
    } else {
      const double opt_bytes = (double)on * ((c->oc.kind == 0 ? 24.0 : (c->oc.kind == 3 ? 8.0 : 16.0)) + c->ges + (pbf ? 2.0 : 0.0));
      LAUNCH(HIFT_K_OPT, opt_bytes, launch_fused_opt(c->st, c->oc.kind, on, pbf, mst, gsrc, s0, s1, hs, c->gate, c->gbf));
    }
  }

  // ---------------- state back to the host (step k)
  if (c->offload) {
    c->note(cudaEventRecord(sr->ev_opt, c->st));
    c->note(cudaStreamWaitEvent(c->st_d2h, sr->ev_opt, 0));
    c->note(cudaEventRecord(c->tl[5], c->st_d2h));
    c->step_d2h = 0;
    for (size_t gi = 0; gi < act.groups.size(); ++gi) {
      GroupRec& gr = c->groups[act.groups[gi]];
      if (gr.blob_bytes) c->note(cudaMemcpyAsync(gr.blob, sr->mem + act.slot_base[gi], gr.blob_bytes, cudaMemcpyDeviceToHost, c->st_d2h));
      c->step_d2h += gr.blob_bytes;
    }
    c->note(cudaEventRecord(c->tl[6], c->st_d2h));
    c->note(cudaEventRecord(sr->ev_d2h, c->st_d2h));
    c->tl_valid = true;
    sr->d2h_pending = true;
  }
}

// Publishes the step's scalars, waits for the compute stream, and turns what it finds into a status.
// `updated`: the optimizer was enqueued too, so the published gate word says whether it ran.
hift_status finish_step(hift_ctx* c, float* loss_host, bool updated) {
  // the loss goes to mapped host memory by a kernel store: a copy would queue behind the state transfers
  publish_scalars_kernel<<<1, 32, 0, c->st>>>(c->scal, c->mixed ? gemm_tc_error_device_ptr() : nullptr, c->scal_host_dev);
  c->note(cudaGetLastError());
  c->note(cudaStreamSynchronize(c->st));
  c->prof_collect();
  if (c->first_err != cudaSuccess) return HIFT_ERR_CUDA;
  int tc_err, bad_h, gate_h;
  memcpy(&tc_err, &c->scal_host[3], sizeof(int));
  memcpy(&bad_h, &c->scal_host[2], sizeof(int));
  memcpy(&gate_h, &c->scal_host[4], sizeof(int));
  const float loss = c->scal_host[0];
  if (tc_err != 0) return HIFT_ERR_TIMEOUT;
  if (loss_host) *loss_host = loss;
  if (bad_h) return HIFT_ERR_INPUT;
  if (!isfinite(loss)) return HIFT_ERR_NONFINITE;
  if (updated && gate_h != 0)      // nothing wrong here, yet the update was called off: a peer's step failed
    return gate_h == 100 ? HIFT_ERR_INPUT : (gate_h == 101 ? HIFT_ERR_NONFINITE : HIFT_ERR_TIMEOUT);
  return HIFT_OK;
}
// A step that failed changed nothing on the device (the gate kept the optimizer out, the write-back
// carried unchanged bytes): take back the update count; t stays, so the same group is next.
void step_failed(hift_ctx* c) {
  for (int g : c->act.groups) if (c->groups[g].tau > 0) c->groups[g].tau -= 1;
}

hift_status do_step(hift_ctx* c, const int32_t* tok, const int32_t* lab, float* loss_host) {
  if (c->pending_update) return HIFT_ERR_CFG;       // hift_step_begin without hift_step_end
  hift_status s = enqueue_forward_backward(c, tok, lab);
  if (s != HIFT_OK) return s;
  enqueue_update(c);
  s = finish_step(c, loss_host, true);
  if (s == HIFT_OK) c->t += 1;     // the learning rate is a function of t / k: it moves once per full cycle
  else step_failed(c);
  return s;
}

void sync_all(hift_ctx* c) {
  if (c->st) cudaStreamSynchronize(c->st);
  if (c->st_h2d) cudaStreamSynchronize(c->st_h2d);
  if (c->st_d2h) cudaStreamSynchronize(c->st_d2h);
}

int group_of_unit(const hift_ctx* c, int u) {
  for (size_t g = 0; g < c->groups.size(); ++g)
    if (u >= c->groups[g].unit_lo && u <= c->groups[g].unit_hi) return (int)g;
  return -1;
}
// The part of tensor ti whose master / state this rank holds: tensor elements [t_lo, t_lo + n), found at
// index p of the group's planes (everything unless the optimizer state is sharded over ranks).
struct OwnPart { size_t t_lo, n, p; };
OwnPart own_part(const hift_ctx* c, int ti) {
  const TensorRec& r = c->tens[ti];
  const GroupRec& gr = c->groups[group_of_unit(c, r.unit)];
  const size_t a = r.off - gr.off, b = a + r.numel;
  const size_t lo = std::max(a, gr.own_lo), hi = std::min(b, gr.own_lo + gr.own_n);
  if (hi <= lo) return OwnPart{0, 0, 0};
  return OwnPart{lo - a, hi - lo, lo - gr.own_lo};
}
// start of the fp32 master / state plane `plane` (0 master, 1 s0, 2 s1) of the group's held range
float* plane_base(hift_ctx* c, const GroupRec& gr, int plane, bool* on_host) {
  *on_host = false;
  if (plane == 0 && !c->mixed) return (float*)c->params + gr.off + gr.own_lo;
  if (c->offload) {
    *on_host = true;
    if (c->compact && plane == 0) return nullptr;        // not stored as floats: see master_read / master_write
    const int pl = (c->mixed && !c->compact) ? plane : plane - 1;
    return (float*)gr.blob + (size_t)pl * gr.own_n;
  }
  float* all = plane == 0 ? c->master_all : (plane == 1 ? c->s0_all : c->s1_all);
  return all ? all + gr.off + gr.own_lo : nullptr;
}

// ---- compact master on the host side (same arithmetic as master_pack / master_unpack on the device)
inline void host_master_pack(uint32_t u, uint32_t& p, uint32_t& lo, uint32_t& carry) {
  lo = u & 0xFFFFu;
  if ((u & 0x7F800000u) == 0x7F800000u) {
    p = u >> 16;
    if (lo && !(p & 0x7Fu)) p |= 0x40u;
    carry = 0;
  } else {
    p = (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
    carry = p - (u >> 16);
  }
}
uint16_t* blob_lo16(const hift_ctx* c, const GroupRec& gr) { (void)c; return (uint16_t*)((float*)gr.blob + gr.state_floats); }
uint8_t* blob_carry8(const hift_ctx* c, const GroupRec& gr) { return (uint8_t*)(blob_lo16(c, gr) + gr.own_n); }
// fp32 master values of elements [o, o + n) of a group (inside the range this rank holds), rebuilt from the
// device's bf16 copy and the blob
bool master_read(hift_ctx* c, const GroupRec& gr, size_t o, size_t n, float* dst) {
  std::vector<uint16_t> p(n);
  if (cudaMemcpy(p.data(), c->params + (gr.off + o) * c->es, n * 2, cudaMemcpyDeviceToHost) != cudaSuccess) return false;
  const size_t q = o - gr.own_lo;                      // index in the blob's planes
  const uint16_t* lo = blob_lo16(c, gr) + q;
  const uint8_t* cr = blob_carry8(c, gr);
  for (size_t i = 0; i < n; ++i) {
    const uint32_t carry = (cr[(q + i) >> 3] >> ((q + i) & 7)) & 1u;
    const uint32_t u = (((uint32_t)p[i] - carry) << 16) | lo[i];
    memcpy(dst + i, &u, 4);
  }
  return true;
}
// the blob's share of new master values (the bf16 copy on the device is the caller's job)
void master_write(hift_ctx* c, GroupRec& gr, size_t o, size_t n, const float* src) {
  const size_t q = o - gr.own_lo;
  uint16_t* lo = blob_lo16(c, gr) + q;
  uint8_t* cr = blob_carry8(c, gr);
  for (size_t i = 0; i < n; ++i) {
    uint32_t u, p, l, carry;
    memcpy(&u, src + i, 4);
    host_master_pack(u, p, l, carry);
    lo[i] = (uint16_t)l;
    uint8_t& byte = cr[(q + i) >> 3];
    byte = (uint8_t)((byte & ~(1u << ((q + i) & 7))) | (carry << ((q + i) & 7)));
  }
}

// fp32 staging of up to max_group elements for the set-up calls: the gradient buffer itself, unless gradients are
// kept in bf16 (then it is half the size and a buffer of its own is allocated, and released when training starts)
float* staging(hift_ctx* c) {
  if (!c->gbf) return c->grad;
  if (!c->stage && cudaMalloc((void**)&c->stage, c->max_group * sizeof(float)) != cudaSuccess) { cudaGetLastError(); c->stage = nullptr; }
  return c->stage;
}

}  // namespace

// ====================================================================== C entry points
extern "C" {

const char* hift_strerror(hift_status s) {
  switch (s) {
    case HIFT_OK: return "ok";
    case HIFT_ERR_CFG: return "invalid or unsupported configuration";
    case HIFT_ERR_OOM_DEVICE: return "out of device memory";
    case HIFT_ERR_OOM_PINNED: return "out of pinned host memory";
    case HIFT_ERR_INPUT: return "invalid input (token id / label out of range or NULL pointer)";
    case HIFT_ERR_NONFINITE: return "non-finite loss";
    case HIFT_ERR_TIMEOUT: return "device-side wait timed out";
    case HIFT_ERR_CUDA: return "CUDA error";
    case HIFT_ERR_CAPACITY: return "size exceeds the library's built-in scratch capacity";
  }
  return "unknown";
}

void hift_destroy(hift_ctx* c) {
  if (!c) return;
  sync_all(c);
  for (void* p : c->dev_allocs) cudaFree(p);
  if (c->stage) cudaFree(c->stage);
  for (auto& g : c->groups) if (g.blob) cudaFreeHost(g.blob);
  if (c->scal_host) cudaFreeHost(c->scal_host);
  for (auto e : c->ev_pool) cudaEventDestroy(e);
  for (auto e : c->chunk_events) cudaEventDestroy(e);
  if (c->events_made) {
    for (int i = 0; i < kMaxSlots; ++i) {
      SlotRec& sr = c->slot[i];
      cudaEventDestroy(sr.ev_h2d); cudaEventDestroy(sr.ev_opt); cudaEventDestroy(sr.ev_d2h);
      cudaEventDestroy(sr.tl_h2d0); cudaEventDestroy(sr.tl_h2d1);
    }
    cudaEventDestroy(c->ev_fwd);
    cudaEventDestroy(c->ev_bwd);
    cudaEventDestroy(c->ev_in);
    for (int i = 0; i < 7; ++i) cudaEventDestroy(c->tl[i]);
  }
  if (c->st) cudaStreamDestroy(c->st);
  if (c->st_h2d) cudaStreamDestroy(c->st_h2d);
  if (c->st_d2h) cudaStreamDestroy(c->st_d2h);
  delete c;
}

hift_status hift_create(const hift_model_cfg* m, const hift_group_cfg* gc, const hift_opt_cfg* oc,
                        void* cuda_stream, hift_ctx** out) {
  if (!out) return HIFT_ERR_CFG;
  *out = nullptr;
  if (!m || !gc || !oc) return HIFT_ERR_CFG;
  // ---- validation
  if (m->arch < 0 || m->arch > 2 || m->n_blocks < 1 || m->d_model < 8 || m->n_heads < 1 ||
      m->d_ffn < 8 || m->vocab < 2 || m->batch < 1 || m->seq < 1)
    return HIFT_ERR_CFG;
  if (m->d_model % 8 || m->d_ffn % 8 || m->d_model % m->n_heads) return HIFT_ERR_CFG;
  if (!attention_head_ok(m->d_model / m->n_heads)) return HIFT_ERR_CFG;
  if (m->arch == 2 && (m->d_model / m->n_heads) % 16) return HIFT_ERR_CFG;   // RoPE rotates 8 pairs per thread
  if (m->dtype != 0 && m->dtype != 1) return HIFT_ERR_CFG;
  if (!(m->dropout >= 0.0 && m->dropout < 1.0)) return HIFT_ERR_CFG;
  if (!(m->attn_dropout >= 0.0 && m->attn_dropout < 1.0)) return HIFT_ERR_CFG;
  if (m->arch != 2 && m->max_pos < m->seq) return HIFT_ERR_CFG;
  if (m->arch == 1 && (m->n_classes < 2 || m->tie_head)) return HIFT_ERR_CFG;
  // several kernels launch one block per token, and the attention grids put the batch on z
  if ((int64_t)m->batch * m->seq > 65536 || m->batch > 65535) return HIFT_ERR_CFG;
  if (gc->layers_per_group < 1 || gc->order < 0 || gc->order > 2) return HIFT_ERR_CFG;
  if (gc->group_sizes != nullptr) {
    if (gc->n_group_sizes < 1) return HIFT_ERR_CFG;
    int64_t sum = 0;
    for (int i = 0; i < gc->n_group_sizes; ++i) {
      if (gc->group_sizes[i] < 1) return HIFT_ERR_CFG;
      sum += gc->group_sizes[i];
    }
    if (sum != (int64_t)m->n_blocks + 2) return HIFT_ERR_CFG;
  }
  if (oc->kind < 0 || oc->kind > 4 || oc->sched < 0 || oc->sched > 1) return HIFT_ERR_CFG;
  if (oc->prefetch_groups < 0 || oc->prefetch_groups > kMaxSlots - 1) return HIFT_ERR_CFG;
  if (oc->shard_world > 1 && (oc->shard_rank < 0 || oc->shard_rank >= oc->shard_world || oc->kind == 4)) return HIFT_ERR_CFG;
  if (oc->grad_bf16 != 0 && (m->dtype != 1 || oc->kind == 4)) return HIFT_ERR_CFG;      // bf16 gradients: bf16 model, fused optimizers
  if (gc->literal_queue != 0 && (gc->group_sizes != nullptr || gc->split_emb_head || oc->shard_world > 1)) return HIFT_ERR_CFG;
  if (oc->sched == 1 && (oc->total_cycles < 1 || oc->warmup_cycles < 0 || oc->warmup_cycles >= oc->total_cycles)) return HIFT_ERR_CFG;
  if (!(oc->lr >= 0.0)) return HIFT_ERR_CFG;

  hift_ctx* c = new hift_ctx();
  c->m = *m; c->gc = *gc; c->oc = *oc;
  if (gc->group_sizes != nullptr) c->group_sizes.assign(gc->group_sizes, gc->group_sizes + gc->n_group_sizes);
  c->gc.group_sizes = nullptr; c->gc.n_group_sizes = 0;   // the caller's array is not kept
  c->caller = (cudaStream_t)cuda_stream;
  c->mixed = m->dtype == 1;
  c->es = c->mixed ? 2 : 4;
  c->L = m->n_blocks; c->d = m->d_model; c->f = m->d_ffn; c->fa = m->arch == 2 ? 2 * m->d_ffn : m->d_ffn;
  c->H = m->n_heads; c->dh = m->d_model / m->n_heads; c->B = m->batch; c->S = m->seq; c->T = m->batch * m->seq;
  c->V = m->vocab; c->Vp = (int)align_up(m->vocab, 128);
  c->af = oc->kind == 4;
  c->n_state = oc->kind == 0 ? 2 : (oc->kind >= 3 ? 0 : 1);
  // plain SGD on fp32 parameters has nothing to page (the paper's "no state, zero traffic" case)
  c->offload = oc->offload_state != 0 && ((m->dtype == 1 ? 1 : 0) + c->n_state + (c->af ? 1 : 0)) > 0;
  // prefetch_groups p: 0 = one slot, upload after the forward pass; 1 = two slots, upload at the start of
  // the group's own step; p >= 2 = p + 1 slots, uploads issued p - 1 steps ahead
  c->n_slots = c->offload ? 1 + oc->prefetch_groups : 1;
  c->lookahead = c->offload && oc->prefetch_groups >= 2 ? oc->prefetch_groups - 1 : 0;
  const bool drifting = gc->literal_queue != 0 && (m->n_blocks + 2) % gc->layers_per_group != 0 && gc->layers_per_group < m->n_blocks + 2;
  // drifting sets share units with one another: one slot, so that an upload always follows the last write-back
  if (drifting) { c->n_slots = 1; c->lookahead = 0; }
  // bf16 parameters + a fused optimizer: page 17 bits of master per element instead of 32
  c->compact = c->mixed && c->offload && !c->af;
  c->recompute = oc->recompute != 0;
  c->gbf = oc->grad_bf16 != 0;
  c->ges = c->gbf ? 2 : 4;
  c->drop_on = m->dropout > 0.0;
  c->drop_thr = (uint32_t)floor(m->dropout * 4294967296.0);
  c->drop_scale = (float)(1.0 / (1.0 - m->dropout));
  c->adrop_thr = (uint32_t)floor(m->attn_dropout * 4294967296.0);
  c->adrop_scale = (float)(1.0 / (1.0 - m->attn_dropout));
  c->checked = g_checked_arena != 0;
  memset(c->prof_launches, 0, sizeof(c->prof_launches));
  memset(c->prof_ms, 0, sizeof(c->prof_ms));
  memset(c->prof_work, 0, sizeof(c->prof_work));
  // the literal queue only differs from the fixed partition when m does not divide n
  c->queue = gc->literal_queue != 0 && gc->group_sizes == nullptr && !gc->split_emb_head &&
             (m->n_blocks + 2) % gc->layers_per_group != 0 && gc->layers_per_group < m->n_blocks + 2;
  build_layout(c);
  c->shard_world = oc->shard_world > 1 ? oc->shard_world : 1;
  c->shard_rank = c->shard_world > 1 ? oc->shard_rank : 0;
  {
    size_t base = 0;
    for (auto& g : c->groups) {
      // the contiguous piece of the group whose master and state this rank holds: pieces of whole 128-element lines
      const size_t piece = align_up((g.numel + c->shard_world - 1) / c->shard_world, kAlignElems);
      g.own_lo = std::min((size_t)c->shard_rank * piece, g.numel);
      g.own_n = std::min(piece, g.numel - g.own_lo);
      g.state_floats = (size_t)c->n_state * g.own_n;
      if (c->af) {
        size_t o = 0;
        for (int u = g.unit_lo; u <= g.unit_hi; ++u)
          for (int ti : c->unit_tens[u]) {
            c->tens[ti].af_off = o;
            o = align_up(o + af_state_floats(c->tens[ti].rows, c->tens[ti].cols), 4);
          }
        g.state_floats = o;
        g.af_base = base;
        base += o;
      }
    }
  }

  hift_status rc = HIFT_OK;
  auto fail = [&](hift_status s) { hift_destroy(c); return s; };
  for (int i = 0; i < kMaxSlots; ++i) {
    SlotRec& sr = c->slot[i];
    cudaEventCreateWithFlags(&sr.ev_h2d, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&sr.ev_opt, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&sr.ev_d2h, cudaEventDisableTiming);
    cudaEventCreate(&sr.tl_h2d0);
    cudaEventCreate(&sr.tl_h2d1);
  }
  cudaEventCreateWithFlags(&c->ev_fwd, cudaEventDisableTiming);
  cudaEventCreateWithFlags(&c->ev_bwd, cudaEventDisableTiming);
  for (int i = 0; i < 7; ++i) cudaEventCreate(&c->tl[i]);
  c->events_made = true;
  cudaEventCreateWithFlags(&c->ev_in, cudaEventDisableTiming);
  // The step runs on a stream of its own: work in the legacy default stream would order itself after
  // the state transfers still in flight from the previous step.
  if (cudaStreamCreateWithFlags(&c->st, cudaStreamNonBlocking) != cudaSuccess) return fail(HIFT_ERR_CUDA);
  if (cudaStreamCreateWithFlags(&c->st_h2d, cudaStreamNonBlocking) != cudaSuccess) return fail(HIFT_ERR_CUDA);
  if (cudaStreamCreateWithFlags(&c->st_d2h, cudaStreamNonBlocking) != cudaSuccess) return fail(HIFT_ERR_CUDA);

  // ---- parameters, gradients, optimizer state
  auto blob_bytes_of = [&](const GroupRec& g) {
    if (c->compact) return g.state_floats * sizeof(float) + g.own_n * 2 + g.own_n / 8;     // own_n is a multiple of 128
    return ((c->mixed ? g.own_n : 0) + g.state_floats) * sizeof(float);
  };
  size_t slot_bytes_max = 0, af_total = 0, grad_max = c->max_group;
  for (auto& g : c->groups) { g.blob_bytes = c->offload ? blob_bytes_of(g) : 0; af_total += c->af ? g.state_floats : 0; }
  for (int sid = 0; sid < c->n_sets; ++sid) {       // the largest set decides the gradient buffer and the state slots
    ActiveSet a;
    fill_set(c, sid, &a);
    slot_bytes_max = std::max(slot_bytes_max, a.slot_bytes);
    grad_max = std::max(grad_max, a.grad_numel);
  }
  if ((rc = dev_alloc(c, (void**)&c->params, c->total * c->es)) != HIFT_OK) return fail(rc);
  cudaMemsetAsync(c->params, 0, c->total * c->es, c->st);
  if ((rc = dev_alloc(c, (void**)&c->grad, grad_max * c->ges)) != HIFT_OK) return fail(rc);
  if (c->offload) {
    for (int s = 0; s < c->n_slots; ++s) {
      if ((rc = dev_alloc(c, (void**)&c->slot[s].mem, slot_bytes_max)) != HIFT_OK) return fail(rc);
      cudaMemsetAsync(c->slot[s].mem, 0, slot_bytes_max, c->st);
    }
    for (auto& g : c->groups) {
      if (pinned_alloc((void**)&g.blob, g.blob_bytes ? g.blob_bytes : 256, cudaHostAllocDefault) != cudaSuccess) {
        cudaGetLastError();
        g.blob = nullptr;
        return fail(HIFT_ERR_OOM_PINNED);
      }
      memset(g.blob, 0, g.blob_bytes);
      c->pinned_bytes += g.blob_bytes;
    }
  } else {
    if (c->mixed) {
      if ((rc = dev_alloc(c, (void**)&c->master_all, c->total * sizeof(float))) != HIFT_OK) return fail(rc);
      cudaMemsetAsync(c->master_all, 0, c->total * sizeof(float), c->st);
    }
    if (c->n_state >= 1) {
      if ((rc = dev_alloc(c, (void**)&c->s0_all, c->total * sizeof(float))) != HIFT_OK) return fail(rc);
      cudaMemsetAsync(c->s0_all, 0, c->total * sizeof(float), c->st);
    }
    if (c->n_state == 2) {
      if ((rc = dev_alloc(c, (void**)&c->s1_all, c->total * sizeof(float))) != HIFT_OK) return fail(rc);
      cudaMemsetAsync(c->s1_all, 0, c->total * sizeof(float), c->st);
    }
    if (c->af) {
      if ((rc = dev_alloc(c, (void**)&c->af_all, af_total * sizeof(float))) != HIFT_OK) return fail(rc);
      cudaMemsetAsync(c->af_all, 0, af_total * sizeof(float), c->st);
    }
  }
  if (c->af) {
    size_t mx = 0;
    for (auto& r : c->tens) mx = std::max(mx, af_scratch_floats(r.rows, r.cols));
    if ((rc = dev_alloc(c, (void**)&c->af_scratch, mx * sizeof(float))) != HIFT_OK) return fail(rc);
  }
  // four scalars the step publishes, then a staging row for the key-length table
  if (pinned_alloc((void**)&c->scal_host, (kScalWords + (size_t)c->B) * sizeof(float), cudaHostAllocMapped) != cudaSuccess) { cudaGetLastError(); c->scal_host = nullptr; return fail(HIFT_ERR_OOM_PINNED); }
  if (cudaHostGetDevicePointer((void**)&c->scal_host_dev, c->scal_host, 0) != cudaSuccess) return fail(HIFT_ERR_CUDA);

  // ---- activation arena: fixed work buffers, one scratch copy of every slot, then the
  //      per-group kept activations (sized for the worst group)
  const size_t T = c->T, d = c->d, es = c->es;
  c->slots.assign(c->L + 1, std::vector<char*>(S_NUM, nullptr));
  for (int pass = 0; pass < 2; ++pass) {
    c->arena_off = 0;
    c->guards.clear();
    c->record_guards = c->checked && pass == 1;
    c->tok_dev = (int32_t*)arena_take(c, T * sizeof(int32_t));
    c->lab_dev = (int32_t*)arena_take(c, T * sizeof(int32_t));
    c->lens_dev = (int32_t*)arena_take(c, (size_t)c->B * sizeof(int32_t));
    c->dxa = (float*)arena_take(c, T * d * 4); c->dxb = (float*)arena_take(c, T * d * 4);
    c->dxa_a = arena_take(c, T * d * es); c->dxb_a = arena_take(c, T * d * es); c->dt1 = arena_take(c, T * d * es);
    c->dqkv = arena_take(c, T * 3 * d * es);
    c->dbig = arena_take(c, T * (size_t)c->fa * es);
    c->dsw = m->arch == 2 ? arena_take(c, T * (size_t)c->f * es) : nullptr;
    c->x_final = (float*)arena_take(c, T * d * 4);
    c->pp[0] = (float*)arena_take(c, T * d * 4); c->pp[1] = (float*)arena_take(c, T * d * 4);
    if (m->arch == 1) {
      c->x_final_a = arena_take(c, T * d * es);
      c->ppa[0] = arena_take(c, T * d * es); c->ppa[1] = arena_take(c, T * d * es);
      c->emb_e = (float*)arena_take(c, T * d * 4);
      c->st_e = (float*)arena_take(c, 2 * T * sizeof(float));
      c->logits = arena_take(c, (size_t)c->B * m->n_classes * es);
    } else {
      c->xf = arena_take(c, T * d * es);
      c->stf = (float*)arena_take(c, 2 * T * sizeof(float));
      c->logits = arena_take(c, T * (size_t)c->Vp * es);
    }
    c->dsum = (float*)arena_take(c, T * c->H * sizeof(float));
    const size_t maxcols = std::max<size_t>(std::max<size_t>(3 * d, c->fa), 8);
    c->partial = (float*)arena_take(c, 2 * kColChunks * maxcols * sizeof(float));
    c->rowloss = (float*)arena_take(c, T * sizeof(float));
    c->scal = (float*)arena_take(c, kScalWords * sizeof(float));
    c->gate = (int*)(c->scal + 4);
    if (m->arch == 2) c->rope_cs = (float*)arena_take(c, 2 * (size_t)c->S * (c->dh / 2) * sizeof(float));
    for (int s = 0; s < S_NUM; ++s)
      c->slots[c->L][s] = (slot_min_level(m->arch, s) == 99 || s == S_XIN || s == S_XINA)
                              ? nullptr : arena_take(c, slot_bytes(c, s));
    c->arena_fixed = c->arena_off;
    c->record_guards = false;
    c->n_fixed_guards = c->guards.size();
    if (pass == 0) {
      size_t worst = c->arena_fixed;
      for (int sid = 0; sid < c->n_sets; ++sid) {
        ActiveSet a;
        fill_set(c, sid, &a);
        worst = std::max(worst, plan_slots(c, a, false));
      }
      c->arena_cap = worst;
      if ((rc = dev_alloc(c, (void**)&c->arena, c->arena_cap)) != HIFT_OK) return fail(rc);
    }
  }
  if (m->arch == 2) {
    const int half = c->dh / 2;
    std::vector<float> cs(2 * (size_t)c->S * half);
    for (int p = 0; p < c->S; ++p)
      for (int j = 0; j < half; ++j) {
        const double ang = (double)p * pow(m->rope_base, -2.0 * j / (double)c->dh);
        cs[(size_t)p * half + j] = (float)cos(ang);
        cs[(size_t)c->S * half + (size_t)p * half + j] = (float)sin(ang);
      }
    cudaMemcpyAsync(c->rope_cs, cs.data(), cs.size() * sizeof(float), cudaMemcpyHostToDevice, c->st);
    cudaStreamSynchronize(c->st);
  }
  if (cudaStreamSynchronize(c->st) != cudaSuccess) return fail(HIFT_ERR_CUDA);
  gemm_tc_init();   // if unavailable, gemm_tc_eligible() answers false and CUDA cores are used
  *out = c;
  return HIFT_OK;
}

hift_status hift_step(hift_ctx* c, const int32_t* tok, const int32_t* lab, float* loss_host) {
  if (!c || !tok || !lab) return HIFT_ERR_INPUT;
  return do_step(c, tok, lab, loss_host);
}

hift_status hift_step_begin(hift_ctx* c, const int32_t* tok, const int32_t* lab, float* loss_host) {
  if (!c || !tok || !lab) return HIFT_ERR_INPUT;
  if (c->pending_update) return HIFT_ERR_CFG;
  hift_status s = enqueue_forward_backward(c, tok, lab);
  if (s != HIFT_OK) return s;
  s = finish_step(c, loss_host, false);
  if (s == HIFT_OK) c->pending_update = true;
  return s;
}
hift_status hift_grad_view(hift_ctx* c, void** grad_dev, size_t* n) {
  if (!c || !grad_dev || !n || c->last_group < 0) return HIFT_ERR_CFG;
  *grad_dev = c->grad;
  *n = c->act.grad_numel;
  return HIFT_OK;
}
hift_status hift_step_begin_async(hift_ctx* c, const int32_t* tok, const int32_t* lab) {
  if (!c || !tok || !lab) return HIFT_ERR_INPUT;
  if (c->pending_update) return HIFT_ERR_CFG;
  const hift_status s = enqueue_forward_backward(c, tok, lab);
  if (s != HIFT_OK) return s;
  c->pending_update = true;
  return c->first_err == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
int32_t hift_grad_num_chunks(const hift_ctx* c) { return c && c->pending_update ? (int32_t)c->chunks.size() : 0; }
hift_status hift_grad_chunk(const hift_ctx* c, int32_t i, size_t* offset, size_t* n) {
  if (!c || !c->pending_update || i < 0 || i >= (int)c->chunks.size() || !offset || !n) return HIFT_ERR_CFG;
  *offset = c->chunks[i].off; *n = c->chunks[i].n;
  return HIFT_OK;
}
hift_status hift_grad_chunk_wait(hift_ctx* c, int32_t i, void* stream) {
  if (!c || !c->pending_update || i < 0 || i >= (int)c->chunks.size()) return HIFT_ERR_CFG;
  cudaError_t e = cudaStreamWaitEvent((cudaStream_t)stream, c->chunks[i].ev, 0);
  if (e == cudaSuccess && i + 1 == (int)c->chunks.size()) e = cudaStreamWaitEvent((cudaStream_t)stream, c->ev_bwd, 0);
  return e == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_gate_view(hift_ctx* c, int32_t** gate_dev) {
  if (!c || !gate_dev) return HIFT_ERR_CFG;
  *gate_dev = c->gate;
  return HIFT_OK;
}
hift_status hift_shard_range(const hift_ctx* c, int32_t g, int32_t rank, size_t* lo, size_t* n) {
  if (!c || c->queue || g < 0 || g >= (int)c->groups.size() || rank < 0 || rank >= c->shard_world || !lo || !n) return HIFT_ERR_CFG;
  const GroupRec& gr = c->groups[g];
  const size_t piece = align_up((gr.numel + c->shard_world - 1) / c->shard_world, kAlignElems);
  *lo = std::min((size_t)rank * piece, gr.numel);
  *n = std::min(piece, gr.numel - *lo);
  return HIFT_OK;
}
hift_status hift_param_view(hift_ctx* c, void** param_dev, size_t* n, int32_t* elem_bytes) {
  if (!c || !param_dev || !n || c->last_group < 0 || c->act.groups.size() != 1) return HIFT_ERR_CFG;
  const GroupRec& gr = c->groups[c->act.groups[0]];
  *param_dev = c->params + gr.off * c->es;
  *n = gr.numel;
  if (elem_bytes) *elem_bytes = c->es;
  return HIFT_OK;
}
hift_status hift_set_grad_chunk_bytes(hift_ctx* c, size_t bytes) {
  if (!c || c->pending_update) return HIFT_ERR_CFG;
  c->chunk_min_elems = bytes / sizeof(float) ? bytes / sizeof(float) : 1;
  return HIFT_OK;
}
hift_status hift_step_finish(hift_ctx* c, float* loss_host) {
  if (!c || !c->pending_update) return HIFT_ERR_CFG;
  c->note(cudaEventRecord(c->ev_in, c->caller));
  c->note(cudaStreamWaitEvent(c->st, c->ev_in, 0));
  enqueue_update(c);
  c->pending_update = false;
  const hift_status s = finish_step(c, loss_host, true);
  if (s == HIFT_OK) c->t += 1;
  else step_failed(c);
  return s;
}
// Host-only: the chunk plan for a span of tensors and a completion order (no GPU involved).
int32_t hift_plan_grad_chunks(const size_t* offsets, const size_t* sizes, int32_t n_tensors, size_t span_elems,
                              const int32_t* completion_order, int32_t n_completed, size_t min_chunk_elems,
                              size_t* chunk_off, size_t* chunk_n, int32_t* chunk_after, int32_t max_chunks) {
  if (!offsets || !sizes || n_tensors < 1 || (n_completed > 0 && !completion_order) || !chunk_off || !chunk_n || max_chunks < 1) return -1;
  GradChunkPlanner p;
  p.reset(span_elems, min_chunk_elems);
  for (int i = 0; i < n_tensors; ++i) p.add(offsets[i], sizes[i]);
  int32_t nc = 0;
  size_t off, n;
  for (int i = 0; i < n_completed; ++i)
    if (p.complete(completion_order[i], &off, &n)) {
      if (nc == max_chunks) return -1;
      chunk_off[nc] = off; chunk_n[nc] = n; if (chunk_after) chunk_after[nc] = i; ++nc;
    }
  if (p.flush(&off, &n)) {
    if (nc == max_chunks) return -1;
    chunk_off[nc] = off; chunk_n[nc] = n; if (chunk_after) chunk_after[nc] = n_completed; ++nc;
  }
  return nc;
}
int32_t hift_grad_elem_bytes(const hift_ctx* c) { return c ? c->ges : 0; }
hift_status hift_step_end(hift_ctx* c) { return hift_step_finish(c, nullptr); }
hift_status hift_step_abort(hift_ctx* c) {
  if (!c || !c->pending_update) return HIFT_ERR_CFG;
  c->pending_update = false;       // the gradient is dropped; the state uploaded for the step stays resident
  return HIFT_OK;
}

namespace {
__global__ void copy_i32_kernel(const int32_t* __restrict__ src, int32_t* __restrict__ dst, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) dst[i] = src[i];
}
// A step's token ids and labels are a few kilobytes.  From pinned (or registered) host memory a copy would be a
// DMA job and could queue on a copy engine behind the gigabytes of optimizer state in flight; a kernel reads such
// memory directly instead.  From pageable memory the runtime stages the bytes itself and no engine queue is involved.
void upload_i32(hift_ctx* c, int32_t* dst, const int32_t* src, size_t n) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, src) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer != nullptr) {
    copy_i32_kernel<<<(unsigned)((n + 255) / 256 < 64 ? (n + 255) / 256 : 64), 256, 0, c->st>>>((const int32_t*)at.devicePointer, dst, n);
    c->note(cudaGetLastError());
    return;
  }
  cudaGetLastError();
  c->note(cudaMemcpyAsync(dst, src, n * sizeof(int32_t), cudaMemcpyHostToDevice, c->st));
}
}  // namespace

hift_status hift_set_key_lengths(hift_ctx* c, const int32_t* lens_host) {
  if (!c) return HIFT_ERR_INPUT;
  if (c->pending_update) return HIFT_ERR_CFG;            // not between the two halves of a step
  if (lens_host == nullptr) { c->use_lens = false; return HIFT_OK; }
  for (int b = 0; b < c->B; ++b) if (lens_host[b] < 1 || lens_host[b] > c->S) return HIFT_ERR_INPUT;
  c->note(cudaStreamSynchronize(c->st));                 // nothing enqueued earlier still reads the staging row
  memcpy(c->scal_host + kScalWords, lens_host, (size_t)c->B * sizeof(int32_t));
  copy_i32_kernel<<<1, 256, 0, c->st>>>((const int32_t*)(c->scal_host_dev + kScalWords), c->lens_dev, (size_t)c->B);
  c->note(cudaGetLastError());
  c->note(cudaStreamSynchronize(c->st));
  c->use_lens = c->first_err == cudaSuccess;
  return c->use_lens ? HIFT_OK : HIFT_ERR_CUDA;
}

hift_status hift_step_host(hift_ctx* c, const int32_t* tok, const int32_t* lab, float* loss_host) {
  if (!c || !tok || !lab) return HIFT_ERR_INPUT;
  const size_t nlab = c->m.arch == 1 ? c->B : c->T;
  for (int i = 0; i < c->T; ++i) if (tok[i] < 0 || tok[i] >= c->V) return HIFT_ERR_INPUT;
  const int nl = c->m.arch == 1 ? c->m.n_classes : c->V;
  for (size_t i = 0; i < nlab; ++i) if (lab[i] >= nl) return HIFT_ERR_INPUT;
  upload_i32(c, c->tok_dev, tok, (size_t)c->T);
  upload_i32(c, c->lab_dev, lab, nlab);
  return do_step(c, c->tok_dev, c->lab_dev, loss_host);
}

int32_t hift_active_group(const hift_ctx* c) { return group_at(c, c->t); }
int32_t hift_num_groups(const hift_ctx* c) { return (int32_t)c->k_cycle; }
int32_t hift_num_sets(const hift_ctx* c) { return (int32_t)c->n_sets; }
hift_status hift_set_units(const hift_ctx* c, int32_t set_id, int32_t* units, int32_t cap, int32_t* n_units) {
  if (!c || set_id < 0 || set_id >= c->n_sets || !units || !n_units) return HIFT_ERR_CFG;
  ActiveSet a;
  fill_set(c, set_id, &a);
  int n = 0;
  for (int g : a.groups)
    for (int u = c->groups[g].unit_lo; u <= c->groups[g].unit_hi; ++u) {
      if (n == cap) return HIFT_ERR_CFG;
      units[n++] = u;
    }
  *n_units = n;
  return HIFT_OK;
}
int64_t hift_step_count(const hift_ctx* c) { return c->t; }
double hift_current_lr(const hift_ctx* c) { return lr_for_cycle(c->oc, c->t / (int64_t)c->k_cycle); }
hift_status hift_group_units(const hift_ctx* c, int32_t g, int32_t* lo, int32_t* hi) {
  if (g < 0 || g >= c->n_sets) return HIFT_ERR_CFG;
  ActiveSet a;
  fill_set(c, g, &a);
  *lo = c->groups[a.groups.front()].unit_lo; *hi = c->groups[a.groups.back()].unit_hi;
  // a set of the drifting queue may wrap around (the top unit together with the bottom one): not an interval
  for (size_t i = 1; i < a.groups.size(); ++i)
    if (c->groups[a.groups[i]].unit_lo != c->groups[a.groups[i - 1]].unit_hi + 1) return HIFT_ERR_CFG;
  return HIFT_OK;
}
hift_status hift_force_group(hift_ctx* c, int32_t g) {
  if (g < -1 || g >= c->n_sets) return HIFT_ERR_CFG;
  if (g != c->forced) drop_reservations(c);     // uploads made for the schedule's coming steps stay resident, unreserved
  c->forced = g;
  return HIFT_OK;
}
hift_status hift_force_sequence(hift_ctx* c, const int32_t* groups, int32_t n) {
  if (!c || n < 0 || (n > 0 && !groups)) return HIFT_ERR_CFG;
  for (int i = 0; i < n; ++i) if (groups[i] < 0 || groups[i] >= c->n_sets) return HIFT_ERR_CFG;
  drop_reservations(c);
  c->forced_seq.assign(groups, groups + n);
  c->forced_seq_t0 = c->t;
  return HIFT_OK;
}
size_t hift_peak_hbm_bytes(const hift_ctx* c) { return c->dev_bytes; }
size_t hift_pinned_host_bytes(const hift_ctx* c) { return c->pinned_bytes; }

int32_t hift_num_tensors(const hift_ctx* c) { return (int32_t)c->tens.size(); }
hift_status hift_tensor_info(const hift_ctx* c, int32_t ti, char* name, int32_t* unit, int64_t* rows, int64_t* cols) {
  if (ti < 0 || ti >= (int)c->tens.size()) return HIFT_ERR_CFG;
  const TensorRec& r = c->tens[ti];
  if (name) memcpy(name, r.name, 64);
  if (unit) *unit = r.unit;
  if (rows) *rows = r.rows;
  if (cols) *cols = r.cols;
  return HIFT_OK;
}

hift_status hift_load_weights(hift_ctx* c, const char* path, int32_t strict, int32_t* n_loaded) {
  if (!c || !path || c->pending_update) return HIFT_ERR_CFG;
  FILE* f = fopen(path, "rb");
  if (!f) return HIFT_ERR_INPUT;
  char magic[8];
  uint32_t n = 0;
  bool ok = fread(magic, 8, 1, f) == 1 && memcmp(magic, "HIFTWTS1", 8) == 0 && fread(&n, 4, 1, f) == 1;
  std::vector<char> seen(c->tens.size(), 0);
  std::vector<float> vals;
  std::vector<uint16_t> half;
  int loaded = 0;
  hift_status rc = HIFT_OK;
  for (uint32_t r = 0; ok && r < n; ++r) {
    char name[64];
    uint32_t dtype = 0;
    uint64_t rows = 0, cols = 0;
    ok = fread(name, 64, 1, f) == 1 && fread(&dtype, 4, 1, f) == 1 && fread(&rows, 8, 1, f) == 1 && fread(&cols, 8, 1, f) == 1;
    if (!ok) break;
    name[63] = 0;
    int ti = -1;
    for (size_t i = 0; i < c->tens.size(); ++i) if (strcmp(c->tens[i].name, name) == 0) { ti = (int)i; break; }
    // unknown tensor, a second record for the same tensor, a wrong shape or element type: refuse the file
    if (ti < 0 || seen[ti] || dtype > 1 || rows != (uint64_t)c->tens[ti].rows || cols != (uint64_t)c->tens[ti].cols) { rc = HIFT_ERR_INPUT; break; }
    const size_t cnt = c->tens[ti].numel;
    vals.resize(cnt);
    if (dtype == 1) {
      half.resize(cnt);
      ok = fread(half.data(), 2, cnt, f) == cnt;
      for (size_t i = 0; ok && i < cnt; ++i) { const uint32_t u = (uint32_t)half[i] << 16; memcpy(&vals[i], &u, 4); }
    } else ok = fread(vals.data(), 4, cnt, f) == cnt;
    if (!ok) break;
    rc = hift_set_param(c, ti, vals.data(), cnt);
    if (rc != HIFT_OK) break;
    seen[ti] = 1;
    ++loaded;
  }
  fclose(f);
  if (n_loaded) *n_loaded = loaded;
  if (rc != HIFT_OK) return rc;
  if (!ok) return HIFT_ERR_INPUT;
  if (strict && loaded != (int)c->tens.size()) return HIFT_ERR_INPUT;
  return HIFT_OK;
}

hift_status hift_set_param(hift_ctx* c, int32_t ti, const float* src, size_t n) {
  if (ti < 0 || ti >= (int)c->tens.size() || !src || n != c->tens[ti].numel) return HIFT_ERR_CFG;
  sync_all(c);
  invalidate_slots(c);
  GroupRec& gr = c->groups[group_of_unit(c, c->tens[ti].unit)];
  const OwnPart op = own_part(c, ti);
  // every copy goes through the context's stream, so the cast below is ordered after its input
  if (op.n) {
    bool on_host;
    float* base = plane_base(c, gr, 0, &on_host);
    if (c->compact) master_write(c, gr, (c->tens[ti].off - gr.off) + op.t_lo, op.n, src + op.t_lo);
    else if (on_host) memcpy(base + op.p, src + op.t_lo, op.n * sizeof(float));
    else if (cudaMemcpyAsync(base + op.p, src + op.t_lo, op.n * sizeof(float), cudaMemcpyHostToDevice, c->st) != cudaSuccess) return HIFT_ERR_CUDA;
  }
  if (c->mixed) {
    // stage the fp32 values in the gradient buffer (any tensor fits in the largest group)
    float* stg = staging(c);
    if (!stg) return HIFT_ERR_OOM_DEVICE;
    if (cudaMemcpyAsync(stg, src, n * sizeof(float), cudaMemcpyHostToDevice, c->st) != cudaSuccess) return HIFT_ERR_CUDA;
    cast_from_f32_kernel<bf16><<<grid_for(n, 256), 256, 0, c->st>>>(stg, (bf16*)c->P(ti), n);
  } else if (op.n != n) {
    // fp32 parameters are their own master: the part another rank updates is still this rank's model value
    if (cudaMemcpyAsync(c->P(ti), src, n * sizeof(float), cudaMemcpyHostToDevice, c->st) != cudaSuccess) return HIFT_ERR_CUDA;
  }
  return cudaStreamSynchronize(c->st) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_get_param(hift_ctx* c, int32_t ti, float* dst, size_t n) {
  if (ti < 0 || ti >= (int)c->tens.size() || !dst || n != c->tens[ti].numel) return HIFT_ERR_CFG;
  sync_all(c);
  if (!c->mixed) return cudaMemcpy(dst, c->P(ti), n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
  const GroupRec& gr = c->groups[group_of_unit(c, c->tens[ti].unit)];
  const OwnPart op = own_part(c, ti);
  if (op.n != n) {                  // sharded state: outside this rank's part only the model value is known
    const hift_status s = hift_get_model_param(c, ti, dst, n);
    if (s != HIFT_OK) return s;
  }
  if (!op.n) return HIFT_OK;
  if (c->compact) return master_read(c, gr, (c->tens[ti].off - gr.off) + op.t_lo, op.n, dst + op.t_lo) ? HIFT_OK : HIFT_ERR_CUDA;
  bool on_host;
  float* base = plane_base(c, const_cast<GroupRec&>(gr), 0, &on_host);
  if (on_host) memcpy(dst + op.t_lo, base + op.p, op.n * sizeof(float));
  else if (cudaMemcpy(dst + op.t_lo, base + op.p, op.n * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) return HIFT_ERR_CUDA;
  return HIFT_OK;
}
hift_status hift_get_model_param(hift_ctx* c, int32_t ti, float* dst, size_t n) {
  if (ti < 0 || ti >= (int)c->tens.size() || !dst || n != c->tens[ti].numel) return HIFT_ERR_CFG;
  sync_all(c);
  if (!c->mixed) return cudaMemcpy(dst, c->P(ti), n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
  float* tmp = nullptr;
  if (cudaMalloc((void**)&tmp, n * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return HIFT_ERR_OOM_DEVICE; }
  cast_to_f32_kernel<bf16><<<grid_for(n, 256), 256, 0, c->st>>>((const bf16*)c->P(ti), tmp, n);
  cudaError_t e = cudaMemcpyAsync(dst, tmp, n * sizeof(float), cudaMemcpyDeviceToHost, c->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->st);
  cudaFree(tmp);
  return e == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_get_state(hift_ctx* c, int32_t ti, int32_t which, float* dst, size_t n) {
  if (ti < 0 || ti >= (int)c->tens.size() || !dst || n != c->tens[ti].numel) return HIFT_ERR_CFG;
  if (which < 0 || which >= c->n_state) return HIFT_ERR_CFG;
  sync_all(c);
  const GroupRec& gr = c->groups[group_of_unit(c, c->tens[ti].unit)];
  const OwnPart op = own_part(c, ti);
  if (op.n != n) memset(dst, 0, n * sizeof(float));      // sharded state: zeros outside this rank's part
  if (!op.n) return HIFT_OK;
  bool on_host;
  float* base = plane_base(c, gr, 1 + which, &on_host);
  if (!base) return HIFT_ERR_CFG;
  if (on_host) memcpy(dst + op.t_lo, base + op.p, op.n * sizeof(float));
  else if (cudaMemcpy(dst + op.t_lo, base + op.p, op.n * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) return HIFT_ERR_CUDA;
  return HIFT_OK;
}
hift_status hift_get_factored_state(hift_ctx* c, int32_t ti, int32_t which, float* dst, size_t n) {
  if (!c || !c->af || ti < 0 || ti >= (int)c->tens.size() || !dst || which < 0 || which > 1) return HIFT_ERR_CFG;
  const TensorRec& r = c->tens[ti];
  const bool vec = r.rows == 1;
  if (vec && which == 1) return HIFT_ERR_CFG;
  const size_t want = vec ? (size_t)r.cols : (which == 0 ? (size_t)r.rows : (size_t)r.cols);
  if (n != want) return HIFT_ERR_CFG;
  sync_all(c);
  const GroupRec& gr = c->groups[group_of_unit(c, r.unit)];
  const size_t o = r.af_off + ((!vec && which == 1) ? (size_t)r.rows : 0);
  if (c->offload) {
    memcpy(dst, (float*)gr.blob + (c->mixed ? gr.numel : 0) + o, n * sizeof(float));
    return HIFT_OK;
  }
  return cudaMemcpy(dst, c->af_all + gr.af_base + o, n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}

hift_status hift_get_grad(hift_ctx* c, int32_t ti, float* dst, size_t n) {
  if (ti < 0 || ti >= (int)c->tens.size() || !dst || n != c->tens[ti].numel) return HIFT_ERR_CFG;
  if (c->last_group < 0 || c->grad_off.size() != c->tens.size() || c->grad_off[ti] == SIZE_MAX) return HIFT_ERR_CFG;
  sync_all(c);
  if (!c->gbf) return cudaMemcpy(dst, c->G(ti), n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
  std::vector<uint16_t> h(n);
  if (cudaMemcpy(h.data(), c->G(ti), n * 2, cudaMemcpyDeviceToHost) != cudaSuccess) return HIFT_ERR_CUDA;
  for (size_t i = 0; i < n; ++i) { const uint32_t u = (uint32_t)h[i] << 16; memcpy(dst + i, &u, 4); }
  return HIFT_OK;
}

hift_status hift_init_synthetic(hift_ctx* c, uint64_t seed, double stdv) {
  sync_all(c);
  invalidate_slots(c);
  float* stg = c->compact ? staging(c) : nullptr;
  if (c->compact && !stg) return HIFT_ERR_OOM_DEVICE;
  for (size_t g = 0; g < c->groups.size(); ++g) {
    GroupRec& gr = c->groups[g];
    if (c->offload) cudaMemsetAsync(c->slot[0].mem, 0, gr.blob_bytes, c->st);
    if (c->compact) cudaMemsetAsync(stg, 0, gr.numel * sizeof(float), c->st);     // alignment gaps pack to zero
    for (int u = gr.unit_lo; u <= gr.unit_hi; ++u) {
      for (int ti : c->unit_tens[u]) {
        const TensorRec& r = c->tens[ti];
        float* mp = nullptr;
        if (c->compact) mp = stg + (r.off - gr.off);           // staged as floats, packed below
        else if (c->mixed) mp = c->offload ? (float*)c->slot[0].mem + (r.off - gr.off) : c->master_all + r.off;
        const uint64_t sd = seed * 0x9E3779B97F4A7C15ull + (uint64_t)ti * 0xD1B54A32D192ED03ull;
        if (c->mixed) init_tensor_kernel<bf16><<<grid_for(r.numel, 256), 256, 0, c->st>>>((bf16*)c->P(ti), mp, r.numel, r.init_kind, (float)stdv, sd);
        else init_tensor_kernel<float><<<grid_for(r.numel, 256), 256, 0, c->st>>>((float*)c->P(ti), nullptr, r.numel, r.init_kind, (float)stdv, sd);
      }
    }
    if (c->compact) {
      uint16_t* lo16 = (uint16_t*)((float*)c->slot[0].mem + gr.state_floats);
      if (gr.own_n)
        master_pack_kernel<<<grid_for(gr.own_n / 8, 256), 256, 0, c->st>>>(stg + gr.own_lo, lo16, (uint8_t*)(lo16 + gr.own_n), gr.own_n / 8);
    }
    if (c->offload) {
      cudaMemcpyAsync(gr.blob, c->slot[0].mem, gr.blob_bytes, cudaMemcpyDeviceToHost, c->st);
      if (cudaStreamSynchronize(c->st) != cudaSuccess) return HIFT_ERR_CUDA;
    }
    gr.tau = 0;
  }
  if (!c->offload) {
    if (c->s0_all) cudaMemsetAsync(c->s0_all, 0, c->total * sizeof(float), c->st);
    if (c->s1_all) cudaMemsetAsync(c->s1_all, 0, c->total * sizeof(float), c->st);
    if (c->af_all) {
      size_t tot = 0;
      for (auto& g : c->groups) tot += g.state_floats;
      cudaMemsetAsync(c->af_all, 0, tot * sizeof(float), c->st);
    }
  }
  return cudaStreamSynchronize(c->st) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}

// ---------------------------------------------------------------- checkpoint
namespace {
struct CkptHeader {
  char magic[8];            // "HIFTCKPT"
  uint32_t version;
  uint32_t kind, dtype, n_groups;
  uint64_t total, t;
};
// device or pinned location of the group's fp32 master (or fp32 parameters) and of its state
void group_locations(hift_ctx* c, GroupRec& gr, float** master, bool* master_host, float** state, bool* state_host) {
  *master_host = false; *state_host = false;
  if (!c->mixed) *master = (float*)c->params + gr.off;
  else if (c->compact) { *master = nullptr; *master_host = true; }       // rebuilt / packed by the caller
  else if (c->offload) { *master = (float*)gr.blob; *master_host = true; }
  else *master = c->master_all + gr.off;
  if (c->offload) { *state = (float*)gr.blob + ((c->mixed && !c->compact) ? gr.numel : 0); *state_host = true; }
  else if (c->af) *state = c->af_all + gr.af_base;
  else *state = nullptr;      // two separate planes, handled by the caller
}
}  // namespace

hift_status hift_save(hift_ctx* c, const char* path) {
  if (!c || !path || c->pending_update || c->shard_world > 1) return HIFT_ERR_CFG;
  sync_all(c);
  FILE* f = fopen(path, "wb");
  if (!f) return HIFT_ERR_INPUT;
  CkptHeader h;
  memset(&h, 0, sizeof(h));
  memcpy(h.magic, "HIFTCKPT", 8);
  h.version = 2; h.kind = (uint32_t)c->oc.kind; h.dtype = (uint32_t)c->m.dtype; h.n_groups = (uint32_t)c->groups.size();
  h.total = c->total; h.t = (uint64_t)c->t;
  bool ok = fwrite(&h, sizeof(h), 1, f) == 1;
  std::vector<float> tmp;
  for (auto& gr : c->groups) {
    if (!ok) break;
    const uint64_t span[2] = {(uint64_t)gr.off, (uint64_t)gr.numel};   // the partition is part of the format
    ok = fwrite(span, sizeof(span), 1, f) == 1 && fwrite(&gr.tau, sizeof(gr.tau), 1, f) == 1;
    float *mp, *sp; bool mh, sh;
    group_locations(c, gr, &mp, &mh, &sp, &sh);
    auto put = [&](const float* p, bool host, size_t n) {
      if (!ok || n == 0) return;
      if (host) { ok = fwrite(p, sizeof(float), n, f) == n; return; }
      tmp.resize(n);
      ok = cudaMemcpy(tmp.data(), p, n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess &&
           fwrite(tmp.data(), sizeof(float), n, f) == n;
    };
    if (c->compact) {
      // the file always holds fp32 master values, whatever the paged form
      std::vector<float> mv(gr.numel);
      ok = ok && master_read(c, gr, 0, gr.numel, mv.data());
      put(mv.data(), true, gr.numel);
    } else put(mp, mh, gr.numel);
    if (sp) put(sp, sh, gr.state_floats);
    else {
      if (c->s0_all) put(c->s0_all + gr.off, false, gr.numel);
      if (c->s1_all) put(c->s1_all + gr.off, false, gr.numel);
    }
  }
  ok = (fclose(f) == 0) && ok;
  return ok ? HIFT_OK : HIFT_ERR_INPUT;
}

hift_status hift_load(hift_ctx* c, const char* path) {
  if (!c || !path || c->pending_update || c->shard_world > 1) return HIFT_ERR_CFG;
  sync_all(c);
  FILE* f = fopen(path, "rb");
  if (!f) return HIFT_ERR_INPUT;
  CkptHeader h;
  bool ok = fread(&h, sizeof(h), 1, f) == 1 && memcmp(h.magic, "HIFTCKPT", 8) == 0 && h.version == 2;
  if (ok && (h.kind != (uint32_t)c->oc.kind || h.dtype != (uint32_t)c->m.dtype || h.n_groups != c->groups.size() ||
             h.total != c->total)) { fclose(f); return HIFT_ERR_CFG; }
  std::vector<float> tmp;
  for (auto& gr : c->groups) {
    if (!ok) break;
    uint64_t span[2] = {0, 0};
    ok = fread(span, sizeof(span), 1, f) == 1;
    if (ok && (span[0] != (uint64_t)gr.off || span[1] != (uint64_t)gr.numel)) { fclose(f); return HIFT_ERR_CFG; }   // other grouping
    ok = ok && fread(&gr.tau, sizeof(gr.tau), 1, f) == 1;
    float *mp, *sp; bool mh, sh;
    group_locations(c, gr, &mp, &mh, &sp, &sh);
    auto get = [&](float* p, bool host, size_t n) {
      if (!ok || n == 0) return;
      if (host) { ok = fread(p, sizeof(float), n, f) == n; return; }
      tmp.resize(n);
      ok = fread(tmp.data(), sizeof(float), n, f) == n &&
           cudaMemcpy(p, tmp.data(), n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess;
    };
    std::vector<float> mv;
    if (c->compact) {
      mv.resize(gr.numel);
      get(mv.data(), true, gr.numel);
      if (ok) master_write(c, gr, 0, gr.numel, mv.data());
      mp = mv.data();
    } else get(mp, mh, gr.numel);
    if (sp) get(sp, sh, gr.state_floats);
    else {
      if (c->s0_all) get(c->s0_all + gr.off, false, gr.numel);
      if (c->s1_all) get(c->s1_all + gr.off, false, gr.numel);
    }
    if (ok && c->mixed) {
      // rebuild the bf16 model copy of this group from its master values
      const float* src = mp;
      if (mh) {
        float* stg = staging(c);
        ok = stg != nullptr && cudaMemcpyAsync(stg, mp, gr.numel * sizeof(float), cudaMemcpyHostToDevice, c->st) == cudaSuccess;
        src = stg;
      }
      cast_from_f32_kernel<bf16><<<grid_for(gr.numel, 256), 256, 0, c->st>>>(src, (bf16*)(c->params + gr.off * c->es), gr.numel);
      ok = ok && cudaStreamSynchronize(c->st) == cudaSuccess;
    }
  }
  fclose(f);
  if (!ok) return HIFT_ERR_INPUT;
  c->t = (int64_t)h.t;
  invalidate_slots(c);
  return HIFT_OK;
}

hift_status hift_profile_enable(hift_ctx* c, int32_t on) {
  sync_all(c);
  c->prof_on = on != 0;
  memset(c->prof_launches, 0, sizeof(c->prof_launches));
  memset(c->prof_ms, 0, sizeof(c->prof_ms));
  memset(c->prof_work, 0, sizeof(c->prof_work));
  return HIFT_OK;
}
hift_status hift_profile(hift_ctx* c, int32_t cls, int64_t* launches, double* ms, double* work) {
  if (cls < 0 || cls >= HIFT_K_NUM) return HIFT_ERR_CFG;
  if (launches) *launches = c->prof_launches[cls];
  if (ms) *ms = c->prof_ms[cls];
  if (work) *work = c->prof_work[cls];
  return HIFT_OK;
}
int64_t hift_last_step_launches(const hift_ctx* c) { return c->step_launches; }
hift_status hift_last_step_paging(const hift_ctx* c, size_t* h2d, size_t* d2h) {
  if (h2d) *h2d = c->step_h2d;
  if (d2h) *d2h = c->step_d2h;
  return HIFT_OK;
}

hift_status hift_last_step_timeline(hift_ctx* c, double* ms6) {
  if (!c || !ms6) return HIFT_ERR_CFG;
  for (int i = 0; i < 6; ++i) ms6[i] = nan("");
  if (!c->offload || !c->tl_valid) return HIFT_OK;
  sync_all(c);
  const SlotRec& sr = c->slot[c->cur_sl];
  const cudaEvent_t ev[6] = {sr.tl_h2d0, sr.tl_h2d1, c->tl[3], c->tl[4], c->tl[5], c->tl[6]};
  for (int i = 0; i < 6; ++i) {
    if (i < 2 && sr.h2d_for_step < 0) continue;        // never uploaded
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->tl[0], ev[i]) == cudaSuccess) ms6[i] = ms;
    else cudaGetLastError();
  }
  return HIFT_OK;
}

int32_t hift_test_switch(int32_t which, int32_t value) {
  if (which == 4) { const int old = g_fail_pinned_in; g_fail_pinned_in = value; return old; }
  if (which == 5) { const int old = g_checked_arena; if (value >= 0) g_checked_arena = value; return old; }
  return gemm_tc_switch(which, value);
}

int64_t hift_check_arena(hift_ctx* c) {
  if (!c || !c->checked) return -1;
  sync_all(c);
  std::vector<unsigned char> buf(kGuardBytes);
  int64_t bad = 0;
  for (size_t o : c->guards) {
    if (cudaMemcpy(buf.data(), c->arena + o, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    for (unsigned char b : buf) if (b != kGuardByte) { ++bad; break; }
  }
  return bad;
}
int64_t hift_arena_guard_count(const hift_ctx* c) { return c && c->checked ? (int64_t)c->guards.size() : -1; }

int32_t hift_tc_error_flag(int32_t set_value) {
  if (gemm_tc_init() != 0) return -1;
  cudaDeviceSynchronize();
  if (set_value >= 0 && gemm_tc_set_error(set_value) != 0) return -1;
  return gemm_tc_poll_error();
}

// ---------------------------------------------------------------- optimizer on flat buffers
hift_status hift_opt_step(int32_t kind, size_t n, void* param_bf16, float* master, const float* grad,
                          float* s0, float* s1, double lr, double b1, double b2, double eps,
                          double wd, double mu, int64_t tau, void* stream) {
  if (kind < 0 || kind > 3 || !master || !grad || (kind != 3 && !s0) || (kind == 0 && !s1) || tau < 1) return HIFT_ERR_CFG;
  const uintptr_t al = (uintptr_t)master | (uintptr_t)grad | (uintptr_t)s0 | (uintptr_t)s1 | (uintptr_t)param_bf16;
  if (al & 15) return HIFT_ERR_CFG;
  const OptScalars h = make_opt_scalars(kind, lr, b1, b2, eps, wd, mu, tau);
  launch_fused_opt((cudaStream_t)stream, kind, n, param_bf16, master, grad, s0, s1, h);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}

hift_status hift_adafactor_step(int64_t rows, int64_t cols, void* param_bf16, float* master, const float* grad,
                                float* state, float* scratch, double lr, double eps1, double wd, int64_t tau,
                                void* stream) {
  if (rows < 1 || cols < 1 || !master || !grad || !state || !scratch || tau < 1) return HIFT_ERR_CFG;
  launch_adafactor_tensor((cudaStream_t)stream, rows, cols, param_bf16, master, grad, state, scratch, lr, eps1, wd, tau);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}

// ---------------------------------------------------------------- single kernels
hift_status hift_k_linear(int32_t form, int32_t dtype, int32_t path, int64_t M, int64_t N, int64_t K,
                          const void* a, const void* b, void* out, const void* bias,
                          const float* residual, void* stream) {
  if (form < 0 || form > 2 || dtype < 0 || dtype > 1 || M < 1 || N < 1 || K < 1) return HIFT_ERR_CFG;
  const bool f32o = residual != nullptr;
  GemmArgs g;
  if (form == 0) g = GemmArgs{(int)M, (int)N, (int)K, a, K, 1, b, 1, K, out, N, bias, residual, N, f32o};
  else if (form == 1) g = GemmArgs{(int)M, (int)K, (int)N, a, N, 1, b, K, 1, out, K, nullptr, residual, K, f32o};
  else g = GemmArgs{(int)N, (int)K, (int)M, a, 1, N, b, K, 1, out, K, nullptr, nullptr, 0, true};
  const bool tc_ok = dtype == 1 && gemm_tc_init() == 0 && gemm_tc_eligible(g);
  if (path == 2 && !tc_ok) return HIFT_ERR_CFG;
  if (path != 1 && tc_ok) {
    if (gemm_tc_launch((cudaStream_t)stream, g) != cudaSuccess) return HIFT_ERR_CUDA;
    return HIFT_OK;
  }
  launch_gemm_simt((cudaStream_t)stream, dtype, g);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_linear_swiglu(int64_t M, int64_t f, int64_t K, const void* a, const void* b, void* gu, void* sact,
                                 const void* bias, void* stream) {
  if (M < 1 || f < 1 || K < 1 || !sact) return HIFT_ERR_CFG;
  GemmArgs g{(int)M, (int)(2 * f), (int)K, a, K, 1, b, 1, K, gu, 2 * f, bias, nullptr, 0, false};
  g.swiglu_out = sact;
  if (gemm_tc_init() != 0 || !gemm_tc_eligible(g)) return HIFT_ERR_CFG;
  return gemm_tc_launch((cudaStream_t)stream, g) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_linear_dx_swiglu_bwd(int64_t M, int64_t N, int64_t f, const void* dy, const void* w, const void* gu,
                                        void* dgu, void* stream) {
  if (M < 1 || N < 1 || f < 1 || !gu || !dgu) return HIFT_ERR_CFG;
  GemmArgs g{(int)M, (int)f, (int)N, dy, N, 1, w, f, 1, dgu, 2 * f, nullptr, nullptr, 0, false};
  g.swiglu_bwd_gu = gu;
  if (gemm_tc_init() != 0 || !gemm_tc_eligible(g)) return HIFT_ERR_CFG;
  return gemm_tc_launch((cudaStream_t)stream, g) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_linear_gelu(int64_t M, int64_t N, int64_t K, const void* a, const void* b, void* pre, void* act,
                               const void* bias, void* stream) {
  if (M < 1 || N < 1 || K < 1 || !act) return HIFT_ERR_CFG;
  GemmArgs g{(int)M, (int)N, (int)K, a, K, 1, b, 1, K, pre, N, bias, nullptr, 0, false};
  g.gelu_out = act;
  if (gemm_tc_init() != 0 || !gemm_tc_eligible(g)) return HIFT_ERR_CFG;
  return gemm_tc_launch((cudaStream_t)stream, g) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_linear_dx_gelu_bwd(int64_t M, int64_t N, int64_t f, const void* dy, const void* w, const void* pre,
                                      void* da, void* stream) {
  if (M < 1 || N < 1 || f < 1 || !pre || !da) return HIFT_ERR_CFG;
  GemmArgs g{(int)M, (int)f, (int)N, dy, N, 1, w, f, 1, da, f, nullptr, nullptr, 0, false};
  g.gelu_bwd_a = pre;
  if (gemm_tc_init() != 0 || !gemm_tc_eligible(g)) return HIFT_ERR_CFG;
  return gemm_tc_launch((cudaStream_t)stream, g) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_attention_fwd(int32_t dtype, int32_t B, int32_t S, int32_t H, int32_t dh, int32_t causal,
                                 const void* qkv, void* o, float* lse, const int32_t* key_lens, void* stream) {
  if (!attention_head_ok(dh) || dtype < 0 || dtype > 1) return HIFT_ERR_CFG;
  launch_attention_fwd((cudaStream_t)stream, dtype, B, S, H, dh, causal, qkv, o, lse, key_lens);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_attention_bwd(int32_t dtype, int32_t B, int32_t S, int32_t H, int32_t dh, int32_t causal,
                                 const void* qkv, const void* o, const float* lse, const void* dout,
                                 void* dqkv, float* dsum, const int32_t* key_lens, void* stream) {
  if (!attention_head_ok(dh) || dtype < 0 || dtype > 1) return HIFT_ERR_CFG;
  launch_attention_bwd((cudaStream_t)stream, dtype, B, S, H, dh, causal, qkv, o, lse, dout, dqkv, dsum, key_lens);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
static DropArgs attn_drop_of(double p, uint64_t seed, int32_t site, int64_t step) {
  DropArgs a;
  a.k0 = (uint32_t)seed; a.k1 = (uint32_t)(seed >> 32); a.site = (uint32_t)site; a.step = (uint32_t)step;
  a.thr = (uint32_t)floor(p * 4294967296.0); a.scale = (float)(1.0 / (1.0 - p));
  return a;
}
hift_status hift_k_attention_fwd_drop(int32_t dtype, int32_t B, int32_t S, int32_t H, int32_t dh, int32_t causal,
                                      const void* qkv, void* o, float* lse, const int32_t* key_lens, double p,
                                      uint64_t seed, int32_t site, int64_t step, void* stream) {
  if (!attention_head_ok(dh) || dtype < 0 || dtype > 1 || !(p >= 0.0 && p < 1.0)) return HIFT_ERR_CFG;
  launch_attention_fwd((cudaStream_t)stream, dtype, B, S, H, dh, causal, qkv, o, lse, key_lens, attn_drop_of(p, seed, site, step));
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_attention_bwd_drop(int32_t dtype, int32_t B, int32_t S, int32_t H, int32_t dh, int32_t causal,
                                      const void* qkv, const void* o, const float* lse, const void* dout,
                                      void* dqkv, float* dsum, const int32_t* key_lens, double p, uint64_t seed,
                                      int32_t site, int64_t step, void* stream) {
  if (!attention_head_ok(dh) || dtype < 0 || dtype > 1 || !(p >= 0.0 && p < 1.0)) return HIFT_ERR_CFG;
  launch_attention_bwd((cudaStream_t)stream, dtype, B, S, H, dh, causal, qkv, o, lse, dout, dqkv, dsum, key_lens,
                       attn_drop_of(p, seed, site, step));
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_linear_rope(int64_t M, int64_t N, int64_t K, const void* a, const void* b, void* out, const void* bias,
                               const float* cs, int32_t seq, int32_t d_head, int64_t rope_cols, void* stream) {
  if (M < 1 || N < 1 || K < 1 || !cs || seq < 1) return HIFT_ERR_CFG;
  GemmArgs g{(int)M, (int)N, (int)K, a, K, 1, b, 1, K, out, N, bias, nullptr, 0, false};
  g.rope_cs = cs; g.rope_seq = seq; g.rope_dh = d_head; g.rope_cols = rope_cols;
  if (gemm_tc_init() != 0 || !gemm_tc_eligible(g)) return HIFT_ERR_CFG;
  return gemm_tc_launch((cudaStream_t)stream, g) == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_norm_fwd(int32_t dtype, int32_t kind, int64_t rows, int64_t cols, double eps,
                            const float* x, const void* gain, const void* bias, void* y, float* stats,
                            void* stream) {
  if (cols % 8 || kind < 0 || kind > 1 || dtype < 0 || dtype > 1) return HIFT_ERR_CFG;
  launch_norm_fwd((cudaStream_t)stream, dtype, kind, rows, (int)cols, (float)eps, x, gain, bias, y, nullptr, stats);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_norm_bwd(int32_t dtype, int32_t kind, int64_t rows, int64_t cols, const void* dy,
                            const float* x, const float* stats, const void* gain, const float* add,
                            float* dx, float* dgain, float* dbias, float* partial, void* stream) {
  if (cols % 8 || kind < 0 || kind > 1 || dtype < 0 || dtype > 1) return HIFT_ERR_CFG;
  if (dgain && !partial) return HIFT_ERR_CFG;
  if ((dx || dgain) && (!dy || !x || !stats || !gain)) return HIFT_ERR_INPUT;
  cudaStream_t st = (cudaStream_t)stream;
  if (dx) launch_norm_bwd_dx(st, dtype, kind, false, rows, (int)cols, dy, x, stats, gain, add, dx, nullptr);
  if (dgain) launch_colreduce(st, dtype == 1, kind == 0 ? 1 : 2, rows, (int)cols, dy, cols, x, stats, partial, dgain, dbias);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
hift_status hift_k_cross_entropy(int32_t dtype, int64_t rows, int64_t vocab, int64_t ld, void* logits,
                                 const int32_t* labels, float* rowloss, float* loss, void* stream) {
  if (dtype < 0 || dtype > 1 || ld < vocab) return HIFT_ERR_CFG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaMemsetAsync(loss, 0, 4 * sizeof(float), st);
  launch_cross_entropy(st, dtype, rows, vocab, ld, logits, labels, rowloss, (int*)(loss + 1), (int*)(loss + 2), loss);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}

}  // extern "C"

// ====================================================================== allocation-free variant
// Column-reduction scratch for hift_k_norm_bwd_static: [2 planes][kColChunks][max cols] fp32,
// resident in every GPU context that loads this library.  In host code `g_static_partial` is
// only a handle for the runtime's symbol lookup, never a device address: the address the
// kernels get comes from cudaGetSymbolAddress, once per device.
namespace {
constexpr int kStaticMaxDevices = 64;
static __device__ __align__(256) float g_static_partial[2 * kColChunks * HIFT_STATIC_SCRATCH_MAX_COLS];
std::atomic<float*> g_static_partial_addr[kStaticMaxDevices];     // zero-initialised; one slot per device ordinal
}  // namespace

extern "C" hift_status hift_k_norm_bwd_static(int32_t dtype, int32_t kind, int64_t rows, int64_t cols,
                                              const void* dy, const float* x, const float* stats,
                                              const void* gain, const float* add, float* dx,
                                              float* dgain, float* dbias, void* stream) {
  if (cols % 8 || cols < 8 || rows < 1 || kind < 0 || kind > 1 || dtype < 0 || dtype > 1) return HIFT_ERR_CFG;
  if (cols > HIFT_STATIC_SCRATCH_MAX_COLS) return HIFT_ERR_CAPACITY;
  if ((dx || dgain) && (!dy || !x || !stats || !gain)) return HIFT_ERR_INPUT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return HIFT_ERR_CUDA;
  float* partial = g_static_partial_addr[dev].load(std::memory_order_relaxed);
  if (!partial) {
    // first call on this device (which is current): resolve the array's device address.  Two host threads
    // racing here both get the same answer from the runtime, so a relaxed store is enough.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_partial) != cudaSuccess || !p) { cudaGetLastError(); return HIFT_ERR_CUDA; }
    partial = (float*)p;
    g_static_partial_addr[dev].store(partial, std::memory_order_relaxed);
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (dx) launch_norm_bwd_dx(st, dtype, kind, false, rows, (int)cols, dy, x, stats, gain, add, dx, nullptr);
  if (dgain) launch_colreduce(st, dtype == 1, kind == 0 ? 1 : 2, rows, (int)cols, dy, cols, x, stats, partial, dgain, dbias);
  return cudaGetLastError() == cudaSuccess ? HIFT_OK : HIFT_ERR_CUDA;
}
