// C ABI of the MixLoRA FFN library: argument checks, workspace layout, and the sequence of
// kernel launches of the forward and backward passes.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace mixlora {

WsLayout ws_layout(const mixlora_shape_t& s, bool allow_fold) {
  WsLayout L;
  memset(&L, 0, sizeof(L));
  const size_t T = (size_t)s.tokens, d = (size_t)s.d_model, f = (size_t)s.d_ff, N = (size_t)s.n_experts,
               k = (size_t)s.top_k, r = (size_t)s.rank;
  const size_t E = act_size(s);
  const size_t nblk = (size_t)route_blocks(s.tokens);
  const size_t mt = (size_t)max_seg_tiles(s.tokens, s.top_k, s.n_experts);
  const size_t NP = (size_t)round_up8(s.n_experts);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + (bytes ? bytes : 1), 256);
    return o;
  };
  L.status = take(64 * 4);
  L.splitk_cnt = take(kSplitCounters * 4);
  L.probs = take(T * N * 4);
  L.expert_idx = take(T * k * 4);
  L.gates = take(T * k * 4);
  L.low_margin = take(T);
  L.perm = take(T * k * 4);
  L.inv = take(T * k * 4);
  L.pos_token = take(T * k * 4);
  L.pos_expert = take(T * k * 4);
  L.seg_off = take((N + 1) * 4);
  L.blk_counts = take(nblk * N * 4);
  L.blk_off = take(nblk * N * 4);
  L.stat_F = take(N * 4);
  L.stat_P = take(N * 4);
  L.stat_raw = take(2 * N * 4);
  L.stat_part = take((size_t)router_part_blocks(s.tokens) * 2 * N * 4);
  L.tile_info = take((mt * 4 + 4) * 4);
  L.G = take(T * f * E);
  L.U = take(T * f * E);
  L.zga = take(T * N * r * E);
  L.zua = take(T * N * r * E);
  const bool fold_zd = allow_fold && grouped_fwd_folds_zd(s);
  L.zd_all = take(fold_zd ? 0 : T * k * N * r * E);
  L.zd_part = take(fold_zd ? (size_t)grouped_fwd_max_groups(s.d_ff) * T * k * r * 4 : 0);
  L.Zs = take(T * N * r * E);
  L.bd_cat = take(d * N * r * E);
  L.bg_cat = take(f * N * r * E);
  L.bu_cat = take(f * N * r * E);
  L.Zg_pos = take(T * k * N * r * E);
  L.Zu_pos = take(T * k * N * r * E);
  const size_t rp = (size_t)pad_rank(s.rank);
  {
    L.zg_s = take(T * k * rp * E);
    L.zu_s = take(T * k * rp * E);
    const size_t padded = rp != r ? N * f * rp * E : 0;
    L.bgp = take(padded);
    L.bup = take(padded);
    L.adp = take(padded);
  }
  L.h_sorted = take(T * k * f * E);
  L.hbar = take(T * f * E);
  L.work_count = take(8 * 4);
  L.work_rows1 = take((size_t)rows_worklist_max(s.tokens * s.top_k, s.n_experts, 1) * 32);
  // rows of the tallest product (the per-slot ones of the weight-decomposed variant), columns of the widest (gate/up)
  L.splitk_bytes = s.dtype == MIXLORA_DTYPE_BF16 ? splitk_part_bytes((long long)(T * k), (long long)(2 * f + 2 * N * r)) : 0;
  L.splitk_part = take(L.splitk_bytes);
  L.total_fwd = off;
  L.D = L.hbar;                      // hbar (forward scratch) is dead once y is written; D = dy W_d takes its place
  L.spd = take(T * N * r * E);
  L.da_sorted = take(T * k * f * E);
  L.db_sorted = take(T * k * f * E);
  L.dabar = take(T * f * E);
  L.dbbar = take(T * f * E);
  L.p_s = take(T * k * rp * E);
  L.dZd_pos = take(T * k * N * r * E);
  L.dgate_part = take((size_t)grouped_swiglu_bwd_col_tiles(s.d_ff) * T * k * 4);
  const bool fold_dz = allow_fold && grouped_bwd_folds_dz(s);
  L.dzg_all = take(fold_dz ? 0 : T * k * N * r * E);
  L.dzu_all = take(fold_dz ? 0 : T * k * N * r * E);
  L.dz_part = take(fold_dz ? (size_t)grouped_bwd_max_groups(s.tokens, s.d_ff) * T * k * 2 * r * 4 : 0);
  L.dZg = take(T * N * r * E);
  L.dZu = take(T * N * r * E);
  L.dgate = take(T * k * 4);
  L.dlogits = take(T * N * 4);
  L.dl_act = take(T * NP * E);
  L.wr_act = take(NP * d * E);
  L.work_rows2 = take((size_t)rows_worklist_max(s.tokens * s.top_k, s.n_experts, 2) * 32);
  L.work_red = take((size_t)reduce_worklist_max(s.d_ff, s.n_experts, 3) * 32);
  L.total_bwd = off;
  return L;
}

namespace {

// ---- opt-in per-stage device timing and launch counting (host-side bookkeeping only) ----
enum Stage {
  ST_ROUTER, ST_DISPATCH, ST_GEMM_GATE_UP, ST_LORA_B_SWIGLU, ST_LORA_A_DOWN, ST_COMBINE_H, ST_GEMM_DOWN,
  ST_GEMM_DGRAD_DOWN, ST_SWIGLU_BWD, ST_LORA_DZ, ST_LORA_WGRAD, ST_ROUTER_BWD, ST_COMBINE_BWD, ST_GEMM_DX, ST_NORM, ST_COUNT
};
const char* const kStageNames[ST_COUNT] = {
    "router", "dispatch", "gemm_gate_up", "lora_b_swiglu", "lora_a_down", "combine_h", "gemm_down",
    "gemm_dgrad_down", "swiglu_bwd", "lora_dz", "lora_wgrad", "router_bwd", "combine_bwd", "gemm_dx", "norm"};

struct StageRec { int stage; cudaEvent_t a, b; };
struct Profiler {
  bool on = false;
  std::mutex mu;                                       // host threads may call into the library side by side
  std::vector<StageRec> recs;
  long long launches[ST_COUNT] = {0};
};
Profiler g_prof;

struct StageScope {
  int stage; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr; bool on;
  StageScope(int stage_, cudaStream_t st_, int launches) : stage(stage_), st(st_), on(g_prof.on) {
    { std::lock_guard<std::mutex> lock(g_prof.mu); g_prof.launches[stage] += launches; }
    if (on) {
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
      cudaEventRecord(a, st);
    }
  }
  ~StageScope() {
    if (on) {
      cudaEventRecord(b, st);
      std::lock_guard<std::mutex> lock(g_prof.mu);
      g_prof.recs.push_back({stage, a, b});
    }
  }
};

// ---- side streams ----
// Steps that do not depend on each other (the router and the dispatch beside the shared projections; the per-adapter
// steps of different adapters) are spread over a few library-owned streams between two points where everything is
// back on the caller's stream.  A call borrows a set of streams and events from a per-device list for the time
// between its fork and its join; the list's lock is held only while a set is picked or handed back, never across
// launches, so host threads that drive different layers or devices do not wait for each other.  Sets are created on
// first need (up to kMaxSideSets per device, kept until exit); with none free the call runs on the caller's stream.
constexpr int kSideStreams = 4;
constexpr int kMaxSideSets = 8;
constexpr int kMaxDevices = 64;
struct SideSet {
  cudaStream_t s[kSideStreams];
  cudaEvent_t fork, join[kSideStreams];
  bool busy = false;
};
struct DeviceSides {
  std::mutex mu;
  std::vector<SideSet*> sets;
};
DeviceSides g_sides[kMaxDevices];
std::atomic<int> g_serial{-1};                          // MIXLORA_OPT_SERIAL; -1 = take the default from the environment

bool serial_mode() {
  int v = g_serial.load(std::memory_order_relaxed);
  if (v < 0) {
    const char* e = getenv("MIXLORA_SERIAL");
    v = (e && e[0] == '1') ? 1 : 0;
    g_serial.store(v, std::memory_order_relaxed);
  }
  return v != 0;
}

SideSet* acquire_side_set(int* dev_out) {
  if (serial_mode()) return nullptr;                   // everything on the caller's stream, for measurements
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  *dev_out = dev;
  DeviceSides& D = g_sides[dev];
  std::lock_guard<std::mutex> lock(D.mu);
  for (SideSet* p : D.sets)
    if (!p->busy) { p->busy = true; return p; }
  if ((int)D.sets.size() >= kMaxSideSets) return nullptr;
  SideSet* p = new SideSet();
  bool ok = cudaEventCreateWithFlags(&p->fork, cudaEventDisableTiming) == cudaSuccess;
  int made = 0;
  for (int i = 0; i < kSideStreams && ok; ++i) {
    ok = cudaStreamCreateWithFlags(&p->s[i], cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&p->join[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok) ++made;
  }
  if (!ok) {                                           // nothing half-made stays behind
    for (int i = 0; i < made; ++i) { cudaStreamDestroy(p->s[i]); cudaEventDestroy(p->join[i]); }
    delete p;
    return nullptr;
  }
  p->busy = true;
  D.sets.push_back(p);
  return p;
}

void release_side_set(SideSet* p, int dev) {
  if (!p) return;
  std::lock_guard<std::mutex> lock(g_sides[dev].mu);
  p->busy = false;
}

// Runs fn(adapter context, index) for every adapter, on side streams when `spread` holds (and no stage timing
// is being taken, which needs one stream), else in turn on the caller's stream.  With `later` set the caller's
// stream is not made to wait yet: join_adapters() does that later, so that work enqueued on the caller's stream in
// between runs beside the adapters' steps.
struct Forked { SideSet* pool = nullptr; int used = 0; int dev = 0; };

mixlora_status_t join_adapters(cudaStream_t main_st, Forked& fk) {
  mixlora_status_t st = MIXLORA_OK;
  for (int j = 0; fk.pool && j < fk.used; ++j)
    if (cudaEventRecord(fk.pool->join[j], fk.pool->s[j]) != cudaSuccess ||
        cudaStreamWaitEvent(main_st, fk.pool->join[j], 0) != cudaSuccess)
      st = MIXLORA_ERR_CUDA;
  // the waits above are enqueued: later users of the set are ordered behind this call's work on its streams
  release_side_set(fk.pool, fk.dev);
  fk.pool = nullptr;
  return st;
}

template <typename F>
mixlora_status_t for_each_adapter(const Ctx* cs, int n, bool spread, F fn, Forked* later = nullptr) {
  Forked fk;
  SideSet* pool = (spread && !g_prof.on) ? acquire_side_set(&fk.dev) : nullptr;
  mixlora_status_t st = MIXLORA_OK;
  if (!pool) {
    for (int m = 0; m < n && st == MIXLORA_OK; ++m) st = fn(cs[m], m);
    return st;
  }
  cudaStream_t main_st = cs[0].st;
  if (cudaEventRecord(pool->fork, main_st) != cudaSuccess) {
    release_side_set(pool, fk.dev);
    return MIXLORA_ERR_CUDA;
  }
  fk.pool = pool;
  fk.used = n < kSideStreams ? n : kSideStreams;
  for (int j = 0; j < fk.used; ++j)
    if (cudaStreamWaitEvent(pool->s[j], pool->fork, 0) != cudaSuccess) st = MIXLORA_ERR_CUDA;
  for (int m = 0; m < n && st == MIXLORA_OK; ++m) {
    Ctx c = cs[m];
    c.st = pool->s[m % kSideStreams];
    st = fn(c, m);
  }
  if (later && st == MIXLORA_OK) {
    *later = fk;
    return st;
  }
  // rejoin at once (always after an error, so that no stream is left dangling)
  mixlora_status_t js = join_adapters(main_st, fk);
  return st == MIXLORA_OK ? js : st;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

mixlora_status_t check_shape(const mixlora_shape_t* s) {
  if (!s || s->struct_size != sizeof(mixlora_shape_t)) return MIXLORA_ERR_INVALID_ARG;
  if (s->tokens < 0 || s->d_model <= 0 || s->d_ff <= 0 || s->n_experts <= 0 || s->top_k <= 0 || s->rank <= 0)
    return MIXLORA_ERR_INVALID_ARG;
  if (s->top_k > s->n_experts) return MIXLORA_ERR_INVALID_ARG;
  if (s->dtype != MIXLORA_DTYPE_BF16 && s->dtype != MIXLORA_DTYPE_FP32) return MIXLORA_ERR_INVALID_ARG;
  if (!(s->lora_alpha == s->lora_alpha)) return MIXLORA_ERR_INVALID_ARG;
  if (s->aux_f_mode != 0 && s->aux_f_mode != 1) return MIXLORA_ERR_INVALID_ARG;
  if (s->renormalize != 0 && s->renormalize != 1) return MIXLORA_ERR_INVALID_ARG;
  if (s->d_model % 8 || s->d_ff % 8) return MIXLORA_ERR_UNSUPPORTED;
  if (s->n_experts > MIXLORA_MAX_EXPERTS || s->top_k > MIXLORA_MAX_TOP_K || s->rank > MIXLORA_MAX_RANK)
    return MIXLORA_ERR_UNSUPPORTED;
  if (s->dtype == MIXLORA_DTYPE_BF16 && s->rank % 8) return MIXLORA_ERR_UNSUPPORTED;
  if (s->dtype == MIXLORA_DTYPE_FP32 && s->rank % 4) return MIXLORA_ERR_UNSUPPORTED;
  if ((long long)s->tokens * s->top_k > 4000000LL) return MIXLORA_ERR_UNSUPPORTED;
  return MIXLORA_OK;
}

mixlora_status_t check_params(const mixlora_params_t* p) {
  if (!p) return MIXLORA_ERR_INVALID_ARG;
  const void* req[] = {p->x, p->w_gate, p->w_up, p->w_down, p->w_router, p->a_gate, p->b_gate,
                       p->a_up, p->b_up, p->a_down, p->b_down};
  for (const void* q : req)
    if (!q || !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
  if (p->router_bias && (reinterpret_cast<uintptr_t>(p->router_bias) & 3u)) return MIXLORA_ERR_INVALID_ARG;
  return MIXLORA_OK;
}

#define MIXLORA_CUDA(expr)                              \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) return MIXLORA_ERR_CUDA;    \
  } while (0)

Ctx make_ctx(const mixlora_shape_t* s, const mixlora_params_t* p, void* ws, void* stream) {
  Ctx c;
  c.s = *s;
  if (p) c.p = *p; else memset(&c.p, 0, sizeof(c.p));
  c.L = ws_layout(*s);
  c.ws = reinterpret_cast<char*>(ws);
  c.st = reinterpret_cast<cudaStream_t>(stream);
  c.bf16 = (s->dtype == MIXLORA_DTYPE_BF16);
  c.scale = s->lora_alpha / (float)s->rank;
  return c;
}

SGemm sgemm_base(const Ctx& c, void* C, long long c_sm, long long c_sn, int c_bf16, int M, int N) {
  SGemm g;
  memset(&g, 0, sizeof(g));
  g.C = C; g.c_sm = c_sm; g.c_sn = c_sn; g.c_sg = 0; g.c_is_bf16 = c_bf16;
  g.M = M; g.N = N; g.groups = 1; g.group_mode = 0; g.alpha = 1.f; g.accumulate = 0; g.nseg = 0;
  g.seg_off = c.at<int>(c.L.seg_off);
  return g;
}

void add_seg(SGemm& g, const SOperand& A, const SOperand& B, int K) {
  g.A[g.nseg] = A; g.B[g.nseg] = B; g.K[g.nseg] = K; ++g.nseg;
}

// Dense product on the tensor-core kernel when it takes the shape, else on the SIMT kernel.
// `split`: the launch may share the reductions of its last round's tiles among the CTA pairs that round would leave
// idle, through the workspace's split scratch: the frozen-projection products, which follow each other on the
// caller's stream (one such launch at a time per workspace).
cudaError_t dense_product(const Ctx& c, int M, const TcOut* outs, int nout, const TcWork* wl = nullptr,
                          bool split = false) {
  if (nout == 0 || M <= 0) return cudaSuccess;
  if (c.bf16 && tc_gemm_supported(M, outs, nout)) {
    TcSplit sp{c.at<float>(c.L.splitk_part), c.L.splitk_bytes, c.at<int>(c.L.splitk_cnt), kSplitCounters};
    return launch_tc_gemm(M, outs, nout, c.at<int>(c.L.status), c.st, wl,   // the SIMT kernel below computes every block
                          split && c.L.splitk_bytes ? &sp : nullptr);
  }
  for (int o = 0; o < nout; ++o) {
    const TcOut& t = outs[o];
    const int Mo = t.M > 0 ? t.M : M;
    SGemm g = t.mode == 0 ? sgemm_base(c, t.C, t.ldc, 1, c.bf16, Mo, t.N) : sgemm_base(c, t.C, t.s_m, t.s_n, 0, Mo, t.N);
    g.alpha = t.alpha;
    if (t.mode == 1) { g.c_nb = t.nb; g.c_sblk = t.s_blk; g.accumulate = t.accumulate; }
    for (int i = 0; i < t.nseg; ++i) {
      const TcSeg& sg = t.seg[i];
      SOperand A = sg.a_mn ? soperand(sg.A, 1, sg.lda, c.bf16) : soperand(sg.A, sg.lda, 1, c.bf16);
      SOperand B = sg.b_kn ? soperand(sg.B, 1, sg.ldb, c.bf16) : soperand(sg.B, sg.ldb, 1, c.bf16);
      add_seg(g, A, B, sg.K);
    }
    cudaError_t e = launch_simt_gemm(g, c.st);
    if (e != cudaSuccess) return e;
    if (t.mode == 0 && t.R && (e = launch_residual_add(c, t.C, t.ldc, t.R, t.ldr, Mo, t.N)) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// The LoRA-side products against every expert's block are scheduled block-sparsely (device-built work lists) once
// the N r columns span more than one 128-column tile; up to one tile the dense form does no extra loads and has
// fewer, longer work items, which measured faster.
bool block_sparse(const Ctx& c) { return c.s.n_experts * c.s.rank > 128; }

int dense_launches(const Ctx& c, int M, const TcOut* outs, int nout) {
  if (nout == 0 || M <= 0) return 0;
  return (c.bf16 && tc_gemm_supported(M, outs, nout)) ? 1 : nout;
}

// activation-type output [M, N] row-major
TcOut tc_out(void* C, long long ldc, int N) {
  TcOut o;
  memset(&o, 0, sizeof(o));
  o.C = C; o.ldc = ldc; o.N = N; o.mode = 0; o.alpha = 1.f; o.nseg = 0;
  return o;
}
// fp32 output at C + (n / nb) * s_blk + (n % nb) * s_n + m * s_m
TcOut tc_out_f32(float* C, int N, long long s_m, long long s_n, int nb, long long s_blk, float alpha, int accumulate) {
  TcOut o;
  memset(&o, 0, sizeof(o));
  o.C = C; o.N = N; o.mode = 1; o.s_m = s_m; o.s_n = s_n; o.nb = nb; o.s_blk = s_blk; o.alpha = alpha;
  o.accumulate = accumulate; o.nseg = 0;
  return o;
}
void tc_add(TcOut& o, const void* A, long long lda, int K, const void* B, long long ldb, int b_kn, int a_mn = 0,
            int b_cols = 0) {
  TcSeg& s = o.seg[o.nseg++];
  s.A = A; s.lda = lda; s.a_mn = a_mn; s.K = K; s.B = B; s.ldb = ldb; s.b_kn = b_kn; s.b_cols = b_cols;
}

}  // namespace
}  // namespace mixlora

using namespace mixlora;

extern "C" {

void mixlora_limits(mixlora_limits_t* out) {
  if (!out) return;
  out->max_experts = MIXLORA_MAX_EXPERTS;
  out->max_top_k = MIXLORA_MAX_TOP_K;
  out->max_rank = MIXLORA_MAX_RANK;
}

const char* mixlora_status_string(mixlora_status_t st) {
  switch (st) {
    case MIXLORA_OK: return "ok";
    case MIXLORA_ERR_INVALID_ARG: return "invalid argument";
    case MIXLORA_ERR_UNSUPPORTED: return "size outside the supported limits";
    case MIXLORA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MIXLORA_ERR_CUDA: return "CUDA call failed";
    case MIXLORA_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
  }
  return "unknown status";
}

size_t mixlora_workspace_bytes(const mixlora_shape_t* shape, int for_backward) {
  if (check_shape(shape) != MIXLORA_OK) return 0;
  WsLayout L = ws_layout(*shape);
  return for_backward ? L.total_bwd : L.total_fwd;
}

// ---- forward, in three steps so that several adapters can share the frozen-projection launch ----
static mixlora_status_t fwd_check(const mixlora_shape_t* shape, const mixlora_params_t* params, void* y,
                                  void* workspace, size_t workspace_bytes, void* stream, Ctx* out) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  st = check_params(params);
  if (st != MIXLORA_OK) return st;
  if (!y || !aligned16(y)) return MIXLORA_ERR_INVALID_ARG;
  *out = make_ctx(shape, params, workspace, stream);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < out->L.total_fwd)
    return MIXLORA_ERR_WORKSPACE;
  return MIXLORA_OK;
}

// router (Eq. 7) and dispatch
static mixlora_status_t fwd_clear_status(const Ctx& c) {
  MIXLORA_CUDA(cudaMemsetAsync(c.ws + c.L.status, 0, 256 + kSplitCounters * 4, c.st));   // status, then the split counters
  return MIXLORA_OK;
}
static mixlora_status_t fwd_route_only(const Ctx& c) {
  if (c.s.tokens == 0) return MIXLORA_OK;
  { StageScope ss(ST_ROUTER, c.st, 2); MIXLORA_CUDA(launch_router(c)); }
  { StageScope ss(ST_DISPATCH, c.st, 3); MIXLORA_CUDA(launch_dispatch(c)); }
  return MIXLORA_OK;
}
// repacks that depend on the parameters only (s B_d, s B_g, s B_u with all experts' blocks side by side); the
// backward pass finds them in the workspace
static mixlora_status_t fwd_repacks(const Ctx& c) {
  if (c.s.tokens == 0) return MIXLORA_OK;
  { StageScope ss(ST_DISPATCH, c.st, 3); MIXLORA_CUDA(launch_bd_cat(c)); MIXLORA_CUDA(launch_bgu_cat(c)); }
  return MIXLORA_OK;
}
static mixlora_status_t fwd_route(const Ctx& c) {
  const mixlora_status_t st = fwd_route_only(c);
  return st == MIXLORA_OK ? fwd_repacks(c) : st;
}
// One adapter: the routing chain and the repacks do not depend on each other and take a side stream each.
static mixlora_status_t fwd_route_forked(const Ctx& c, Forked* fk) {
  const Ctx two[2] = {c, c};
  return for_each_adapter(two, 2, true, [&](const Ctx& cc, int m) { return m == 0 ? fwd_route_only(cc) : fwd_repacks(cc); },
                          fk);
}

// Shared gate / up projections, once per token (Section 3.3 (I)), for one adapter (then the LoRA-A columns of every
// expert ride along in the same pass over x) or for two adapters that share W1, W3 (Section 3.3 (II): their tokens
// go through the frozen weights in one launch; each adapter's LoRA-A product follows on its own).
static mixlora_status_t fwd_shared_projections(const Ctx* cs, int n) {
  TcOut outs[4];
  int no = 0, Tmax = 0;
  for (int i = 0; i < n; ++i) {
    const Ctx& c = cs[i];
    const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff;
    if (T == 0) continue;
    Tmax = T > Tmax ? T : Tmax;
    outs[no] = tc_out(c.ws + c.L.G, f, f); outs[no].M = T; tc_add(outs[no++], c.p.x, d, d, c.p.w_gate, d, 0);
    outs[no] = tc_out(c.ws + c.L.U, f, f); outs[no].M = T; tc_add(outs[no++], c.p.x, d, d, c.p.w_up, d, 0);
  }
  if (no == 0) return MIXLORA_OK;
  const Ctx& c0 = cs[0].s.tokens ? cs[0] : cs[n - 1];
  if (n == 1) {
    const Ctx& c = cs[0];
    const int T = c.s.tokens, d = c.s.d_model, Nr = c.s.n_experts * c.s.rank;
    outs[2] = tc_out(c.ws + c.L.zga, Nr, Nr); tc_add(outs[2], c.p.x, d, d, c.p.a_gate, d, 0);
    outs[3] = tc_out(c.ws + c.L.zua, Nr, Nr); tc_add(outs[3], c.p.x, d, d, c.p.a_up, d, 0);
    StageScope ss(ST_GEMM_GATE_UP, c.st, dense_launches(c, T, outs, 4));
    MIXLORA_CUDA(dense_product(c, T, outs, 4, nullptr, true));
    return MIXLORA_OK;
  }
  {
    StageScope ss(ST_GEMM_GATE_UP, c0.st, dense_launches(c0, Tmax, outs, no));
    MIXLORA_CUDA(dense_product(c0, Tmax, outs, no, nullptr, true));
  }
  for (int i = 0; i < n; ++i) {
    const Ctx& c = cs[i];
    const int T = c.s.tokens, d = c.s.d_model, Nr = c.s.n_experts * c.s.rank;
    if (T == 0) continue;
    TcOut z[2];
    z[0] = tc_out(c.ws + c.L.zga, Nr, Nr); tc_add(z[0], c.p.x, d, d, c.p.a_gate, d, 0);
    z[1] = tc_out(c.ws + c.L.zua, Nr, Nr); tc_add(z[1], c.p.x, d, d, c.p.a_up, d, 0);
    StageScope ss(ST_GEMM_GATE_UP, c.st, dense_launches(c, T, z, 2));
    MIXLORA_CUDA(dense_product(c, T, z, 2));
  }
  return MIXLORA_OK;
}

// everything after the shared projections: per-expert deltas, SwiGLU, down projection, combine
// `residual` (optional, [T, d] of the activation type) is added to y in the down product's epilogue (Eq. 6).
static mixlora_status_t fwd_experts_main(const Ctx& c, void* y, const void* residual, bool zpos_here);
// `zpos_aside`: the scatter of zg, zu into the slots' expert blocks, which only the backward pass reads, goes to a
// side stream that joins the caller's stream at the end (not for callers that already run on a side stream).
static mixlora_status_t fwd_experts(const Ctx& c, void* y, const void* residual = nullptr, bool zpos_aside = false) {
  if (c.s.tokens == 0) return MIXLORA_OK;
  if (!zpos_aside) return fwd_experts_main(c, y, residual, true);
  Forked fk;
  mixlora_status_t st = for_each_adapter(&c, 1, true, [&](const Ctx& cc, int) -> mixlora_status_t {
    StageScope ss(ST_LORA_B_SWIGLU, cc.st, 1);
    MIXLORA_CUDA(launch_zpos(cc));
    return MIXLORA_OK;
  }, &fk);
  if (st == MIXLORA_OK) st = fwd_experts_main(c, y, residual, false);
  const mixlora_status_t js = join_adapters(c.st, fk);
  return st != MIXLORA_OK ? st : js;
}
static mixlora_status_t fwd_experts_main(const Ctx& c, void* y, const void* residual, bool zpos_here) {
  const mixlora_params_t* params = &c.p;
  const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank, k = c.s.top_k;
  const int Nr = N * r;
  // per-slot LoRA-B expansion + SwiGLU
  {
    StageScope ss(ST_LORA_B_SWIGLU, c.st, zpos_here ? 3 : 2);
    if (zpos_here) MIXLORA_CUDA(launch_zpos(c));
    if (grouped_swiglu_supported(c)) {
      MIXLORA_CUDA(launch_zcompact(c));
      MIXLORA_CUDA(launch_grouped_swiglu_fwd(c));
    } else {
      MIXLORA_CUDA(launch_lora_b_swiglu(c));
    }
  }
  // zd = A_d h per slot, against every expert's A_d (the slot's own block is picked up by the combine); not when
  // the grouped kernel above has formed it from the tiles it held
  if (!ctx_folds_zd(c)) {
    TcOut out = tc_out(c.ws + c.L.zd_all, Nr, Nr);
    tc_add(out, c.ws + c.L.h_sorted, f, f, params->a_down, f, 0);
    StageScope ss(ST_LORA_A_DOWN, c.st, (block_sparse(c) ? 1 : 0) + dense_launches(c, T * k, &out, 1));
    // only the block of a slot's own expert is needed: schedule (row tile, expert) pairs that exist
    TcWork wl = {c.at<int>(c.L.work_rows1), c.at<int>(c.L.work_count) + 0, rows_worklist_max(T * k, N, 1), r};
    if (block_sparse(c))
      MIXLORA_CUDA(launch_rows_worklist(c, tc_gemm_tile_rows(T * k), 1, (f + 63) / 64, c.at<int>(c.L.work_rows1),
                                        c.at<int>(c.L.work_count) + 0));
    MIXLORA_CUDA(dense_product(c, T * k, &out, 1, block_sparse(c) ? &wl : nullptr));
  }
  { StageScope ss(ST_COMBINE_H, c.st, c.bf16 ? 2 : 1); MIXLORA_CUDA(launch_combine_h(c)); }
  // y = [hbar | Zs] [W_d | s B_d]^T : the frozen down projection acts once on the gate-weighted sum of a
  // token's slots (W_d is linear and shared), its LoRA rides along as extra reduction columns
  {
    TcOut out = tc_out(y, d, d);
    out.R = residual; out.ldr = d;
    tc_add(out, c.ws + c.L.hbar, f, f, params->w_down, f, 0);
    tc_add(out, c.ws + c.L.Zs, Nr, Nr, c.ws + c.L.bd_cat, Nr, 0);
    StageScope ss(ST_GEMM_DOWN, c.st, dense_launches(c, T, &out, 1));
    MIXLORA_CUDA(dense_product(c, T, &out, 1, nullptr, true));
  }
  return MIXLORA_OK;
}

mixlora_status_t mixlora_ffn_forward(const mixlora_shape_t* shape, const mixlora_params_t* params, void* y,
                                     void* workspace, size_t workspace_bytes, void* stream) {
  Ctx c;
  mixlora_status_t st = fwd_check(shape, params, y, workspace, workspace_bytes, stream, &c);
  if (st != MIXLORA_OK) return st;
  if ((st = fwd_clear_status(c)) != MIXLORA_OK) return st;
  // the router and the dispatch need only x: they run on a side stream beside the shared projections
  Forked fk;
  if ((st = fwd_route_forked(c, &fk)) != MIXLORA_OK)
    return st;
  st = fwd_shared_projections(&c, 1);
  mixlora_status_t js = join_adapters(c.st, fk);
  if (st != MIXLORA_OK || js != MIXLORA_OK) return st != MIXLORA_OK ? st : js;
  return fwd_experts(c, y, nullptr, true);
}

static bool same_frozen_ffn(const Ctx& a, const Ctx& b) {
  return a.s.d_model == b.s.d_model && a.s.d_ff == b.s.d_ff && a.s.dtype == b.s.dtype && a.p.w_gate == b.p.w_gate &&
         a.p.w_up == b.p.w_up && a.p.w_down == b.p.w_down;
}

mixlora_status_t mixlora_multi_ffn_forward(int32_t n_models, const mixlora_shape_t* shapes,
                                           const mixlora_params_t* params, void* const* y, void* const* workspaces,
                                           const size_t* workspace_bytes, void* stream) {
  if (n_models < 1 || n_models > MIXLORA_MAX_MODELS || !shapes || !params || !y || !workspaces || !workspace_bytes)
    return MIXLORA_ERR_INVALID_ARG;
  Ctx cs[MIXLORA_MAX_MODELS];
  for (int m = 0; m < n_models; ++m) {
    mixlora_status_t st = fwd_check(&shapes[m], &params[m], y[m], workspaces[m], workspace_bytes[m], stream, &cs[m]);
    if (st != MIXLORA_OK) return st;
    if (!same_frozen_ffn(cs[0], cs[m])) return MIXLORA_ERR_INVALID_ARG;   // the adapters must share one frozen FFN
    for (int o = 0; o < m; ++o)
      if (workspaces[o] == workspaces[m] || y[o] == y[m]) return MIXLORA_ERR_INVALID_ARG;
  }
  mixlora_status_t st;
  for (int m = 0; m < n_models; ++m)
    if ((st = fwd_clear_status(cs[m])) != MIXLORA_OK) return st;
  Forked fk;
  if ((st = for_each_adapter(cs, n_models, true, [&](const Ctx& c, int) { return fwd_route(c); }, &fk)) != MIXLORA_OK)
    return st;
  for (int m = 0; m < n_models && st == MIXLORA_OK; m += 2)
    st = fwd_shared_projections(&cs[m], n_models - m >= 2 ? 2 : 1);
  mixlora_status_t js = join_adapters(cs[0].st, fk);
  if (st != MIXLORA_OK || js != MIXLORA_OK) return st != MIXLORA_OK ? st : js;
  return for_each_adapter(cs, n_models, n_models > 1, [&](const Ctx& c, int m) { return fwd_experts(c, y[m]); });
}

mixlora_status_t mixlora_aux_loss(const mixlora_shape_t* shape, const void* workspace, float coef, float* loss,
                                  float* F, float* P, void* stream) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MIXLORA_ERR_WORKSPACE;
  if (!loss) return MIXLORA_ERR_INVALID_ARG;
  Ctx c = make_ctx(shape, nullptr, const_cast<void*>(workspace), stream);
  if (shape->tokens == 0) {
    MIXLORA_CUDA(cudaMemsetAsync(loss, 0, sizeof(float), c.st));
    if (F) MIXLORA_CUDA(cudaMemsetAsync(F, 0, sizeof(float) * shape->n_experts, c.st));
    if (P) MIXLORA_CUDA(cudaMemsetAsync(P, 0, sizeof(float) * shape->n_experts, c.st));
    return MIXLORA_OK;
  }
  { StageScope ss(ST_ROUTER, c.st, 1); MIXLORA_CUDA(launch_aux_loss(c, coef, loss, F, P)); }
  return MIXLORA_OK;
}

mixlora_status_t mixlora_aux_stats(const mixlora_shape_t* shape, const void* workspace, float* prob_sum, float* count,
                                   void* stream) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MIXLORA_ERR_WORKSPACE;
  if (!prob_sum || !count) return MIXLORA_ERR_INVALID_ARG;
  Ctx c = make_ctx(shape, nullptr, const_cast<void*>(workspace), stream);
  const size_t nb = sizeof(float) * shape->n_experts;
  if (shape->tokens == 0) {
    MIXLORA_CUDA(cudaMemsetAsync(prob_sum, 0, nb, c.st));
    MIXLORA_CUDA(cudaMemsetAsync(count, 0, nb, c.st));
    return MIXLORA_OK;
  }
  const float* raw = c.at<float>(c.L.stat_raw);
  MIXLORA_CUDA(cudaMemcpyAsync(prob_sum, raw, nb, cudaMemcpyDeviceToDevice, c.st));
  MIXLORA_CUDA(cudaMemcpyAsync(count, raw + shape->n_experts, nb, cudaMemcpyDeviceToDevice, c.st));
  return MIXLORA_OK;
}

mixlora_status_t mixlora_aux_loss_global(const mixlora_shape_t* shape, void* workspace, float coef,
                                         const float* prob_sum, const float* count, int64_t total_tokens, float* loss,
                                         float* F, float* P, void* stream) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MIXLORA_ERR_WORKSPACE;
  if (!loss || !prob_sum || !count || total_tokens < shape->tokens || total_tokens <= 0) return MIXLORA_ERR_INVALID_ARG;
  Ctx c = make_ctx(shape, nullptr, workspace, stream);
  { StageScope ss(ST_ROUTER, c.st, 1); MIXLORA_CUDA(launch_aux_loss_global(c, coef, prob_sum, count, total_tokens, loss, F, P)); }
  return MIXLORA_OK;
}

// ---- backward, split the same way: checks, the shared dy W_d launch, the rest ----
static mixlora_status_t bwd_check(const mixlora_shape_t* shape, const mixlora_params_t* params, const void* dy,
                                  void* workspace, size_t workspace_bytes, const mixlora_grads_t* grads, void* stream,
                                  Ctx* out) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  st = check_params(params);
  if (st != MIXLORA_OK) return st;
  if (!dy || !aligned16(dy) || !grads) return MIXLORA_ERR_INVALID_ARG;
  {
    const void* outs[] = {grads->d_a_gate, grads->d_b_gate, grads->d_a_up, grads->d_b_up, grads->d_a_down,
                          grads->d_b_down, grads->d_w_router, grads->d_x};
    for (const void* q : outs)
      if (q && !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
    if (grads->accumulate != 0 && grads->accumulate != 1) return MIXLORA_ERR_INVALID_ARG;
  }
  *out = make_ctx(shape, params, workspace, stream);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < out->L.total_bwd)
    return MIXLORA_ERR_WORKSPACE;
  return MIXLORA_OK;
}

// D = dy W_d (shared by a token's slots) and s B_d^T dy for every expert; two adapters that share W_d send their
// dy through it in one launch
static mixlora_status_t bwd_shared_dgrad(const Ctx* cs, const void* const* dys, int n) {
  if (n == 1) {
    const Ctx& c = cs[0];
    const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff, Nr = c.s.n_experts * c.s.rank;
    if (T == 0) return MIXLORA_OK;
    TcOut outs[2];
    outs[0] = tc_out(c.ws + c.L.D, f, f);      tc_add(outs[0], dys[0], d, d, c.p.w_down, f, 1);
    outs[1] = tc_out(c.ws + c.L.spd, Nr, Nr);  tc_add(outs[1], dys[0], d, d, c.ws + c.L.bd_cat, Nr, 1);
    StageScope ss(ST_GEMM_DGRAD_DOWN, c.st, dense_launches(c, T, outs, 2));
    MIXLORA_CUDA(dense_product(c, T, outs, 2, nullptr, true));   // bd_cat is the forward pass's
    return MIXLORA_OK;
  }
  TcOut outs[2];
  int no = 0, Tmax = 0, last = 0;
  for (int i = 0; i < n; ++i) {
    const Ctx& c = cs[i];
    const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff;
    if (T == 0) continue;
    Tmax = T > Tmax ? T : Tmax;
    last = i;
    outs[no] = tc_out(c.ws + c.L.D, f, f); outs[no].M = T; tc_add(outs[no++], dys[i], d, d, c.p.w_down, f, 1);
  }
  if (no == 0) return MIXLORA_OK;
  {
    const Ctx& c0 = cs[last];
    StageScope ss(ST_GEMM_DGRAD_DOWN, c0.st, dense_launches(c0, Tmax, outs, no));
    MIXLORA_CUDA(dense_product(c0, Tmax, outs, no, nullptr, true));
  }
  for (int i = 0; i < n; ++i) {
    const Ctx& c = cs[i];
    const int T = c.s.tokens, d = c.s.d_model, Nr = c.s.n_experts * c.s.rank;
    if (T == 0) continue;
    TcOut z = tc_out(c.ws + c.L.spd, Nr, Nr);
    tc_add(z, dys[i], d, d, c.ws + c.L.bd_cat, Nr, 1);
    StageScope ss(ST_GEMM_DGRAD_DOWN, c.st, dense_launches(c, T, &z, 1));
    MIXLORA_CUDA(dense_product(c, T, &z, 1));
  }
  return MIXLORA_OK;
}

static mixlora_status_t bwd_zero_tokens(const Ctx& c, const mixlora_grads_t* grads) {
  const int d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank;
  if (!grads->accumulate) {
    struct { float* p; size_t n; } z[] = {
        {grads->d_a_gate, (size_t)N * r * d}, {grads->d_b_gate, (size_t)N * f * r}, {grads->d_a_up, (size_t)N * r * d},
        {grads->d_b_up, (size_t)N * f * r},   {grads->d_a_down, (size_t)N * r * f}, {grads->d_b_down, (size_t)N * d * r},
        {grads->d_w_router, (size_t)N * d},   {grads->d_router_bias, (size_t)N}};
    for (auto& q : z)
      if (q.p) MIXLORA_CUDA(cudaMemsetAsync(q.p, 0, q.n * sizeof(float), c.st));
  }
  return MIXLORA_OK;
}

// `param_grads_ready` (optional cudaEvent_t) is recorded once every LoRA / router gradient has been enqueued, before
// the input-gradient product: a caller's gradient all-reduce can then overlap that product.
// `may_fork`: the gate-gradient reduction and the router's backward step may go to a side stream beside the dense
// products that do not need them (not when this call already runs on a side stream).
static mixlora_status_t bwd_experts(const Ctx& c, const void* dy, float aux_coef, const mixlora_grads_t* grads,
                                    void* param_grads_ready = nullptr, bool may_fork = true) {
  const mixlora_params_t* params = &c.p;
  const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank, k = c.s.top_k;
  const int Nr = N * r, NP = round_up8(N);
  const int acc = grads->accumulate;
  const int want_dx = grads->d_x != nullptr;
  if (T == 0) {
    mixlora_status_t zs = bwd_zero_tokens(c, grads);
    if (zs == MIXLORA_OK && param_grads_ready)
      MIXLORA_CUDA(cudaEventRecord(reinterpret_cast<cudaEvent_t>(param_grads_ready), c.st));
    return zs;
  }
  int dgate_tiles = 0;                                 // > 0: the per-column-tile partial sums still have to be added
  {
    StageScope ss(ST_SWIGLU_BWD, c.st, 2);
    MIXLORA_CUDA(launch_slot_prep_bwd(c));
    if (grouped_swiglu_supported(c)) {
      MIXLORA_CUDA(launch_grouped_swiglu_bwd(c));
      dgate_tiles = grouped_swiglu_bwd_col_tiles(f);
    } else {
      MIXLORA_CUDA(launch_swiglu_bwd(c));
    }
  }
  // router: gate gradients -> probabilities -> logits.  Nothing before the d-sized weight gradients needs the
  // result, so these small launches run beside the dense products below.
  Forked router_fk;
  {
    mixlora_status_t st = for_each_adapter(
        &c, 1, may_fork,
        [&](const Ctx& cc, int) {
          if (dgate_tiles > 0) {
            StageScope ss(ST_SWIGLU_BWD, cc.st, 1);
            MIXLORA_CUDA(launch_dgate_reduce(cc, dgate_tiles));
          }
          StageScope ss(ST_ROUTER_BWD, cc.st, 1 + (grads->d_router_bias ? 1 : 0) + (want_dx ? 1 : 0));
          MIXLORA_CUDA(launch_router_bwd(cc, aux_coef, grads->d_router_bias, acc, want_dx));
          return MIXLORA_OK;
        },
        &router_fk);
    if (st != MIXLORA_OK) return st;
  }
  // from here to the join every early return has to hand the side stream back
#define MIXLORA_CUDA_FK(expr)                                   \
  do {                                                          \
    if ((expr) != cudaSuccess) {                                \
      join_adapters(c.st, router_fk);                           \
      return MIXLORA_ERR_CUDA;                                  \
    }                                                           \
  } while (0)
  // dzg = da (s B_g), dzu = db (s B_u), against every expert (the slot's own block is used); not when the grouped
  // kernel above has formed them from the tiles it held
  if (!ctx_folds_dz(c)) {
    TcOut outs[2];
    outs[0] = tc_out(c.ws + c.L.dzg_all, Nr, Nr); tc_add(outs[0], c.ws + c.L.da_sorted, f, f, c.ws + c.L.bg_cat, Nr, 1);
    outs[1] = tc_out(c.ws + c.L.dzu_all, Nr, Nr); tc_add(outs[1], c.ws + c.L.db_sorted, f, f, c.ws + c.L.bu_cat, Nr, 1);
    StageScope ss(ST_LORA_DZ, c.st, (block_sparse(c) ? 1 : 0) + dense_launches(c, T * k, outs, 2));
    TcWork wl = {c.at<int>(c.L.work_rows2), c.at<int>(c.L.work_count) + 1, rows_worklist_max(T * k, N, 2), r};
    if (block_sparse(c))
      MIXLORA_CUDA_FK(launch_rows_worklist(c, tc_gemm_tile_rows(T * k), 2, (f + 63) / 64, c.at<int>(c.L.work_rows2),
                                           c.at<int>(c.L.work_count) + 1));
    MIXLORA_CUDA_FK(dense_product(c, T * k, outs, 2, block_sparse(c) ? &wl : nullptr));
  }
  { StageScope ss(ST_COMBINE_BWD, c.st, (c.bf16 && want_dx) ? 2 : 1); MIXLORA_CUDA_FK(launch_combine_bwd(c, want_dx)); }
  // LoRA and router weight gradients.  Reduction over the sorted slots (f-sized matrices) ...
  {
    TcOut outs[3];
    int n = 0;
    if (grads->d_b_gate) {   // dB_g[e][f'][rr] = s sum_pos da[pos][f'] zg[pos][rr]
      outs[n] = tc_out_f32(grads->d_b_gate, Nr, r, 1, r, (long long)f * r, c.scale, acc);
      tc_add(outs[n++], c.ws + c.L.da_sorted, f, T * k, c.ws + c.L.Zg_pos, Nr, 1, 1);
    }
    if (grads->d_b_up) {
      outs[n] = tc_out_f32(grads->d_b_up, Nr, r, 1, r, (long long)f * r, c.scale, acc);
      tc_add(outs[n++], c.ws + c.L.db_sorted, f, T * k, c.ws + c.L.Zu_pos, Nr, 1, 1);
    }
    if (grads->d_a_down) {   // dA_d[e][rr][f'] = sum_pos (g s pd)[pos][rr] h[pos][f']
      outs[n] = tc_out_f32(grads->d_a_down, Nr, 1, f, 0, 0, 1.f, acc);
      tc_add(outs[n++], c.ws + c.L.h_sorted, f, T * k, c.ws + c.L.dZd_pos, Nr, 1, 1);
    }
    StageScope ss(ST_LORA_WGRAD, c.st, (block_sparse(c) ? 1 : 0) + dense_launches(c, f, outs, n));
    if (n > 0) {
      // each expert's block is a sum over that expert's segment of sorted slots only
      TcWork wl = {c.at<int>(c.L.work_red), c.at<int>(c.L.work_count) + 2, reduce_worklist_max(f, N, n), r};
      if (block_sparse(c))
        MIXLORA_CUDA_FK(launch_reduce_worklist(c, f, tc_gemm_tile_rows(f), n, c.at<int>(c.L.work_red),
                                               c.at<int>(c.L.work_count) + 2));
      MIXLORA_CUDA_FK(dense_product(c, f, outs, n, block_sparse(c) ? &wl : nullptr));
    }
  }
#undef MIXLORA_CUDA_FK
  if (join_adapters(c.st, router_fk) != MIXLORA_OK) return MIXLORA_ERR_CUDA;   // dl and the router terms are needed now
  // ... and over the tokens (d-sized matrices and the router weight)
  {
    TcOut outs[4];
    int n = 0;
    if (grads->d_a_gate) {   // dA_g[e][rr][c] = sum_t dzg[t][e*r+rr] x[t][c]
      outs[n] = tc_out_f32(grads->d_a_gate, Nr, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dZg, Nr, 1, 1);
    }
    if (grads->d_a_up) {
      outs[n] = tc_out_f32(grads->d_a_up, Nr, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dZu, Nr, 1, 1);
    }
    if (grads->d_b_down) {   // dB_d[e][c][rr] = s sum_t dy[t][c] (g zd)[t][e*r+rr]
      outs[n] = tc_out_f32(grads->d_b_down, Nr, r, 1, r, (long long)d * r, c.scale, acc);
      tc_add(outs[n++], dy, d, T, c.ws + c.L.Zs, Nr, 1, 1);
    }
    if (grads->d_w_router) {   // dW_r[i][c] = sum_t dl[t][i] x[t][c]
      outs[n] = tc_out_f32(grads->d_w_router, N, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dl_act, NP, 1, 1, NP);
    }
    StageScope ss(ST_LORA_WGRAD, c.st, dense_launches(c, d, outs, n));
    MIXLORA_CUDA(dense_product(c, d, outs, n));
  }
  if (param_grads_ready) MIXLORA_CUDA(cudaEventRecord(reinterpret_cast<cudaEvent_t>(param_grads_ready), c.st));
  if (want_dx) {
    // dx = [dabar | dbbar | dZg | dZu | dl] [W_g ; W_u ; A_g ; A_u ; W_r]
    TcOut out = tc_out(grads->d_x, d, d);
    tc_add(out, c.ws + c.L.dabar, f, f, params->w_gate, d, 1);
    tc_add(out, c.ws + c.L.dbbar, f, f, params->w_up, d, 1);
    tc_add(out, c.ws + c.L.dZg, Nr, Nr, params->a_gate, d, 1);
    tc_add(out, c.ws + c.L.dZu, Nr, Nr, params->a_up, d, 1);
    tc_add(out, c.ws + c.L.dl_act, NP, NP, c.ws + c.L.wr_act, d, 1);
    StageScope ss(ST_GEMM_DX, c.st, dense_launches(c, T, &out, 1));
    MIXLORA_CUDA(dense_product(c, T, &out, 1, nullptr, true));
  }
  return MIXLORA_OK;
}

mixlora_status_t mixlora_ffn_backward(const mixlora_shape_t* shape, const mixlora_params_t* params, const void* dy,
                                      float aux_coef, void* workspace, size_t workspace_bytes,
                                      const mixlora_grads_t* grads, void* stream) {
  Ctx c;
  mixlora_status_t st = bwd_check(shape, params, dy, workspace, workspace_bytes, grads, stream, &c);
  if (st != MIXLORA_OK) return st;
  if ((st = bwd_shared_dgrad(&c, &dy, 1)) != MIXLORA_OK) return st;
  return bwd_experts(c, dy, aux_coef, grads);
}

mixlora_status_t mixlora_ffn_backward_overlap(const mixlora_shape_t* shape, const mixlora_params_t* params,
                                              const void* dy, float aux_coef, void* workspace, size_t workspace_bytes,
                                              const mixlora_grads_t* grads, void* param_grads_ready, void* stream) {
  Ctx c;
  mixlora_status_t st = bwd_check(shape, params, dy, workspace, workspace_bytes, grads, stream, &c);
  if (st != MIXLORA_OK) return st;
  if ((st = bwd_shared_dgrad(&c, &dy, 1)) != MIXLORA_OK) return st;
  return bwd_experts(c, dy, aux_coef, grads, param_grads_ready);
}

mixlora_status_t mixlora_multi_ffn_backward(int32_t n_models, const mixlora_shape_t* shapes,
                                            const mixlora_params_t* params, const void* const* dy,
                                            const float* aux_coef, void* const* workspaces,
                                            const size_t* workspace_bytes, const mixlora_grads_t* grads, void* stream) {
  if (n_models < 1 || n_models > MIXLORA_MAX_MODELS || !shapes || !params || !dy || !aux_coef || !workspaces ||
      !workspace_bytes || !grads)
    return MIXLORA_ERR_INVALID_ARG;
  Ctx cs[MIXLORA_MAX_MODELS];
  for (int m = 0; m < n_models; ++m) {
    mixlora_status_t st = bwd_check(&shapes[m], &params[m], dy[m], workspaces[m], workspace_bytes[m], &grads[m], stream,
                                    &cs[m]);
    if (st != MIXLORA_OK) return st;
    if (!same_frozen_ffn(cs[0], cs[m])) return MIXLORA_ERR_INVALID_ARG;
    for (int o = 0; o < m; ++o)
      if (workspaces[o] == workspaces[m]) return MIXLORA_ERR_INVALID_ARG;
  }
  mixlora_status_t st;
  for (int m = 0; m < n_models; m += 2)
    if ((st = bwd_shared_dgrad(&cs[m], &dy[m], n_models - m >= 2 ? 2 : 1)) != MIXLORA_OK) return st;
  return for_each_adapter(cs, n_models, n_models > 1,
                          [&](const Ctx& c, int m) {
                            return bwd_experts(c, dy[m], aux_coef[m], &grads[m], nullptr, n_models == 1);
                          });
}


// ---- the block inside its layer (Eq. 5 / Eq. 6) ----
static mixlora_status_t layer_check(const mixlora_shape_t* shape, const mixlora_params_t* params, const void* norm_weight,
                                    float eps, const void* xn, const float* inv_rms) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if (!params || !norm_weight || !xn || !inv_rms || !aligned16(norm_weight) || !aligned16(xn) ||
      (reinterpret_cast<uintptr_t>(inv_rms) & 3u) || !(eps >= 0.f))
    return MIXLORA_ERR_INVALID_ARG;
  if (xn == params->x) return MIXLORA_ERR_INVALID_ARG;   // the residual stream is read again after xn is written
  if (shape->d_model > rmsnorm_max_width(shape->dtype == MIXLORA_DTYPE_BF16)) return MIXLORA_ERR_UNSUPPORTED;
  return MIXLORA_OK;
}

mixlora_status_t mixlora_layer_forward(const mixlora_shape_t* shape, const mixlora_params_t* params,
                                       const void* norm_weight, float eps, void* xn, float* inv_rms, void* h,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  mixlora_status_t st = layer_check(shape, params, norm_weight, eps, xn, inv_rms);
  if (st != MIXLORA_OK) return st;
  if (h == xn) return MIXLORA_ERR_INVALID_ARG;
  mixlora_params_t inner = *params;                    // the block itself sees the normalised input
  inner.x = xn;
  Ctx c;
  if ((st = fwd_check(shape, &inner, h, workspace, workspace_bytes, stream, &c)) != MIXLORA_OK) return st;
  if (!params->x || !aligned16(params->x)) return MIXLORA_ERR_INVALID_ARG;
  {
    StageScope ss(ST_NORM, c.st, shape->tokens > 0 ? 1 : 0);
    MIXLORA_CUDA(launch_rmsnorm_fwd(c, params->x, norm_weight, eps, xn, inv_rms));
  }
  if ((st = fwd_clear_status(c)) != MIXLORA_OK) return st;
  Forked fk;
  if ((st = fwd_route_forked(c, &fk)) != MIXLORA_OK)
    return st;
  st = fwd_shared_projections(&c, 1);
  mixlora_status_t js = join_adapters(c.st, fk);
  if (st != MIXLORA_OK || js != MIXLORA_OK) return st != MIXLORA_OK ? st : js;
  return fwd_experts(c, h, params->x, true);
}

mixlora_status_t mixlora_layer_backward(const mixlora_shape_t* shape, const mixlora_params_t* params,
                                        const void* norm_weight, float eps, const void* xn, const float* inv_rms,
                                        const void* dh, float aux_coef, void* workspace, size_t workspace_bytes,
                                        const mixlora_grads_t* grads, void* stream) {
  mixlora_status_t st = layer_check(shape, params, norm_weight, eps, xn, inv_rms);
  if (st != MIXLORA_OK) return st;
  mixlora_params_t inner = *params;
  inner.x = xn;
  Ctx c;
  if ((st = bwd_check(shape, &inner, dh, workspace, workspace_bytes, grads, stream, &c)) != MIXLORA_OK) return st;
  if (!params->x || !aligned16(params->x)) return MIXLORA_ERR_INVALID_ARG;
  if (grads->d_x && (grads->d_x == dh || grads->d_x == params->x || grads->d_x == xn)) return MIXLORA_ERR_INVALID_ARG;
  if ((st = bwd_shared_dgrad(&c, &dh, 1)) != MIXLORA_OK) return st;
  if ((st = bwd_experts(c, dh, aux_coef, grads)) != MIXLORA_OK) return st;
  if (grads->d_x) {
    // d_x holds dL/dxn now; the norm's Jacobian and the residual path turn it into dL/dz in place
    StageScope ss(ST_NORM, c.st, shape->tokens > 0 ? 1 : 0);
    MIXLORA_CUDA(launch_rmsnorm_bwd(c, params->x, norm_weight, inv_rms, grads->d_x, dh, grads->d_x));
  }
  return MIXLORA_OK;
}

// ---- MixDoRA (Section 4.1 / Table 1): every expert projection is diag(m / n) (W + s B A) ----
namespace {
struct DoraLayout {
  size_t cg, cu, cd, inv_g, inv_u, inv_d, rowsq_g, rowsq_u, rowsq_d, wa_g, wa_u, wa_d, aat_g, aat_u, aat_d;
  size_t Zd_pos, gZd_pos, o_pre, total_fwd;
  size_t dO, D_s, spd_s, dmp_g, dmp_u, dmp_d, total_bwd;
};
// the MixLoRA layout (sized for both passes, without the grouped kernel's partial sums) followed by the extra regions
DoraLayout dora_layout(const mixlora_shape_t& s, const WsLayout& L) {
  DoraLayout D;
  const size_t T = (size_t)s.tokens, d = (size_t)s.d_model, f = (size_t)s.d_ff, N = (size_t)s.n_experts,
               k = (size_t)s.top_k, r = (size_t)s.rank, E = act_size(s);
  const size_t mt = (size_t)max_seg_tiles(s.tokens, s.top_k, s.n_experts);
  size_t off = L.total_bwd;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + (bytes ? bytes : 1), 256); return o; };
  D.cg = take(N * f * 4); D.cu = take(N * f * 4); D.cd = take(N * d * 4);
  D.inv_g = take(N * f * 4); D.inv_u = take(N * f * 4); D.inv_d = take(N * d * 4);
  D.rowsq_g = take(f * 4); D.rowsq_u = take(f * 4); D.rowsq_d = take(d * 4);
  D.wa_g = take(f * N * r * 4); D.wa_u = take(f * N * r * 4); D.wa_d = take(d * N * r * 4);
  D.aat_g = take(N * r * N * r * 4); D.aat_u = take(N * r * N * r * 4); D.aat_d = take(N * r * N * r * 4);
  D.Zd_pos = take(T * k * N * r * E); D.gZd_pos = take(T * k * N * r * E);
  D.o_pre = take(T * k * d * E);
  D.total_fwd = off;
  D.dO = take(T * k * d * E);
  D.D_s = take(T * k * f * E);
  D.spd_s = take(T * k * N * r * E);
  D.dmp_g = take(4 * mt * f * 4); D.dmp_u = take(4 * mt * f * 4); D.dmp_d = take(mt * d * 4);
  D.total_bwd = off;
  return D;
}

mixlora_status_t dora_setup(const mixlora_shape_t* shape, const mixlora_params_t* params,
                            const mixlora_dora_t* magn, void* workspace, size_t workspace_bytes, int for_backward,
                            void* stream, Ctx* c, DoraCtx* dc) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if ((st = check_params(params)) != MIXLORA_OK) return st;
  if (!magn || !magn->m_gate || !magn->m_up || !magn->m_down) return MIXLORA_ERR_INVALID_ARG;
  const void* mq[] = {magn->m_gate, magn->m_up, magn->m_down};
  for (const void* q : mq)
    if (reinterpret_cast<uintptr_t>(q) & 3u) return MIXLORA_ERR_INVALID_ARG;
  *c = make_ctx(shape, params, workspace, stream);
  c->L = ws_layout(*shape, false);
  c->no_fold = 1;
  const DoraLayout D = dora_layout(*shape, c->L);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      workspace_bytes < (for_backward ? D.total_bwd : D.total_fwd))
    return MIXLORA_ERR_WORKSPACE;
  dc->m = *magn;
  dc->cg = c->at<float>(D.cg); dc->cu = c->at<float>(D.cu); dc->cd = c->at<float>(D.cd);
  dc->inv_g = c->at<float>(D.inv_g); dc->inv_u = c->at<float>(D.inv_u); dc->inv_d = c->at<float>(D.inv_d);
  dc->rowsq_g = c->at<float>(D.rowsq_g); dc->rowsq_u = c->at<float>(D.rowsq_u); dc->rowsq_d = c->at<float>(D.rowsq_d);
  dc->wa_g = c->at<float>(D.wa_g); dc->wa_u = c->at<float>(D.wa_u); dc->wa_d = c->at<float>(D.wa_d);
  dc->aat_g = c->at<float>(D.aat_g); dc->aat_u = c->at<float>(D.aat_u); dc->aat_d = c->at<float>(D.aat_d);
  dc->Zd_pos = c->ws + D.Zd_pos; dc->gZd_pos = c->ws + D.gZd_pos; dc->o_pre = c->ws + D.o_pre;
  dc->dO = c->ws + D.dO; dc->D_s = c->ws + D.D_s; dc->spd_s = c->ws + D.spd_s;
  dc->dmp_g = c->at<float>(D.dmp_g); dc->dmp_u = c->at<float>(D.dmp_u); dc->dmp_d = c->at<float>(D.dmp_d);
  return MIXLORA_OK;
}
}  // namespace

size_t mixlora_dora_workspace_bytes(const mixlora_shape_t* shape, int for_backward) {
  if (check_shape(shape) != MIXLORA_OK) return 0;
  const WsLayout L = ws_layout(*shape, false);
  const DoraLayout D = dora_layout(*shape, L);
  return for_backward ? D.total_bwd : D.total_fwd;
}

mixlora_status_t mixlora_dora_ffn_forward(const mixlora_shape_t* shape, const mixlora_params_t* params,
                                          const mixlora_dora_t* magnitudes, void* y, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  Ctx c;
  DoraCtx dc;
  mixlora_status_t st = dora_setup(shape, params, magnitudes, workspace, workspace_bytes, 0, stream, &c, &dc);
  if (st != MIXLORA_OK) return st;
  if (!y || !aligned16(y)) return MIXLORA_ERR_INVALID_ARG;
  const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank, k = c.s.top_k;
  const int Nr = N * r;
  if ((st = fwd_clear_status(c)) != MIXLORA_OK) return st;
  if (T == 0) return MIXLORA_OK;
  // the router and the dispatch need only x, the repacks and the row norms of the frozen weights only parameters:
  // on a side stream each beside the dense products of the norms and the shared projections
  Forked fk;
  {
    const Ctx two[2] = {c, c};
    st = for_each_adapter(two, 2, true, [&](const Ctx& cc, int m) -> mixlora_status_t {
      if (m == 0) return fwd_route_only(cc);
      const mixlora_status_t rs = fwd_repacks(cc);
      if (rs != MIXLORA_OK) return rs;
      StageScope ss(ST_NORM, cc.st, 3);
      MIXLORA_CUDA(launch_dora_rowsq(cc, dc));
      return MIXLORA_OK;
    }, &fk);
    if (st != MIXLORA_OK) return st;
  }
  st = [&]() -> mixlora_status_t {
  // the scales c = m / n of the three projections: |W_o + s B_o A|^2 = |W_o|^2 + 2 s B_o . (W A^T)_o + s^2 B_o (A A^T) B_o^T
  {
    StageScope ss(ST_NORM, c.st, 6);
    TcOut gu[2];
    gu[0] = tc_out_f32(dc.wa_g, Nr, Nr, 1, 0, 0, 1.f, 0); tc_add(gu[0], params->w_gate, d, d, params->a_gate, d, 0);
    gu[1] = tc_out_f32(dc.wa_u, Nr, Nr, 1, 0, 0, 1.f, 0); tc_add(gu[1], params->w_up, d, d, params->a_up, d, 0);
    MIXLORA_CUDA(dense_product(c, f, gu, 2));
    TcOut dn = tc_out_f32(dc.wa_d, Nr, Nr, 1, 0, 0, 1.f, 0);
    tc_add(dn, params->w_down, f, f, params->a_down, f, 0);
    MIXLORA_CUDA(dense_product(c, d, &dn, 1));
    TcOut aa[2];
    aa[0] = tc_out_f32(dc.aat_g, Nr, Nr, 1, 0, 0, 1.f, 0); tc_add(aa[0], params->a_gate, d, d, params->a_gate, d, 0);
    aa[1] = tc_out_f32(dc.aat_u, Nr, Nr, 1, 0, 0, 1.f, 0); tc_add(aa[1], params->a_up, d, d, params->a_up, d, 0);
    MIXLORA_CUDA(dense_product(c, Nr, aa, 2));
    TcOut ad = tc_out_f32(dc.aat_d, Nr, Nr, 1, 0, 0, 1.f, 0);
    tc_add(ad, params->a_down, f, f, params->a_down, f, 0);
    MIXLORA_CUDA(dense_product(c, Nr, &ad, 1));
  }
  return fwd_shared_projections(&c, 1);   // W1 x, W3 x once per token, A_g x, A_u x
  }();
  {
    const mixlora_status_t js = join_adapters(c.st, fk);   // always: no side stream is left dangling after an error
    if (st != MIXLORA_OK || js != MIXLORA_OK) return st != MIXLORA_OK ? st : js;
  }
  { StageScope ss(ST_NORM, c.st, 3); MIXLORA_CUDA(launch_dora_scales(c, dc)); }   // needs the row norms and the products
  {
    StageScope ss(ST_LORA_B_SWIGLU, c.st, 2);
    if (grouped_swiglu_supported(c)) {      // the tensor-core kernel of the MixLoRA path with the two scale vectors
      MIXLORA_CUDA(launch_zcompact(c));
      MIXLORA_CUDA(launch_grouped_swiglu_dora_fwd(c, dc));
    } else {
      MIXLORA_CUDA(launch_dora_swiglu_fwd(c, dc));
    }
  }
  {   // zd = A_d h against every expert, then the slot's own block (and gate times it)
    StageScope ss(ST_LORA_A_DOWN, c.st, 2);
    TcOut out = tc_out(c.ws + c.L.zd_all, Nr, Nr);
    tc_add(out, c.ws + c.L.h_sorted, f, f, params->a_down, f, 0);
    MIXLORA_CUDA(dense_product(c, T * k, &out, 1));
    MIXLORA_CUDA(launch_dora_own_block(c, c.ws + c.L.zd_all, dc.Zd_pos, dc.gZd_pos));
  }
  {   // o_pre = [h | Zd] [W2 | s B_d]^T per sorted slot: W2 cannot act on the gate-weighted sum of a token's slots
      // here, because the scale of its output differs between the token's experts
    StageScope ss(ST_GEMM_DOWN, c.st, 1);
    TcOut out = tc_out(dc.o_pre, d, d);
    tc_add(out, c.ws + c.L.h_sorted, f, f, params->w_down, f, 0);
    tc_add(out, dc.Zd_pos, Nr, Nr, c.ws + c.L.bd_cat, Nr, 0);
    MIXLORA_CUDA(dense_product(c, T * k, &out, 1, nullptr, true));
  }
  { StageScope ss(ST_COMBINE_H, c.st, 1); MIXLORA_CUDA(launch_dora_combine_y(c, dc, y)); }
  return MIXLORA_OK;
}

mixlora_status_t mixlora_dora_ffn_backward(const mixlora_shape_t* shape, const mixlora_params_t* params,
                                           const mixlora_dora_t* magnitudes, const void* dy, float aux_coef,
                                           void* workspace, size_t workspace_bytes, const mixlora_grads_t* grads,
                                           const mixlora_dora_grads_t* mgrads, void* stream) {
  Ctx c;
  DoraCtx dc;
  mixlora_status_t st = dora_setup(shape, params, magnitudes, workspace, workspace_bytes, 1, stream, &c, &dc);
  if (st != MIXLORA_OK) return st;
  if (!dy || !aligned16(dy) || !grads || !mgrads) return MIXLORA_ERR_INVALID_ARG;
  {
    const void* outs[] = {grads->d_a_gate, grads->d_b_gate, grads->d_a_up, grads->d_b_up, grads->d_a_down,
                          grads->d_b_down, grads->d_w_router, grads->d_x};
    for (const void* q : outs)
      if (q && !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
    if (grads->accumulate != 0 && grads->accumulate != 1) return MIXLORA_ERR_INVALID_ARG;
  }
  const int T = c.s.tokens, d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank, k = c.s.top_k;
  const int Nr = N * r, NP = round_up8(N), acc = grads->accumulate, want_dx = grads->d_x != nullptr;
  if (T == 0) {
    if ((st = bwd_zero_tokens(c, grads)) != MIXLORA_OK) return st;
    if (!acc) {
      if (mgrads->d_m_gate) MIXLORA_CUDA(cudaMemsetAsync(mgrads->d_m_gate, 0, sizeof(float) * N * f, c.st));
      if (mgrads->d_m_up) MIXLORA_CUDA(cudaMemsetAsync(mgrads->d_m_up, 0, sizeof(float) * N * f, c.st));
      if (mgrads->d_m_down) MIXLORA_CUDA(cudaMemsetAsync(mgrads->d_m_down, 0, sizeof(float) * N * d, c.st));
    }
    return MIXLORA_OK;
  }
  // dO = c_d * dy per sorted slot (and the down magnitude's shares), then D = dO W2 and s B_d^T dO per slot
  { StageScope ss(ST_COMBINE_BWD, c.st, 1); MIXLORA_CUDA(launch_dora_dout(c, dc, dy)); }
  {
    StageScope ss(ST_GEMM_DGRAD_DOWN, c.st, 1);
    TcOut outs[2];
    outs[0] = tc_out(dc.D_s, f, f);      tc_add(outs[0], dc.dO, d, d, params->w_down, f, 1);
    outs[1] = tc_out(dc.spd_s, Nr, Nr);  tc_add(outs[1], dc.dO, d, d, c.ws + c.L.bd_cat, Nr, 1);
    MIXLORA_CUDA(dense_product(c, T * k, outs, 2, nullptr, true));
  }
  const bool tc_swiglu = grouped_swiglu_supported(c);
  { StageScope ss(ST_SWIGLU_BWD, c.st, 3);
    if (tc_swiglu) {
      MIXLORA_CUDA(launch_dora_pcompact(c, dc));
      MIXLORA_CUDA(launch_grouped_swiglu_dora_bwd(c, dc));
      MIXLORA_CUDA(launch_dgate_reduce(c, grouped_swiglu_bwd_col_tiles(f)));
    } else {
      MIXLORA_CUDA(launch_dora_swiglu_bwd(c, dc));
      MIXLORA_CUDA(launch_dgate_reduce(c, dora_bwd_col_chunks(f)));
    } }
  MIXLORA_CUDA(launch_router_bwd(c, aux_coef, grads->d_router_bias, acc, want_dx));
  const int dm_sub = tc_swiglu ? 4 : 1;    // partial rows per tile of the gate / up magnitude shares
  if (mgrads->d_m_gate) MIXLORA_CUDA(launch_dora_dm_reduce(c, dc.dmp_g, dc.inv_g, mgrads->d_m_gate, f, acc, dm_sub));
  if (mgrads->d_m_up) MIXLORA_CUDA(launch_dora_dm_reduce(c, dc.dmp_u, dc.inv_u, mgrads->d_m_up, f, acc, dm_sub));
  if (mgrads->d_m_down) MIXLORA_CUDA(launch_dora_dm_reduce(c, dc.dmp_d, dc.inv_d, mgrads->d_m_down, d, acc));
  {   // dzg = da (s B_g), dzu = db (s B_u) with da, db the gradients of the pre-scale activations
    TcOut outs[2];
    outs[0] = tc_out(c.ws + c.L.dzg_all, Nr, Nr); tc_add(outs[0], c.ws + c.L.da_sorted, f, f, c.ws + c.L.bg_cat, Nr, 1);
    outs[1] = tc_out(c.ws + c.L.dzu_all, Nr, Nr); tc_add(outs[1], c.ws + c.L.db_sorted, f, f, c.ws + c.L.bu_cat, Nr, 1);
    MIXLORA_CUDA(dense_product(c, T * k, outs, 2));
  }
  MIXLORA_CUDA(launch_combine_bwd(c, want_dx));
  MIXLORA_CUDA(launch_zpos(c));
  // dZd_pos = gate * (s B_d^T dO) in the slot's own block
  MIXLORA_CUDA(launch_dora_own_block(c, dc.spd_s, nullptr, c.ws + c.L.dZd_pos));
  {
    TcOut outs[3];
    int n = 0;
    if (grads->d_b_gate) {
      outs[n] = tc_out_f32(grads->d_b_gate, Nr, r, 1, r, (long long)f * r, c.scale, acc);
      tc_add(outs[n++], c.ws + c.L.da_sorted, f, T * k, c.ws + c.L.Zg_pos, Nr, 1, 1);
    }
    if (grads->d_b_up) {
      outs[n] = tc_out_f32(grads->d_b_up, Nr, r, 1, r, (long long)f * r, c.scale, acc);
      tc_add(outs[n++], c.ws + c.L.db_sorted, f, T * k, c.ws + c.L.Zu_pos, Nr, 1, 1);
    }
    if (grads->d_a_down) {
      outs[n] = tc_out_f32(grads->d_a_down, Nr, 1, f, 0, 0, 1.f, acc);
      tc_add(outs[n++], c.ws + c.L.h_sorted, f, T * k, c.ws + c.L.dZd_pos, Nr, 1, 1);
    }
    MIXLORA_CUDA(dense_product(c, f, outs, n));
  }
  if (grads->d_b_down) {   // dB_d[e][c][rr] = s sum over slots of dO[slot][c] (g zd)[slot][e r + rr]
    TcOut out = tc_out_f32(grads->d_b_down, Nr, r, 1, r, (long long)d * r, c.scale, acc);
    tc_add(out, dc.dO, d, T * k, dc.gZd_pos, Nr, 1, 1);
    MIXLORA_CUDA(dense_product(c, d, &out, 1));
  }
  {
    TcOut outs[3];
    int n = 0;
    if (grads->d_a_gate) {
      outs[n] = tc_out_f32(grads->d_a_gate, Nr, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dZg, Nr, 1, 1);
    }
    if (grads->d_a_up) {
      outs[n] = tc_out_f32(grads->d_a_up, Nr, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dZu, Nr, 1, 1);
    }
    if (grads->d_w_router) {
      outs[n] = tc_out_f32(grads->d_w_router, N, 1, d, 0, 0, 1.f, acc);
      tc_add(outs[n++], params->x, d, T, c.ws + c.L.dl_act, NP, 1, 1, NP);
    }
    MIXLORA_CUDA(dense_product(c, d, outs, n));
  }
  if (want_dx) {
    TcOut out = tc_out(grads->d_x, d, d);
    tc_add(out, c.ws + c.L.dabar, f, f, params->w_gate, d, 1);
    tc_add(out, c.ws + c.L.dbbar, f, f, params->w_up, d, 1);
    tc_add(out, c.ws + c.L.dZg, Nr, Nr, params->a_gate, d, 1);
    tc_add(out, c.ws + c.L.dZu, Nr, Nr, params->a_up, d, 1);
    tc_add(out, c.ws + c.L.dl_act, NP, NP, c.ws + c.L.wr_act, d, 1);
    MIXLORA_CUDA(dense_product(c, T, &out, 1, nullptr, true));
  }
  return MIXLORA_OK;
}

mixlora_status_t mixlora_routing_view(const mixlora_shape_t* shape, const void* workspace, const int32_t** expert_idx,
                                      const float** gates, const int32_t** perm, const int32_t** seg_off,
                                      const uint8_t** low_margin, const float** probs) {
  mixlora_status_t st = check_shape(shape);
  if (st != MIXLORA_OK) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MIXLORA_ERR_WORKSPACE;
  WsLayout L = ws_layout(*shape);
  const char* ws = reinterpret_cast<const char*>(workspace);
  if (expert_idx) *expert_idx = reinterpret_cast<const int32_t*>(ws + L.expert_idx);
  if (gates) *gates = reinterpret_cast<const float*>(ws + L.gates);
  if (perm) *perm = reinterpret_cast<const int32_t*>(ws + L.perm);
  if (seg_off) *seg_off = reinterpret_cast<const int32_t*>(ws + L.seg_off);
  if (low_margin) *low_margin = reinterpret_cast<const uint8_t*>(ws + L.low_margin);
  if (probs) *probs = reinterpret_cast<const float*>(ws + L.probs);
  return MIXLORA_OK;
}

mixlora_status_t mixlora_device_status(const void* workspace, int32_t* code, void* stream) {
  if (!workspace || !code) return MIXLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int32_t v = 0;
  MIXLORA_CUDA(cudaMemcpyAsync(&v, workspace, sizeof(v), cudaMemcpyDeviceToHost, st));
  MIXLORA_CUDA(cudaStreamSynchronize(st));
  *code = v;
  return MIXLORA_OK;
}

mixlora_status_t mixlora_set_option(int32_t option, int32_t value) {
  if (value != 0 && value != 1) return MIXLORA_ERR_INVALID_ARG;
  switch (option) {
    case MIXLORA_OPT_SERIAL: g_serial.store(value, std::memory_order_relaxed); return MIXLORA_OK;
    case MIXLORA_OPT_TC_SINGLE: tc_set_force_single(value); return MIXLORA_OK;
  }
  return MIXLORA_ERR_INVALID_ARG;
}

mixlora_status_t mixlora_selftest_wait_timeout(void* workspace, uint32_t wait_rounds, void* stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MIXLORA_ERR_WORKSPACE;
  if (wait_rounds == 0 || wait_rounds > (1u << 20)) return MIXLORA_ERR_INVALID_ARG;
  MIXLORA_CUDA(launch_wait_timeout_selftest(reinterpret_cast<int*>(workspace), wait_rounds,
                                            reinterpret_cast<cudaStream_t>(stream)));
  return MIXLORA_OK;
}

mixlora_status_t mixlora_stage_timing(int32_t enable) {
  std::lock_guard<std::mutex> lock(g_prof.mu);
  for (auto& r : g_prof.recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  g_prof.recs.clear();
  for (int i = 0; i < ST_COUNT; ++i) g_prof.launches[i] = 0;
  g_prof.on = enable != 0;
  return MIXLORA_OK;
}

int32_t mixlora_stage_timing_read(int32_t max_stages, const char** names, float* ms, int64_t* launches) {
  std::lock_guard<std::mutex> lock(g_prof.mu);
  float acc[ST_COUNT] = {0};
  for (auto& r : g_prof.recs) {
    float t = 0.f;
    if (cudaEventSynchronize(r.b) == cudaSuccess && cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) acc[r.stage] += t;
  }
  int n = max_stages < ST_COUNT ? max_stages : ST_COUNT;
  for (int i = 0; i < n; ++i) {
    if (names) names[i] = kStageNames[i];
    if (ms) ms[i] = acc[i];
    if (launches) launches[i] = g_prof.launches[i];
  }
  return ST_COUNT;
}

// ---- plain LoRA on a linear layer (Eq. 1; the attention projections of Section 3.2) ----
namespace {
struct LinearLayout { size_t status, zs, dzs, total; };
LinearLayout linear_layout(const mixlora_linear_shape_t& s) {
  const size_t el = s.dtype == MIXLORA_DTYPE_BF16 ? 2 : 4;
  LinearLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
  L.status = take(256);
  L.zs = take((size_t)(s.tokens > 0 ? s.tokens : 1) * s.rank * el);
  L.dzs = take((size_t)(s.tokens > 0 ? s.tokens : 1) * s.rank * el);
  L.total = off;
  return L;
}
bool linear_shape_ok(const mixlora_linear_shape_t* s) {
  return s && s->struct_size == sizeof(mixlora_linear_shape_t) && s->tokens >= 0 && s->d_in > 0 && s->d_out > 0 &&
         s->rank > 0 && s->rank <= MIXLORA_MAX_RANK && s->d_in % 8 == 0 && s->d_out % 8 == 0 && s->rank % 8 == 0 &&
         (s->dtype == MIXLORA_DTYPE_BF16 || s->dtype == MIXLORA_DTYPE_FP32) && s->lora_alpha == s->lora_alpha;
}
// the dense-product helpers only need the type, the stream and a status word from the context
Ctx linear_ctx(const mixlora_linear_shape_t& s, void* workspace, void* stream) {
  Ctx c;
  memset(&c.s, 0, sizeof(c.s));
  memset(&c.p, 0, sizeof(c.p));
  memset(&c.L, 0, sizeof(c.L));
  c.s.dtype = s.dtype;
  c.s.tokens = s.tokens;
  c.ws = reinterpret_cast<char*>(workspace);
  c.st = reinterpret_cast<cudaStream_t>(stream);
  c.bf16 = s.dtype == MIXLORA_DTYPE_BF16;
  c.scale = s.lora_alpha / (float)s.rank;
  return c;
}
}  // namespace

size_t mixlora_lora_linear_workspace_bytes(const mixlora_linear_shape_t* shape) {
  return linear_shape_ok(shape) ? linear_layout(*shape).total : 0;
}

mixlora_status_t mixlora_lora_linear_forward(const mixlora_linear_shape_t* shape, const void* x, const void* w,
                                             const void* a, const void* b, void* y, void* workspace,
                                             size_t workspace_bytes, void* stream) {
  if (!linear_shape_ok(shape)) return MIXLORA_ERR_INVALID_ARG;
  const void* req[] = {x, w, a, b, y};
  for (const void* q : req)
    if (!q || !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
  const LinearLayout L = linear_layout(*shape);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total)
    return MIXLORA_ERR_WORKSPACE;
  const Ctx c = linear_ctx(*shape, workspace, stream);
  const int T = shape->tokens, din = shape->d_in, dout = shape->d_out, r = shape->rank;
  MIXLORA_CUDA(cudaMemsetAsync(c.ws + L.status, 0, 256, c.st));
  if (T == 0) return MIXLORA_OK;
  {   // zs = s x A^T
    TcOut z = tc_out(c.ws + L.zs, r, r);
    z.alpha = c.scale;
    tc_add(z, x, din, din, a, din, 0);
    MIXLORA_CUDA(dense_product(c, T, &z, 1));
  }
  // y = [x | zs] [W | B]^T : the low-rank term rides along as r extra reduction columns of the frozen product
  TcOut out = tc_out(y, dout, dout);
  tc_add(out, x, din, din, w, din, 0);
  tc_add(out, c.ws + L.zs, r, r, b, r, 0);
  MIXLORA_CUDA(dense_product(c, T, &out, 1));
  return MIXLORA_OK;
}

mixlora_status_t mixlora_lora_linear_backward(const mixlora_linear_shape_t* shape, const void* x, const void* w,
                                              const void* a, const void* b, const void* dy, void* workspace,
                                              size_t workspace_bytes, float* d_a, float* d_b, void* d_x,
                                              int32_t accumulate, void* stream) {
  if (!linear_shape_ok(shape)) return MIXLORA_ERR_INVALID_ARG;
  const void* req[] = {x, w, a, b, dy};
  for (const void* q : req)
    if (!q || !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
  const void* opt[] = {d_a, d_b, d_x};
  for (const void* q : opt)
    if (q && !aligned16(q)) return MIXLORA_ERR_INVALID_ARG;
  if (accumulate != 0 && accumulate != 1) return MIXLORA_ERR_INVALID_ARG;
  const LinearLayout L = linear_layout(*shape);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total)
    return MIXLORA_ERR_WORKSPACE;
  const Ctx c = linear_ctx(*shape, workspace, stream);
  const int T = shape->tokens, din = shape->d_in, dout = shape->d_out, r = shape->rank;
  if (T == 0) {
    if (!accumulate) {
      if (d_a) MIXLORA_CUDA(cudaMemsetAsync(d_a, 0, sizeof(float) * (size_t)r * din, c.st));
      if (d_b) MIXLORA_CUDA(cudaMemsetAsync(d_b, 0, sizeof(float) * (size_t)dout * r, c.st));
    }
    return MIXLORA_OK;
  }
  {   // dzs = s dy B
    TcOut z = tc_out(c.ws + L.dzs, r, r);
    z.alpha = c.scale;
    tc_add(z, dy, dout, dout, b, r, 1);
    MIXLORA_CUDA(dense_product(c, T, &z, 1));
  }
  if (d_x) {   // dx = [dy | dzs] [W ; A]
    TcOut out = tc_out(d_x, din, din);
    tc_add(out, dy, dout, dout, w, din, 1);
    tc_add(out, c.ws + L.dzs, r, r, a, din, 1);
    MIXLORA_CUDA(dense_product(c, T, &out, 1));
  }
  if (d_a) {   // dA[rr][c] = sum_t dzs[t][rr] x[t][c]
    TcOut out = tc_out_f32(d_a, r, 1, din, 0, 0, 1.f, accumulate);
    tc_add(out, x, din, T, c.ws + L.dzs, r, 1, 1);
    MIXLORA_CUDA(dense_product(c, din, &out, 1));
  }
  if (d_b) {   // dB[c][rr] = sum_t dy[t][c] zs[t][rr]   (zs carries the scale s)
    TcOut out = tc_out_f32(d_b, r, r, 1, 0, 0, 1.f, accumulate);
    tc_add(out, dy, dout, T, c.ws + L.zs, r, 1, 1);
    MIXLORA_CUDA(dense_product(c, dout, &out, 1));
  }
  return MIXLORA_OK;
}

int32_t mixlora_lora_linear_status(const void* workspace, void* stream) {
  int v = 0;
  if (!workspace) return (int32_t)MIXLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&v, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return (int32_t)MIXLORA_ERR_CUDA;
  return v;
}

mixlora_status_t mixlora_gemm_bf16(const void* A, const void* B, void* C, int32_t M, int32_t N, int32_t K,
                                   int32_t b_is_kn, int32_t* status_word, void* stream) {
  if (!A || !B || !C || !aligned16(A) || !aligned16(B) || !aligned16(C)) return MIXLORA_ERR_INVALID_ARG;
  if (M < 0 || N <= 0 || K <= 0 || (b_is_kn != 0 && b_is_kn != 1)) return MIXLORA_ERR_INVALID_ARG;
  if (N % 8 || K % 8) return MIXLORA_ERR_UNSUPPORTED;
  if (M == 0) return MIXLORA_OK;
  TcOut out = tc_out(C, N, N);
  tc_add(out, A, K, K, B, b_is_kn ? N : K, b_is_kn);
  if (!tc_gemm_supported(M, &out, 1)) return MIXLORA_ERR_UNSUPPORTED;
  MIXLORA_CUDA(launch_tc_gemm(M, &out, 1, status_word, reinterpret_cast<cudaStream_t>(stream)));
  return MIXLORA_OK;
}

}  // extern "C"
