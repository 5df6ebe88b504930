// Shared declarations of the MixLoRA FFN library: workspace layout, launch helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "mixlora.h"

namespace mixlora {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------------------
// Workspace layout.  Every region starts on a 256-byte boundary.  "act" regions hold
// elements of the activation type (bf16 or fp32 according to shape.dtype).
// The regions up to total_fwd are what a forward call needs; the rest is backward scratch.
// ---------------------------------------------------------------------------------------
struct WsLayout {
  size_t status;      // int32[64]; [0] = device status word; bytes 8..15: int64 token count of the whole batch when
                      //            the auxiliary loss was evaluated over data-parallel shards (0 = this call's tokens)
  size_t splitk_cnt;  // i32 [kSplitCounters]  arrival counters of a split reduction, zero between launches
  size_t probs;       // f32 [T, N]        softmax probabilities (Eq. 7)
  size_t expert_idx;  // i32 [T, k]
  size_t gates;       // f32 [T, k]
  size_t low_margin;  // u8  [T]
  size_t perm;        // i32 [T*k]         slot id at sorted position
  size_t inv;         // i32 [T*k]         sorted position of slot id
  size_t pos_token;   // i32 [T*k]         token of sorted position
  size_t pos_expert;  // i32 [T*k]         expert of sorted position
  size_t seg_off;     // i32 [N+1]
  size_t blk_counts;  // i32 [nblk, N]
  size_t blk_off;     // i32 [nblk, N]
  size_t stat_F;      // f32 [N]           F_i of Eq. 9
  size_t stat_P;      // f32 [N]           P_i of Eq. 9
  size_t stat_raw;    // f32 [2N]          un-normalised sums of Eq. 9: probability per expert, then selections per expert
  size_t stat_part;   // f32 [router blocks, 2N]  the same sums per block of the router kernel
  size_t tile_info;   // i32 [max_tiles, 4] (expert, first position, rows, 0) of kSegTile-row segment tiles;
                      //                    the int after the table holds the tile count
  size_t G, U;        // act [T, f]        shared W1 / W3 projections (Section 3.3 (I))
  size_t zga, zua;    // act [T, N*r]      A_g x and A_u x for every expert
  size_t zd_all;      // act [T*k, N*r]    A_d h of every expert per sorted slot (the slot's own block is used)
  size_t Zs;          // act [T, N*r]      gate * zd scattered to the slot's expert block
  size_t bd_cat;      // act [d, N*r]      s * B_d laid out [c][e*r + rr]
  size_t bg_cat, bu_cat;  // act [f, N*r]  s * B_g, s * B_u laid out [f'][e*r + rr]
  size_t Zg_pos, Zu_pos;  // act [T*k, N*r]  zg / zu of the slot in its expert block, zero elsewhere
  size_t zg_s, zu_s;  // act [T*k, pad_rank(r)]  s * zg, s * zu of the slot's own expert, zero padded
  size_t bgp, bup;    // act [N*f, pad_rank(r)]  B_g, B_u zero padded (used when pad_rank(r) != r)
  size_t adp;         // act [N*pad_rank(r), f]  A_d with each expert's rows zero padded (same condition)
  size_t h_sorted;    // act [T*k, f]
  size_t hbar;        // act [T, f]        sum_j g_j h_j
  size_t work_count;  // i32 [8]  item counts of the work lists below; [3] = column groups the backward grouped
                      //          kernel used (rows of dz_part); [4] = the same of the forward kernel (zd_part)
  size_t work_rows1;  // i32 [.., 8]  rows list with one output (A_d h)
  size_t splitk_part; // f32 partial tiles of a split reduction ([T, d] products of a short batch), splitk_bytes long
  size_t splitk_bytes;
  size_t total_fwd;
  size_t D;           // act [T, f]        dy W_d
  size_t spd;         // act [T, N*r]      s * B_d^T dy for every expert
  size_t da_sorted, db_sorted;  // act [T*k, f]
  size_t dabar, dbbar;          // act [T, f]
  size_t p_s;                   // act [T*k, pad_rank(r)]  s * pd of the slot's own expert, zero padded
  size_t dZd_pos;               // act [T*k, N*r]  gate * s * pd of the slot in its expert block, zero elsewhere
  size_t dgate_part;            // f32 [ceil(f/64), T*k]  per column tile partial <Dt, h> of the fused backward
  size_t dzg_all, dzu_all;      // act [T*k, N*r]  da (s B_g) and db (s B_u) against every expert (not when the
                                //                 grouped kernel forms them, see dz_part)
  size_t dz_part;               // f32 [groups, T*k, 2, r]  per column group: dzg, dzu of the slot's own expert
  size_t zd_part;               // f32 [groups, T*k, r]  per column group: zd = A_d h of the slot's own expert (forward;
                                //                 takes the place of zd_all where the grouped kernel forms it)
  size_t dZg, dZu;    // act [T, N*r]      dzg / dzu scattered dense
  size_t dgate;       // f32 [T*k]         by slot id
  size_t dlogits;     // f32 [T, N]
  size_t dl_act;      // act [T, NP]       dlogits in the activation type, NP = N rounded up to 8
  size_t wr_act;      // act [NP, d]       router weight in the activation type
  size_t work_rows2;  // i32 [.., 8]  rows list with two outputs (da sB_g, db sB_u)
  size_t work_red;    // i32 [.., 8]  reduce list of the f-sized weight gradients
  size_t total_bwd;
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static const int kRouteBlockTokens = 256;  // tokens per block in the dispatch kernels
static const int kSegTile = 128;           // rows of a segment tile

static inline int route_blocks(int T) { return (T + kRouteBlockTokens - 1) / kRouteBlockTokens; }
static inline int max_seg_tiles(int T, int k, int N) { return (int)(((long long)T * k + kSegTile - 1) / kSegTile) + N; }
static inline int round_up8(int v) { return (v + 7) / 8 * 8; }
// rank-r operands of the grouped SwiGLU kernels are rows of 32, 64 or 128 bytes (or two 128-byte blocks): other
// ranks are zero-padded to the next of these widths
static inline int pad_rank(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : (r <= 64 ? 64 : 128)); }

// `allow_fold` = false sizes every region for the path that does not form dzg / dzu inside the grouped kernel
WsLayout ws_layout(const mixlora_shape_t& s, bool allow_fold = true);

// Column tiles of the backward grouped SwiGLU kernel (64 columns each) and the widest group of them whose pieces of
// G, U and D (tokens x columns x 3 matrices) stay well inside L2 while every segment tile of the group is worked on;
// never narrower than 4 tiles (beyond about 14 000 tokens at the 7B width the group then outgrows that share of L2,
// which measured cheaper than giving the fold up: 3.04 -> 2.64 ms for the three backward stages at 32768 tokens).
static inline int grouped_bwd_col_tiles(int f) { return (f + 63) / 64; }
static inline int grouped_bwd_col_group_max(int tokens, int f) {
  const long long cols = (32ll << 20) / ((long long)(tokens > 0 ? tokens : 1) * 2 * 3);
  const long long g = cols / 64;
  const int ct = grouped_bwd_col_tiles(f);
  return (int)(g < 4 ? 4 : (g > ct ? ct : g));
}
// The backward grouped kernel also forms dzg = da (s B_g), dzu = db (s B_u) of a slot's own expert (summed over the
// column tiles of a group in TMEM, one fp32 partial per group) when the rank divides a 64-column operand block.
static inline bool grouped_bwd_folds_dz(const mixlora_shape_t& s) {
  return s.dtype == MIXLORA_DTYPE_BF16 && s.tokens > 0 && (s.rank == 8 || s.rank == 16 || s.rank == 32) &&
         (long long)s.tokens * s.d_ff < (1ll << 31);
}
// the kernel may narrow the groups down to 4 tiles to even out the CTAs' shares (with few tokens there are few segment
// tiles, and wide groups would leave most CTAs without a unit): narrowest width, and the bound of the group count
static inline int grouped_bwd_col_group_min(int tokens, int f) {
  (void)tokens; (void)f;
  return 4;
}
// The forward grouped kernel forms zd = h A_d[e]^T (the input of the LoRA of W2) the same way, on 64-column tiles,
// for ranks up to 32: widest column group (tokens x columns x 2 matrices G, U inside L2) and the condition.  The
// narrower tile costs the kernel about as much as the dense product it replaces at 8192 tokens of the 7B width
// (measured), and less below, so the fold is taken up to 4096 tokens there (groups of at least 32 tiles).
static inline int grouped_fwd_col_group_max(int tokens, int f) {
  const long long cols = (32ll << 20) / ((long long)(tokens > 0 ? tokens : 1) * 2 * 2);
  const long long g = cols / 64;
  const int ct = grouped_bwd_col_tiles(f);
  return (int)(g < 1 ? 1 : (g > ct ? ct : g));
}
static inline bool grouped_fwd_folds_zd(const mixlora_shape_t& s) {
  return s.dtype == MIXLORA_DTYPE_BF16 && s.tokens > 0 && s.rank % 8 == 0 && s.rank <= 32 &&
         grouped_fwd_col_group_max(s.tokens, s.d_ff) >= 32 && (long long)s.tokens * s.d_ff < (1ll << 31);
}
static inline int grouped_fwd_max_groups(int f) { return (grouped_bwd_col_tiles(f) + 3) / 4; }
static inline int grouped_bwd_max_groups(int tokens, int f) {
  const int cg_min = grouped_bwd_col_group_min(tokens, f);
  return (grouped_bwd_col_tiles(f) + cg_min - 1) / cg_min;
}

static inline size_t act_size(const mixlora_shape_t& s) { return s.dtype == MIXLORA_DTYPE_BF16 ? 2 : 4; }

// ---------------------------------------------------------------------------------------
// Generic SIMT product with fp32 accumulation:
//   C[g][m, n] (+)= alpha * sum_seg sum_k A_seg(m, k) * B_seg(n, k)
// Operand element (i, k) of group g sits at p + g*sg + I(i)*si + K(k)*sk, where I / K are
// optional gather tables.  group_mode 1 takes the row range of group g from
// seg_off[g..g+1] (rows are absolute positions), group_mode 2 takes the reduction range of
// the first K-segment from seg_off instead.
// ---------------------------------------------------------------------------------------
struct SOperand {
  const void* p;
  const int* gi;  // gather on the row / column index, or nullptr
  const int* gk;  // gather on the reduction index, or nullptr
  long long si, sk, sg;
  int is_bf16;
};

static const int kMaxKSeg = 5;

struct SGemm {
  SOperand A[kMaxKSeg], B[kMaxKSeg];
  int K[kMaxKSeg];
  int nseg;
  void* C;
  long long c_sm, c_sn, c_sg;
  int c_nb;             // > 0: column n sits at (n / c_nb) * c_sblk + (n % c_nb) * c_sn
  long long c_sblk;
  int c_is_bf16;
  int M, N;            // for group_mode 1, M is the upper bound of rows over all groups
  const int* seg_off;  // device
  int group_mode;
  int groups;
  float alpha;
  int accumulate;
};

cudaError_t launch_simt_gemm(const SGemm& g, cudaStream_t st);

static inline SOperand soperand(const void* p, long long si, long long sk, int is_bf16, long long sg = 0,
                                const int* gi = nullptr, const int* gk = nullptr) {
  SOperand o;
  o.p = p; o.gi = gi; o.gk = gk; o.si = si; o.sk = sk; o.sg = sg; o.is_bf16 = is_bf16;
  return o;
}

// ---------------------------------------------------------------------------------------
// Kernel launchers (router.cu, elementwise.cu, tc_gemm.cu)
// ---------------------------------------------------------------------------------------
struct Ctx {
  mixlora_shape_t s;
  mixlora_params_t p;
  WsLayout L;
  char* ws;
  cudaStream_t st;
  int bf16;  // activation type is bf16
  int no_fold = 0;   // 1: the workspace was laid out with allow_fold = false (MixDoRA path)
  float scale;
  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

static inline bool ctx_folds_dz(const Ctx& c) { return !c.no_fold && grouped_bwd_folds_dz(c.s); }
static inline bool ctx_folds_zd(const Ctx& c) { return !c.no_fold && grouped_fwd_folds_zd(c.s); }

cudaError_t launch_router(const Ctx& c);              // probs, expert_idx, gates, low_margin, stats
cudaError_t launch_dispatch(const Ctx& c);            // perm, inv, pos_token, pos_expert, seg_off, tile_info
cudaError_t launch_aux_loss(const Ctx& c, float coef, float* loss, float* F, float* P);
cudaError_t launch_aux_loss_global(const Ctx& c, float coef, const float* prob_sum, const float* count,
                                   long long total_tokens, float* loss, float* F, float* P);
int router_part_blocks(int tokens);                   // upper bound of the router kernel's blocks
cudaError_t launch_bd_cat(const Ctx& c);
cudaError_t launch_bgu_cat(const Ctx& c);              // bg_cat, bu_cat
cudaError_t launch_zpos(const Ctx& c);                 // Zg_pos, Zu_pos
cudaError_t launch_dgate_reduce(const Ctx& c, int col_tiles);   // dgate from dgate_part
cudaError_t launch_zcompact(const Ctx& c);             // zg_s, zu_s (and bgp, bup, adp when the rank is padded)
bool grouped_swiglu_supported(const Ctx& c);
int grouped_swiglu_bwd_col_tiles(int f);
cudaError_t launch_grouped_swiglu_fwd(const Ctx& c);   // per-expert tiles, K = r (grouped_swiglu.cu)
cudaError_t launch_grouped_swiglu_bwd(const Ctx& c);
cudaError_t launch_lora_b_swiglu(const Ctx& c);       // h_sorted from G, U, zga, zua, B_g, B_u
cudaError_t launch_combine_h(const Ctx& c);           // hbar, Zs
cudaError_t launch_swiglu_bwd(const Ctx& c);          // h_sorted, da_sorted, db_sorted, dgate, Zg_pos, Zu_pos
cudaError_t launch_slot_prep_bwd(const Ctx& c);       // dZd_pos, p_s
cudaError_t launch_combine_bwd(const Ctx& c, int want_dx);  // dZg, dZu and, for dx, dabar, dbbar
cudaError_t launch_router_bwd(const Ctx& c, float aux_coef, float* d_bias, int accumulate, int want_dx);
// the block inside its layer (Eq. 5 / Eq. 6)
int rmsnorm_max_width(int bf16_mode);   // widest model the norm kernels take (8192 bf16, 4096 fp32)
cudaError_t launch_rmsnorm_fwd(const Ctx& c, const void* z, const void* w_norm, float eps, void* xn, float* inv_rms);
cudaError_t launch_rmsnorm_bwd(const Ctx& c, const void* z, const void* w_norm, const float* inv_rms, const void* dxn,
                               const void* dh, void* dz);
cudaError_t launch_residual_add(const Ctx& c, void* C, long long ldc, const void* R, long long ldr, int M, int N);

// MixDoRA (dora.cu): pointers into the extra regions of its workspace, and the launchers of its kernels
struct DoraCtx {
  mixlora_dora_t m;
  float *cg, *cu, *cd;                 // [N, f], [N, f], [N, d]  c = m / n
  float *inv_g, *inv_u, *inv_d;        // 1 / n
  float *rowsq_g, *rowsq_u, *rowsq_d;  // [f], [f], [d]  squared row norms of the frozen weights
  float *wa_g, *wa_u, *wa_d;           // [f, N r], [f, N r], [d, N r]  W times every expert's A^T
  float *aat_g, *aat_u, *aat_d;        // [N r, N r]  A_cat A_cat^T (diagonal blocks used)
  void *Zd_pos, *gZd_pos;              // act [T k, N r]  zd (and gate * zd) of the slot in its expert block
  void *o_pre;                         // act [T k, d]   W2 h + s B_d zd per sorted slot, before the scale
  void *dO;                            // act [T k, d]   c_d * dy per sorted slot
  void *D_s;                           // act [T k, f]   dO W2 per sorted slot
  void *spd_s;                         // act [T k, N r] s B_d^T dO for every expert, per sorted slot
  float *dmp_g, *dmp_u, *dmp_d;        // [4 tiles, f], [4 tiles, f], [tiles, d]  per-tile shares of the magnitude
                                       // gradients (gate / up: per tile and lane quarter from the tensor-core kernel,
                                       // one row per tile from the SIMT kernel)
};
int dora_bwd_col_chunks(int f);
cudaError_t launch_dora_rowsq(const Ctx& c, const DoraCtx& dc);    // squared row norms of the three frozen weights
cudaError_t launch_dora_scales(const Ctx& c, const DoraCtx& dc);   // c = m / n from the row norms and the W A^T, A A^T products
cudaError_t launch_dora_swiglu_fwd(const Ctx& c, const DoraCtx& dc);
cudaError_t launch_dora_own_block(const Ctx& c, const void* in, void* own, void* gown);
cudaError_t launch_dora_combine_y(const Ctx& c, const DoraCtx& dc, void* y);
cudaError_t launch_dora_dout(const Ctx& c, const DoraCtx& dc, const void* dy);
cudaError_t launch_dora_swiglu_bwd(const Ctx& c, const DoraCtx& dc);
cudaError_t launch_dora_dm_reduce(const Ctx& c, const float* part, const float* inv_n, float* dm, int width,
                                  int accumulate, int sub = 1);
cudaError_t launch_dora_pcompact(const Ctx& c, const DoraCtx& dc);
cudaError_t launch_grouped_swiglu_dora_fwd(const Ctx& c, const DoraCtx& dora);   // grouped_swiglu.cu
cudaError_t launch_grouped_swiglu_dora_bwd(const Ctx& c, const DoraCtx& dora);

// Dense product (tensor-core kernel in tc_gemm.cu, SIMT kernel otherwise), fp32 accumulation:
//   C_o[M, N_o] = sum_seg op(A_o,seg) * op(B_o,seg)
// A is [M, K] row-major (a_mn = 0) or [K, M] row-major (a_mn = 1); B is [N, K] row-major
// (b_kn = 0) or [K, N] row-major (b_kn = 1).  Reduction segments are concatenated; several
// outputs share one launch.  The tensor-core kernel wants bf16 operands.
// Output mode 0: activation type, row-major with pitch ldc.  Mode 1: fp32 at
//   C + (n / nb) * s_blk + (n % nb) * s_n + m * s_m   (nb = 0: C + n * s_n + m * s_m),
// value alpha * acc, added to the old value when accumulate is set.
struct TcSeg {
  const void* A; long long lda; int a_mn; int K;
  const void* B; long long ldb; int b_kn;
  int b_cols;   // columns (b_kn = 1) or rows (b_kn = 0) that exist in B when fewer than N_o rounded up; 0 = N_o
};
struct TcOut {
  void* C; long long ldc; int N;
  int M;        // rows of this output when it differs from the launch's M (0 = same)
  int mode; long long s_m, s_n, s_blk; int nb; float alpha; int accumulate;
  const void* R; long long ldr;   // mode 0 only: optional [M, N] matrix of the output's type added to the product
  TcSeg seg[kMaxKSeg]; int nseg;
};
// Optional block-sparse schedule built on the device from the segment offsets (router.cu): only the listed
// (row tile, column block) items are computed, each with its own range of 64-deep reduction blocks and its own
// window of stored columns.  Items are 8 ints {output, m0, n0, kb_begin, kb_end, n_lo, n_hi, 0}.
struct TcWork {
  const int* items;   // device
  const int* count;   // device, number of items
  int max_items;      // bound used to size the launch
  int block_cols;     // columns of one block (the LoRA rank)
};
bool tc_gemm_supported(int M, const TcOut* outs, int nout);
void tc_set_force_single(int v);   // 1: single-CTA tensor-core kernel for every shape (measurement switch)
cudaError_t launch_wait_timeout_selftest(int* status, unsigned limit, cudaStream_t st);
int tc_gemm_tile_rows(int M);   // rows of the tiles the tensor-core kernel will use for a problem with M rows
// Optional scratch for a split reduction: the tiles of a launch's last, partial round of CTA pairs (every tile when
// the launch has fewer tiles than pairs) are given to 2..kSplitKMax pairs each, which exchange fp32 partials through
// `part`; `counters` must be zero at the launch and are zero again after it.  One launch at a time per scratch.
constexpr int kSplitKMax = 4;
constexpr int kSplitCounters = 1024;                         // ints; 8 per split tile
constexpr size_t kSplitTileBytes = 256 * 256 * 4;            // one fp32 partial of a 256 x 256 tile
constexpr int kSplitMaxItems = 222;                          // shares in flight: three rounds of 74 CTA pairs
struct TcSplit {
  float* part; size_t part_bytes;
  int* counters; int n_counters;
};
// Bytes of `part` that serve every launch whose outputs have at most `rows` rows and `cols` columns in total
// (0 where the CTA-pair kernel is not used).
static inline size_t splitk_part_bytes(long long rows, long long cols) {
  if (rows < 256) return 0;
  long long tiles = ((rows + 255) / 256) * ((cols + 255) / 256 + 4);   // a few narrow outputs beside the wide ones
  long long items = tiles * kSplitKMax;
  if (items > kSplitMaxItems) items = kSplitMaxItems;
  return (size_t)items * kSplitTileBytes;
}
cudaError_t launch_tc_gemm(int M, const TcOut* outs, int nout, int* status_word, cudaStream_t st,
                           const TcWork* wl = nullptr, const TcSplit* split = nullptr);
// Work lists over the sorted slots (need seg_off of the dispatch step):
//   rows list : for every tile of `tile_rows` sorted slots and every expert with slots in it, `nout` items that
//               compute that expert's block of r columns for the tile's rows (all k-blocks);
//   reduce list: for every output, expert and tile of `tile_rows` output rows, one item whose reduction runs over
//               the k-blocks that touch the expert's segment of sorted slots.
cudaError_t launch_rows_worklist(const Ctx& c, int tile_rows, int nout, int kblocks, int* items, int* count);
cudaError_t launch_reduce_worklist(const Ctx& c, int out_rows, int tile_rows, int nout, int* items, int* count);
static inline int rows_worklist_max(int slots, int N, int nout) { return ((slots + kSegTile - 1) / kSegTile + N) * nout; }
static inline int reduce_worklist_max(int out_rows, int N, int nout) { return ((out_rows + kSegTile - 1) / kSegTile) * N * nout; }

}  // namespace mixlora
