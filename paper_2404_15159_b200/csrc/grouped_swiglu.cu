// Per-expert LoRA-B expansion fused with SwiGLU over the permuted token segments, forward and
// backward, on the tensor cores (Algorithm 1, the steps inside the expert loop up to the down projection).
//
// Work item = (segment tile, column tile): up to 128 consecutive sorted slots of ONE expert e (the
// dispatch kernel cuts every expert's segment into such tiles) times COLS columns of the FFN width.
//   producer warp : TMA loads of the rank-r operands: the tile's rows of zg / zu (/ s pd) and the COLS rows of
//                   B_g[e] / B_u[e] (/ the r rows of A_d[e]); a few KB per item
//   MMA warp      : da = zg B_g[e]^T, db = zu B_u[e]^T (, dd = (s pd) A_d[e]) as tcgen05.mma with K = r into TMEM
//   gather warps  : fetch the shared projections G, U (and D = dy W_d) of the tile's tokens with cp.async, four
//                   rows of 128 contiguous bytes per warp instruction, into a ring of 128B-swizzled smem tiles,
//                   up to three items ahead of the epilogue; they also look up the item's slot range and gates
//   16 (8 backward) epilogue warps: a = G + da, b = U + db, h = SiLU(a) b (backward: Dt = D + dd, dgate, d a, d b as well) in
//                   packed fp32 pairs, into one of two swizzled output tiles; one CTA-wide barrier per item
//   store warp    : after that barrier, sends full tiles out by TMA, waits until the copy has read the tile and
//                   hands it back; the last, shorter tile of a segment (whose remaining rows belong to the next
//                   expert) is copied out by the epilogue threads with predicated stores instead
// The TMA stores of these 128-byte-wide boxes drain at about 15 cycles per row and SM, which paces the kernel; both
// other ways out (coalesced stores from the smem tile, 32-byte stores straight from the registers) measured slower.
// All waits are bounded as in the dense product.
//
// Backward with FOLD: the kernel also forms the rank-r gradients dzg = da (s B_g[e]), dzu = db (s B_u[e]) of every
// slot.  A CTA then takes units of work (one segment tile x one group of column tiles) instead of single items and
// walks the unit's column tiles in turn; after the barrier of an item the store warp's thread multiplies the da and
// db tiles, still in shared memory, with the matching 64 x 64 blocks of s B_g, s B_u (all experts' blocks side by
// side, so the block holds the tile's expert) into two accumulators of 64 TMEM columns that live for the whole unit.
// At the unit's end the gather warps write the expert's own r columns as one fp32 partial per column group; a
// later kernel adds the groups in a fixed order.  da and db are then not read again for this product.
// Forward with FOLD: the same for zd = h A_d[e]^T (the input of the LoRA of W2): 64-column tiles like the backward
// kernel's, which leaves TMEM columns for one accumulator of up to 128; B = the r x 64 block of A_d[e].
// DORA (the weight-decomposed variant, Section 4.1): a = c_g[e] (G + da), b = c_u[e] (U + db) with one scale per
// expert and column; the epilogue threads load their columns' scales, the backward kernel gathers D per sorted slot,
// stores the gradients of the pre-scale values and leaves, per (segment tile, lane quarter), the sums over rows of
// d a * a_pre and d b * b_pre (formed inside each warp by halving shuffle exchanges).
#include <algorithm>
#include <type_traits>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace mixlora {

namespace {

using namespace tc;

// epilogue warps per TMEM lane quarter: 4 forward (16 warps, 80 registers per thread); 2 backward, whose heavier
// per-element arithmetic gains a little more from 128 registers per thread (8 warps) than from the extra warps
// (measured at C3: forward 0.217 ms with 4 against 0.235 with 2, backward 0.472 with 4 against 0.456 with 2)
template <int BWD> struct Epi {
  static constexpr int kSplit = BWD ? 2 : 4;
  static constexpr int NET = 128 * kSplit;   // epilogue threads
};
constexpr int kStoreWarp = 2;             // issues the TMA stores of the results
constexpr int kGatherWarps = 4;           // warps that fetch the G / U / D rows
constexpr int NGT = 32 * kGatherWarps;
constexpr int kFirstGatherWarp = 3;
constexpr int kFirstEpiWarp = kFirstGatherWarp + kGatherWarps;
template <int BWD> constexpr int kThreadsOf = 32 * kFirstEpiWarp + Epi<BWD>::NET;
constexpr int kRowsPerPass = NGT / 8;     // rows one pass of the gather threads covers
constexpr int kPasses = 128 / kRowsPerPass;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kBufStride = 256;
constexpr int kMaxStages = 4;
constexpr int kMaxSets = 4;               // gathered tiles in flight per CTA
constexpr int kHdrFloats = 128 + 4;       // per set: gates of the 128 rows, first slot, row count, column tile
constexpr uint32_t kBlockBytes = 128 * 128;   // one 64-column block of a 128-row tile
constexpr uint32_t kDzbBytes = 64 * 128;      // one 64 x 64 block of s B_g or s B_u
constexpr int kUnitsAlways = 0;               // 1: whole (segment tile, column group) units without the rank-r products too (measured: no gain)

struct alignas(64) GsParams {
  CUtensorMap a_map[3];    // zg_s, zu_s, p_s : [slots, RP]
  CUtensorMap b_map[3];    // B_g, B_u as [N f, RP] ; A_d as [N r, f]
  CUtensorMap o_map[2];    // h (forward) ; da, db (backward) : [slots, f]
  const bf16* G; const bf16* U; const bf16* D;
  const int* pos_token; const int* perm; const float* gates; const int* tile_info;
  bf16* h; bf16* da; bf16* db;
  float* dgate_part;       // [col_tiles, slots]
  int max_tiles, slots, f, r, row_bytes, kblocks, ksteps, krows, col_tiles, col_group, nstages, nsets, out_sets;
  uint32_t stage_bytes, a_bytes;
  int* status;
  // FOLD only
  CUtensorMap z_map[2];    // s B_g, s B_u with all experts' blocks side by side: [f, N r], boxes of 64 x 64
  float* dz_part;          // [groups, slots, 2, r_true]
  int* groups_used;        // the number of column groups the kernel settled on
  int r_true, cg_min;
  // DORA only (the weight-decomposed variant: a = c_g[e] (G + da), b = c_u[e] (U + db))
  const float* cg; const float* cu;   // [N, f] scales of the gate and up projections
  float* dm_g; float* dm_u;           // backward: [max_tiles * 4, f] per (segment tile, lane quarter) sums over rows of
                                      // d a * a_pre and d b * b_pre (the magnitude gradients before the division by n)
};

// The order in which a CTA takes (segment tile, column tile) items; every role of the CTA walks it the same way.
//   items : groups of col_group column tiles; inside a group every segment tile in turn, its column tiles innermost;
//           consecutive items go to consecutive CTAs.  The slots of a token (they sit in different experts' segments)
//           are then worked on while the token's piece of G / U / D is still in L2, so DRAM sees each piece once.
//   units : the same groups, but a CTA takes a whole (segment tile, group) and walks its column tiles itself.
template <int UNITS>
struct Walk {
  int w;                                    // next item or unit of this CTA
  int tile, ct, ct_end, group;              // units: the unit being walked
  __device__ Walk() : w(blockIdx.x), tile(0), ct(0), ct_end(0), group(0) {}
  // the next item: its segment tile and column tile, and whether it opens / closes a unit
  __device__ __forceinline__ bool next(int ntiles, int col_tiles, int col_group, int& tile_o, int& ct_o, bool& first,
                                       bool& last) {
    if (!UNITS) {
      if (w >= ntiles * col_tiles) return false;
      const int per_group = ntiles * col_group;
      const int g = w / per_group, rem = w - g * per_group;
      const int gw = min(col_group, col_tiles - g * col_group);   // the last group may be narrower
      tile_o = rem / gw;
      ct_o = g * col_group + rem % gw;
      first = last = false;
      w += gridDim.x;
      return true;
    }
    if (ct >= ct_end) {
      const int groups = (col_tiles + col_group - 1) / col_group;
      if (w >= ntiles * groups) return false;
      group = w / ntiles;
      tile = w - group * ntiles;
      ct = group * col_group;
      ct_end = min(ct + col_group, col_tiles);
      w += gridDim.x;
    }
    tile_o = tile;
    ct_o = ct;
    first = ct == group * col_group;
    last = ct == ct_end - 1;
    ++ct;
    return true;
  }
};

// Width of the column groups in units mode: between cg_min and cg_max, the one that leaves the busiest CTA the
// fewest items (a pure function of its arguments: every thread of every CTA gets the same answer).
__device__ __forceinline__ int choose_col_group(int ntiles, int col_tiles, int cg_min, int cg_max, int ctas) {
  int best = cg_max, best_cost = 0x7fffffff;
  for (int cg = cg_max; cg >= cg_min && cg >= 1; --cg) {
    const int groups = (col_tiles + cg - 1) / cg;
    const int rounds = (ntiles * groups + ctas - 1) / ctas;
    const int cost = rounds * cg;
    if (cost < best_cost) { best_cost = cost; best = cg; }
  }
  return best;
}

// Packed fp32 pairs: one add / mul / fma instruction works on both halves of a 64-bit register pair, which halves
// the issue slots of the element-wise math (the kernel is bound by instruction issue, not by a pipe).
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pk2u(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
constexpr uint64_t kHalf2 = 0x3f0000003f000000ull;      // (0.5f, 0.5f)
constexpr uint64_t kOne2 = 0x3f8000003f800000ull;       // (1.0f, 1.0f)
constexpr uint64_t kMinusOne2 = 0xbf800000bf800000ull;  // (-1.0f, -1.0f)
// two bf16 in one word -> two fp32 (exact)
__device__ __forceinline__ uint64_t bf2_to_f2(uint32_t v) { return pk2u(v << 16, v & 0xffff0000u); }
__device__ __forceinline__ uint32_t f2_to_bf2(uint64_t v) {
  float lo, hi;
  upk2(v, lo, hi);
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
// sigmoid(a) = 0.5 tanh(a / 2) + 0.5 with the hardware tanh approximation (one special-function op per value;
// its error is below the bf16 rounding of every value stored from here)
__device__ __forceinline__ uint64_t sigmoid2(uint64_t a) {
  float lo, hi, tl, th;
  upk2(mul2(a, kHalf2), lo, hi);
  asm("tanh.approx.f32 %0, %1;" : "=f"(tl) : "f"(lo));
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(hi));
  return fma2(pk2(tl, th), kHalf2, kHalf2);
}
// Sums over the 32 lanes of a warp of 32 values per lane: on return lane l holds the sum of every lane's v[l].
// Five exchange steps, each halving the number of values a lane still carries (31 shuffles in all).
__device__ __forceinline__ float warp_transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
  for (int st = 0; st < 5; ++st) {
    const int off = 16 >> st, n = 32 >> st;
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float send = up ? v[i] : v[i + n / 2];
      const float keep = up ? v[i + n / 2] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return v[0];
}

template <int BWD, int FOLD, int UNITS, int DORA = 0>
__global__ void __launch_bounds__(kThreadsOf<BWD>, 1) grouped_swiglu_kernel(const __grid_constant__ GsParams p) {
  static_assert(!DORA || !FOLD, "the scaled variant runs without the rank-r products");
  constexpr int kSplit = Epi<BWD>::kSplit, NET = Epi<BWD>::NET;
  constexpr int COLS = (BWD || FOLD) ? 64 : 128;
  constexpr int CB = COLS / 64;                        // 64-column blocks per tile
  constexpr int NSUB = BWD ? 3 : 2;                    // MMAs per item
  constexpr int NMAT = BWD ? 3 : 2;                    // gathered matrices G, U (, D)
  constexpr int NOUT = BWD ? 2 : 1;                    // stored matrices: h forward; da, db backward (the forward's h
                                                       // is still in the workspace and serves the A_d gradient)
  constexpr uint32_t kSetBytes = NMAT * CB * kBlockBytes;
  constexpr uint32_t kOutBytes = NOUT * CB * kBlockBytes;
  constexpr int WCOLS = COLS / kSplit;                 // columns per epilogue thread
  constexpr uint32_t kDzCol0 = 192, kDzCol1 = 448;     // TMEM columns of the dzg / dzu accumulators (64 each): the
                                                       // backward's two buffers use columns 0-191 and 256-447
                                                       // (dz_readout reads them back)
  static_assert(!FOLD || UNITS, "the rank-r products accumulate over a unit of work");
  constexpr uint32_t kZdCol = 128;                     // forward FOLD: TMEM columns of the zd accumulator (up to 128; the
                                                       // forward's two 128-column buffers sit at 0 and 256)

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* gather_smem = smem;                                    // nsets sets
  uint8_t* out_smem = gather_smem + p.nsets * kSetBytes;           // one or two output tiles
  uint8_t* dzb_smem = out_smem + p.out_sets * kOutBytes;           // FOLD: the 64 x 64 blocks of s B_g, s B_u
  uint8_t* stage_smem = dzb_smem + (FOLD ? 2 * kDzbBytes : 0);
  float* dg_smem = reinterpret_cast<float*>(stage_smem + p.nstages * p.stage_bytes);   // [2][kSplit][128]
  float* hdr_smem = dg_smem + (BWD ? 2 * kSplit * BM : 0);                              // [nsets][kHdrFloats]
  uint64_t* bars = reinterpret_cast<uint64_t*>(hdr_smem + p.nsets * kHdrFloats);
  constexpr int kNumBars = 2 * kMaxStages + 6 + 2 * kMaxSets + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* out_hdr = reinterpret_cast<int*>(tmem_slot + 4);   // [2][4]: first slot, rows, column tile of the item in each output tile's turn
  // [2], by item parity: a warp that runs ahead and gives up on the next item cannot change what the others read
  // after this item's barrier
  volatile int* epi_stop = reinterpret_cast<volatile int*>(tmem_slot + 2);
  // FOLD: [gather warp][set][4]: each gather warp's own note of the item it put into a set (closes a unit / column
  // group / expert's column offset, first slot, rows), read back by the same warp when the set returns
  int* gnote = reinterpret_cast<int*>(tmem_slot + 12);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t stage_base = smem_u32(stage_smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 2 + b); };
  auto gfull_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 4 + b); };
  auto gempty_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 4 + kMaxSets + b); };
  auto ofree_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 4 + 2 * kMaxSets + b); };
  // FOLD: the s B blocks of an item have landed; the item's rank-r products are done (they have read the output tile
  // and the blocks); the accumulators of the finished unit have been read out
  const uint32_t dzb_full_bar = bar_base + 8u * (2 * kMaxStages + 6 + 2 * kMaxSets);
  const uint32_t dzdone_bar = dzb_full_bar + 8u, dzfree_bar = dzb_full_bar + 16u;
  // FOLD: a unit's last rank-r products are done.  One arrival per unit, and the next unit cannot get there before
  // this one's accumulators have been read out (dzfree), so a waiter that counts units never sees a later phase.
  const uint32_t dzunit_bar = dzb_full_bar + 24u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4 * kSplit); mbar_init(ofree_bar(b), 1);
    }
    // a set is full when every gather thread's copies have landed (one asynchronous arrival each) and its header
    // is written (one plain arrival each); it is empty again when every epilogue warp has read it
    for (int b = 0; b < kMaxSets; ++b) { mbar_init(gfull_bar(b), 2 * NGT); mbar_init(gempty_bar(b), 4 * kSplit); }
    mbar_init(dzb_full_bar, 1); mbar_init(dzdone_bar, 1); mbar_init(dzfree_bar, kGatherWarps); mbar_init(dzunit_bar, 1);
    *abort_flag = 0;
    epi_stop[0] = 0;
    epi_stop[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int ntiles = min(p.tile_info[p.max_tiles * 4], p.max_tiles);
  const int kb_cols = p.row_bytes / 2;                 // K elements per k-block (16, 32 or 64)
  const int col_group = UNITS ? choose_col_group(ntiles, p.col_tiles, p.cg_min, p.col_group, (int)gridDim.x) : p.col_group;
  if (FOLD && blockIdx.x == 0 && threadIdx.x == 0) *p.groups_used = (p.col_tiles + col_group - 1) / col_group;
  Walk<UNITS> walk;
  int tile, ct;
  bool first, last;

  if (warp == 0) {
    // ---------------- producer: rank-r operands ----------------
    if (lane == 0) {
      for (int s = 0; s < NSUB; ++s) { prefetch_tmap(&p.a_map[s]); prefetch_tmap(&p.b_map[s]); }
      uint32_t it = 0;
      bool ok = true;
      while (ok && walk.next(ntiles, p.col_tiles, col_group, tile, ct, first, last)) {
        const int col0 = ct * COLS;
        const int e = p.tile_info[tile * 4 + 0], p0 = p.tile_info[tile * 4 + 1];
        for (int sub = 0; sub < NSUB && ok; ++sub) {
          for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
            const int st = it % p.nstages;
            const uint32_t ph = (it / p.nstages) & 1u;
            if (!mbar_wait(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = stage_base + st * p.stage_bytes;
            const uint32_t b_dst = a_dst + p.a_bytes;
            const uint32_t b_bytes = (sub < 2) ? (uint32_t)COLS * p.row_bytes : (uint32_t)CB * p.krows * 128;
            mbar_expect_tx(full_bar(st), p.a_bytes + b_bytes);
            tma_load_2d(a_dst, &p.a_map[sub], full_bar(st), kb * kb_cols, p0);
            if (sub < 2) {
              tma_load_2d(b_dst, &p.b_map[sub], full_bar(st), kb * kb_cols, e * p.f + col0);
            } else {
#pragma unroll
              for (int j = 0; j < CB; ++j)
                tma_load_2d(b_dst + j * (p.krows * 128), &p.b_map[2], full_bar(st), col0 + j * 64,
                            e * p.r + kb * p.krows);
            }
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      uint32_t it = 0, wcount = 0;
      bool ok = true;
      const uint32_t idesc_k = make_idesc(COLS, 0, 0), idesc_n = make_idesc(COLS, 0, 1);
      for (; ok && walk.next(ntiles, p.col_tiles, col_group, tile, ct, first, last); ++wcount) {
        const uint32_t buf = wcount & 1u, use = wcount >> 1;
        if (!mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int sub = 0; sub < NSUB && ok; ++sub) {
          const uint32_t d_tmem = tmem_base + buf * kBufStride + sub * COLS;
          for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
            const int st = it % p.nstages;
            const uint32_t ph = (it / p.nstages) & 1u;
            if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = stage_base + st * p.stage_bytes;
            const uint32_t b_addr = a_addr + p.a_bytes;
            for (int k = 0; k < p.ksteps; ++k) {
              const uint64_t ad = make_desc_kmajor_rows(a_addr + k * 32, p.row_bytes);
              const uint64_t bd = (sub < 2) ? make_desc_kmajor_rows(b_addr + k * 32, p.row_bytes)
                                            : make_desc(b_addr + k * 2048, p.krows * 128, 1024);
              umma_bf16(d_tmem, ad, bd, sub < 2 ? idesc_k : idesc_n, (kb | k) != 0);
            }
            umma_commit(empty_bar(st));
          }
        }
        if (ok) umma_commit(tfull_bar(buf));
      }
      if (!ok) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
    }
  } else if (warp == kStoreWarp) {
    // ---------------- store warp ----------------
    if (lane == 0) {
      for (int m = 0; m < NOUT; ++m) prefetch_tmap(&p.o_map[m]);
      if (FOLD) { prefetch_tmap(&p.z_map[0]); if (BWD) prefetch_tmap(&p.z_map[1]); }
    }
    const uint32_t out_base = smem_u32(out_smem);
    const uint32_t dzb_base = smem_u32(dzb_smem);
    // FOLD: fetches the item's 64 x 64 blocks of s B_g, s B_u (rows = the tile's columns of the FFN width, columns =
    // the 64-column block of the N r experts' columns that holds the tile's expert)
    auto load_dzb = [&](int tile_, int ct_) {
      const int e = p.tile_info[tile_ * 4 + 0];
      if (BWD) {
        const int zc = (e * p.r_true) / 64 * 64;
        mbar_expect_tx(dzb_full_bar, 2 * kDzbBytes);
        tma_load_2d(dzb_base, &p.z_map[0], dzb_full_bar, zc, ct_ * COLS);
        tma_load_2d(dzb_base + kDzbBytes, &p.z_map[1], dzb_full_bar, zc, ct_ * COLS);
      } else {                                         // the r x 64 block of A_d[e] under the tile's columns
        mbar_expect_tx(dzb_full_bar, (uint32_t)p.r * 128u);
        tma_load_2d(dzb_base, &p.z_map[0], dzb_full_bar, ct_ * COLS, e * p.r);
      }
    };
    int prev_o = -1;
    uint32_t n = 0, units_done = 0;
    bool have = walk.next(ntiles, p.col_tiles, col_group, tile, ct, first, last);
    bool dz_ok = true;                                 // lane 0 only: no bounded wait of the rank-r products gave up
    if (FOLD && have && lane == 0) load_dzb(tile, ct);
    for (; have; ++n) {
      named_barrier(1, NET + 32);                      // the item's results are complete in its output tile
      if (epi_stop[n & 1u]) break;
      const bool cur_first = first, cur_last = last;
      int ntile = 0, nct = 0;
      have = walk.next(ntiles, p.col_tiles, col_group, ntile, nct, first, last);        // the item after this one (its s B blocks are fetched below)
      if (lane == 0) {
        // every epilogue thread is past the previous item (also past copying a short tile out), that item's
        // TMA stores have read its tile and, with FOLD, so have its rank-r products (both waited for below):
        // the tile may be written again
        if (prev_o >= 0) mbar_arrive(ofree_bar(prev_o));
        const int o = p.out_sets == 2 ? (int)(n & 1u) : 0;
        const int* hdr = reinterpret_cast<const int*>(out_hdr + 4 * (n & 1u));
        const int p0 = hdr[0], rows = hdr[1], col0 = hdr[2] * COLS;
        if (rows == BM) {
#pragma unroll
          for (int m = 0; m < NOUT; ++m)
#pragma unroll
            for (int j = 0; j < CB; ++j)
              tma_store_2d(&p.o_map[m], out_base + o * kOutBytes + (m * CB + j) * kBlockBytes, col0 + j * 64, p0);
        }
        tma_store_commit();
        if (FOLD && dz_ok) {
          // dzg += da_tile (s B_g block), dzu += db_tile (s B_u block): A = the 128 x 64 tile just written (K-major,
          // K = the tile's 64 columns), B = the 64 x 64 block as fetched ([K, N] row-major), four K-steps of 16
          dz_ok = mbar_wait(dzb_full_bar, n & 1u, abort_flag);
          if (dz_ok && cur_first) dz_ok = mbar_wait(dzfree_bar, (units_done & 1u) ^ 1u, abort_flag);
          if (dz_ok) {
            tc_fence_after();
            if (BWD) {
              const uint32_t idesc = make_idesc(64, 0, 1);
#pragma unroll
              for (int m = 0; m < 2; ++m) {
                const uint32_t a_addr = out_base + o * kOutBytes + m * kBlockBytes;
                const uint32_t b_addr = dzb_base + m * kDzbBytes;
                const uint32_t d_tmem = tmem_base + (m == 0 ? kDzCol0 : kDzCol1);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_bf16(d_tmem, make_desc_kmajor_rows(a_addr + k * 32, 128), make_desc(b_addr + k * 2048, 8192, 1024),
                            idesc, (cur_first && k == 0) ? 0u : 1u);
              }
            } else {
              // zd += h_tile A_d[e]^T over the tile's 64 columns: both operands K-major with 128-byte rows
              const uint32_t idesc = make_idesc(p.r, 0, 0);
              const uint32_t a_addr = out_base + o * kOutBytes;
#pragma unroll
              for (int k = 0; k < 4; ++k)
                umma_bf16(tmem_base + kZdCol, make_desc_kmajor_rows(a_addr + k * 32, 128),
                          make_desc_kmajor_rows(dzb_base + k * 32, 128), idesc, (cur_first && k == 0) ? 0u : 1u);
            }
            umma_commit(dzdone_bar);
          }
        }
        tma_store_wait_read<0>();
        if (FOLD) {
          if (dz_ok) dz_ok = mbar_wait(dzdone_bar, n & 1u, abort_flag);
          if (dz_ok && cur_last) mbar_arrive(dzunit_bar);   // the gather warps may read the unit's accumulators
          if (dz_ok && have) load_dzb(ntile, nct);
          if (!dz_ok) {
            // everyone leaves at the next item's barrier (this warp still arrives there)
            *abort_flag = 1;
            if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
            epi_stop[(n + 1) & 1u] = 1;
          }
        }
        prev_o = o;
      }
      if (cur_last) ++units_done;
      if (p.out_sets == 1) {
        // a single output tile is handed back at once: after the copy has read it or, for a short tile, after
        // the epilogue threads have copied it out (they meet the store warp once more)
        const int rows = out_hdr[4 * (n & 1u) + 1];
        if (rows < BM) named_barrier(2, NET + 32);
        if (lane == 0) mbar_arrive(ofree_bar(0));
        prev_o = -1;
      }
      __syncwarp();
    }
    if (lane == 0) tma_store_wait_all<0>();
  } else if (warp < kFirstEpiWarp) {
    // ---------------- gather warps: rows of G, U (, D) of the item's tokens ----------------
    // Thread -> 16-byte chunk g_cb of rows g_r0, g_r0 + kRowsPerPass, ... of every 64-column block, so a warp
    // instruction reads 4 rows x 128 contiguous bytes.  The copies of one item signal gfull[set] when they have
    // landed; the warps run ahead of the epilogue by the depth of the ring and never block on the data.
    const int gt = threadIdx.x - 32 * kFirstGatherWarp;
    const int g_r0 = gt >> 3, g_cb = gt & 7;
    const uint32_t g_dst0 = smem_u32(gather_smem) + g_r0 * 128 + ((g_cb ^ (g_r0 & 7)) << 4);
    int set = 0;
    uint32_t set_use = 0;                              // times the ring has wrapped
    uint32_t gitem = 0;                                // items gathered so far
    bool ok = true;
    // FOLD: the accumulators of a finished unit go out as that column group's partial: the expert's own r columns
    // of dzg and dzu for this thread's row of the tile, then the accumulators are handed back to the store warp.
    // `info`, `zp0`, `zrows` are the note of the unit's last item.  The wait is short: the store warp issues the
    // item's rank-r products right behind the item's barrier, which the epilogue warps have reached (or are about
    // to reach) when the item's gathered set comes back.
    uint32_t gunits = 0;                               // units read out so far
    auto dz_readout = [&](int info, int zp0, int zrows) {
      if (!__all_sync(0xffffffffu, mbar_wait(dzunit_bar, gunits & 1u, abort_flag))) return false;
      ++gunits;
      tc_fence_after();
      const int r = p.r_true;
      const int zrow = (warp & 3) * 32 + lane;         // the TMEM lanes this warp may read
      const uint32_t z_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(info >> 16);
      constexpr int NZ = BWD ? 2 : 1;                  // accumulators: dzg, dzu backward; zd forward
      float* dst = p.dz_part + ((size_t)((info >> 1) & 0x7fff) * p.slots + zp0 + zrow) * NZ * r;
      // 8 columns at a time: the expert's columns may end with the accumulator's (and TMEM's) last column
      for (int m = 0; m < NZ; ++m)
        for (int c = 0; c < r; c += 8) {
          uint32_t v[8];
          tmem_ld8(z_addr + (BWD ? (m == 0 ? kDzCol0 : kDzCol1) : kZdCol) + c, v);
          tmem_ld_wait();
          if (zrow < zrows) {
            *reinterpret_cast<float4*>(dst + m * r + c) = make_float4(__uint_as_float(v[0]), __uint_as_float(v[1]),
                                                                      __uint_as_float(v[2]), __uint_as_float(v[3]));
            *reinterpret_cast<float4*>(dst + m * r + c + 4) = make_float4(__uint_as_float(v[4]), __uint_as_float(v[5]),
                                                                          __uint_as_float(v[6]), __uint_as_float(v[7]));
          }
        }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(dzfree_bar);
      return true;
    };
    while (walk.next(ntiles, p.col_tiles, col_group, tile, ct, first, last)) {
      // everything the item needs from global memory besides the rows themselves is fetched before the wait for
      // a free set, so those dependent loads never delay the copies
      const int col0 = ct * COLS;
      const int p0 = p.tile_info[tile * 4 + 1], rows = p.tile_info[tile * 4 + 2];
      // rows past the tile's end and columns past f are clamped to valid data: what is computed from them is
      // never stored (kRowsPerPass is a multiple of 8, so the swizzle term of a thread's rows is constant)
      // (with FOLD the element offsets fit 32 bits: the groups are only wide enough for it at modest token counts)
      typename std::conditional<FOLD != 0, uint32_t, size_t>::type roff[kPasses];
#pragma unroll
      for (int ps = 0; ps < kPasses; ++ps)
        roff[ps] = (typename std::conditional<FOLD != 0, uint32_t, size_t>::type)
                       p.pos_token[p0 + min(g_r0 + kRowsPerPass * ps, rows - 1)] * p.f;
      // DORA backward: D = dO W2 exists per sorted slot (the output scale differs between a token's experts)
      uint32_t roff_d[(DORA && BWD) ? kPasses : 1];    // element offsets inside the tile's 128 rows of D
      if (DORA && BWD) {
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps)
          roff_d[ps] = (uint32_t)min(g_r0 + kRowsPerPass * ps, rows - 1) * (uint32_t)p.f;
      }
      float gate0 = 0.f, gate1 = 0.f;                  // gates of rows gt and (fewer than 128 gather threads) gt + NGT
      if (BWD) {
        if (gt < rows) gate0 = p.gates[p.perm[p0 + gt]];
        if (NGT < 128 && gt + NGT < rows) gate1 = p.gates[p.perm[p0 + gt + NGT]];
      }
      if (!mbar_wait(gempty_bar(set), (set_use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
      float* hdr = hdr_smem + set * kHdrFloats;
      // FOLD: the set that has just come back held the item nsets items ago, which is finished; this warp's note of
      // it is still there.  If that item closed a unit, the unit's accumulators are read out below, once this
      // item's copies are on their way.
      int old_info = 0, old_p0 = 0, old_rows = 0;
      int* note = gnote + ((warp - kFirstGatherWarp) * kMaxSets + set) * 4;
      if (FOLD) {
        if (gitem >= (uint32_t)p.nsets) { old_info = note[0]; old_p0 = note[1]; old_rows = note[2]; }
        __syncwarp();
        if (lane == 0) {
          note[0] = (last ? 1 : 0) | (walk.group << 1) |
                    ((BWD ? (p.tile_info[tile * 4 + 0] * p.r_true) & 63 : 0) << 16);
          note[1] = p0;
          note[2] = rows;
        }
        __syncwarp();
      }
      if (BWD) {
        hdr[gt] = gate0;
        if (NGT < 128) hdr[gt + NGT] = gate1;
      }
      if (gt == 0) {
        reinterpret_cast<int*>(hdr)[128] = p0;
        reinterpret_cast<int*>(hdr)[129] = rows;
        reinterpret_cast<int*>(hdr)[130] = ct;
        if (DORA) reinterpret_cast<int*>(hdr)[131] = p.tile_info[tile * 4 + 0] | (tile << 8);   // expert, segment tile
      }
      const uint32_t dst_set = g_dst0 + set * kSetBytes;
#pragma unroll
      for (int j = 0; j < CB; ++j) {
        const int col = min(col0 + j * 64 + g_cb * 8, p.f - 8);
        // D is zero-filled past column f: those columns must not add to the row's <Dt, h> (and, with D and the
        // A_d product zero there, da and db come out as zero, so they add nothing to the rank-r products either)
        const uint32_t d_bytes = col0 + j * 64 + g_cb * 8 < p.f ? 16u : 0u;
#pragma unroll
        for (int m = 0; m < NMAT; ++m) {
          const bf16* base = (m == 0 ? p.G : (m == 1 ? p.U : p.D)) + col;
          const uint32_t dst = dst_set + (m * CB + j) * kBlockBytes;
#pragma unroll
          for (int ps = 0; ps < kPasses; ++ps) {
            if (m < 2)
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + ps * kRowsPerPass * 128),
                           "l"(base + roff[ps])
                           : "memory");
            else
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + ps * kRowsPerPass * 128),
                           "l"((DORA && BWD) ? base + (size_t)p0 * p.f + roff_d[ps] : base + roff[ps]), "r"(d_bytes)
                           : "memory");
          }
        }
      }
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(gfull_bar(set)) : "memory");
      mbar_arrive(gfull_bar(set));                     // publishes the header
      if (FOLD && (old_info & 1) && !dz_readout(old_info, old_p0, old_rows)) { ok = false; break; }
      if (FOLD) ++gitem;
      if (++set == p.nsets) { set = 0; ++set_use; }
    }
    if (FOLD && ok) {
      // the last nsets items (fewer if the CTA had fewer): their records are still in the ring, oldest first
      const uint32_t left = gitem < (uint32_t)p.nsets ? gitem : (uint32_t)p.nsets;
      if (gitem < (uint32_t)p.nsets) set = 0;
      for (uint32_t i = gitem - left; i < gitem && ok; ++i) {
        const int* note = gnote + ((warp - kFirstGatherWarp) * kMaxSets + set) * 4;
        if ((note[0] & 1) && !dz_readout(note[0], note[1], note[2])) ok = false;
        if (++set == p.nsets) set = 0;
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
    }
  } else {
    // ---------------- epilogue ----------------
    const int q = warp & 3;                            // TMEM lane quarter this warp may read
    const int part = (warp - kFirstEpiWarp) >> 2;      // column share of the tile
    const int et = threadIdx.x - 32 * kFirstEpiWarp;
    const int row = q * 32 + lane;                     // this thread's row of the tile
    // this thread's columns are 16-byte chunks part * (WCOLS / 8) + ch of the tile; all lie in one 64-column block
    const int jblk = (part * (WCOLS / 8)) >> 3, cb0 = (part * (WCOLS / 8)) & 7, rx = row & 7;
    const uint32_t row_off = jblk * kBlockBytes + row * 128;

    // the items of this CTA are only counted here: what an item is comes with its gathered set's header
    uint32_t n_items = 0;
    if (UNITS) {
      const int groups = (p.col_tiles + col_group - 1) / col_group;
      for (int u = blockIdx.x; u < ntiles * groups; u += gridDim.x)
        n_items += min(col_group, p.col_tiles - (u / ntiles) * col_group);
    } else {
      const int total = ntiles * p.col_tiles;
      n_items = (int)blockIdx.x < total ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    }
    int set = 0;
    uint32_t set_use = 0;
    for (uint32_t wcount = 0; wcount < n_items; ++wcount) {
      const uint32_t buf = wcount & 1u, use = wcount >> 1;
      const int oidx = p.out_sets == 2 ? (int)buf : 0;  // output tile of this item
      const uint32_t o_use = p.out_sets == 2 ? use : wcount;
      const bool got = __all_sync(0xffffffffu, mbar_wait(gfull_bar(set), set_use & 1u, abort_flag) &&
                                                   mbar_wait(tfull_bar(buf), use & 1u, abort_flag) &&
                                                   mbar_wait(ofree_bar(oidx), (o_use & 1u) ^ 1u, abort_flag));
      int pos = 0, p0 = 0, rows = 0, ct = 0;
      if (got) {
        tc_fence_after();
        const float* hdr = hdr_smem + set * kHdrFloats;
        p0 = reinterpret_cast<const int*>(hdr)[128];
        rows = reinterpret_cast<const int*>(hdr)[129];
        ct = reinterpret_cast<const int*>(hdr)[130];
        const int etile = DORA ? reinterpret_cast<const int*>(hdr)[131] : 0;   // expert | segment tile << 8
        pos = p0 + row;
        if (et == 0) {                                 // for the store warp: the set itself is released earlier
          int* oh = out_hdr + 4 * (wcount & 1u);
          oh[0] = p0; oh[1] = rows; oh[2] = ct;
        }
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kBufStride + part * WCOLS;
        const uint8_t* gset = gather_smem + set * kSetBytes;
        uint8_t* oset = out_smem + oidx * kOutBytes;
        uint64_t dg2 = 0;
        const float gate = BWD ? hdr[row] : 0.f;
        const uint64_t gate2 = pk2(gate, gate);
        // DORA: the expert's scales of this thread's columns, and (backward) this row's weight in the column sums
        const int dcol0 = ct * COLS + part * WCOLS;
        const float* cg_row = DORA ? p.cg + (size_t)(etile & 255) * p.f : nullptr;
        const float* cu_row = DORA ? p.cu + (size_t)(etile & 255) * p.f : nullptr;
        const float live = row < rows ? 1.f : 0.f;
        const uint64_t live2 = pk2(live, live);
#pragma unroll
        for (int c16 = 0; c16 < WCOLS; c16 += 16) {
          uint32_t va[16], vb[16], vd[BWD ? 16 : 1];
          uint64_t pg2[(DORA && BWD) ? 8 : 1], pu2[(DORA && BWD) ? 8 : 1];
          constexpr bool kLoad8 = DORA && BWD;          // 8 accumulator columns at a time: the column sums need the registers
          if (!kLoad8) {
            tmem_ld16(t_addr + c16, va);
            tmem_ld16(t_addr + COLS + c16, vb);
            if (BWD) tmem_ld16(t_addr + 2 * COLS + c16, reinterpret_cast<uint32_t(&)[16]>(vd));
            tmem_ld_wait();
          }
#pragma unroll
          for (int hh8 = 0; hh8 < 2; ++hh8) {
            if (kLoad8) {
              uint32_t ta[8], tb[8], td[8];
              tmem_ld8(t_addr + c16 + hh8 * 8, ta);
              tmem_ld8(t_addr + COLS + c16 + hh8 * 8, tb);
              tmem_ld8(t_addr + 2 * COLS + c16 + hh8 * 8, td);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                va[hh8 * 8 + j] = ta[j]; vb[hh8 * 8 + j] = tb[j]; vd[BWD ? hh8 * 8 + j : 0] = td[j];
              }
            }
            const int ch = c16 / 8 + hh8;
            const uint32_t off = row_off + (((cb0 + ch) ^ rx) << 4);
            const uint4 rg = *reinterpret_cast<const uint4*>(gset + 0 * CB * kBlockBytes + off);
            const uint4 ru = *reinterpret_cast<const uint4*>(gset + 1 * CB * kBlockBytes + off);
            const uint32_t wg[4] = {rg.x, rg.y, rg.z, rg.w}, wu[4] = {ru.x, ru.y, ru.z, ru.w};
            uint64_t cg2[DORA ? 4 : 1], cu2[DORA ? 4 : 1];
            if (DORA) {
              const int dcol = dcol0 + c16 + hh8 * 8;
              float4 g0 = make_float4(0.f, 0.f, 0.f, 0.f), g1 = g0, u0 = g0, u1 = g0;
              if (dcol < p.f) {                        // f is a multiple of 8: the chunk is inside the row or past it
                g0 = __ldg(reinterpret_cast<const float4*>(cg_row + dcol));
                g1 = __ldg(reinterpret_cast<const float4*>(cg_row + dcol + 4));
                u0 = __ldg(reinterpret_cast<const float4*>(cu_row + dcol));
                u1 = __ldg(reinterpret_cast<const float4*>(cu_row + dcol + 4));
              }
              cg2[0] = pk2(g0.x, g0.y); cg2[1] = pk2(g0.z, g0.w); cg2[2] = pk2(g1.x, g1.y); cg2[3] = pk2(g1.z, g1.w);
              cu2[0] = pk2(u0.x, u0.y); cu2[1] = pk2(u0.z, u0.w); cu2[2] = pk2(u1.x, u1.y); cu2[3] = pk2(u1.z, u1.w);
            }
            if (!BWD) {
              uint32_t ho[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int v = hh8 * 8 + 2 * i;
                uint64_t a = add2(bf2_to_f2(wg[i]), pk2u(va[v], va[v + 1]));
                uint64_t b = add2(bf2_to_f2(wu[i]), pk2u(vb[v], vb[v + 1]));
                if (DORA) { a = mul2(a, cg2[i]); b = mul2(b, cu2[i]); }
                ho[i] = f2_to_bf2(mul2(mul2(a, sigmoid2(a)), b));
              }
              *reinterpret_cast<uint4*>(oset + off) = make_uint4(ho[0], ho[1], ho[2], ho[3]);
            } else {
              const uint4 rd = *reinterpret_cast<const uint4*>(gset + 2 * CB * kBlockBytes + off);
              const uint32_t wd[4] = {rd.x, rd.y, rd.z, rd.w};
              uint32_t ao[4], bo[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int v = hh8 * 8 + 2 * i;
                const uint64_t a_pre = add2(bf2_to_f2(wg[i]), pk2u(va[v], va[v + 1]));
                const uint64_t b_pre = add2(bf2_to_f2(wu[i]), pk2u(vb[v], vb[v + 1]));
                const uint64_t a = DORA ? mul2(a_pre, cg2[DORA ? i : 0]) : a_pre;
                const uint64_t b = DORA ? mul2(b_pre, cu2[DORA ? i : 0]) : b_pre;
                const uint64_t Dt = add2(bf2_to_f2(wd[i]), pk2u(vd[BWD ? v : 0], vd[BWD ? v + 1 : 0]));
                const uint64_t sg = sigmoid2(a);
                const uint64_t sa = mul2(a, sg);                         // SiLU(a)
                dg2 = fma2(Dt, mul2(sa, b), dg2);                        // <Dt, h>
                const uint64_t dh = mul2(gate2, Dt);
                // SiLU'(a) = sg (1 + a (1 - sg))
                const uint64_t ds = mul2(sg, fma2(a, fma2(sg, kMinusOne2, kOne2), kOne2));
                const uint64_t da = mul2(mul2(dh, b), ds), db = mul2(dh, sa);
                if (DORA) {
                  // with respect to the scaled a, b: the magnitude gradient collects d a * a_pre over the tile's own
                  // rows; what goes downstream is the gradient of the pre-scale value
                  pg2[(DORA && BWD) ? hh8 * 4 + i : 0] = mul2(mul2(da, a_pre), live2);
                  pu2[(DORA && BWD) ? hh8 * 4 + i : 0] = mul2(mul2(db, b_pre), live2);
                  ao[i] = f2_to_bf2(mul2(da, cg2[DORA ? i : 0]));
                  bo[i] = f2_to_bf2(mul2(db, cu2[DORA ? i : 0]));
                } else {
                  ao[i] = f2_to_bf2(da);
                  bo[i] = f2_to_bf2(db);
                }
              }
              *reinterpret_cast<uint4*>(oset + 0 * CB * kBlockBytes + off) = make_uint4(ao[0], ao[1], ao[2], ao[3]);
              *reinterpret_cast<uint4*>(oset + 1 * CB * kBlockBytes + off) = make_uint4(bo[0], bo[1], bo[2], bo[3]);
            }
          }
          if (DORA && BWD) {
            // column sums over this warp's 32 rows of the 16 + 16 products: lane l ends up with column l & 15 of
            // the gate (l < 16) or up (l >= 16) side; one partial row per (segment tile, lane quarter)
            float pv[32];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              upk2(pg2[(DORA && BWD) ? i : 0], pv[2 * i], pv[2 * i + 1]);
              upk2(pu2[(DORA && BWD) ? i : 0], pv[16 + 2 * i], pv[16 + 2 * i + 1]);
            }
            const float csum = warp_transpose_sum32(pv, lane);
            const int col = dcol0 + c16 + (lane & 15);
            if (col < p.f)
              ((lane & 16) ? p.dm_u : p.dm_g)[((size_t)(etile >> 8) * 4 + q) * p.f + col] = csum;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) { mbar_arrive(tempty_bar(buf)); mbar_arrive(gempty_bar(set)); }
        if (BWD) {
          float dlo, dhi;
          upk2(dg2, dlo, dhi);
          dg_smem[(wcount & 1u) * (kSplit * BM) + part * BM + row] = dlo + dhi;
        }
      } else if (lane == 0) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
      fence_proxy_async_smem();                        // the tile written above is read by the TMA unit (and the MMA)
      if (!got) epi_stop[wcount & 1u] = 1;
      // the one CTA-wide barrier of an item (with the store warp): the results are complete in the output tile
      named_barrier(1, NET + 32);
      // every thread sees the same value after the barrier: all of them (and the store warp) leave together, before
      // the second barrier below, if any warp gave up on this item
      if (epi_stop[wcount & 1u]) break;
      if (rows < BM) {
        // a segment's last, shorter tile: the rows behind it belong to the next expert, so the valid rows are
        // copied out of the smem tile one 16-byte chunk per thread and turn
        const uint8_t* otile = out_smem + oidx * kOutBytes;
        const int col0 = ct * COLS;
        for (int idx = et; idx < NOUT * CB * 128 * 8; idx += NET) {
          const int c = idx & 7, rr = (idx >> 3) & 127, blk = idx >> 10;   // blk = matrix * CB + column block
          const int col = col0 + (blk % CB) * 64 + c * 8;
          if (rr < rows && col < p.f) {
            bf16* dst = (BWD ? (blk / CB == 0 ? p.da : p.db) : p.h) + (size_t)(p0 + rr) * p.f + col;
            *reinterpret_cast<uint4*>(dst) =
                *reinterpret_cast<const uint4*>(otile + blk * kBlockBytes + rr * 128 + ((c ^ (rr & 7)) << 4));
          }
        }
      }
      if (p.out_sets == 1 && rows < BM) named_barrier(2, NET + 32);
      if (BWD && part == 0 && row < rows) {     // the row's partial <Dt, h> over this column tile, fixed order
        float sdg = 0.f;
#pragma unroll
        for (int pp = 0; pp < kSplit; ++pp) sdg += dg_smem[(wcount & 1u) * (kSplit * BM) + pp * BM + row];
        p.dgate_part[(size_t)ct * p.slots + pos] = sdg;
      }
      if (++set == p.nsets) { set = 0; ++set_use; }
    }
  }

  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(5000);   // let copies that may still be in flight land
  }
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int BWD>
cudaError_t launch_t(const Ctx& c, const DoraCtx* dora = nullptr) {
  constexpr int NMAT = BWD ? 3 : 2;
  const int slots = c.s.tokens * c.s.top_k, f = c.s.d_ff, r = c.s.rank, N = c.s.n_experts;
  const int rp = pad_rank(r);
  const bool fold = !dora && (BWD ? ctx_folds_dz(c) : ctx_folds_zd(c));
  if (dora && N > 256) return cudaErrorInvalidConfiguration;   // the item header packs the expert into 8 bits
  const int COLS = (BWD || fold) ? 64 : 128, CB = COLS / 64;
  GsParams p;
  memset(&p, 0, sizeof(p));
  p.row_bytes = rp >= 64 ? 128 : rp * 2;               // bytes of one operand row per k-block
  p.kblocks = rp > 64 ? rp / 64 : 1;
  p.ksteps = (p.row_bytes / 2) / 16;
  p.krows = rp >= 64 ? 64 : rp;                        // rows of A_d per k-block
  p.a_bytes = 128 * p.row_bytes;
  const uint32_t b_bytes_k = COLS * p.row_bytes, b_bytes_n = CB * p.krows * 128;
  p.stage_bytes = (uint32_t)align_up(p.a_bytes + (b_bytes_k > b_bytes_n ? b_bytes_k : b_bytes_n), 1024);
  const uint32_t budget = 227 * 1024;
  // two output tiles and as many gathered tiles in flight as fit beside two operand stages (one output tile for
  // wide operands), then as many operand stages as fit
  constexpr int NOUT = BWD ? 2 : 1;
  const uint32_t set_bytes = NMAT * CB * kBlockBytes, out_bytes = NOUT * CB * kBlockBytes;
  constexpr int kSplit = Epi<BWD>::kSplit;
  const uint32_t base = (BWD ? 2 * kSplit * BM * 4 : 0) + 1024 + 640 + (fold ? 2 * kDzbBytes : 0);
  auto need = [&](int ns, int os) { return ns * (set_bytes + kHdrFloats * 4) + os * out_bytes + base + 2 * p.stage_bytes; };
  int nsets = kMaxSets, out_sets = 2;
  while (nsets > 2 && need(nsets, out_sets) > budget) --nsets;
  if (need(nsets, out_sets) > budget) out_sets = 1;
  if (fold && out_sets != 2) return cudaErrorInvalidConfiguration;   // ranks up to 32 always leave room for two
  const uint32_t other = base + nsets * kHdrFloats * 4;
  const uint32_t fixed = nsets * set_bytes + out_sets * out_bytes + other;
  if (fixed + 2 * p.stage_bytes > budget) return cudaErrorInvalidConfiguration;
  int nst = (int)((budget - fixed) / p.stage_bytes);
  if (nst > kMaxStages) nst = kMaxStages;
  p.nsets = nsets;
  p.out_sets = out_sets;
  p.nstages = nst;
  const uint32_t smem_bytes = fixed + nst * p.stage_bytes;

  const int kbc = p.row_bytes / 2;
  // ranks between the native widths work on zero-padded copies of B_g, B_u and A_d (built with the compact z)
  const void* bg = rp != r ? (const void*)(c.ws + c.L.bgp) : c.p.b_gate;
  const void* bu = rp != r ? (const void*)(c.ws + c.L.bup) : c.p.b_up;
  const void* ad = rp != r ? (const void*)(c.ws + c.L.adp) : c.p.a_down;
  bool ok = tc_encode_2d(&p.a_map[0], c.ws + c.L.zg_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
            tc_encode_2d(&p.a_map[1], c.ws + c.L.zu_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
            tc_encode_2d(&p.b_map[0], bg, (long long)N * f, rp, rp, COLS, kbc, p.row_bytes) &&
            tc_encode_2d(&p.b_map[1], bu, (long long)N * f, rp, rp, COLS, kbc, p.row_bytes) &&
            tc_encode_2d(&p.o_map[0], c.ws + c.L.h_sorted, slots, f, f, BM, 64, 128);
  if (BWD)
    ok = ok && tc_encode_2d(&p.a_map[2], c.ws + c.L.p_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
         tc_encode_2d(&p.b_map[2], ad, (long long)N * rp, f, f, p.krows, 64, 128) &&
         tc_encode_2d(&p.o_map[0], c.ws + c.L.da_sorted, slots, f, f, BM, 64, 128) &&
         tc_encode_2d(&p.o_map[1], c.ws + c.L.db_sorted, slots, f, f, BM, 64, 128);
  if (fold && BWD)
    ok = ok && tc_encode_2d(&p.z_map[0], c.ws + c.L.bg_cat, f, (long long)N * r, (long long)N * r, 64, 64, 128) &&
         tc_encode_2d(&p.z_map[1], c.ws + c.L.bu_cat, f, (long long)N * r, (long long)N * r, 64, 64, 128);
  if (fold && !BWD)
    ok = ok && tc_encode_2d(&p.z_map[0], ad, (long long)N * rp, f, f, rp, 64, 128);
  if (!ok) return cudaErrorInvalidValue;
  p.G = c.at<bf16>(c.L.G); p.U = c.at<bf16>(c.L.U); p.D = c.at<bf16>(c.L.D);
  p.pos_token = c.at<int>(c.L.pos_token); p.perm = c.at<int>(c.L.perm); p.gates = c.at<float>(c.L.gates);
  p.tile_info = c.at<int>(c.L.tile_info);
  p.h = c.at<bf16>(c.L.h_sorted); p.da = c.at<bf16>(c.L.da_sorted); p.db = c.at<bf16>(c.L.db_sorted);
  p.dgate_part = c.at<float>(c.L.dgate_part);
  p.max_tiles = max_seg_tiles(c.s.tokens, c.s.top_k, N);
  p.slots = slots; p.f = f; p.r = rp;                  // rows per expert in the A_d operand
  p.col_tiles = (f + COLS - 1) / COLS;
  // columns per group: the group's pieces of the gathered matrices (tokens x columns x NMAT) stay well inside L2
  const long long group_cols = (32ll << 20) / ((long long)c.s.tokens * 2 * NMAT);
  p.col_group = (int)std::min<long long>(std::max<long long>(group_cols / COLS, 1), p.col_tiles);
  p.cg_min = (p.col_group + 1) / 2;                    // units of work: the kernel may settle on narrower groups
  if (fold && BWD) {
    p.col_group = grouped_bwd_col_group_max(c.s.tokens, f);
    p.cg_min = grouped_bwd_col_group_min(c.s.tokens, f);
    p.dz_part = c.at<float>(c.L.dz_part);
    p.groups_used = c.at<int>(c.L.work_count) + 3;
    p.r_true = r;
  }
  if (fold && !BWD) {
    p.col_group = grouped_fwd_col_group_max(c.s.tokens, f);
    p.cg_min = 4;
    p.dz_part = c.at<float>(c.L.zd_part);
    p.groups_used = c.at<int>(c.L.work_count) + 4;
    p.r_true = r;
  }
  if (dora) {
    p.cg = dora->cg; p.cu = dora->cu;
    p.dm_g = dora->dmp_g; p.dm_u = dora->dmp_u;
    if (BWD) p.D = reinterpret_cast<const bf16*>(dora->D_s);
  }
  p.status = c.at<int>(c.L.status);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // the number of segment tiles is only known on the device; every CTA reads it and idles if it has no item
  cudaError_t e;
  if (dora) {
    e = cudaFuncSetAttribute(grouped_swiglu_kernel<BWD, 0, 0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    grouped_swiglu_kernel<BWD, 0, 0, 1><<<sms, kThreadsOf<BWD>, smem_bytes, c.st>>>(p);
  } else if (fold) {
    e = cudaFuncSetAttribute(grouped_swiglu_kernel<BWD, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    grouped_swiglu_kernel<BWD, 1, 1><<<sms, kThreadsOf<BWD>, smem_bytes, c.st>>>(p);
  } else {
    e = cudaFuncSetAttribute(grouped_swiglu_kernel<BWD, 0, kUnitsAlways>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    grouped_swiglu_kernel<BWD, 0, kUnitsAlways><<<sms, kThreadsOf<BWD>, smem_bytes, c.st>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace

// every bf16 rank (a multiple of 8 up to 128): the operand rows are 32, 64 or 128 bytes, or two 128-byte blocks,
// other ranks zero-padded to the next of these
bool grouped_swiglu_supported(const Ctx& c) {
  return c.bf16 && c.s.tokens > 0 && c.s.rank % 8 == 0 && c.s.rank <= 128;
}
int grouped_swiglu_bwd_col_tiles(int f) { return (f + 63) / 64; }
cudaError_t launch_grouped_swiglu_fwd(const Ctx& c) { return launch_t<0>(c); }
cudaError_t launch_grouped_swiglu_bwd(const Ctx& c) { return launch_t<1>(c); }
// The weight-decomposed variant: scales c_g, c_u per (expert, column), D per sorted slot, and (backward) the
// per-(tile, lane quarter) shares of the magnitude gradients in dora.dmp_g / dmp_u ([4 * max tiles, f]).
cudaError_t launch_grouped_swiglu_dora_fwd(const Ctx& c, const DoraCtx& dora) { return launch_t<0>(c, &dora); }
cudaError_t launch_grouped_swiglu_dora_bwd(const Ctx& c, const DoraCtx& dora) { return launch_t<1>(c, &dora); }

}  // namespace mixlora
