// Dense bf16 product on the Blackwell tensor cores (tcgen05 + TMEM), operands staged by TMA.
//
//   C_o[M, N_o] = sum_seg A_seg[M, K_seg] * op(B_o,seg)          fp32 accumulation, bf16 output
//
// One persistent CTA per SM walks 128 x tile_n output tiles (tile_n <= 256).  Warp roles:
//   warp 0    : TMA producer  (one lane)  global -> 128B-swizzled smem ring, kStages deep
//   warp 1    : MMA issuer    (one lane)  tcgen05.mma 128 x tile_n x 16 into one of two TMEM accumulators
//   warps 2-5 : epilogue      tcgen05.ld of the finished accumulator, bf16 convert, global stores,
//               overlapped with the main loop of the next tile (two accumulators of 256 columns)
// Reduction segments are walked back to back into the same accumulator (K-concatenation);
// several outputs (column blocks with their own B and C) share one launch when they share A.
// A launch with few tiles and a deep reduction may split each tile's reduction over several CTA pairs (TcParams).
// Every wait is bounded: when a limit runs out the CTA records MIXLORA_ERR_DEVICE_TIMEOUT in the
// caller's status word, all roles leave their loops, and TMEM is released before exit.
#include <cuda.h>

#include <stdlib.h>

#include <atomic>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace mixlora {

namespace {

using namespace tc;
constexpr int BN_MAX = 256;      // columns per tile (UMMA N)
constexpr int BK = 64;           // reduction elements per stage = one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kMaxSeg = kMaxKSeg;  // A maps
constexpr int kMaxOut = 4;
constexpr int kMaxB = 8;           // B maps (outputs x segments)
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;        // 16 KiB
constexpr uint32_t kBBytes = BN_MAX * BK * 2;    // 32 KiB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr uint32_t kTmemCols = 512;
constexpr int kSplitMinBlocks = 32;     // k-blocks a share of a split reduction keeps at least
constexpr int kSplitShareCost = 24;     // what a share costs beside its loop, in k-blocks' time

struct alignas(64) TcParams {
  CUtensorMap a_map[kMaxB];        // index o * nseg + seg
  CUtensorMap b_map[kMaxB];        // index o * nseg + seg
  void* C[kMaxOut];
  long long ldc[kMaxOut];          // mode 0: row pitch; mode 1: stride of m
  const void* R[kMaxOut];          // mode 0: optional matrix added to the product (a residual stream), or null
  long long ldr[kMaxOut];
  long long s_n[kMaxOut], s_blk[kMaxOut];
  float alpha[kMaxOut];
  int mode[kMaxOut], nb[kMaxOut], accumulate[kMaxOut];
  int vec4[kMaxOut];               // mode 1: groups of four columns may go out as one 16-byte store
  int N[kMaxOut];                  // columns stored
  int tile_n[kMaxOut];
  int tile_start[kMaxOut + 1];     // first tile index of each output
  int kblocks[kMaxSeg];
  int Mo[kMaxOut];                 // rows of each output (outputs of one launch may differ in rows)
  int m_tiles_o[kMaxOut];
  int n_tiles_o[kMaxOut];          // column tiles of each output
  int row_group;                   // > 0: tiles are handed out row group by row group (see tile_coord)
  int nt_total;                    // column tiles of all outputs together
  int nseg, nout, total_tiles, tile_m;
  // Optional device-built work list (block-sparse schedule over the sorted slots): item = 8 ints
  // {output, m0, n0, first k-block, end k-block, first stored column, end stored column, 0}; *work_count items.
  const int* work;
  const int* work_count;
  int* status;
  // Split reduction (CTA-pair kernel, no work list): the tiles from split_from on (those of the last, partial round
  // of CTA pairs; all tiles when there are fewer than pairs) become split_k items each, over equal shares of the
  // concatenated k-blocks, so that the round's idle pairs take part.  An item leaves its fp32 partial in `part`
  // ([split tile][share][CTA of the pair][128 rows][256 columns]); per (split tile, CTA, epilogue warp) a counter
  // tells the warp that arrives last, which adds the shares in index order (the same sum whoever is last), writes
  // the output and sets the counter back to zero.
  int split_from;
  int split_k, total_kb;
  float* part;
  int* counters;
};

struct TileCoord { int o, m0, n0, kb0, kb1, n_lo, n_hi, base, ks; };

__device__ __forceinline__ int tile_total(const TcParams& p) {
  if (!p.work) return p.total_tiles;
  const int n = *p.work_count;
  return n < p.total_tiles ? n : p.total_tiles;
}

__device__ __forceinline__ TileCoord tile_coord(const TcParams& p, int tile) {
  TileCoord t;
  if (p.work) {
    const int4 a = *reinterpret_cast<const int4*>(p.work + (size_t)tile * 8);
    const int4 b = *reinterpret_cast<const int4*>(p.work + (size_t)tile * 8 + 4);
    t.o = a.x; t.m0 = a.y; t.n0 = a.z; t.kb0 = a.w; t.kb1 = b.x; t.n_lo = b.y; t.n_hi = b.z;
    t.base = 0; t.ks = -1;
    return t;
  }
  t.kb0 = 0; t.kb1 = -1;                  // all k-blocks of every segment
  t.base = 0; t.ks = -1;                  // ks >= 0: a share of a split tile, base = index among the split tiles
  if (p.split_k > 1 && tile >= p.split_from) {
    const int j = tile - p.split_from;
    t.base = j / p.split_k;
    t.ks = j - t.base * p.split_k;
    t.kb0 = (int)((long long)t.ks * p.total_kb / p.split_k);
    t.kb1 = (int)((long long)(t.ks + 1) * p.total_kb / p.split_k);
    tile = p.split_from + t.base;
  }
  if (p.row_group > 0) {
    // Row groups (all outputs have the same rows): inside a group of row_group row tiles, rows fastest, then the
    // column tiles of every output in turn.  The CTAs that run together then cover a near-square patch of the
    // output (few distinct A and B tiles per step of the reduction), and when the A rows of one group fit in L2
    // they stay there while the group sweeps every column: DRAM sees A about once and B once per group.
    const int m_tiles = p.m_tiles_o[0];
    const int per_group = p.row_group * p.nt_total;
    const int g = tile / per_group, rem = tile - g * per_group;
    const int rows = min(p.row_group, m_tiles - g * p.row_group);
    int cidx = rem / rows;
    const int mloc = rem - cidx * rows;
    int o = 0;
#pragma unroll
    for (int i = 0; i < kMaxOut - 1; ++i)
      if (o == i && i + 1 < p.nout && cidx >= p.n_tiles_o[i]) { cidx -= p.n_tiles_o[i]; o = i + 1; }
    t.o = o;
    t.m0 = (g * p.row_group + mloc) * p.tile_m;
    t.n0 = cidx * p.tile_n[o];
    t.n_lo = 0; t.n_hi = p.N[o];
    return t;
  }
  int o = 0;
#pragma unroll
  for (int i = 1; i < kMaxOut; ++i)
    if (i < p.nout && tile >= p.tile_start[i]) o = i;
  const int local = tile - p.tile_start[o];
  t.o = o;
  t.m0 = (local % p.m_tiles_o[o]) * p.tile_m;  // rows fastest: neighbouring CTAs share the B tile
  t.n0 = (local / p.m_tiles_o[o]) * p.tile_n[o];
  t.n_lo = 0; t.n_hi = p.N[o];
  return t;
}

// Stores 32 accumulator columns [n0c, n0c + 32) of one row; only columns inside [n_lo, n_hi) are written.
__device__ __forceinline__ void store_chunk32(const TcParams& p, int o, int row, int n0c, int n_lo, int n_hi,
                                              const uint32_t (&v)[32]) {
  if (row >= p.Mo[o]) return;
  if (p.mode[o] == 1) {
    float* base = reinterpret_cast<float*>(p.C[o]) + (size_t)row * p.ldc[o];
    const int nb = p.nb[o];
    const long long sn = p.s_n[o], sb = p.s_blk[o];
    const float alpha = p.alpha[o];
    const int accum = p.accumulate[o];
    const bool vec = p.vec4[o] != 0;                   // four consecutive columns are 16 contiguous, aligned bytes
    // block and offset inside the block of the chunk's first column, carried along instead of divided out per column
    int blk = nb > 0 ? n0c / nb : 0;
    int rem = nb > 0 ? n0c - blk * nb : n0c;
#pragma unroll
    for (int j4 = 0; j4 < 8; ++j4) {
      const int n = n0c + 4 * j4;
      if (vec && n >= n_lo && n + 3 < n_hi) {
        float4* dst = reinterpret_cast<float4*>(base + (size_t)blk * sb + rem);
        float4 val = make_float4(alpha * __uint_as_float(v[4 * j4]), alpha * __uint_as_float(v[4 * j4 + 1]),
                                 alpha * __uint_as_float(v[4 * j4 + 2]), alpha * __uint_as_float(v[4 * j4 + 3]));
        if (accum) {
          const float4 old = *dst;
          val.x += old.x; val.y += old.y; val.z += old.z; val.w += old.w;
        }
        *dst = val;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          int bi = blk, ri = rem + i;
          while (nb > 0 && ri >= nb) { ri -= nb; ++bi; }
          if (n + i >= n_lo && n + i < n_hi) {
            float* dst = base + (size_t)bi * sb + (size_t)ri * sn;
            float val = alpha * __uint_as_float(v[4 * j4 + i]);
            if (accum) val += *dst;
            *dst = val;
          }
        }
      }
      rem += 4;
      while (nb > 0 && rem >= nb) { rem -= nb; ++blk; }
    }
  } else {
    bf16* crow = reinterpret_cast<bf16*>(p.C[o]) + (size_t)row * p.ldc[o];
    const float alpha0 = p.alpha[o];
    const bf16* rrow = p.R[o] ? reinterpret_cast<const bf16*>(p.R[o]) + (size_t)row * p.ldr[o] : nullptr;
#pragma unroll
    for (int g8 = 0; g8 < 4; ++g8) {
      const int col = n0c + g8 * 8;
      if (col >= n_lo && col < n_hi) {
        uint4 q4;
        float w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) w[j] = alpha0 * __uint_as_float(v[g8 * 8 + j]);
        if (rrow) {                                   // fused residual add, in fp32 before the one rounding
          const uint4 r4 = *reinterpret_cast<const uint4*>(rrow + col);
          const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&r4);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 rf = __bfloat1622float2(rp[j]);
            w[2 * j] += rf.x;
            w[2 * j + 1] += rf.y;
          }
        }
        __nv_bfloat162 h0 = __floats2bfloat162_rn(w[0], w[1]);
        __nv_bfloat162 h1 = __floats2bfloat162_rn(w[2], w[3]);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(w[4], w[5]);
        __nv_bfloat162 h3 = __floats2bfloat162_rn(w[6], w[7]);
        q4.x = *reinterpret_cast<uint32_t*>(&h0);
        q4.y = *reinterpret_cast<uint32_t*>(&h1);
        q4.z = *reinterpret_cast<uint32_t*>(&h2);
        q4.w = *reinterpret_cast<uint32_t*>(&h3);
        *reinterpret_cast<uint4*>(crow + col) = q4;
      }
    }
  }
}

template <int A_MN, int B_KN>
__global__ void __launch_bounds__(kThreads, 1) tc_gemm_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  // bars[0..kStages) full, [kStages..2kStages) empty, then tmem_full[2], tmem_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
    *abort_flag = 0;
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

  int total_kb = 0;
  for (int s = 0; s < p.nseg; ++s) total_kb += p.kblocks[s];
  const int total = tile_total(p);

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      for (int s = 0; s < p.nseg * p.nout; ++s) { prefetch_tmap(&p.a_map[s]); prefetch_tmap(&p.b_map[s]); }
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        const TileCoord tc = tile_coord(p, tile);
        const int tn = p.tile_n[tc.o];
        const uint32_t tx = kABytes + (uint32_t)tn * BK * 2;
        int seg_first = 0;
        for (int sg = 0; sg < p.nseg && ok; ++sg) {
          const CUtensorMap* am = &p.a_map[tc.o * p.nseg + sg];
          const CUtensorMap* bm = &p.b_map[tc.o * p.nseg + sg];
          // an item's k-range counts the 64-deep blocks of all segments back to back
          const int nk = p.kblocks[sg];
          const int kb_begin = tc.kb1 < 0 ? 0 : max(tc.kb0 - seg_first, 0);
          const int kb_end = tc.kb1 < 0 ? nk : min(tc.kb1 - seg_first, nk);
          seg_first += nk;
          for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
            const int st = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = smem_base + st * kStageBytes;
            const uint32_t b_dst = a_dst + kABytes;
            mbar_expect_tx(full_bar(st), tx);
            if (A_MN == 0) {
              tma_load_2d(a_dst, am, full_bar(st), kb * BK, tc.m0);
            } else {
              tma_load_2d(a_dst, am, full_bar(st), tc.m0, kb * BK);
              tma_load_2d(a_dst + BK * 128, am, full_bar(st), tc.m0 + 64, kb * BK);
            }
            if (B_KN == 0) {
              tma_load_2d(b_dst, bm, full_bar(st), kb * BK, tc.n0);
            } else {
              for (int j = 0; j < tn / 64; ++j)
                tma_load_2d(b_dst + j * (BK * 128), bm, full_bar(st), tc.n0 + j * 64, kb * BK);
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
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++tcount) {
        const TileCoord tc = tile_coord(p, tile);
        const int tn = p.tile_n[tc.o];
        const int nkb = tc.kb1 < 0 ? total_kb : tc.kb1 - tc.kb0;
        const uint32_t idesc = make_idesc(tn, A_MN, B_KN);
        const uint32_t buf = tcount & 1u;
        const uint32_t use = tcount >> 1;                 // how often this accumulator was used before
        if (!mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN_MAX;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int st = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_base + st * kStageBytes;
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = (A_MN == 0) ? make_desc(a_addr + k * (UMMA_K * 2), 16, 1024)
                                            : make_desc(a_addr + k * (UMMA_K * 128), BK * 128, 1024);
            const uint64_t bd = (B_KN == 0) ? make_desc(b_addr + k * (UMMA_K * 2), 16, 1024)
                                            : make_desc(b_addr + k * (UMMA_K * 128), BK * 128, 1024);
            umma_bf16(d_tmem, ad, bd, idesc, (kb | k) != 0);
          }
          umma_commit(empty_bar(st));                      // frees the smem stage when the MMAs retire
        }
        if (ok) umma_commit(tfull_bar(buf));               // accumulator complete
      }
      if (!ok) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> bf16 -> global ----------------
    const int q = warp & 3;                                // TMEM lane quarter this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++tcount) {
      const TileCoord tc = tile_coord(p, tile);
      const int tn = p.tile_n[tc.o];
      const bool empty = tc.kb1 >= 0 && tc.kb1 <= tc.kb0;   // no k-block: the result is zero, TMEM holds nothing for it
      const uint32_t buf = tcount & 1u;
      const uint32_t use = tcount >> 1;
      // the decision must be the same for the whole warp: the TMEM loads below are warp-collective
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const int row = tc.m0 + q * 32 + lane;
      const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN_MAX;
      for (int c = 0; c < tn; c += 32) {
        uint32_t v[32];
        if (empty) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        } else {
          tmem_ld32(t_addr + c, v);
          tmem_ld_wait();
        }
        store_chunk32(p, tc.o, row, tc.n0 + c, tc.n_lo, tc.n_hi, v);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(buf));         // 4 arrivals release the accumulator
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
    }
  }

  __syncthreads();
  if (*abort_flag) {
    // a wait gave up: give copies that may still be in flight time to land before the CTA's smem goes away
    for (int i = 0; i < 200; ++i) __nanosleep(5000);
  }
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- CTA-pair variant ------------------------------------------------------------------------
// Two CTAs of a cluster work on one 256 x tile_n output tile with cta_group::2 MMAs: each CTA stages its own 128 rows
// of A and HALF of the B tile, so the operand bytes per CTA and k-block drop from 48 KB to 32 KB and the same shared
// memory holds a 6-stage ring.  Protocol (every CTA issues its own loads):
//   - both CTAs allocate TMEM (cta_group::2) and run a producer warp; every load signals the LEADER's full barrier,
//     on which the leader's producer has posted the byte count of both CTAs;
//   - the leader's MMA thread issues the MMAs for the pair and commits onto both CTAs' empty barriers at once
//     (stage free) and accumulator-full barriers;
//   - each CTA's epilogue warps drain that CTA's 128 accumulator rows and arrive on the leader's accumulator-empty
//     barrier through its cluster address;
//   - a cluster barrier at the end keeps either CTA's smem and barriers alive until both are done.
constexpr int kStages2 = 6;
constexpr uint32_t kBBytes2 = 128 * BK * 2;              // half of a 256-column B tile
constexpr uint32_t kStageBytes2 = kABytes + kBBytes2;    // 32 KiB
constexpr uint32_t kSmemBytes2 = kStages2 * kStageBytes2 + 1024 + 256;

template <int A_MN, int B_KN>
__global__ void __launch_bounds__(kThreads, 1) tc_gemm_pair_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages2 * kStageBytes2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages2 + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader of the pair
  const bool leader = rank == 0;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages2 + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kStages2 + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kStages2 + 2 + b); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 8); }   // 4 warps of each CTA
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  int total_kb = 0;
  for (int s = 0; s < p.nseg; ++s) total_kb += p.kblocks[s];
  const int total = tile_total(p);
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      for (int s = 0; s < p.nseg * p.nout; ++s) { prefetch_tmap(&p.a_map[s]); prefetch_tmap(&p.b_map[s]); }
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; tile < total && ok; tile += npairs) {
        const TileCoord tc = tile_coord(p, tile);
        const int tn = p.tile_n[tc.o], half = tn >> 1;
        const int m0 = tc.m0 + (int)rank * BM;
        const int n0 = tc.n0 + (int)rank * half;
        const uint32_t tx_pair = 2u * (kABytes + (uint32_t)half * BK * 2);
        int seg_first = 0;
        for (int sg = 0; sg < p.nseg && ok; ++sg) {
          const CUtensorMap* am = &p.a_map[tc.o * p.nseg + sg];
          const CUtensorMap* bm = &p.b_map[tc.o * p.nseg + sg];
          // an item's k-range counts the 64-deep blocks of all segments back to back
          const int nk = p.kblocks[sg];
          const int kb_begin = tc.kb1 < 0 ? 0 : max(tc.kb0 - seg_first, 0);
          const int kb_end = tc.kb1 < 0 ? nk : min(tc.kb1 - seg_first, nk);
          seg_first += nk;
          for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
            const int st = it % kStages2;
            const uint32_t ph = (it / kStages2) & 1u;
            if (!mbar_wait(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = smem_base + st * kStageBytes2;
            const uint32_t b_dst = a_dst + kABytes;
            const uint32_t lbar = map_to_cta(full_bar(st), 0);
            if (leader) mbar_expect_tx(full_bar(st), tx_pair);
            if (A_MN == 0) {
              tma_load_2d_pair(a_dst, am, lbar, kb * BK, m0);
            } else {
              tma_load_2d_pair(a_dst, am, lbar, m0, kb * BK);
              tma_load_2d_pair(a_dst + BK * 128, am, lbar, m0 + 64, kb * BK);
            }
            if (B_KN == 0) {
              tma_load_2d_pair(b_dst, bm, lbar, kb * BK, n0);
            } else {
              for (int j = 0; j < half / 64; ++j)
                tma_load_2d_pair(b_dst + j * (BK * 128), bm, lbar, n0 + j * 64, kb * BK);
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
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && leader) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < total && ok; tile += npairs, ++tcount) {
        const TileCoord tc = tile_coord(p, tile);
        const int tn = p.tile_n[tc.o];
        const int nkb = tc.kb1 < 0 ? total_kb : tc.kb1 - tc.kb0;
        const uint32_t idesc = make_idesc_m(2 * BM, tn, A_MN, B_KN);
        const uint32_t buf = tcount & 1u;
        const uint32_t use = tcount >> 1;
        if (!mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN_MAX;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int st = it % kStages2;
          const uint32_t ph = (it / kStages2) & 1u;
          if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_base + st * kStageBytes2;
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = (A_MN == 0) ? make_desc(a_addr + k * (UMMA_K * 2), 16, 1024)
                                            : make_desc(a_addr + k * (UMMA_K * 128), BK * 128, 1024);
            const uint64_t bd = (B_KN == 0) ? make_desc(b_addr + k * (UMMA_K * 2), 16, 1024)
                                            : make_desc(b_addr + k * (UMMA_K * 128), BK * 128, 1024);
            umma_bf16_pair(d_tmem, ad, bd, idesc, (kb | k) != 0);
          }
          umma_commit_pair(empty_bar(st), 3);            // frees the stage in both CTAs
        }
        if (ok) umma_commit_pair(tfull_bar(buf), 3);     // accumulator complete, for both CTAs' epilogues
      }
      if (!ok) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
    }
  } else {
    // ---------------- epilogue (both CTAs, own 128 rows) ----------------
    const int q = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < total && ok; tile += npairs, ++tcount) {
      const TileCoord tc = tile_coord(p, tile);
      const int tn = p.tile_n[tc.o];
      const bool empty = tc.kb1 >= 0 && tc.kb1 <= tc.kb0;
      const uint32_t buf = tcount & 1u;
      const uint32_t use = tcount >> 1;
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const int row = tc.m0 + (int)rank * BM + q * 32 + lane;
      const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN_MAX;
      if (tc.ks >= 0) {
        // this item's share of the reduction goes to the partial array; the warp that completes the tile adds up.
        // A warp's 32 rows x 256 columns of a share are laid out [32-column chunk][4-column group][lane]: every
        // store and load instruction of the warp covers 512 contiguous bytes.
        const size_t slab = (size_t)BM * BN_MAX;                       // floats of one CTA's half of a tile
        const size_t wofs = (size_t)q * 32 * BN_MAX + (size_t)lane * 4;   // this warp's region, this lane's float4
        float* mine = p.part + ((size_t)(tc.base * p.split_k + tc.ks) * 2 + rank) * slab + wofs;
        for (int c = 0; c < tn; c += 32) {
          uint32_t v[32];
          if (empty) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
          } else {
            tmem_ld32(t_addr + c, v);
            tmem_ld_wait();
          }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(mine + (size_t)(c / 32 * 8 + j) * 128) =
                make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
        tc_fence_before();
        __threadfence();                                               // the partial is visible before the count
        __syncwarp();
        int* counter = p.counters + (tc.base * 2 + (int)rank) * 4 + q;
        int seen = 0;
        if (lane == 0) {
          mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0));         // the accumulator is free again
          seen = atomicAdd(counter, 1);
        }
        seen = __shfl_sync(0xffffffffu, seen, 0);
        if (seen == p.split_k - 1) {
          __threadfence();
          const float* first = p.part + ((size_t)(tc.base * p.split_k) * 2 + rank) * slab + wofs;
          const int nshare = p.split_k;
          for (int c = 0; c < tn; c += 32) {
            // all shares' loads of the chunk are issued before the first sum (one round trip to L2 per chunk)
            float4 w[kSplitKMax][8];
#pragma unroll
            for (int sidx = 0; sidx < kSplitKMax; ++sidx)
#pragma unroll
              for (int j = 0; j < 8; ++j)
                w[sidx][j] = sidx < nshare
                                 ? __ldcg(reinterpret_cast<const float4*>(first + (size_t)sidx * 2 * slab +
                                                                          (size_t)(c / 32 * 8 + j) * 128))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 a = w[0][j];
#pragma unroll
              for (int sidx = 1; sidx < kSplitKMax; ++sidx)
                if (sidx < nshare) { a.x += w[sidx][j].x; a.y += w[sidx][j].y; a.z += w[sidx][j].z; a.w += w[sidx][j].w; }
              v[4 * j] = __float_as_uint(a.x); v[4 * j + 1] = __float_as_uint(a.y);
              v[4 * j + 2] = __float_as_uint(a.z); v[4 * j + 3] = __float_as_uint(a.w);
            }
            store_chunk32(p, tc.o, row, tc.n0 + c, tc.n_lo, tc.n_hi, v);
          }
          if (lane == 0) *counter = 0;                                 // ready for the next launch
        }
        continue;
      }
      for (int c = 0; c < tn; c += 32) {
        uint32_t v[32];
        if (empty) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        } else {
          tmem_ld32(t_addr + c, v);
          tmem_ld_wait();
        }
        store_chunk32(p, tc.o, row, tc.n0 + c, tc.n_lo, tc.n_hi, v);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0));   // 8 arrivals release the accumulator
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
    }
  }

  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(5000);     // let copies that may still be in flight land
  }
  tc_fence_before();
  cluster_sync_all();                                    // neither CTA leaves while its peer may still touch it
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(f);
  });
  return fn;
}

// 2-D bf16 tensor [rows, cols] row-major with leading dimension ld (elements); box = [box_rows, box_cols].
// A tensor map is a pure function of the address and the geometry, and the same few dozen (frozen weights, workspace
// regions) come back on every call, so encoded maps are kept in a small table keyed by exactly those arguments.
struct MapKey {
  const void* ptr; long long rows, cols, ld; int box_rows, box_cols, swizzle;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows &&
           box_cols == o.box_cols && swizzle == o.swizzle;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = reinterpret_cast<size_t>(k.ptr) * 0x9E3779B97F4A7C15ull;
    auto mix = [&](long long v) { h ^= (size_t)v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2); };
    mix(k.rows); mix(k.cols); mix(k.ld); mix(k.box_rows); mix(k.box_cols); mix(k.swizzle);
    return h;
  }
};
std::mutex g_map_mu;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_map_cache;
constexpr size_t kMapCacheMax = 4096;

bool encode_2d(CUtensorMap* map, const void* ptr, long long rows, long long cols, long long ld, int box_rows,
               int box_cols, int swizzle_bytes = 128) {
  EncodeFn fn = get_encode();
  if (!fn) return false;
  const MapKey key{ptr, rows, cols, ld, box_rows, box_cols, swizzle_bytes};
  {
    std::lock_guard<std::mutex> lock(g_map_mu);
    auto it = g_map_cache.find(key);
    if (it != g_map_cache.end()) { *map = it->second; return true; }
  }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                       : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B),
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  std::lock_guard<std::mutex> lock(g_map_mu);
  if (g_map_cache.size() >= kMapCacheMax) g_map_cache.clear();
  g_map_cache.emplace(key, *map);
  return true;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device
constexpr int kMaxDev = 64;
template <typename K>
cudaError_t ensure_smem_attr(K kernel, bool (&done)[kMaxDev], uint32_t bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDev && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0 && dev < kMaxDev) done[dev] = true;   // a race only repeats the call
  return e;
}

int round_up(int v, int a) { return (v + a - 1) / a * a; }

}  // namespace

bool tc_encode_2d(CUtensorMap* map, const void* ptr, long long rows, long long cols, long long ld, int box_rows,
                  int box_cols, int swizzle_bytes) {
  return encode_2d(map, ptr, rows, cols, ld, box_rows, box_cols, swizzle_bytes);
}

bool tc_gemm_supported(int M, const TcOut* outs, int nout) {
  if (M <= 0 || nout <= 0 || nout > kMaxOut) return false;
  const int nseg = outs[0].nseg;
  if (nseg <= 0 || nseg > kMaxSeg || nseg * nout > kMaxB) return false;
  if (!get_encode()) return false;
  const int a_mn = outs[0].seg[0].a_mn, b_kn = outs[0].seg[0].b_kn;
  if (a_mn && M % 8) return false;
  for (int o = 0; o < nout; ++o) {
    const TcOut& t = outs[o];
    if (t.nseg != nseg || t.N <= 0 || !t.C) return false;
    if (t.mode == 0) {
      if (t.N % 8 || t.ldc % 8 || (reinterpret_cast<uintptr_t>(t.C) & 15u)) return false;
      if (t.R && (t.ldr % 8 || (reinterpret_cast<uintptr_t>(t.R) & 15u))) return false;
    } else if (t.mode != 1 || (reinterpret_cast<uintptr_t>(t.C) & 3u)) {
      return false;
    }
    for (int s = 0; s < nseg; ++s) {
      const TcSeg& g = t.seg[s];
      if (g.K <= 0 || g.lda % 8 || g.ldb % 8) return false;   // row pitches are multiples of 16 bytes
      if ((reinterpret_cast<uintptr_t>(g.A) & 15u) || (reinterpret_cast<uintptr_t>(g.B) & 15u)) return false;
      if (g.b_kn != b_kn || g.a_mn != a_mn) return false;
      if (g.K != outs[0].seg[s].K) return false;
    }
  }
  return true;
}

namespace {

template <int A_MN, int B_KN>
cudaError_t launch_variant(const TcParams& p, int grid, cudaStream_t st) {
  static bool done[kMaxDev] = {false};
  cudaError_t e = ensure_smem_attr(tc_gemm_kernel<A_MN, B_KN>, done, kSmemBytes);
  if (e != cudaSuccess) return e;
  tc_gemm_kernel<A_MN, B_KN><<<grid, kThreads, kSmemBytes, st>>>(p);
  return cudaGetLastError();
}

template <int A_MN, int B_KN>
cudaError_t launch_pair_variant(const TcParams& p, int grid, cudaStream_t st) {
  static bool done[kMaxDev] = {false};
  cudaError_t e = ensure_smem_attr(tc_gemm_pair_kernel<A_MN, B_KN>, done, kSmemBytes2);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes2;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tc_gemm_pair_kernel<A_MN, B_KN>, p);
}

// CTA pairs are used whenever the problem has at least 256 rows; the option MIXLORA_OPT_TC_SINGLE keeps the
// single-CTA kernel for every shape (a measurement switch; MIXLORA_TC_SINGLE=1 in the environment sets its default)
std::atomic<int> g_force_single{-1};
bool tc_force_single() {
  int v = g_force_single.load(std::memory_order_relaxed);
  if (v < 0) {
    const char* e = getenv("MIXLORA_TC_SINGLE");
    v = (e && e[0] == '1') ? 1 : 0;
    g_force_single.store(v, std::memory_order_relaxed);
  }
  return v != 0;
}

// A kernel whose only job is to let a bounded wait run out: one thread waits, with the given limit, on an mbarrier
// that nothing arrives on (no copy is in flight, nothing else is touched) and records the status the production
// kernels record in that case.
__global__ void wait_timeout_selftest_kernel(int* status, uint32_t limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_limit(smem_u32(&bar), 0, &abort_flag, limit)) atomicExch(status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
  }
}

}  // namespace

void tc_set_force_single(int v) { g_force_single.store(v ? 1 : 0, std::memory_order_relaxed); }

cudaError_t launch_wait_timeout_selftest(int* status, unsigned limit, cudaStream_t st) {
  wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(status, limit);
  return cudaGetLastError();
}

int tc_gemm_tile_rows(int M) { return (!tc_force_single() && M >= 2 * BM) ? 2 * BM : BM; }

cudaError_t launch_tc_gemm(int M, const TcOut* outs, int nout, int* status_word, cudaStream_t st, const TcWork* wl,
                           const TcSplit* split) {
  TcParams p;
  memset(&p, 0, sizeof(p));
  const int nseg = outs[0].nseg;
  const int a_mn = outs[0].seg[0].a_mn, b_kn = outs[0].seg[0].b_kn;
  const bool pair = !tc_force_single() && M >= 2 * BM;
  const int tile_m = pair ? 2 * BM : BM;
  p.nseg = nseg; p.nout = nout; p.status = status_word;
  p.tile_m = tile_m;
  if (wl) {
    if (nseg != 1) return cudaErrorInvalidValue;   // a work list carries one k-range per item
    p.work = wl->items; p.work_count = wl->count;
  }
  for (int s = 0; s < nseg; ++s) p.kblocks[s] = (outs[0].seg[s].K + BK - 1) / BK;
  int tiles = 0;
  for (int o = 0; o < nout; ++o) {
    const TcOut& t = outs[o];
    // the operand tile covers whole groups of columns (16 for a K-major B, 64 for an N-major B, per CTA); columns
    // past N read as zero through the tensor map and are never stored
    const int cols = t.mode == 0 ? t.N : round_up(t.N, 8);
    const int gran = (b_kn ? 64 : 16) * (pair ? 2 : 1);
    // with a work list every item covers one block of `block_cols` columns, rounded up to the tile granularity
    const int want = wl ? wl->block_cols : cols;
    const int tn = want >= BN_MAX ? BN_MAX : round_up(want, gran);
    if (wl && wl->block_cols > BN_MAX) return cudaErrorInvalidValue;
    const int Mrows = t.M > 0 ? t.M : M;
    p.Mo[o] = Mrows; p.m_tiles_o[o] = (Mrows + tile_m - 1) / tile_m;
    p.C[o] = t.C; p.N[o] = t.N; p.tile_n[o] = tn;
    p.mode[o] = t.mode;
    p.ldc[o] = t.mode == 0 ? t.ldc : t.s_m;
    p.R[o] = t.mode == 0 ? t.R : nullptr; p.ldr[o] = t.ldr;
    p.s_n[o] = t.s_n; p.s_blk[o] = t.s_blk; p.nb[o] = t.nb; p.alpha[o] = t.alpha; p.accumulate[o] = t.accumulate;
    p.vec4[o] = t.mode == 1 && t.s_n == 1 && t.nb % 4 == 0 && t.s_m % 4 == 0 && t.s_blk % 4 == 0 &&
                (reinterpret_cast<uintptr_t>(t.C) & 15u) == 0;
    p.tile_start[o] = tiles;
    p.n_tiles_o[o] = (t.N + tn - 1) / tn;
    p.nt_total += p.n_tiles_o[o];
    tiles += p.m_tiles_o[o] * p.n_tiles_o[o];
    const int b_rows = pair ? tn / 2 : tn;               // rows of a K-major B tile held by one CTA
    for (int s = 0; s < nseg; ++s) {
      const TcSeg& g = t.seg[s];
      bool ok = a_mn ? encode_2d(&p.a_map[o * nseg + s], g.A, g.K, Mrows, g.lda, BK, 64)
                     : encode_2d(&p.a_map[o * nseg + s], g.A, Mrows, g.K, g.lda, BM, BK);
      if (!ok) return cudaErrorInvalidValue;
      ok = b_kn ? encode_2d(&p.b_map[o * nseg + s], g.B, g.K, g.b_cols > 0 ? g.b_cols : t.N, g.ldb, BK, 64)
                : encode_2d(&p.b_map[o * nseg + s], g.B, g.b_cols > 0 ? g.b_cols : t.N, g.K, g.ldb, b_rows, BK);
      if (!ok) return cudaErrorInvalidValue;
    }
  }
  for (int o = nout; o <= kMaxOut; ++o) p.tile_start[o] = tiles;
  if (!wl) {
    bool uniform = true;
    for (int o = 1; o < nout; ++o) uniform = uniform && p.m_tiles_o[o] == p.m_tiles_o[0];
    const int m_tiles = p.m_tiles_o[0];
    long long k_total = 0;
    for (int s = 0; s < nseg; ++s) k_total += outs[0].seg[s].K;
    const long long slice = (long long)tile_m * k_total * 2;          // bytes of A behind one row tile
    if (uniform && m_tiles > 1 && slice * m_tiles > (24ll << 20)) {   // A does not simply stay in L2
      const long long resident = (40ll << 20) / slice;                // row tiles whose A rows fit in L2 together
      int rg;
      if (resident >= 8) {
        const int groups = (int)((m_tiles + resident - 1) / resident);
        rg = (m_tiles + groups - 1) / groups;                         // balanced groups
      } else {
        rg = 8;                                                        // deep reductions: near-square waves of CTAs
      }
      if (rg < m_tiles) p.row_group = rg;
    }
  }
  p.total_tiles = wl ? wl->max_items : tiles;
  tiles = p.total_tiles;

  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  for (int s = 0; s < nseg; ++s) p.total_kb += p.kblocks[s];
  if (split && pair && !wl && split->part && split->counters && tiles > 0) {
    // the tiles of the last, partial round of CTA pairs (all tiles when there are fewer tiles than pairs) share their
    // reductions: with `rest` such tiles split `sk` ways the round takes ceil(rest sk / pairs) passes of
    // total_kb / sk k-blocks plus what a share costs on top (partial out, fence, count, and the adding up: measured
    // at about 24 k-blocks' time); the split must win a tenth of the round to be taken
    const int pairs = sms / 2;
    const int rest = tiles % pairs;
    int best = 1;
    if (rest > 0) {
      long long best_cost = (long long)p.total_kb * 9 / 10;
      for (int sk = 2; sk <= kSplitKMax; ++sk) {
        if (sk > p.total_kb / kSplitMinBlocks) break;                 // every share keeps a deep enough loop
        if ((size_t)rest * sk * kSplitTileBytes > split->part_bytes || rest * 8 > split->n_counters) break;
        const long long passes = (rest * sk + pairs - 1) / pairs;
        const long long cost = passes * (p.total_kb / sk + kSplitShareCost);
        if (cost < best_cost) { best_cost = cost; best = sk; }
      }
    }
    if (best >= 2) {
      p.split_k = best;
      p.split_from = tiles - rest;
      p.part = split->part;
      p.counters = split->counters;
      p.total_tiles = p.split_from + rest * best;
      tiles = p.total_tiles;
    }
  }
  if (pair) {
    const int pairs = tiles < sms / 2 ? tiles : sms / 2;
    if (a_mn) return b_kn ? launch_pair_variant<1, 1>(p, 2 * pairs, st) : launch_pair_variant<1, 0>(p, 2 * pairs, st);
    return b_kn ? launch_pair_variant<0, 1>(p, 2 * pairs, st) : launch_pair_variant<0, 0>(p, 2 * pairs, st);
  }
  const int grid = tiles < sms ? tiles : sms;
  if (a_mn) return b_kn ? launch_variant<1, 1>(p, grid, st) : launch_variant<1, 0>(p, grid, st);
  return b_kn ? launch_variant<0, 1>(p, grid, st) : launch_variant<0, 0>(p, grid, st);
}

}  // namespace mixlora
