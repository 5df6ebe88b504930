// Per-expert LoRA-B expansion fused with SwiGLU over the permuted token segments, forward and
// backward, on the tensor cores (Algorithm 1, the steps inside the expert loop up to the down projection).
//
// Work item = (segment tile, column tile): up to 128 consecutive sorted slots of ONE expert e (the
// dispatch kernel cuts every expert's segment into such tiles) times COLS columns of the FFN width.
//   producer warp : TMA loads of the rank-r operands: the tile's rows of zg / zu (/ s pd) and the COLS rows of
//                   B_g[e] / B_u[e] (/ the r rows of A_d[e]); a few KB per item
//   MMA warp      : da = zg B_g[e]^T, db = zu B_u[e]^T (, dd = (s pd) A_d[e]) as tcgen05.mma with K = r into TMEM
//   16 epilogue warps:
//     - gather the shared projections G, U (and D = dy W_d) of the tile's tokens with cp.async, four rows of 128
//       contiguous bytes per warp instruction, one item ahead, into 128B-swizzled smem tiles
//     - a = G + da, b = U + db, h = SiLU(a) b            (backward: Dt = D + dd, dgate, d a, d b as well)
//     - results go to swizzled smem tiles and leave with TMA tile stores (full tiles) or predicated stores
//       (the last, shorter tile of a segment, whose remaining rows belong to the next expert)
// All waits are bounded as in the dense product; the epilogue warps leave their loop together.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace mixlora {

namespace {

using namespace tc;

constexpr int kSplit = 4;                 // epilogue warps per TMEM lane quarter
constexpr int NET = 128 * kSplit;         // epilogue threads
constexpr int kThreads = 64 + NET;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kBufStride = 256;
constexpr int kMaxStages = 4;
constexpr uint32_t kBlockBytes = 128 * 128;   // one 64-column block of a 128-row tile

struct alignas(64) GsParams {
  CUtensorMap a_map[3];    // zg_s, zu_s, p_s : [slots, RP]
  CUtensorMap b_map[3];    // B_g, B_u as [N f, RP] ; A_d as [N r, f]
  CUtensorMap o_map[3];    // h, da, db : [slots, f]
  const bf16* G; const bf16* U; const bf16* D;
  const int* pos_token; const int* perm; const float* gates; const int* tile_info;
  bf16* h; bf16* da; bf16* db;
  float* dgate_part;       // [col_tiles, slots]
  int max_tiles, slots, f, r, row_bytes, kblocks, ksteps, krows, col_tiles, nstages, out_sets;
  uint32_t stage_bytes, a_bytes;
  int* status;
};

__device__ __forceinline__ void unpack8(const uint4& raw, float* o) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 v = __bfloat1622float2(p[i]);
    o[2 * i] = v.x;
    o[2 * i + 1] = v.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float* v) {
  uint4 r;
  __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 h2 = __floats2bfloat162_rn(v[4], v[5]), h3 = __floats2bfloat162_rn(v[6], v[7]);
  r.x = *reinterpret_cast<uint32_t*>(&h0); r.y = *reinterpret_cast<uint32_t*>(&h1);
  r.z = *reinterpret_cast<uint32_t*>(&h2); r.w = *reinterpret_cast<uint32_t*>(&h3);
  return r;
}
// sigmoid(a) = 0.5 tanh(a / 2) + 0.5 with the hardware tanh approximation (one special-function op;
// its error is below the bf16 rounding of every value stored from here)
__device__ __forceinline__ float fast_sigmoid(float a) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * a));
  return fmaf(t, 0.5f, 0.5f);
}
template <int BWD>
__global__ void __launch_bounds__(kThreads, 1) grouped_swiglu_kernel(const __grid_constant__ GsParams p) {
  constexpr int COLS = BWD ? 64 : 128;
  constexpr int CB = COLS / 64;                        // 64-column blocks per tile
  constexpr int NSUB = BWD ? 3 : 2;                    // MMAs per item
  constexpr int NMAT = BWD ? 3 : 2;                    // gathered matrices G, U (, D)
  constexpr int NOUT = BWD ? 2 : 1;                    // stored matrices: h forward; da, db backward (the forward's h
                                                       // is still in the workspace and serves the A_d gradient)
  constexpr uint32_t kSetBytes = NMAT * CB * kBlockBytes;
  constexpr uint32_t kOutBytes = NOUT * CB * kBlockBytes;
  constexpr int WCOLS = COLS / kSplit;                 // columns per epilogue thread
  constexpr int NCH = WCOLS / 8;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* gather_smem = smem;                                    // two sets
  uint8_t* out_smem = gather_smem + 2 * kSetBytes;
  uint8_t* stage_smem = out_smem + p.out_sets * kOutBytes;          // one or two output tiles
  float* dg_smem = reinterpret_cast<float*>(stage_smem + p.nstages * p.stage_bytes);   // [kSplit][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(dg_smem + (BWD ? kSplit * BM : 0));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_stop = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t stage_base = smem_u32(stage_smem);
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kMaxStages + 2 + b); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4 * kSplit); }
    *abort_flag = 0;
    *epi_stop = 0;
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
  const int total = ntiles * p.col_tiles;
  const int kb_cols = p.row_bytes / 2;                 // K elements per k-block (16, 32 or 64)

  if (warp == 0) {
    // ---------------- producer: rank-r operands ----------------
    if (lane == 0) {
      for (int s = 0; s < NSUB; ++s) { prefetch_tmap(&p.a_map[s]); prefetch_tmap(&p.b_map[s]); }
      uint32_t it = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
        const int tile = w / p.col_tiles, col0 = (w % p.col_tiles) * COLS;
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
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++wcount) {
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
  } else {
    // ---------------- epilogue ----------------
    const int q = warp & 3;                            // TMEM lane quarter this warp may read
    const int part = (warp - 2) >> 2;                  // column share of the tile
    const int et = threadIdx.x - 64;
    const int row = q * 32 + lane;                     // this thread's row of the tile
    const uint32_t gs_base = smem_u32(gather_smem);
    const uint32_t out_base = smem_u32(out_smem);

    // Cooperative gather of item w into `set`.  Thread -> rows g_r0 and g_r0 + 64 of every 64-column block and the
    // 16-byte chunk g_cb of those rows, so a warp instruction reads 4 rows x 128 contiguous bytes.  Everything
    // that does not depend on the item is computed once here.
    const int g_r0 = et >> 3, g_cb = et & 7;
    const uint32_t g_dst0 = gs_base + g_r0 * 128 + ((g_cb ^ (g_r0 & 7)) << 4);
    auto gather = [&](int w, int set) {
      const int tile = w / p.col_tiles, col0 = (w % p.col_tiles) * COLS;
      const int p0 = p.tile_info[tile * 4 + 1], rows = p.tile_info[tile * 4 + 2];
      const bool in0 = g_r0 < rows, in1 = g_r0 + 64 < rows;
      const size_t row0 = (size_t)(in0 ? p.pos_token[p0 + g_r0] : 0) * p.f + col0 + g_cb * 8;
      const size_t row1 = (size_t)(in1 ? p.pos_token[p0 + g_r0 + 64] : 0) * p.f + col0 + g_cb * 8;
      const uint32_t dst_set = g_dst0 + set * kSetBytes;
#pragma unroll
      for (int m = 0; m < NMAT; ++m) {
        const bf16* base = m == 0 ? p.G : (m == 1 ? p.U : p.D);
#pragma unroll
        for (int j = 0; j < CB; ++j) {
          const bool cin = col0 + j * 64 + g_cb * 8 < p.f;
          const uint32_t dst = dst_set + (m * CB + j) * kBlockBytes;
          const bool a0 = in0 && cin, a1 = in1 && cin;
          const bf16* s0 = a0 ? base + row0 + j * 64 : base;
          const bf16* s1 = a1 ? base + row1 + j * 64 : base;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(s0), "r"(a0 ? 16 : 0) : "memory");
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 64 * 128), "l"(s1), "r"(a1 ? 16 : 0)
                       : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };

    uint32_t wcount = 0;
    if ((int)blockIdx.x < total) gather(blockIdx.x, 0);
    for (int w = blockIdx.x; w < total; w += gridDim.x, ++wcount) {
      const int tile = w / p.col_tiles, ct = w % p.col_tiles;
      const int col0 = ct * COLS;
      const int p0 = p.tile_info[tile * 4 + 1], rows = p.tile_info[tile * 4 + 2];
      const uint32_t buf = wcount & 1u, use = wcount >> 1;
      const int set = wcount & 1u;
      const bool valid = row < rows;
      const bool full_tile = rows == BM;
      const int pos = p0 + row;
      float gate = 0.f;
      if (BWD && valid) gate = p.gates[p.perm[pos]];

      if (w + (int)gridDim.x < total) gather(w + gridDim.x, set ^ 1);
      else asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 1;" ::: "memory");
      const int oidx = p.out_sets == 2 ? set : 0;      // output tile of this item
      if (et == 0) {                                   // earlier stores have finished reading that tile
        if (p.out_sets == 2) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
      }
      named_barrier(1, NET);                           // this item's gathers are visible; the output tile is free

      const bool got = __all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abort_flag));
      if (got) {
        tc_fence_after();
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kBufStride + part * WCOLS;
        const uint8_t* gset = gather_smem + set * kSetBytes;
        uint8_t* oset = out_smem + oidx * kOutBytes;
        // this thread's columns are chunks c8 = part * NCH + ch of the tile; all lie in one 64-column block
        const int jblk = (part * NCH) >> 3, cb0 = (part * NCH) & 7, rx = row & 7;
        const uint32_t row_off = jblk * kBlockBytes + row * 128;
        float dg = 0.f;
#pragma unroll
        for (int c16 = 0; c16 < WCOLS; c16 += 16) {
          uint32_t va[16], vb[16], vd[BWD ? 16 : 1];
          tmem_ld16(t_addr + c16, va);
          tmem_ld16(t_addr + COLS + c16, vb);
          if (BWD) tmem_ld16(t_addr + 2 * COLS + c16, reinterpret_cast<uint32_t(&)[16]>(vd));
          tmem_ld_wait();
#pragma unroll
          for (int hh8 = 0; hh8 < 2; ++hh8) {
            const int ch = c16 / 8 + hh8;
            const uint32_t off = row_off + (((cb0 + ch) ^ rx) << 4);
            float gv[8], uv[8], hv[8];
            unpack8(*reinterpret_cast<const uint4*>(gset + 0 * CB * kBlockBytes + off), gv);
            unpack8(*reinterpret_cast<const uint4*>(gset + 1 * CB * kBlockBytes + off), uv);
            const int col = col0 + (part * NCH + ch) * 8;
            const size_t gdst = (size_t)pos * p.f + col;
            const bool direct = !full_tile && valid && col < p.f;
            if (!BWD) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float a = gv[i] + __uint_as_float(va[hh8 * 8 + i]);
                const float b = uv[i] + __uint_as_float(vb[hh8 * 8 + i]);
                hv[i] = a * fast_sigmoid(a) * b;
              }
              const uint4 ho = pack8(hv);
              if (full_tile) *reinterpret_cast<uint4*>(oset + off) = ho;
              else if (direct) *reinterpret_cast<uint4*>(p.h + gdst) = ho;
            } else {
              float dv[8], dav[8], dbv[8];
              unpack8(*reinterpret_cast<const uint4*>(gset + 2 * CB * kBlockBytes + off), dv);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float a = gv[i] + __uint_as_float(va[hh8 * 8 + i]);
                const float b = uv[i] + __uint_as_float(vb[hh8 * 8 + i]);
                const float sg = fast_sigmoid(a);
                const float sa = a * sg;
                const float hh = sa * b;
                const float Dt = dv[i] + __uint_as_float(vd[BWD ? hh8 * 8 + i : 0]);
                dg = fmaf(Dt, hh, dg);
                const float dh = gate * Dt;
                dav[i] = dh * b * sg * (1.f + a * (1.f - sg));
                dbv[i] = dh * sa;
              }
              const uint4 ao = pack8(dav), bo = pack8(dbv);
              if (full_tile) {
                *reinterpret_cast<uint4*>(oset + 0 * CB * kBlockBytes + off) = ao;
                *reinterpret_cast<uint4*>(oset + 1 * CB * kBlockBytes + off) = bo;
              } else if (direct) {
                *reinterpret_cast<uint4*>(p.da + gdst) = ao;
                *reinterpret_cast<uint4*>(p.db + gdst) = bo;
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(buf));
        if (BWD) dg_smem[part * BM + row] = dg;
      } else if (lane == 0) {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
      }
      fence_proxy_async_smem();                        // the tile written above is read by the TMA unit
      if (et == 0 && *abort_flag) *epi_stop = 1;
      named_barrier(1, NET);
      if (et == 0 && got && full_tile) {
#pragma unroll
        for (int m = 0; m < NOUT; ++m)
#pragma unroll
          for (int j = 0; j < CB; ++j)
            tma_store_2d(&p.o_map[m], out_base + oidx * kOutBytes + (m * CB + j) * kBlockBytes, col0 + j * 64, p0);
      }
      if (et == 0) tma_store_commit();                 // one group per item, also when nothing was stored
      if (BWD && got && part == 0 && valid) {          // the row's partial <Dt, h> over this column tile, fixed order
        float sdg = 0.f;
#pragma unroll
        for (int pp = 0; pp < kSplit; ++pp) sdg += dg_smem[pp * BM + row];
        p.dgate_part[(size_t)ct * p.slots + pos] = sdg;
      }
      if (*epi_stop) break;                            // same value for every epilogue thread after the barrier
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (et == 0) tma_store_wait_all<0>();
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
cudaError_t launch_t(const Ctx& c) {
  constexpr int COLS = BWD ? 64 : 128;
  constexpr int CB = COLS / 64;
  constexpr int NMAT = BWD ? 3 : 2, NOUT = BWD ? 2 : 1;
  const int slots = c.s.tokens * c.s.top_k, f = c.s.d_ff, r = c.s.rank, N = c.s.n_experts;
  const int rp = r < 16 ? 16 : r;
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
  p.out_sets = 2;
  uint32_t fixed = 2 * NMAT * CB * kBlockBytes + 2 * NOUT * CB * kBlockBytes + (BWD ? kSplit * BM * 4 : 0) + 1024 + 256;
  if (fixed + 2 * p.stage_bytes > budget) {            // wide operands: fall back to one output tile
    p.out_sets = 1;
    fixed -= NOUT * CB * kBlockBytes;
  }
  int nst = (int)((budget - fixed) / p.stage_bytes);
  if (nst > kMaxStages) nst = kMaxStages;
  if (nst < 2) return cudaErrorInvalidConfiguration;
  p.nstages = nst;
  const uint32_t smem_bytes = fixed + nst * p.stage_bytes;

  const int kbc = p.row_bytes / 2;
  const void* bg = r < 16 ? (const void*)(c.ws + c.L.bgp) : c.p.b_gate;
  const void* bu = r < 16 ? (const void*)(c.ws + c.L.bup) : c.p.b_up;
  bool ok = tc_encode_2d(&p.a_map[0], c.ws + c.L.zg_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
            tc_encode_2d(&p.a_map[1], c.ws + c.L.zu_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
            tc_encode_2d(&p.b_map[0], bg, (long long)N * f, rp, rp, COLS, kbc, p.row_bytes) &&
            tc_encode_2d(&p.b_map[1], bu, (long long)N * f, rp, rp, COLS, kbc, p.row_bytes) &&
            tc_encode_2d(&p.o_map[0], c.ws + c.L.h_sorted, slots, f, f, BM, 64, 128);
  if (BWD)
    ok = ok && tc_encode_2d(&p.a_map[2], c.ws + c.L.p_s, slots, rp, rp, BM, kbc, p.row_bytes) &&
         tc_encode_2d(&p.b_map[2], c.p.a_down, (long long)N * r, f, f, p.krows, 64, 128) &&
         tc_encode_2d(&p.o_map[0], c.ws + c.L.da_sorted, slots, f, f, BM, 64, 128) &&
         tc_encode_2d(&p.o_map[1], c.ws + c.L.db_sorted, slots, f, f, BM, 64, 128);
  if (!ok) return cudaErrorInvalidValue;
  p.G = c.at<bf16>(c.L.G); p.U = c.at<bf16>(c.L.U); p.D = c.at<bf16>(c.L.D);
  p.pos_token = c.at<int>(c.L.pos_token); p.perm = c.at<int>(c.L.perm); p.gates = c.at<float>(c.L.gates);
  p.tile_info = c.at<int>(c.L.tile_info);
  p.h = c.at<bf16>(c.L.h_sorted); p.da = c.at<bf16>(c.L.da_sorted); p.db = c.at<bf16>(c.L.db_sorted);
  p.dgate_part = c.at<float>(c.L.dgate_part);
  p.max_tiles = max_seg_tiles(c.s.tokens, c.s.top_k, N);
  p.slots = slots; p.f = f; p.r = r;
  p.col_tiles = (f + COLS - 1) / COLS;
  p.status = c.at<int>(c.L.status);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(grouped_swiglu_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  // the number of segment tiles is only known on the device; every CTA reads it and idles if it has no item
  grouped_swiglu_kernel<BWD><<<sms, kThreads, smem_bytes, c.st>>>(p);
  return cudaGetLastError();
}

}  // namespace

// ranks this kernel takes: the operand rows must be 32, 64 or 128 bytes, or two 128-byte blocks
bool grouped_swiglu_supported(const Ctx& c) {
  const int r = c.s.rank;
  return c.bf16 && c.s.tokens > 0 && (r == 8 || r == 16 || r == 32 || r == 64 || r == 128);
}
int grouped_swiglu_bwd_col_tiles(int f) { return (f + 63) / 64; }
cudaError_t launch_grouped_swiglu_fwd(const Ctx& c) { return launch_t<0>(c); }
cudaError_t launch_grouped_swiglu_bwd(const Ctx& c) { return launch_t<1>(c); }

}  // namespace mixlora
