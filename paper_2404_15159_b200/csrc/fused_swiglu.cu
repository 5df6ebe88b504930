// Per-slot LoRA-B expansion fused with SwiGLU, forward and backward, on the tensor cores.
//
// For a tile of 128 sorted slots and COLS columns of the FFN width the kernel forms
//   da = Zg_pos  (s B_g)^T     db = Zu_pos  (s B_u)^T     [backward also]  dd = P_pos  A_d
// as tcgen05 MMAs into TMEM.  Zg_pos / Zu_pos / P_pos hold a slot's rank-r vector inside the block
// of its own expert and zeros elsewhere, so one K = N r product applies every slot's own expert
// without splitting tiles at expert boundaries.  The epilogue threads (one slot each) then gather
// the shared projections G, U (and D = dy W_d) of the slot's token and finish
//   forward :  a = G + da, b = U + db, h = SiLU(a) b                                (Algorithm 1, expert loop)
//   backward:  Dt = D + dd, dgate += <Dt, h>, dh = g Dt, d a = dh b SiLU'(a), d b = dh SiLU(a)
// Warp roles, smem ring, mbarrier protocol and bounded waits are those of the dense product.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace mixlora {

namespace {

using namespace tc;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
// epilogue warps per TMEM lane quarter (each takes COLS / split columns of a tile)
constexpr int epi_split(int bwd) { return bwd ? 2 : 4; }
constexpr int threads_of(int bwd) { return 64 + 128 * epi_split(bwd); }
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kBufStride = 256;

struct alignas(64) FsParams {
  CUtensorMap a_map[3];    // Zg_pos, Zu_pos, P_pos : [slots, N r], box 128 x 64
  CUtensorMap b_map[3];    // bg_cat, bu_cat : [f, N r] box COLS x 64 ; a_down as [N r, f] box 64 x 64
  const bf16* G; const bf16* U; const bf16* D;
  const int* pos_token; const int* perm; const float* gates;
  bf16* h; bf16* da; bf16* db;
  float* dgate_part;       // [col_tiles, slots]
  int slots, f, kblocks, row_tiles, col_tiles, total;
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

template <int BWD>
__global__ void __launch_bounds__(threads_of(BWD), 1) fused_swiglu_kernel(const __grid_constant__ FsParams p) {
  constexpr int COLS = BWD ? 64 : 128;
  constexpr int kEpiSplit = epi_split(BWD);
  constexpr int NSUB = BWD ? 3 : 2;
  constexpr uint32_t kBBytes = COLS * BK * 2;
  constexpr uint32_t kStageBytes = kABytes + kBBytes;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
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
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4 * kEpiSplit); }
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

  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < NSUB; ++s) { prefetch_tmap(&p.a_map[s]); prefetch_tmap(&p.b_map[s]); }
      uint32_t it = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < p.total && ok; w += gridDim.x) {
        const int row0 = (w / p.col_tiles) * BM, col0 = (w % p.col_tiles) * COLS;
        for (int sub = 0; sub < NSUB && ok; ++sub) {
          for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
            const int st = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(empty_bar(st), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = smem_base + st * kStageBytes;
            const uint32_t b_dst = a_dst + kABytes;
            mbar_expect_tx(full_bar(st), kStageBytes);
            tma_load_2d(a_dst, &p.a_map[sub], full_bar(st), kb * BK, row0);
            if (sub < 2) {
              tma_load_2d(b_dst, &p.b_map[sub], full_bar(st), kb * BK, col0);
            } else {
#pragma unroll
              for (int j = 0; j < COLS / 64; ++j)
                tma_load_2d(b_dst + j * (BK * 128), &p.b_map[2], full_bar(st), col0 + j * 64, kb * BK);
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
    if (lane == 0) {
      uint32_t it = 0, wcount = 0;
      bool ok = true;
      const uint32_t idesc_k = make_idesc(COLS, 0, 0), idesc_n = make_idesc(COLS, 0, 1);
      for (int w = blockIdx.x; w < p.total && ok; w += gridDim.x, ++wcount) {
        const uint32_t buf = wcount & 1u, use = wcount >> 1;
        if (!mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int sub = 0; sub < NSUB && ok; ++sub) {
          const uint32_t d_tmem = tmem_base + buf * kBufStride + sub * COLS;
          for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
            const int st = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(full_bar(st), ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = smem_base + st * kStageBytes;
            const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint64_t ad = make_desc(a_addr + k * (UMMA_K * 2), 16, 1024);
              const uint64_t bd = (sub < 2) ? make_desc(b_addr + k * (UMMA_K * 2), 16, 1024)
                                            : make_desc(b_addr + k * (UMMA_K * 128), BK * 128, 1024);
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
    constexpr int WCOLS = COLS / kEpiSplit;            // columns this warp handles
    const int q = warp & 3;                            // TMEM lane quarter this warp may read
    const int part = (warp - 2) >> 2;                  // which column share of the tile
    uint32_t wcount = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < p.total && ok; w += gridDim.x, ++wcount) {
      const int ct = w % p.col_tiles;
      const int row0 = (w / p.col_tiles) * BM, col0 = ct * COLS + part * WCOLS;
      const uint32_t buf = wcount & 1u, use = wcount >> 1;
      const int pos = row0 + q * 32 + lane;
      const bool valid = pos < p.slots;
      // routing of this thread's slot (independent of the accumulator: fetched before the wait)
      const int tok = valid ? p.pos_token[pos] : 0;
      float gate = 0.f;
      if (BWD && valid) gate = p.gates[p.perm[pos]];
      const size_t src = (size_t)tok * p.f + col0;
      const size_t dst = (size_t)pos * p.f + col0;
      // the token's G, U (and D) values of this column tile do not depend on the accumulator: fetch the whole
      // row segment now, so that the gathers are in flight while the MMAs finish
      uint4 gq[WCOLS / 8], uq[WCOLS / 8], dq[BWD ? WCOLS / 8 : 1];
#pragma unroll
      for (int i = 0; i < WCOLS / 8; ++i) {
        const bool in = valid && (col0 + i * 8 < p.f);
        gq[i] = in ? __ldg(reinterpret_cast<const uint4*>(p.G + src + i * 8)) : make_uint4(0, 0, 0, 0);
        uq[i] = in ? __ldg(reinterpret_cast<const uint4*>(p.U + src + i * 8)) : make_uint4(0, 0, 0, 0);
        if (BWD) dq[i] = in ? __ldg(reinterpret_cast<const uint4*>(p.D + src + i * 8)) : make_uint4(0, 0, 0, 0);
      }
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kBufStride + part * WCOLS;
      float dg = 0.f;
#pragma unroll
      for (int c = 0; c < WCOLS; c += 16) {
        uint32_t va[16], vb[16], vd[16];
        tmem_ld16(t_addr + c, va);
        tmem_ld16(t_addr + COLS + c, vb);
        if (BWD) tmem_ld16(t_addr + 2 * COLS + c, vd);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int g8 = 0; g8 < 2; ++g8) {
            const int col = col0 + c + g8 * 8;
            if (col < p.f) {
              float gv[8], uv[8], hv[8];
              unpack8(gq[c / 8 + g8], gv);
              unpack8(uq[c / 8 + g8], uv);
              if (!BWD) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float a = gv[i] + __uint_as_float(va[g8 * 8 + i]);
                  const float b = uv[i] + __uint_as_float(vb[g8 * 8 + i]);
                  hv[i] = __fdividef(a, 1.f + __expf(-a)) * b;
                }
                *reinterpret_cast<uint4*>(p.h + dst + c + g8 * 8) = pack8(hv);
              } else {
                float dv[8], dav[8], dbv[8];
                unpack8(dq[c / 8 + g8], dv);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float a = gv[i] + __uint_as_float(va[g8 * 8 + i]);
                  const float b = uv[i] + __uint_as_float(vb[g8 * 8 + i]);
                  const float sg = __fdividef(1.f, 1.f + __expf(-a));
                  const float sa = a * sg;
                  const float hh = sa * b;
                  const float Dt = dv[i] + __uint_as_float(vd[g8 * 8 + i]);
                  dg = fmaf(Dt, hh, dg);
                  const float dh = gate * Dt;
                  hv[i] = hh;
                  dav[i] = dh * b * sg * (1.f + a * (1.f - sg));
                  dbv[i] = dh * sa;
                }
                *reinterpret_cast<uint4*>(p.h + dst + c + g8 * 8) = pack8(hv);
                *reinterpret_cast<uint4*>(p.da + dst + c + g8 * 8) = pack8(dav);
                *reinterpret_cast<uint4*>(p.db + dst + c + g8 * 8) = pack8(dbv);
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(buf));
      if (BWD && valid) p.dgate_part[(size_t)(ct * kEpiSplit + part) * p.slots + pos] = dg;
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (p.status) atomicExch(p.status, (int)MIXLORA_ERR_DEVICE_TIMEOUT);
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
cudaError_t launch_t(const Ctx& c) {
  constexpr int COLS = BWD ? 64 : 128;
  constexpr uint32_t kStageBytes = kABytes + COLS * BK * 2;
  constexpr uint32_t kSmem = kStages * kStageBytes + 1024 + 256;
  const int slots = c.s.tokens * c.s.top_k, f = c.s.d_ff, Nr = c.s.n_experts * c.s.rank;
  FsParams p;
  memset(&p, 0, sizeof(p));
  bool ok = tc_encode_2d(&p.a_map[0], c.ws + c.L.Zg_pos, slots, Nr, Nr, BM, BK) &&
            tc_encode_2d(&p.a_map[1], c.ws + c.L.Zu_pos, slots, Nr, Nr, BM, BK) &&
            tc_encode_2d(&p.b_map[0], c.ws + c.L.bg_cat, f, Nr, Nr, COLS, BK) &&
            tc_encode_2d(&p.b_map[1], c.ws + c.L.bu_cat, f, Nr, Nr, COLS, BK);
  if (BWD)
    ok = ok && tc_encode_2d(&p.a_map[2], c.ws + c.L.P_pos, slots, Nr, Nr, BM, BK) &&
         tc_encode_2d(&p.b_map[2], c.p.a_down, Nr, f, f, BK, 64);
  if (!ok) return cudaErrorInvalidValue;
  p.G = c.at<bf16>(c.L.G); p.U = c.at<bf16>(c.L.U); p.D = c.at<bf16>(c.L.D);
  p.pos_token = c.at<int>(c.L.pos_token); p.perm = c.at<int>(c.L.perm); p.gates = c.at<float>(c.L.gates);
  p.h = c.at<bf16>(c.L.h_sorted); p.da = c.at<bf16>(c.L.da_sorted); p.db = c.at<bf16>(c.L.db_sorted);
  p.dgate_part = c.at<float>(c.L.dgate_part);
  p.slots = slots; p.f = f; p.kblocks = (Nr + BK - 1) / BK;
  p.row_tiles = (slots + BM - 1) / BM; p.col_tiles = (f + COLS - 1) / COLS;
  p.total = p.row_tiles * p.col_tiles;
  p.status = c.at<int>(c.L.status);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(fused_swiglu_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  if (e != cudaSuccess) return e;
  const int grid = p.total < sms ? p.total : sms;
  fused_swiglu_kernel<BWD><<<grid, threads_of(BWD), kSmem, c.st>>>(p);
  return cudaGetLastError();
}

}  // namespace

bool fused_swiglu_supported(const Ctx& c) { return c.bf16 && c.s.tokens > 0; }
int fused_swiglu_bwd_col_tiles(int f) { return (f + 63) / 64 * epi_split(1); }
cudaError_t launch_fused_swiglu_fwd(const Ctx& c) { return launch_t<0>(c); }
cudaError_t launch_fused_swiglu_bwd(const Ctx& c) { return launch_t<1>(c); }

}  // namespace mixlora
