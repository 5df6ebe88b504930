// Router (Eq. 7), load-balance statistics (Eq. 8-9) and the dispatch of slots to experts:
// histogram, prefix scan and stable permutation in the order "expert ascending, token ascending".
#include "common.cuh"

namespace mixlora {

namespace {

constexpr int kRWarps = 8;            // warps per block of the router kernel
constexpr int kRCols = 256;           // features per step: 32 lanes x 8
constexpr float kMarginFlag = 1e-4f;

// 8 consecutive features of one row, as loaded (16 bytes of bf16, 32 bytes of fp32) and as floats
template <typename T> struct Raw8;
template <> struct Raw8<bf16> { uint4 v; };
template <> struct Raw8<float> { float4 lo, hi; };
__device__ __forceinline__ void ld_raw8(const bf16* p, Raw8<bf16>& r) { r.v = __ldg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void ld_raw8(const float* p, Raw8<float>& r) {
  r.lo = __ldg(reinterpret_cast<const float4*>(p));
  r.hi = __ldg(reinterpret_cast<const float4*>(p) + 1);
}
__device__ __forceinline__ void zero_raw8(Raw8<bf16>& r) { r.v = make_uint4(0u, 0u, 0u, 0u); }
__device__ __forceinline__ void zero_raw8(Raw8<float>& r) { r.lo = r.hi = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void cvt_raw8(const Raw8<bf16>& r, float (&o)[8]) {
  const uint32_t w[4] = {r.v.x, r.v.y, r.v.z, r.v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {                     // a bf16 is the upper half of the fp32 with the same value
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void cvt_raw8(const Raw8<float>& r, float (&o)[8]) {
  o[0] = r.lo.x; o[1] = r.lo.y; o[2] = r.lo.z; o[3] = r.lo.w;
  o[4] = r.hi.x; o[5] = r.hi.y; o[6] = r.hi.z; o[7] = r.hi.w;
}

// Router (Eq. 7).  A block of kRWarps warps handles kRWarps * TOK tokens; a warp handles TOK tokens and NE (>= N)
// logits per token, TOK * NE accumulators per lane, and each lane covers 8 consecutive features per step of 256.
// x is read once, 16 bytes per lane and token, one step ahead of its use.  The router weight goes through shared
// memory in chunks of 256 features (staged by all threads, laid out so that a lane's two 16-byte pieces of an
// expert's row are read without bank conflicts), so a block reads W_r once for all its tokens and each weight
// register serves TOK tokens.  The block also leaves the sums over its tokens that Eq. 9 needs (probability per
// expert, selections per expert) in `part`, in a fixed order.
template <typename T, int NE, int TOK>
__global__ void __launch_bounds__(kRWarps * 32)
router_kernel(const T* __restrict__ x, const float* __restrict__ w_router, const float* __restrict__ bias,
              float* __restrict__ probs, int* __restrict__ expert_idx, float* __restrict__ gates,
              uint8_t* __restrict__ low_margin, float* __restrict__ part, int tokens, int d, int N, int k,
              int renorm, int f_mode) {
  constexpr int WPT = NE / 4;                          // 16-byte pieces of a weight chunk staged per thread
  constexpr int BT = kRWarps * TOK;                    // tokens per block
  __shared__ float4 wsm[NE * 2 * 32];                  // [expert][half of the lane's 8 features][lane]
  __shared__ float sp[BT][NE];                         // probabilities of the block's tokens
  __shared__ unsigned ssel[BT];                        // bit e set: expert e counts for F_i of this token
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t0 = (blockIdx.x * kRWarps + warp) * TOK;

  float acc[TOK][NE];
#pragma unroll
  for (int a = 0; a < TOK; ++a)
#pragma unroll
    for (int e = 0; e < NE; ++e) acc[a][e] = 0.f;

  float4 wn[WPT];
  Raw8<T> xr[TOK];
  auto load_w = [&](int ch) {
#pragma unroll
    for (int i = 0; i < WPT; ++i) {
      const int j = threadIdx.x + i * (kRWarps * 32), e = j >> 6, c = ch * kRCols + (j & 63) * 4;
      wn[i] = (e < N && c < d) ? __ldg(reinterpret_cast<const float4*>(w_router + (size_t)e * d + c))
                               : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto load_x = [&](int ch) {
    const int c = ch * kRCols + lane * 8;
#pragma unroll
    for (int a = 0; a < TOK; ++a) {
      const int t = min(t0 + a, tokens - 1);           // rows past the end repeat the last token; never written
      if (c < d) ld_raw8(x + (size_t)t * d + c, xr[a]); else zero_raw8(xr[a]);
    }
  };
  const int nchunk = (d + kRCols - 1) / kRCols;
  load_w(0);
  load_x(0);
  for (int ch = 0; ch < nchunk; ++ch) {
    __syncthreads();                                   // the previous chunk has been read by every warp
#pragma unroll
    for (int i = 0; i < WPT; ++i) {
      const int j = threadIdx.x + i * (kRWarps * 32), e = j >> 6, q = j & 63;
      wsm[(e * 2 + (q & 1)) * 32 + (q >> 1)] = wn[i];
    }
    __syncthreads();
    float xv[TOK][8];
#pragma unroll
    for (int a = 0; a < TOK; ++a) cvt_raw8(xr[a], xv[a]);
    if (ch + 1 < nchunk) { load_w(ch + 1); load_x(ch + 1); }
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      if (e < N) {
        const float4 w0 = wsm[(e * 2) * 32 + lane], w1 = wsm[(e * 2 + 1) * 32 + lane];
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int a = 0; a < TOK; ++a)
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[a][e] = fmaf(xv[a][i], w[i], acc[a][e]);
      }
    }
  }
#pragma unroll
  for (int a = 0; a < TOK; ++a)
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      float v = acc[a][e];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      acc[a][e] = v;
    }

  // every lane now holds all logits; lane a finishes token t0 + a
#pragma unroll
  for (int a = 0; a < TOK; ++a) {
    const int t = t0 + a;
    if (lane != a) continue;
    const int bt = warp * TOK + a;
    if (t >= tokens) {
      ssel[bt] = 0u;
#pragma unroll
      for (int e = 0; e < NE; ++e) sp[bt][e] = 0.f;
      continue;
    }
    float l[NE];
    float mx = -INFINITY;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      l[e] = (e < N) ? acc[a][e] + (bias ? bias[e] : 0.f) : -INFINITY;
      mx = fmaxf(mx, l[e]);
    }
    float p[NE];
    float sum = 0.f;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      p[e] = (e < N) ? expf(l[e] - mx) : 0.f;
      sum += p[e];
    }
    const float inv_sum = 1.f / sum;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      p[e] *= inv_sum;
      sp[bt][e] = p[e];
      if (e < N) probs[(size_t)t * N + e] = p[e];
    }
    // top-k on the logits, ties to the lower index.  Each round starts from the lowest expert not taken yet, so
    // the k choices are distinct whatever the logits are (NaN or -inf rows included: those show up in the
    // values, never as a repeated index)
    const unsigned all = (N >= 32) ? 0xffffffffu : ((1u << N) - 1u);
    unsigned taken = 0;
    float qsum = 0.f, first = 0.f, second = 0.f, last = 0.f;
    int sel[MIXLORA_MAX_TOP_K];
    float selp[MIXLORA_MAX_TOP_K];
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
      if (j < k) {
        int bi = __ffs(~taken & all) - 1;
        float best = -INFINITY, bp = 0.f;
#pragma unroll
        for (int e = 0; e < NE; ++e)
          if (e == bi) { best = l[e]; bp = p[e]; }
#pragma unroll
        for (int e = 0; e < NE; ++e) {
          const bool free_e = !((taken >> e) & 1u) && e < N;
          if (free_e && l[e] > best) { best = l[e]; bi = e; bp = p[e]; }
        }
        taken |= 1u << bi;
        sel[j] = bi;
        selp[j] = bp;
        qsum += bp;
        if (j == 0) first = best;
        if (j == 1) second = best;
        last = best;
      }
    }
    float next = -INFINITY;  // largest logit left out
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      const bool free_e = !((taken >> e) & 1u) && e < N;
      if (free_e && l[e] > next) next = l[e];
    }
    float margin = INFINITY;
    if (k < N) margin = fminf(margin, last - next);
    if (N > 1) margin = fminf(margin, first - ((k >= 2) ? second : next));
    low_margin[t] = (margin < kMarginFlag) ? 1 : 0;
    ssel[bt] = f_mode == 0 ? (1u << sel[0]) : taken;
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
      if (j < k) {
        expert_idx[(size_t)t * k + j] = sel[j];
        gates[(size_t)t * k + j] = renorm ? selp[j] / qsum : selp[j];  // k = 1 gives exactly 1
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < N) {                                // the block's sums for Eq. 9, tokens in order
    const int e = threadIdx.x;
    float ps = 0.f, cnt = 0.f;
    for (int i = 0; i < BT; ++i) {
      ps += sp[i][e];
      cnt += (float)((ssel[i] >> e) & 1u);
    }
    part[(size_t)blockIdx.x * 2 * N + e] = ps;
    part[(size_t)blockIdx.x * 2 * N + N + e] = cnt;
  }
}

// F_i and P_i of Eq. 9 from the blocks' partial sums: warp e adds expert e's entries in a fixed order.  Also keeps
// the un-normalised sums (for callers that add them over data-parallel shards first).
__global__ void __launch_bounds__(1024)
router_stats_kernel(const float* __restrict__ part, int nblocks, float* __restrict__ F, float* __restrict__ P,
                    float* __restrict__ raw /* [2N]: probability sums, then counts */, int tokens, int N, int k,
                    int f_mode) {
  const int e = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (e >= N) return;
  float ps = 0.f, cnt = 0.f;
  for (int b = lane; b < nblocks; b += 32) {
    ps += part[(size_t)b * 2 * N + e];
    cnt += part[(size_t)b * 2 * N + N + e];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ps += __shfl_xor_sync(0xffffffffu, ps, o);
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  }
  if (lane == 0) {
    const float denom = (f_mode == 0) ? (float)tokens : (float)tokens * (float)k;
    F[e] = tokens > 0 ? cnt / denom : 0.f;
    P[e] = tokens > 0 ? ps / (float)tokens : 0.f;
    raw[e] = ps;
    raw[N + e] = cnt;
  }
}

__global__ void aux_loss_kernel(const float* __restrict__ Fs, const float* __restrict__ Ps, float coef, int N,
                                float* loss, float* F, float* P) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float acc = 0.f;
    for (int e = 0; e < N; ++e) {
      acc += Fs[e] * Ps[e];
      if (F) F[e] = Fs[e];
      if (P) P[e] = Ps[e];
    }
    *loss = coef * (float)N * acc;
  }
}

// Eq. 8-9 over a batch that is spread over several shards: `psum`, `count` are the shards' sums added up,
// `total_tokens` the size of the whole batch.  Leaves F, P of the whole batch and its token count in the workspace,
// where the backward pass picks them up for the gradient of the auxiliary loss.
__global__ void aux_loss_global_kernel(const float* __restrict__ psum, const float* __restrict__ count,
                                       long long total_tokens, int N, int k, int f_mode, float coef, float* ws_F,
                                       float* ws_P, long long* ws_tokens, float* loss, float* F, float* P) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    const float tt = (float)total_tokens;
    const float denom = f_mode == 0 ? tt : tt * (float)k;
    float acc = 0.f;
    for (int e = 0; e < N; ++e) {
      const float fe = count[e] / denom, pe = psum[e] / tt;
      acc += fe * pe;
      ws_F[e] = fe;
      ws_P[e] = pe;
      if (F) F[e] = fe;
      if (P) P[e] = pe;
    }
    *ws_tokens = total_tokens;
    *loss = coef * (float)N * acc;
  }
}

// ---- dispatch ---------------------------------------------------------------------------
// Step 1: slots per expert inside each block of kRouteBlockTokens tokens.
__global__ void __launch_bounds__(kRouteBlockTokens)
dispatch_count_kernel(const int* __restrict__ expert_idx, int* __restrict__ blk_counts, int tokens, int N, int k) {
  __shared__ int cnt[MIXLORA_MAX_EXPERTS];
  if (threadIdx.x < MIXLORA_MAX_EXPERTS) cnt[threadIdx.x] = 0;
  __syncthreads();
  const int t = blockIdx.x * kRouteBlockTokens + threadIdx.x;
  if (t < tokens)
    for (int j = 0; j < k; ++j) atomicAdd(&cnt[expert_idx[(size_t)t * k + j]], 1);   // the router's indices: valid, distinct
  __syncthreads();
  if (threadIdx.x < N) blk_counts[blockIdx.x * N + threadIdx.x] = cnt[threadIdx.x];
}

// Step 2: exclusive scan of the (expert-major, block-minor) count table; segment offsets;
// table of kSegTile-row tiles that never straddle a segment.
__global__ void __launch_bounds__(1024)
dispatch_scan_kernel(const int* __restrict__ blk_counts, int* __restrict__ blk_off, int* __restrict__ seg_off,
                     int* __restrict__ tile_info, int max_tiles, int nblk, int N) {
  __shared__ int part[1024];
  const int n = nblk * N;
  const int per = (n + 1023) / 1024;
  const int q0 = threadIdx.x * per;
  int s = 0;
  for (int q = q0; q < q0 + per && q < n; ++q) s += blk_counts[(q % nblk) * N + (q / nblk)];
  part[threadIdx.x] = s;
  __syncthreads();
  // inclusive scan of the 1024 partial sums
  for (int o = 1; o < 1024; o <<= 1) {
    int v = (threadIdx.x >= o) ? part[threadIdx.x - o] : 0;
    __syncthreads();
    part[threadIdx.x] += v;
    __syncthreads();
  }
  int run = (threadIdx.x == 0) ? 0 : part[threadIdx.x - 1];
  for (int q = q0; q < q0 + per && q < n; ++q) {
    const int e = q / nblk, b = q % nblk;
    blk_off[b * N + e] = run;
    if (b == 0) seg_off[e] = run;
    run += blk_counts[b * N + e];
  }
  if (threadIdx.x == 1023) seg_off[N] = part[1023];
  __syncthreads();
  if (threadIdx.x == 0) {
    int nt = 0;
    for (int e = 0; e < N; ++e) {
      int b = seg_off[e], en = seg_off[e + 1];
      for (int p = b; p < en && nt < max_tiles; p += kSegTile) {
        tile_info[nt * 4 + 0] = e;
        tile_info[nt * 4 + 1] = p;
        tile_info[nt * 4 + 2] = min(kSegTile, en - p);
        tile_info[nt * 4 + 3] = 0;
        ++nt;
      }
    }
    tile_info[max_tiles * 4] = nt;
  }
}

// Step 3: rank of each slot inside its (block, expert) bucket by warp ballots, then scatter.
__global__ void __launch_bounds__(kRouteBlockTokens)
dispatch_scatter_kernel(const int* __restrict__ expert_idx, const int* __restrict__ blk_off, int* __restrict__ perm,
                        int* __restrict__ inv, int* __restrict__ pos_token, int* __restrict__ pos_expert, int tokens,
                        int N, int k) {
  constexpr int W = kRouteBlockTokens / 32;
  __shared__ int wcnt[W][MIXLORA_MAX_EXPERTS];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int t = blockIdx.x * kRouteBlockTokens + threadIdx.x;
  int mine[MIXLORA_MAX_TOP_K];
  int rank[MIXLORA_MAX_TOP_K];
#pragma unroll
  for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
    mine[j] = (t < tokens && j < k) ? expert_idx[(size_t)t * k + j] : -1;
    rank[j] = 0;
  }
  for (int e = 0; e < N; ++e) {
    bool has = false;
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) has |= (mine[j] == e);
    unsigned b = __ballot_sync(0xffffffffu, has);
    int r = __popc(b & ((1u << lane) - 1u));
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j)
      if (mine[j] == e) rank[j] = r;
    if (lane == 0) wcnt[w][e] = __popc(b);
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
    if (mine[j] < 0) continue;
    const int e = mine[j];
    int before = 0;
    for (int ww = 0; ww < w; ++ww) before += wcnt[ww][e];
    const int pos = blk_off[blockIdx.x * N + e] + before + rank[j];
    const int slot = t * k + j;
    perm[pos] = slot;
    inv[slot] = pos;
    pos_token[pos] = t;
    pos_expert[pos] = e;
  }
}

// ---- work lists for the block-sparse dense products ------------------------------------------
__global__ void rows_worklist_kernel(const int* __restrict__ seg_off, int N, int slots, int tile_rows, int r, int nout,
                                     int kblocks, int max_items, int* __restrict__ items, int* __restrict__ count) {
  const int m_tiles = (slots + tile_rows - 1) / tile_rows;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= m_tiles * N) return;
  const int mt = idx / N, e = idx % N;
  const int lo = mt * tile_rows, hi = min(lo + tile_rows, slots);
  const int sb = seg_off[e], se = seg_off[e + 1];
  if (se <= sb || se <= lo || sb >= hi) return;            // expert e has no slot in this tile
  const int at = atomicAdd(count, nout);                   // the order of items does not affect any result
  if (at + nout > max_items) return;
  for (int o = 0; o < nout; ++o) {
    int* it = items + (size_t)(at + o) * 8;
    it[0] = o; it[1] = lo; it[2] = e * r; it[3] = 0; it[4] = kblocks; it[5] = e * r; it[6] = e * r + r; it[7] = 0;
  }
}

__global__ void reduce_worklist_kernel(const int* __restrict__ seg_off, int N, int out_rows, int tile_rows, int r,
                                       int nout, int* __restrict__ items, int* __restrict__ count) {
  const int m_tiles = (out_rows + tile_rows - 1) / tile_rows;
  const int total = nout * N * m_tiles;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx == 0) *count = total;
  if (idx >= total) return;
  // tile index fastest, then expert, then output: neighbouring CTAs work on the same expert's operand rows
  const int mt = idx % m_tiles, e = (idx / m_tiles) % N, o = idx / (m_tiles * N);
  const int sb = seg_off[e], se = seg_off[e + 1];
  int* it = items + (size_t)idx * 8;
  it[0] = o; it[1] = mt * tile_rows; it[2] = e * r;
  it[3] = sb / 64; it[4] = se > sb ? (se + 63) / 64 : sb / 64;   // k-blocks that touch the segment (none if empty)
  it[5] = e * r; it[6] = e * r + r; it[7] = 0;
}

template <typename T>
cudaError_t launch_router_t(const Ctx& c) {
  const mixlora_shape_t& s = c.s;
  const T* x = reinterpret_cast<const T*>(c.p.x);
  float* probs = c.at<float>(c.L.probs);
  int* idx = c.at<int>(c.L.expert_idx);
  float* gates = c.at<float>(c.L.gates);
  uint8_t* flags = c.at<uint8_t>(c.L.low_margin);
  int blocks = 0;
#define MIXLORA_ROUTER_LAUNCH(NE, TOK)                                                                         \
  {                                                                                                            \
    blocks = (s.tokens + kRWarps * TOK - 1) / (kRWarps * TOK);                                                 \
    router_kernel<T, NE, TOK><<<blocks, kRWarps * 32, 0, c.st>>>(                                              \
        x, c.p.w_router, c.p.router_bias, probs, idx, gates, flags, c.at<float>(c.L.stat_part), s.tokens,      \
        s.d_model, s.n_experts, s.top_k, s.renormalize, s.aux_f_mode);                                         \
  }
  if (s.n_experts <= 8) MIXLORA_ROUTER_LAUNCH(8, 4)
  else if (s.n_experts <= 16) MIXLORA_ROUTER_LAUNCH(16, 4)
  else MIXLORA_ROUTER_LAUNCH(32, 2)
#undef MIXLORA_ROUTER_LAUNCH
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  router_stats_kernel<<<1, 1024, 0, c.st>>>(c.at<float>(c.L.stat_part), blocks, c.at<float>(c.L.stat_F),
                                            c.at<float>(c.L.stat_P), c.at<float>(c.L.stat_raw), s.tokens, s.n_experts,
                                            s.top_k, s.aux_f_mode);
  return cudaGetLastError();
}

}  // namespace

int router_part_blocks(int tokens) { return (tokens + kRWarps * 2 - 1) / (kRWarps * 2); }   // the smallest block

cudaError_t launch_router(const Ctx& c) { return c.bf16 ? launch_router_t<bf16>(c) : launch_router_t<float>(c); }

cudaError_t launch_dispatch(const Ctx& c) {
  const mixlora_shape_t& s = c.s;
  const int nblk = route_blocks(s.tokens);
  int* idx = c.at<int>(c.L.expert_idx);
  dispatch_count_kernel<<<nblk, kRouteBlockTokens, 0, c.st>>>(idx, c.at<int>(c.L.blk_counts), s.tokens, s.n_experts,
                                                              s.top_k);
  dispatch_scan_kernel<<<1, 1024, 0, c.st>>>(c.at<int>(c.L.blk_counts), c.at<int>(c.L.blk_off), c.at<int>(c.L.seg_off),
                                             c.at<int>(c.L.tile_info), max_seg_tiles(s.tokens, s.top_k, s.n_experts),
                                             nblk, s.n_experts);
  dispatch_scatter_kernel<<<nblk, kRouteBlockTokens, 0, c.st>>>(idx, c.at<int>(c.L.blk_off), c.at<int>(c.L.perm),
                                                                c.at<int>(c.L.inv), c.at<int>(c.L.pos_token),
                                                                c.at<int>(c.L.pos_expert), s.tokens, s.n_experts,
                                                                s.top_k);
  return cudaGetLastError();
}

cudaError_t launch_rows_worklist(const Ctx& c, int tile_rows, int nout, int kblocks, int* items, int* count) {
  const int slots = c.s.tokens * c.s.top_k, N = c.s.n_experts;
  const int m_tiles = (slots + tile_rows - 1) / tile_rows;
  cudaError_t e = cudaMemsetAsync(count, 0, sizeof(int), c.st);
  if (e != cudaSuccess) return e;
  const int n = m_tiles * N;
  rows_worklist_kernel<<<(n + 255) / 256, 256, 0, c.st>>>(c.at<int>(c.L.seg_off), N, slots, tile_rows, c.s.rank, nout,
                                                         kblocks, rows_worklist_max(slots, N, nout), items, count);
  return cudaGetLastError();
}

cudaError_t launch_reduce_worklist(const Ctx& c, int out_rows, int tile_rows, int nout, int* items, int* count) {
  const int N = c.s.n_experts;
  const int n = nout * N * ((out_rows + tile_rows - 1) / tile_rows);
  reduce_worklist_kernel<<<(n + 255) / 256, 256, 0, c.st>>>(c.at<int>(c.L.seg_off), N, out_rows, tile_rows, c.s.rank,
                                                           nout, items, count);
  return cudaGetLastError();
}

cudaError_t launch_aux_loss(const Ctx& c, float coef, float* loss, float* F, float* P) {
  aux_loss_kernel<<<1, 32, 0, c.st>>>(c.at<float>(c.L.stat_F), c.at<float>(c.L.stat_P), coef, c.s.n_experts, loss, F,
                                      P);
  return cudaGetLastError();
}

cudaError_t launch_aux_loss_global(const Ctx& c, float coef, const float* prob_sum, const float* count,
                                   long long total_tokens, float* loss, float* F, float* P) {
  aux_loss_global_kernel<<<1, 32, 0, c.st>>>(prob_sum, count, total_tokens, c.s.n_experts, c.s.top_k, c.s.aux_f_mode,
                                             coef, c.at<float>(c.L.stat_F), c.at<float>(c.L.stat_P),
                                             reinterpret_cast<long long*>(c.ws + c.L.status + 8), loss, F, P);
  return cudaGetLastError();
}

}  // namespace mixlora
