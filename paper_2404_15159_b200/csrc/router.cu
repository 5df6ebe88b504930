// Router (Eq. 7), load-balance statistics (Eq. 8-9) and the dispatch of slots to experts:
// histogram, prefix scan and stable permutation in the order "expert ascending, token ascending".
#include "common.cuh"

namespace mixlora {

namespace {

constexpr int kWarpsPerBlock = 4;
constexpr float kMarginFlag = 1e-4f;

// VEC consecutive features of one row as floats (16-byte load)
template <int VEC> struct FeatVec { float v[VEC]; };
__device__ __forceinline__ FeatVec<4> ld_feat(const float* p) {
  const float4 r = *reinterpret_cast<const float4*>(p);
  FeatVec<4> o; o.v[0] = r.x; o.v[1] = r.y; o.v[2] = r.z; o.v[3] = r.w;
  return o;
}
__device__ __forceinline__ FeatVec<8> ld_feat(const bf16* p) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
  FeatVec<8> o;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(h[i]);
    o.v[2 * i] = f.x; o.v[2 * i + 1] = f.y;
  }
  return o;
}
template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int value = 4; };
template <> struct VecOf<bf16> { static constexpr int value = 8; };

// One warp handles TOK tokens at a time and NE (>= N) logits per token, TOK * NE = 32
// accumulators per lane.  Each lane covers VEC consecutive features (one 16-byte load of x)
// per step of 32 * VEC features.
template <typename T, int NE, int TOK>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
router_kernel(const T* __restrict__ x, const float* __restrict__ w_router, const float* __restrict__ bias,
              float* __restrict__ probs, int* __restrict__ expert_idx, float* __restrict__ gates,
              uint8_t* __restrict__ low_margin, int tokens, int d, int N, int k, int renorm) {
  constexpr int VEC = VecOf<T>::value;
  const int lane = threadIdx.x & 31;
  const int warp = (blockIdx.x * kWarpsPerBlock) + (threadIdx.x >> 5);
  const int t0 = warp * TOK;
  if (t0 >= tokens) return;

  float acc[TOK][NE];
#pragma unroll
  for (int a = 0; a < TOK; ++a)
#pragma unroll
    for (int e = 0; e < NE; ++e) acc[a][e] = 0.f;

  for (int c = lane * VEC; c < d; c += 32 * VEC) {
    FeatVec<VEC> xv[TOK];
#pragma unroll
    for (int a = 0; a < TOK; ++a) {
      const int t = min(t0 + a, tokens - 1);       // rows past the end repeat the last token; never written
      xv[a] = ld_feat(x + (size_t)t * d + c);
    }
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      if (e < N) {
        float w[VEC];
#pragma unroll
        for (int i = 0; i < VEC; i += 4) {
          const float4 r = __ldg(reinterpret_cast<const float4*>(w_router + (size_t)e * d + c + i));
          w[i] = r.x; w[i + 1] = r.y; w[i + 2] = r.z; w[i + 3] = r.w;
        }
#pragma unroll
        for (int a = 0; a < TOK; ++a)
#pragma unroll
          for (int i = 0; i < VEC; ++i) acc[a][e] = fmaf(xv[a].v[i], w[i], acc[a][e]);
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
    if (t >= tokens || lane != a) continue;
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
      if (e < N) probs[(size_t)t * N + e] = p[e];
    }
    // top-k on the logits, ties to the lower index
    unsigned taken = 0;
    float qsum = 0.f, first = 0.f, second = 0.f, last = 0.f;
    int sel[MIXLORA_MAX_TOP_K];
    float selp[MIXLORA_MAX_TOP_K];
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
      if (j < k) {
        float best = -INFINITY;
        int bi = 0;
        float bp = 0.f;
#pragma unroll
        for (int e = 0; e < NE; ++e) {
          bool free_e = !((taken >> e) & 1u) && e < N;
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
      bool free_e = !((taken >> e) & 1u) && e < N;
      if (free_e && l[e] > next) next = l[e];
    }
    float margin = INFINITY;
    if (k < N) margin = fminf(margin, last - next);
    if (N > 1) margin = fminf(margin, first - ((k >= 2) ? second : next));
    low_margin[t] = (margin < kMarginFlag) ? 1 : 0;
    
#pragma unroll
    for (int j = 0; j < MIXLORA_MAX_TOP_K; ++j) {
      if (j < k) {
        expert_idx[(size_t)t * k + j] = sel[j];
        gates[(size_t)t * k + j] = renorm ? selp[j] / qsum : selp[j];  // k = 1 gives exactly 1
      }
    }
  }
}

// F_i and P_i of Eq. 9, one block per expert, fixed summation order (deterministic).
__global__ void __launch_bounds__(1024)
router_stats_kernel(const float* __restrict__ probs, const int* __restrict__ expert_idx, float* __restrict__ F,
                    float* __restrict__ P, int tokens, int N, int k, int f_mode) {
  __shared__ float sp[1024];
  __shared__ int sc[1024];
  const int e = blockIdx.x;
  float ps = 0.f;
  int cnt = 0;
  for (int t = threadIdx.x; t < tokens; t += 1024) {
    ps += probs[(size_t)t * N + e];
    if (f_mode == 0) {
      cnt += (expert_idx[(size_t)t * k] == e);
    } else {
      for (int j = 0; j < k; ++j) cnt += (expert_idx[(size_t)t * k + j] == e);
    }
  }
  sp[threadIdx.x] = ps;
  sc[threadIdx.x] = cnt;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sp[threadIdx.x] += sp[threadIdx.x + o];
      sc[threadIdx.x] += sc[threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float denom = (f_mode == 0) ? (float)tokens : (float)tokens * (float)k;
    F[e] = tokens > 0 ? (float)sc[0] / denom : 0.f;
    P[e] = tokens > 0 ? sp[0] / (float)tokens : 0.f;
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

// ---- dispatch ---------------------------------------------------------------------------
// Step 1: slots per expert inside each block of kRouteBlockTokens tokens.
__global__ void __launch_bounds__(kRouteBlockTokens)
dispatch_count_kernel(const int* __restrict__ expert_idx, int* __restrict__ blk_counts, int tokens, int N, int k) {
  __shared__ int cnt[MIXLORA_MAX_EXPERTS];
  if (threadIdx.x < MIXLORA_MAX_EXPERTS) cnt[threadIdx.x] = 0;
  __syncthreads();
  const int t = blockIdx.x * kRouteBlockTokens + threadIdx.x;
  if (t < tokens)
    for (int j = 0; j < k; ++j) atomicAdd(&cnt[expert_idx[(size_t)t * k + j]], 1);
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
#define MIXLORA_ROUTER_LAUNCH(NE, TOK)                                                                         \
  {                                                                                                            \
    int warps = (s.tokens + TOK - 1) / TOK;                                                                    \
    int blocks = (warps + kWarpsPerBlock - 1) / kWarpsPerBlock;                                                \
    router_kernel<T, NE, TOK><<<blocks, kWarpsPerBlock * 32, 0, c.st>>>(                                       \
        x, c.p.w_router, c.p.router_bias, probs, idx, gates, flags, s.tokens, s.d_model, s.n_experts, s.top_k, \
        s.renormalize);                                                                                        \
  }
  if (s.n_experts <= 8) MIXLORA_ROUTER_LAUNCH(8, 2)
  else if (s.n_experts <= 16) MIXLORA_ROUTER_LAUNCH(16, 2)
  else MIXLORA_ROUTER_LAUNCH(32, 1)
#undef MIXLORA_ROUTER_LAUNCH
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_router(const Ctx& c) {
  cudaError_t e = c.bf16 ? launch_router_t<bf16>(c) : launch_router_t<float>(c);
  if (e != cudaSuccess) return e;
  router_stats_kernel<<<c.s.n_experts, 1024, 0, c.st>>>(c.at<float>(c.L.probs), c.at<int>(c.L.expert_idx),
                                                       c.at<float>(c.L.stat_F), c.at<float>(c.L.stat_P), c.s.tokens,
                                                       c.s.n_experts, c.s.top_k, c.s.aux_f_mode);
  return cudaGetLastError();
}

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

}  // namespace mixlora
