// MixDoRA: the memory-bound kernels that the weight-decomposed variant of the block adds to the MixLoRA path
// (Section 4.1 / Table 1 name the variant).  Each expert projection is diag(m / n) (W + s B A) with n the row norm
// of the merged weight, so the per-expert scale c = m / n multiplies output rows: the shared W1 x, W3 x and the
// dense products stay as they are, and these kernels apply c, build it, and collect the magnitude gradients.
// Work over the sorted slots is cut by the dispatch step's table of single-expert tiles of up to 128 rows.
// In bf16 the scaled SwiGLU itself (forward and backward) runs on the grouped tensor-core kernel
// (grouped_swiglu.cu); the SwiGLU kernels here serve fp32.
#include "common.cuh"

namespace mixlora {

namespace {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16(v); }
__device__ __forceinline__ float sigmoidf_(float v) { return 1.f / (1.f + expf(-v)); }

constexpr int kCols = 256;   // columns (threads) per block of the tile kernels

// 8 consecutive values of a row as floats (16-byte loads; the row start is 16-byte aligned when r % 8 == 0)
__device__ __forceinline__ void load8(const bf16* p, float (&o)[8]) {
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8(const float* p, float (&o)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}

// rowsq[o] = sum_c W[o, c]^2, one warp per row
template <typename T>
__global__ void rowsq_kernel(const T* __restrict__ w, float* __restrict__ rowsq, int rows, int cols) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float s = 0.f;
  for (int c = lane; c < cols; c += 32) {
    const float v = to_f(w[(size_t)row * cols + c]);
    s = fmaf(v, v, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) rowsq[row] = s;
}

// n^2 = |W_o|^2 + 2 s B_o . (W A^T)_o + s^2 B_o (A A^T) B_o^T for expert e and output row o;
// inv_n = 1 / n, c = m / n.  wa is [rows, N r] (W times every expert's A^T), aat is [N r, N r] (A_cat A_cat^T, of
// which the diagonal r x r blocks are used), b is [N, rows, r].
template <typename T>
__global__ void dora_scale_kernel(const float* __restrict__ rowsq, const float* __restrict__ wa,
                                  const float* __restrict__ aat, const T* __restrict__ b, const float* __restrict__ m,
                                  float* __restrict__ c_out, float* __restrict__ inv_n, int rows, int N, int r, float s) {
  const long long n = (long long)N * rows;
  const int nr = N * r;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int e = (int)(i / rows), o = (int)(i % rows);
    const T* bo = b + ((size_t)e * rows + o) * r;
    float cross = 0.f, quad = 0.f;
    for (int p = 0; p < r; ++p) {
      const float bp = to_f(bo[p]);
      cross = fmaf(bp, wa[(size_t)o * nr + e * r + p], cross);
      float inner = 0.f;
      for (int q = 0; q < r; ++q) inner = fmaf(aat[(size_t)(e * r + p) * nr + e * r + q], to_f(bo[q]), inner);
      quad = fmaf(bp, inner, quad);
    }
    const float n2 = rowsq[o] + 2.f * s * cross + s * s * quad;
    const float inv = rsqrtf(fmaxf(n2, 1e-30f));
    inv_n[i] = inv;
    c_out[i] = m[i] * inv;
  }
}

// Forward, per single-expert tile and chunk of 256 columns (a thread per column, 8 rows at a time in registers so
// that a column's rows of B_g[e], B_u[e] are read once per 8 slots): a = c_g[e] (G_t + s B_g[e] zg),
// b = c_u[e] (U_t + s B_u[e] zu), h = SiLU(a) b.
template <typename T>
__global__ void __launch_bounds__(kCols)
dora_swiglu_fwd_kernel(const T* __restrict__ G, const T* __restrict__ U, const T* __restrict__ zga,
                       const T* __restrict__ zua, const T* __restrict__ b_gate, const T* __restrict__ b_up,
                       const float* __restrict__ cg, const float* __restrict__ cu, const int* __restrict__ pos_token,
                       const int* __restrict__ tile_info, int max_tiles, T* __restrict__ h_sorted, int f, int N, int r,
                       float s) {
  constexpr int RB = 8;
  extern __shared__ float sm[];
  float* zg = sm;                                // [RB][r], already scaled by s
  float* zu = zg + RB * r;
  __shared__ int tok[kSegTile];
  const int tile = blockIdx.x;
  const int c = blockIdx.y * kCols + threadIdx.x;
  if (tile >= min(tile_info[max_tiles * 4], max_tiles)) return;
  const int e = tile_info[tile * 4 + 0], p0 = tile_info[tile * 4 + 1], rows = tile_info[tile * 4 + 2];
  for (int i = threadIdx.x; i < rows; i += kCols) tok[i] = pos_token[p0 + i];
  const bool live = c < f;
  const int cc = live ? c : f - 1;               // threads past the width read valid data and store nothing
  const T* bg = b_gate + ((size_t)e * f + cc) * r;
  const T* bu = b_up + ((size_t)e * f + cc) * r;
  const float cgv = cg[(size_t)e * f + cc], cuv = cu[(size_t)e * f + cc];
  for (int i0 = 0; i0 < rows; i0 += RB) {
    __syncthreads();                             // tok is set; the previous rows' vectors are no longer read
    for (int i = threadIdx.x; i < RB * r; i += kCols) {
      const int sl = i / r, rr = i % r;
      float vg = 0.f, vu = 0.f;
      if (i0 + sl < rows) {
        const size_t o = ((size_t)tok[i0 + sl] * N + e) * r + rr;
        vg = s * to_f(zga[o]);
        vu = s * to_f(zua[o]);
      }
      zg[rr * RB + sl] = vg; zu[rr * RB + sl] = vu;      // [rr][row]: a step of the rank reads 8 rows as two float4
    }
    __syncthreads();
    float ea[RB], eb[RB];
#pragma unroll
    for (int i = 0; i < RB; ++i) { ea[i] = 0.f; eb[i] = 0.f; }
    auto rank_step = [&](int rr, float wg, float wu) {
      const float4 g0 = *reinterpret_cast<const float4*>(zg + rr * RB), g1 = *reinterpret_cast<const float4*>(zg + rr * RB + 4);
      const float4 u0 = *reinterpret_cast<const float4*>(zu + rr * RB), u1 = *reinterpret_cast<const float4*>(zu + rr * RB + 4);
      const float zgv[RB] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      const float zuv[RB] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
      for (int i = 0; i < RB; ++i) {
        ea[i] = fmaf(zgv[i], wg, ea[i]);
        eb[i] = fmaf(zuv[i], wu, eb[i]);
      }
    };
    if (r % 8 == 0) {
      for (int r0 = 0; r0 < r; r0 += 8) {
        float wg[8], wu[8];
        load8(bg + r0, wg);
        load8(bu + r0, wu);
#pragma unroll
        for (int q = 0; q < 8; ++q) rank_step(r0 + q, wg[q], wu[q]);
      }
    } else {
      for (int rr = 0; rr < r; ++rr) rank_step(rr, to_f(bg[rr]), to_f(bu[rr]));
    }
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      if (i0 + i < rows && live) {
        const size_t go = (size_t)tok[i0 + i] * f + c;
        const float a = cgv * (to_f(G[go]) + ea[i]);
        const float b = cuv * (to_f(U[go]) + eb[i]);
        h_sorted[(size_t)(p0 + i0 + i) * f + c] = from_f<T>(a * sigmoidf_(a) * b);
      }
    }
  }
}

// own[pos][q] = in[pos][q] inside the slot's expert block of r columns, zero elsewhere; gown = gate * own (optional)
template <typename T>
__global__ void dora_own_block_kernel(const T* __restrict__ in, const float* __restrict__ gates,
                                      const int* __restrict__ perm, const int* __restrict__ pos_expert,
                                      T* __restrict__ own, T* __restrict__ gown, int slots, int N, int r) {
  const long long nr = (long long)N * r, n = (long long)slots * nr;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / nr), q = (int)(i % nr);
    const bool mine = (q / r) == pos_expert[pos];
    const float v = mine ? to_f(in[i]) : 0.f;
    if (own) own[i] = from_f<T>(v);
    if (gown) gown[i] = from_f<T>(mine ? gates[perm[pos]] * v : 0.f);
  }
}

// y_t = sum_j g_tj c_d[e_tj] * o_pre[position of slot (t, j)]   (Eq. 6 with the scaled down projection)
template <typename T>
__global__ void __launch_bounds__(kCols)
dora_combine_y_kernel(const T* __restrict__ o_pre, const float* __restrict__ cd, const float* __restrict__ gates,
                      const int* __restrict__ inv, const int* __restrict__ expert_idx, T* __restrict__ y, int d, int k) {
  const int t = blockIdx.x;
  __shared__ int pos[MIXLORA_MAX_TOP_K], ex[MIXLORA_MAX_TOP_K];
  __shared__ float g[MIXLORA_MAX_TOP_K];
  if (threadIdx.x < k) {
    pos[threadIdx.x] = inv[(size_t)t * k + threadIdx.x];
    ex[threadIdx.x] = expert_idx[(size_t)t * k + threadIdx.x];
    g[threadIdx.x] = gates[(size_t)t * k + threadIdx.x];
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += kCols) {
    float acc = 0.f;
    for (int j = 0; j < k; ++j)
      acc = fmaf(g[j] * cd[(size_t)ex[j] * d + c], to_f(o_pre[(size_t)pos[j] * d + c]), acc);
    y[(size_t)t * d + c] = from_f<T>(acc);
  }
}

// Backward, first step, per single-expert tile (a thread per column o): dO[pos] = c_d[e] * dy_t (no gate) and the
// tile's share of the magnitude gradient, sum over its rows of g * dy_t[o] * o_pre[pos][o].
template <typename T>
__global__ void __launch_bounds__(kCols)
dora_dout_kernel(const T* __restrict__ dy, const T* __restrict__ o_pre, const float* __restrict__ cd,
                 const float* __restrict__ gates, const int* __restrict__ perm, const int* __restrict__ pos_token,
                 const int* __restrict__ tile_info, int max_tiles, T* __restrict__ dO, float* __restrict__ dm_part,
                 int d) {
  const int tile = blockIdx.x;
  const int c = blockIdx.y * kCols + threadIdx.x;
  if (tile >= min(tile_info[max_tiles * 4], max_tiles)) return;
  const int e = tile_info[tile * 4 + 0], p0 = tile_info[tile * 4 + 1], rows = tile_info[tile * 4 + 2];
  __shared__ int tok[kSegTile];
  __shared__ float gt[kSegTile];
  for (int i = threadIdx.x; i < rows; i += kCols) {
    tok[i] = pos_token[p0 + i];
    gt[i] = gates[perm[p0 + i]];
  }
  __syncthreads();
  if (c >= d) return;
  const float cv = cd[(size_t)e * d + c];
  float acc = 0.f;
  for (int i = 0; i < rows; ++i) {
    const float dyv = to_f(dy[(size_t)tok[i] * d + c]);
    dO[(size_t)(p0 + i) * d + c] = from_f<T>(cv * dyv);
    acc = fmaf(gt[i] * dyv, to_f(o_pre[(size_t)(p0 + i) * d + c]), acc);
  }
  dm_part[(size_t)tile * d + c] = acc;
}

// Backward of the scaled SwiGLU, per single-expert tile and chunk of 256 columns (a thread per column).  Re-computes
// a_pre = G_t + s B_g[e] zg, b_pre likewise, a = c_g a_pre, b = c_u b_pre, h; Dt = D[pos] + A_d[e]^T (s pd) is the
// gradient of the slot's h before the gate; dgate partial = <Dt, h> over the chunk; dh = g Dt;
// da = dh b SiLU'(a), db = dh SiLU(a) (with respect to the scaled a, b); stores c_g da and c_u db (the gradients of
// a_pre, b_pre, which everything downstream works on) and the tile's shares of the magnitude gradients,
// sum over rows of da * a_pre and db * b_pre.
template <typename T>
__global__ void __launch_bounds__(kCols)
dora_swiglu_bwd_kernel(const T* __restrict__ G, const T* __restrict__ U, const T* __restrict__ D,
                       const T* __restrict__ zga, const T* __restrict__ zua, const T* __restrict__ spd,
                       const T* __restrict__ b_gate, const T* __restrict__ b_up, const T* __restrict__ a_down,
                       const float* __restrict__ cg, const float* __restrict__ cu, const float* __restrict__ gates,
                       const int* __restrict__ perm, const int* __restrict__ pos_token,
                       const int* __restrict__ tile_info, int max_tiles, T* __restrict__ da_sorted,
                       T* __restrict__ db_sorted, float* __restrict__ dgate_part, float* __restrict__ dm_part_g,
                       float* __restrict__ dm_part_u, int slots, int f, int N, int r, float s) {
  constexpr int RB = 8;                          // rows whose rank-r vectors sit in shared memory at a time
  extern __shared__ float sm[];
  float* zg = sm;                                // [RB][r] scaled by s
  float* zu = zg + RB * r;
  float* pd = zu + RB * r;                       // [RB][r] = s pd
  __shared__ int tok[kSegTile];
  __shared__ float gt[kSegTile];
  __shared__ float red[RB][kCols / 32];
  const int tile = blockIdx.x;
  const int c = blockIdx.y * kCols + threadIdx.x;
  if (tile >= min(tile_info[max_tiles * 4], max_tiles)) return;
  const int e = tile_info[tile * 4 + 0], p0 = tile_info[tile * 4 + 1], rows = tile_info[tile * 4 + 2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < rows; i += kCols) {
    tok[i] = pos_token[p0 + i];
    gt[i] = gates[perm[p0 + i]];
  }
  const bool live = c < f;
  const int cc = live ? c : f - 1;               // threads past the width read valid data and store nothing
  const T* bg = b_gate + ((size_t)e * f + cc) * r;
  const T* bu = b_up + ((size_t)e * f + cc) * r;
  const T* ad = a_down + (size_t)e * r * f + cc;
  const float cgv = cg[(size_t)e * f + cc], cuv = cu[(size_t)e * f + cc];
  float mg = 0.f, mu = 0.f;
  for (int i0 = 0; i0 < rows; i0 += RB) {
    __syncthreads();                             // tok / gt are set; the previous rows' vectors are no longer read
    for (int i = threadIdx.x; i < RB * r; i += kCols) {
      const int sl = i / r, rr = i % r;
      float vg = 0.f, vu = 0.f, vp = 0.f;
      if (i0 + sl < rows) {
        const size_t o = ((size_t)tok[i0 + sl] * N + e) * r + rr;
        vg = s * to_f(zga[o]);
        vu = s * to_f(zua[o]);
        vp = to_f(spd[((size_t)(p0 + i0 + sl) * N + e) * r + rr]);
      }
      zg[rr * RB + sl] = vg; zu[rr * RB + sl] = vu; pd[rr * RB + sl] = vp;   // [rr][row]
    }
    __syncthreads();
    float ea[RB], eb[RB], ed[RB];
#pragma unroll
    for (int i = 0; i < RB; ++i) { ea[i] = 0.f; eb[i] = 0.f; ed[i] = 0.f; }
    auto rank_step = [&](int rr, float wg, float wu) {
      const float wd = to_f(ad[(size_t)rr * f]);
      const float4 g0 = *reinterpret_cast<const float4*>(zg + rr * RB), g1 = *reinterpret_cast<const float4*>(zg + rr * RB + 4);
      const float4 u0 = *reinterpret_cast<const float4*>(zu + rr * RB), u1 = *reinterpret_cast<const float4*>(zu + rr * RB + 4);
      const float4 d0 = *reinterpret_cast<const float4*>(pd + rr * RB), d1 = *reinterpret_cast<const float4*>(pd + rr * RB + 4);
      const float zgv[RB] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      const float zuv[RB] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
      const float pdv[RB] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
      for (int i = 0; i < RB; ++i) {
        ea[i] = fmaf(zgv[i], wg, ea[i]);
        eb[i] = fmaf(zuv[i], wu, eb[i]);
        ed[i] = fmaf(pdv[i], wd, ed[i]);
      }
    };
    if (r % 8 == 0) {
      for (int r0 = 0; r0 < r; r0 += 8) {
        float wg[8], wu[8];
        load8(bg + r0, wg);
        load8(bu + r0, wu);
#pragma unroll
        for (int q = 0; q < 8; ++q) rank_step(r0 + q, wg[q], wu[q]);
      }
    } else {
      for (int rr = 0; rr < r; ++rr) rank_step(rr, to_f(bg[rr]), to_f(bu[rr]));
    }
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      float dgv = 0.f;
      if (i0 + i < rows && live) {
        const size_t go = (size_t)tok[i0 + i] * f + c;
        const size_t so = (size_t)(p0 + i0 + i) * f + c;
        const float a_pre = to_f(G[go]) + ea[i], b_pre = to_f(U[go]) + eb[i];
        const float a = cgv * a_pre, b = cuv * b_pre;
        const float sg = sigmoidf_(a), sa = a * sg;
        const float Dt = to_f(D[so]) + ed[i];
        dgv = Dt * sa * b;
        const float dh = gt[i0 + i] * Dt;
        const float da = dh * b * sg * (1.f + a * (1.f - sg));
        const float db = dh * sa;
        mg = fmaf(da, a_pre, mg);
        mu = fmaf(db, b_pre, mu);
        da_sorted[so] = from_f<T>(cgv * da);
        db_sorted[so] = from_f<T>(cuv * db);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dgv += __shfl_xor_sync(0xffffffffu, dgv, o);
      if (lane == 0) red[i][warp] = dgv;
    }
    __syncthreads();
    if (threadIdx.x < RB && i0 + threadIdx.x < rows) {
      float v = 0.f;
      for (int w = 0; w < kCols / 32; ++w) v += red[threadIdx.x][w];      // fixed order
      dgate_part[(size_t)blockIdx.y * slots + p0 + i0 + threadIdx.x] = v;
    }
  }
  if (live) {
    dm_part_g[(size_t)tile * f + c] = mg;
    dm_part_u[(size_t)tile * f + c] = mu;
  }
}

// p_s[pos][c] = spd_s[pos][e r + c] for c < r (e the slot's expert), zero up to the padded width rp: the rank-r
// operand s B_d[e]^T dO of the grouped backward kernel, per sorted slot
template <typename T>
__global__ void dora_pcompact_kernel(const T* __restrict__ spd_s, const int* __restrict__ pos_expert,
                                     T* __restrict__ p_s, int slots, int N, int r, int rp) {
  const long long n = (long long)slots * rp;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / rp), cidx = (int)(i % rp);
    p_s[i] = cidx < r ? spd_s[((size_t)pos * N + pos_expert[pos]) * r + cidx] : from_f<T>(0.f);
  }
}

// d_m[e][o] (+)= inv_n[e][o] * sum over the expert's tiles (in table order) of part[tile][o]; with sub > 1 a tile
// has `sub` partial rows (part[tile * sub + j][o]), added in the order of j
__global__ void dora_dm_reduce_kernel(const float* __restrict__ part, const float* __restrict__ inv_n,
                                      const int* __restrict__ tile_info, int max_tiles, float* __restrict__ dm,
                                      int N, int width, int accumulate, int sub) {
  const int e = blockIdx.y;
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= width) return;
  const int ntiles = min(tile_info[max_tiles * 4], max_tiles);
  float s = 0.f;
  for (int t = 0; t < ntiles; ++t)
    if (tile_info[t * 4 + 0] == e)
      for (int j = 0; j < sub; ++j) s += part[((size_t)t * sub + j) * width + o];
  const size_t i = (size_t)e * width + o;
  const float v = inv_n[i] * s;
  dm[i] = accumulate ? dm[i] + v : v;
}

inline int grid_for(long long n, int block) {
  long long g = (n + block - 1) / block;
  return (int)(g < 1 ? 1 : (g > 148 * 16 ? 148 * 16 : g));
}

template <typename T>
cudaError_t rowsq_t(const Ctx& c, const DoraCtx& dc) {
  const int d = c.s.d_model, f = c.s.d_ff;
  rowsq_kernel<T><<<(f + 7) / 8, 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.w_gate), dc.rowsq_g, f, d);
  rowsq_kernel<T><<<(f + 7) / 8, 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.w_up), dc.rowsq_u, f, d);
  rowsq_kernel<T><<<(d + 7) / 8, 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.w_down), dc.rowsq_d, d, f);
  return cudaGetLastError();
}

template <typename T>
cudaError_t scales_t(const Ctx& c, const DoraCtx& dc) {
  const int d = c.s.d_model, f = c.s.d_ff, N = c.s.n_experts, r = c.s.rank;
  dora_scale_kernel<T><<<grid_for((long long)N * f, 256), 256, 0, c.st>>>(
      dc.rowsq_g, dc.wa_g, dc.aat_g, reinterpret_cast<const T*>(c.p.b_gate), dc.m.m_gate, dc.cg, dc.inv_g, f, N, r, c.scale);
  dora_scale_kernel<T><<<grid_for((long long)N * f, 256), 256, 0, c.st>>>(
      dc.rowsq_u, dc.wa_u, dc.aat_u, reinterpret_cast<const T*>(c.p.b_up), dc.m.m_up, dc.cu, dc.inv_u, f, N, r, c.scale);
  dora_scale_kernel<T><<<grid_for((long long)N * d, 256), 256, 0, c.st>>>(
      dc.rowsq_d, dc.wa_d, dc.aat_d, reinterpret_cast<const T*>(c.p.b_down), dc.m.m_down, dc.cd, dc.inv_d, d, N, r, c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t swiglu_fwd_t(const Ctx& c, const DoraCtx& dc) {
  const int mt = max_seg_tiles(c.s.tokens, c.s.top_k, c.s.n_experts);
  dim3 grid(mt, (c.s.d_ff + kCols - 1) / kCols);
  dora_swiglu_fwd_kernel<T><<<grid, kCols, 2 * 8 * c.s.rank * sizeof(float), c.st>>>(
      c.at<T>(c.L.G), c.at<T>(c.L.U), c.at<T>(c.L.zga), c.at<T>(c.L.zua), reinterpret_cast<const T*>(c.p.b_gate),
      reinterpret_cast<const T*>(c.p.b_up), dc.cg, dc.cu, c.at<int>(c.L.pos_token), c.at<int>(c.L.tile_info), mt,
      c.at<T>(c.L.h_sorted), c.s.d_ff, c.s.n_experts, c.s.rank, c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t own_block_t(const Ctx& c, const void* in, void* own, void* gown) {
  const int slots = c.s.tokens * c.s.top_k;
  dora_own_block_kernel<T><<<grid_for((long long)slots * c.s.n_experts * c.s.rank, 256), 256, 0, c.st>>>(
      reinterpret_cast<const T*>(in), c.at<float>(c.L.gates), c.at<int>(c.L.perm), c.at<int>(c.L.pos_expert),
      reinterpret_cast<T*>(own), reinterpret_cast<T*>(gown), slots, c.s.n_experts, c.s.rank);
  return cudaGetLastError();
}

template <typename T>
cudaError_t combine_y_t(const Ctx& c, const DoraCtx& dc, void* y) {
  dora_combine_y_kernel<T><<<c.s.tokens, kCols, 0, c.st>>>(reinterpret_cast<const T*>(dc.o_pre), dc.cd,
                                                          c.at<float>(c.L.gates), c.at<int>(c.L.inv),
                                                          c.at<int>(c.L.expert_idx), reinterpret_cast<T*>(y),
                                                          c.s.d_model, c.s.top_k);
  return cudaGetLastError();
}

template <typename T>
cudaError_t dout_t(const Ctx& c, const DoraCtx& dc, const void* dy) {
  const int mt = max_seg_tiles(c.s.tokens, c.s.top_k, c.s.n_experts);
  dim3 grid(mt, (c.s.d_model + kCols - 1) / kCols);
  dora_dout_kernel<T><<<grid, kCols, 0, c.st>>>(reinterpret_cast<const T*>(dy), reinterpret_cast<const T*>(dc.o_pre),
                                               dc.cd, c.at<float>(c.L.gates), c.at<int>(c.L.perm),
                                               c.at<int>(c.L.pos_token), c.at<int>(c.L.tile_info), mt,
                                               reinterpret_cast<T*>(dc.dO), dc.dmp_d, c.s.d_model);
  return cudaGetLastError();
}

template <typename T>
cudaError_t swiglu_bwd_t(const Ctx& c, const DoraCtx& dc) {
  const int mt = max_seg_tiles(c.s.tokens, c.s.top_k, c.s.n_experts);
  dim3 grid(mt, (c.s.d_ff + kCols - 1) / kCols);
  dora_swiglu_bwd_kernel<T><<<grid, kCols, 3 * 8 * c.s.rank * sizeof(float), c.st>>>(
      c.at<T>(c.L.G), c.at<T>(c.L.U), reinterpret_cast<const T*>(dc.D_s), c.at<T>(c.L.zga), c.at<T>(c.L.zua),
      reinterpret_cast<const T*>(dc.spd_s), reinterpret_cast<const T*>(c.p.b_gate),
      reinterpret_cast<const T*>(c.p.b_up), reinterpret_cast<const T*>(c.p.a_down), dc.cg, dc.cu,
      c.at<float>(c.L.gates), c.at<int>(c.L.perm), c.at<int>(c.L.pos_token), c.at<int>(c.L.tile_info), mt,
      c.at<T>(c.L.da_sorted), c.at<T>(c.L.db_sorted), c.at<float>(c.L.dgate_part), dc.dmp_g, dc.dmp_u,
      c.s.tokens * c.s.top_k, c.s.d_ff, c.s.n_experts, c.s.rank, c.scale);
  return cudaGetLastError();
}

}  // namespace

int dora_bwd_col_chunks(int f) { return (f + kCols - 1) / kCols; }

cudaError_t launch_dora_rowsq(const Ctx& c, const DoraCtx& dc) { return c.bf16 ? rowsq_t<bf16>(c, dc) : rowsq_t<float>(c, dc); }
cudaError_t launch_dora_scales(const Ctx& c, const DoraCtx& dc) { return c.bf16 ? scales_t<bf16>(c, dc) : scales_t<float>(c, dc); }
cudaError_t launch_dora_swiglu_fwd(const Ctx& c, const DoraCtx& dc) {
  return c.bf16 ? swiglu_fwd_t<bf16>(c, dc) : swiglu_fwd_t<float>(c, dc);
}
cudaError_t launch_dora_own_block(const Ctx& c, const void* in, void* own, void* gown) {
  return c.bf16 ? own_block_t<bf16>(c, in, own, gown) : own_block_t<float>(c, in, own, gown);
}
cudaError_t launch_dora_combine_y(const Ctx& c, const DoraCtx& dc, void* y) {
  return c.bf16 ? combine_y_t<bf16>(c, dc, y) : combine_y_t<float>(c, dc, y);
}
cudaError_t launch_dora_dout(const Ctx& c, const DoraCtx& dc, const void* dy) {
  return c.bf16 ? dout_t<bf16>(c, dc, dy) : dout_t<float>(c, dc, dy);
}
cudaError_t launch_dora_swiglu_bwd(const Ctx& c, const DoraCtx& dc) {
  return c.bf16 ? swiglu_bwd_t<bf16>(c, dc) : swiglu_bwd_t<float>(c, dc);
}
cudaError_t launch_dora_dm_reduce(const Ctx& c, const float* part, const float* inv_n, float* dm, int width,
                                  int accumulate, int sub) {
  const int mt = max_seg_tiles(c.s.tokens, c.s.top_k, c.s.n_experts);
  dim3 grid((width + 255) / 256, c.s.n_experts);
  dora_dm_reduce_kernel<<<grid, 256, 0, c.st>>>(part, inv_n, c.at<int>(c.L.tile_info), mt, dm, c.s.n_experts, width,
                                                accumulate, sub);
  return cudaGetLastError();
}

cudaError_t launch_dora_pcompact(const Ctx& c, const DoraCtx& dc) {
  const int slots = c.s.tokens * c.s.top_k, r = c.s.rank, rp = pad_rank(r);
  if (!c.bf16) return cudaErrorInvalidValue;       // only the tensor-core grouped kernel reads the compact form
  dora_pcompact_kernel<bf16><<<grid_for((long long)slots * rp, 256), 256, 0, c.st>>>(
      reinterpret_cast<const bf16*>(dc.spd_s), c.at<int>(c.L.pos_expert), c.at<bf16>(c.L.p_s), slots, c.s.n_experts, r,
      rp);
  return cudaGetLastError();
}

}  // namespace mixlora
