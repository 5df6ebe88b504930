// Memory-bound stages of the block in the order "expert ascending, token ascending":
// LoRA-B expansion + SwiGLU (forward and backward), combine over a token's slots,
// small repacks, router backward.
#include "common.cuh"

namespace mixlora {

namespace {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16(v); }

__device__ __forceinline__ float sigmoidf_(float v) { return 1.f / (1.f + expf(-v)); }

constexpr int SL = 8;      // sorted slots per block in the per-slot kernels
constexpr int ENT = 256;   // threads per block

// cat[c][e*r + rr] = s * B[e][c][rr]   (B is [N, rows, r]; used for B_d with rows = d and B_g, B_u with rows = f)
template <typename T>
__global__ void bd_cat_kernel(const T* __restrict__ b_down, T* __restrict__ bd_cat, int d, int N, int r, float s) {
  const long long n = (long long)d * N * r;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    int rr = (int)(i % r);
    int e = (int)((i / r) % N);
    int c = (int)(i / ((long long)r * N));
    bd_cat[i] = from_f<T>(s * to_f(b_down[((long long)e * d + c) * r + rr]));
  }
}

// Forward, per sorted slot: a = G_t + s B_g[e] zg, b = U_t + s B_u[e] zu, h = SiLU(a) * b
// (Algorithm 1, the three steps inside the expert loop before the down projection).
template <typename T>
__global__ void __launch_bounds__(ENT)
lora_b_swiglu_kernel(const T* __restrict__ G, const T* __restrict__ U, const T* __restrict__ zga,
                     const T* __restrict__ zua, const T* __restrict__ b_gate, const T* __restrict__ b_up,
                     const int* __restrict__ pos_token, const int* __restrict__ pos_expert, T* __restrict__ h_sorted,
                     int slots, int f, int N, int r, float s) {
  extern __shared__ float sm[];
  float* zg = sm;              // [SL][r], already scaled by s
  float* zu = sm + SL * r;     // [SL][r]
  __shared__ int tok[SL], ex[SL];
  const int base = blockIdx.x * SL;
  const int ns = min(SL, slots - base);
  if (threadIdx.x < SL) {
    int i = threadIdx.x;
    tok[i] = (i < ns) ? pos_token[base + i] : 0;
    ex[i] = (i < ns) ? pos_expert[base + i] : -1;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < SL * r; i += ENT) {
    int sl = i / r, rr = i % r;
    float vg = 0.f, vu = 0.f;
    if (sl < ns) {
      size_t o = (size_t)tok[sl] * N * r + (size_t)ex[sl] * r + rr;
      vg = s * to_f(zga[o]);
      vu = s * to_f(zua[o]);
    }
    zg[i] = vg;
    zu[i] = vu;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < f; c += ENT) {
    int i0 = 0;
    while (i0 < ns) {
      const int e = ex[i0];
      int i1 = i0;
      while (i1 < ns && ex[i1] == e) ++i1;
      float ea[SL], eb[SL];
#pragma unroll
      for (int i = 0; i < SL; ++i) { ea[i] = 0.f; eb[i] = 0.f; }
      const T* bg = b_gate + ((size_t)e * f + c) * r;
      const T* bu = b_up + ((size_t)e * f + c) * r;
      for (int rr = 0; rr < r; ++rr) {
        const float wg = to_f(bg[rr]), wu = to_f(bu[rr]);
#pragma unroll
        for (int i = 0; i < SL; ++i) {
          ea[i] = fmaf(zg[i * r + rr], wg, ea[i]);
          eb[i] = fmaf(zu[i * r + rr], wu, eb[i]);
        }
      }
#pragma unroll
      for (int i = 0; i < SL; ++i) {
        if (i >= i0 && i < i1) {
          const size_t go = (size_t)tok[i] * f + c;
          const float a = to_f(G[go]) + ea[i];
          const float b = to_f(U[go]) + eb[i];
          h_sorted[(size_t)(base + i) * f + c] = from_f<T>(a * sigmoidf_(a) * b);
        }
      }
      i0 = i1;
    }
  }
}

// hbar_t = sum_j g_tj h_tj ;  Zs[t, e_j*r + rr] = g_tj * zd_j[rr], zero elsewhere.  With `zd_part` (the forward
// grouped kernel's per-column-group partial sums [groups, slots, r] of the slot's own expert) zd is those partials
// added up in group order; else it is read from zd [slots, N r].
template <typename T>
__global__ void __launch_bounds__(ENT)
combine_h_kernel(const T* __restrict__ h_sorted, const T* __restrict__ zd, const float* __restrict__ zd_part,
                 const int* __restrict__ zd_groups, int slots, const float* __restrict__ gates,
                 const int* __restrict__ inv, const int* __restrict__ expert_idx, T* __restrict__ hbar,
                 T* __restrict__ Zs, int f, int N, int r, int k, int do_wide) {
  const int t = blockIdx.x;
  __shared__ int pos[MIXLORA_MAX_TOP_K], ex[MIXLORA_MAX_TOP_K];
  __shared__ float g[MIXLORA_MAX_TOP_K];
  __shared__ float zds[MIXLORA_MAX_TOP_K * 32];        // fold mode (r <= 32): [slot of the token][r]
  if (threadIdx.x < k) {
    pos[threadIdx.x] = inv[(size_t)t * k + threadIdx.x];
    ex[threadIdx.x] = expert_idx[(size_t)t * k + threadIdx.x];
    g[threadIdx.x] = gates[(size_t)t * k + threadIdx.x];
  }
  __syncthreads();
  if (zd_part) {
    const int groups = *zd_groups;
    const size_t gstride = (size_t)slots * r;
    for (int i = threadIdx.x; i < k * r; i += blockDim.x) {
      const int j = i / r;
      const float* src = zd_part + (size_t)pos[j] * r + (i - j * r);
      float sum = 0.f;
      int gi = 0;
      for (; gi + 8 <= groups; gi += 8) {              // eight groups' loads in flight; the sum keeps group order
        float tv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) tv[u] = __ldg(src + (size_t)(gi + u) * gstride);
#pragma unroll
        for (int u = 0; u < 8; ++u) sum += tv[u];
      }
      for (; gi < groups; ++gi) sum += __ldg(src + (size_t)gi * gstride);
      zds[i] = sum;
    }
    __syncthreads();
  }
  for (int c = threadIdx.x; do_wide && c < f; c += ENT) {
    float acc = 0.f;
    for (int j = 0; j < k; ++j) acc = fmaf(g[j], to_f(h_sorted[(size_t)pos[j] * f + c]), acc);
    hbar[(size_t)t * f + c] = from_f<T>(acc);
  }
  const int nr = N * r;
  for (int q = threadIdx.x; q < nr; q += blockDim.x) {
    const int e = q / r, rr = q % r;
    float v = 0.f;
    for (int j = 0; j < k; ++j)
      if (ex[j] == e) v = g[j] * (zd_part ? to_f(from_f<T>(zds[j * r + rr])) : to_f(zd[(size_t)pos[j] * nr + q]));
    Zs[(size_t)t * nr + q] = from_f<T>(v);
  }
}

// bf16 version of the f-wide part of combine_h, 8 values per thread per step.  K = top-k when it is at most 4
// (all of a chunk's loads are then issued before the first use), else 0 = any k.
template <int K>
__global__ void __launch_bounds__(ENT)
combine_h_vec_kernel(const bf16* __restrict__ h_sorted, const float* __restrict__ gates, const int* __restrict__ inv,
                     bf16* __restrict__ hbar, int f, int k_any) {
  const int k = K > 0 ? K : k_any;
  const int t = blockIdx.x;
  __shared__ int pos[MIXLORA_MAX_TOP_K];
  __shared__ float g[MIXLORA_MAX_TOP_K];
  if (threadIdx.x < k) {
    pos[threadIdx.x] = inv[(size_t)t * k + threadIdx.x];
    g[threadIdx.x] = gates[(size_t)t * k + threadIdx.x];
  }
  __syncthreads();
  for (int c = threadIdx.x * 8; c < f; c += ENT * 8) {
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (K > 0) {
      uint4 raw[K > 0 ? K : 1];
#pragma unroll
      for (int j = 0; j < K; ++j) raw[j] = __ldg(reinterpret_cast<const uint4*>(h_sorted + (size_t)pos[j] * f + c));
#pragma unroll
      for (int j = 0; j < K; ++j) {                    // slot order, as in the generic loop: the same bits
        const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&raw[j]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __bfloat1622float2(pr[i]);
          acc[2 * i] = fmaf(g[j], v.x, acc[2 * i]);
          acc[2 * i + 1] = fmaf(g[j], v.y, acc[2 * i + 1]);
        }
      }
    } else {
      for (int j = 0; j < k; ++j) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(h_sorted + (size_t)pos[j] * f + c));
        const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __bfloat1622float2(pr[i]);
          acc[2 * i] = fmaf(g[j], v.x, acc[2 * i]);
          acc[2 * i + 1] = fmaf(g[j], v.y, acc[2 * i + 1]);
        }
      }
    }
    uint4 o;
    __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) po[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    *reinterpret_cast<uint4*>(hbar + (size_t)t * f + c) = o;
  }
}

// bf16 version of the f-wide part of combine_bwd
__global__ void __launch_bounds__(ENT)
combine_bwd_vec_kernel(const bf16* __restrict__ da_sorted, const bf16* __restrict__ db_sorted,
                       const int* __restrict__ inv, bf16* __restrict__ dabar, bf16* __restrict__ dbbar, int f, int k) {
  const int t = blockIdx.x;
  __shared__ int pos[MIXLORA_MAX_TOP_K];
  if (threadIdx.x < k) pos[threadIdx.x] = inv[(size_t)t * k + threadIdx.x];
  __syncthreads();
  for (int c = threadIdx.x * 8; c < f; c += ENT * 8) {
    float sa[8] = {0, 0, 0, 0, 0, 0, 0, 0}, sb[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int j = 0; j < k; ++j) {
      const uint4 ra = __ldg(reinterpret_cast<const uint4*>(da_sorted + (size_t)pos[j] * f + c));
      const uint4 rb = __ldg(reinterpret_cast<const uint4*>(db_sorted + (size_t)pos[j] * f + c));
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&ra);
      const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&rb);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 va = __bfloat1622float2(pa[i]), vb = __bfloat1622float2(pb[i]);
        sa[2 * i] += va.x; sa[2 * i + 1] += va.y;
        sb[2 * i] += vb.x; sb[2 * i + 1] += vb.y;
      }
    }
    uint4 oa, ob;
    __nv_bfloat162* qa = reinterpret_cast<__nv_bfloat162*>(&oa);
    __nv_bfloat162* qb = reinterpret_cast<__nv_bfloat162*>(&ob);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      qa[i] = __floats2bfloat162_rn(sa[2 * i], sa[2 * i + 1]);
      qb[i] = __floats2bfloat162_rn(sb[2 * i], sb[2 * i + 1]);
    }
    *reinterpret_cast<uint4*>(dabar + (size_t)t * f + c) = oa;
    *reinterpret_cast<uint4*>(dbbar + (size_t)t * f + c) = ob;
  }
}

// Backward, per sorted slot.  Re-computes a, b, h from the saved G, U, zg, zu, then
//   Dt = D_t + A_d[e]^T (s pd)      (gradient of the slot's h before the gate)
//   dgate = <Dt, h> ;  dh = g Dt ;  da = dh * b * SiLU'(a) ;  db = dh * SiLU(a)
template <typename T>
__global__ void __launch_bounds__(ENT)
swiglu_bwd_kernel(const T* __restrict__ G, const T* __restrict__ U, const T* __restrict__ D,
                  const T* __restrict__ zga, const T* __restrict__ zua, const T* __restrict__ spd,
                  const T* __restrict__ b_gate, const T* __restrict__ b_up, const T* __restrict__ a_down,
                  const float* __restrict__ gates, const int* __restrict__ perm, const int* __restrict__ pos_token,
                  const int* __restrict__ pos_expert, T* __restrict__ h_sorted, T* __restrict__ da_sorted,
                  T* __restrict__ db_sorted, float* __restrict__ dgate, int slots, int f, int N, int r, float s) {
  extern __shared__ float sm[];
  float* zg = sm;                 // [SL][r] scaled by s
  float* zu = sm + SL * r;        // [SL][r] scaled by s
  float* pd = sm + 2 * SL * r;    // [SL][r] = s * pd
  __shared__ int tok[SL], ex[SL], slot[SL];
  __shared__ float gt[SL];
  __shared__ float red[SL][ENT / 32];
  const int base = blockIdx.x * SL;
  const int ns = min(SL, slots - base);
  if (threadIdx.x < SL) {
    int i = threadIdx.x;
    tok[i] = (i < ns) ? pos_token[base + i] : 0;
    ex[i] = (i < ns) ? pos_expert[base + i] : -1;
    slot[i] = (i < ns) ? perm[base + i] : 0;
    gt[i] = (i < ns) ? gates[slot[i]] : 0.f;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < SL * r; i += ENT) {
    int sl = i / r, rr = i % r;
    float vg = 0.f, vu = 0.f, vp = 0.f;
    if (sl < ns) {
      size_t o = (size_t)tok[sl] * N * r + (size_t)ex[sl] * r + rr;
      vg = s * to_f(zga[o]);
      vu = s * to_f(zua[o]);
      vp = to_f(spd[o]);
    }
    zg[i] = vg; zu[i] = vu; pd[i] = vp;
  }
  __syncthreads();
  float dg_acc[SL];
#pragma unroll
  for (int i = 0; i < SL; ++i) dg_acc[i] = 0.f;
  for (int c = threadIdx.x; c < f; c += ENT) {
    int i0 = 0;
    while (i0 < ns) {
      const int e = ex[i0];
      int i1 = i0;
      while (i1 < ns && ex[i1] == e) ++i1;
      float ea[SL], eb[SL], ed[SL];
#pragma unroll
      for (int i = 0; i < SL; ++i) { ea[i] = 0.f; eb[i] = 0.f; ed[i] = 0.f; }
      const T* bg = b_gate + ((size_t)e * f + c) * r;
      const T* bu = b_up + ((size_t)e * f + c) * r;
      const T* ad = a_down + (size_t)e * r * f + c;
      for (int rr = 0; rr < r; ++rr) {
        const float wg = to_f(bg[rr]), wu = to_f(bu[rr]), wd = to_f(ad[(size_t)rr * f]);
#pragma unroll
        for (int i = 0; i < SL; ++i) {
          ea[i] = fmaf(zg[i * r + rr], wg, ea[i]);
          eb[i] = fmaf(zu[i * r + rr], wu, eb[i]);
          ed[i] = fmaf(pd[i * r + rr], wd, ed[i]);
        }
      }
#pragma unroll
      for (int i = 0; i < SL; ++i) {
        if (i >= i0 && i < i1) {
          const size_t go = (size_t)tok[i] * f + c;
          const float a = to_f(G[go]) + ea[i];
          const float b = to_f(U[go]) + eb[i];
          const float sg = sigmoidf_(a);
          const float sa = a * sg;
          const float h = sa * b;
          const float Dt = to_f(D[go]) + ed[i];
          dg_acc[i] = fmaf(Dt, h, dg_acc[i]);
          const float dh = gt[i] * Dt;
          const size_t so = (size_t)(base + i) * f + c;
          h_sorted[so] = from_f<T>(h);
          da_sorted[so] = from_f<T>(dh * b * sg * (1.f + a * (1.f - sg)));
          db_sorted[so] = from_f<T>(dh * sa);
        }
      }
      i0 = i1;
    }
  }
  // deterministic block reduction of the gate gradients
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < SL; ++i) {
    float v = dg_acc[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red[i][w] = v;
  }
  __syncthreads();
  if (threadIdx.x < ns) {
    float v = 0.f;
    for (int ww = 0; ww < ENT / 32; ++ww) v += red[threadIdx.x][ww];
    dgate[slot[threadIdx.x]] = v;
  }
}

// dZd_pos[pos][q] = g * (s pd)[token, q] inside the slot's expert block, zero elsewhere
template <typename T>
__global__ void slot_prep_bwd_kernel(const T* __restrict__ spd, const float* __restrict__ gates,
                                     const int* __restrict__ perm, const int* __restrict__ pos_token,
                                     const int* __restrict__ pos_expert,
                                     T* __restrict__ dZd_pos, T* __restrict__ p_s, int slots, int N, int r, int rp) {
  const long long nr = (long long)N * r;
  const long long n = (long long)slots * nr;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / nr), q = (int)(i % nr);
    float v = 0.f;
    if (q / r == pos_expert[pos]) v = gates[perm[pos]] * to_f(spd[(size_t)pos_token[pos] * nr + q]);
    dZd_pos[i] = from_f<T>(v);
  }
  // compact copy: the slot's own r values, zero padded to rp
  const long long n2 = (long long)slots * rp;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n2; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / rp), cidx = (int)(i % rp);
    p_s[i] = cidx < r ? spd[((size_t)pos_token[pos] * N + pos_expert[pos]) * r + cidx] : from_f<T>(0.f);
  }
}

// Zg_pos[pos][q] = zga[token(pos)][q] inside the slot's expert block, zero elsewhere (same for Zu_pos)
template <typename T>
__global__ void zpos_kernel(const T* __restrict__ zga, const T* __restrict__ zua, const int* __restrict__ pos_token,
                            const int* __restrict__ pos_expert, T* __restrict__ Zg_pos, T* __restrict__ Zu_pos,
                            int slots, int N, int r) {
  const long long nr = (long long)N * r;
  const long long n = (long long)slots * nr;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / nr), q = (int)(i % nr);
    const bool own = (q / r) == pos_expert[pos];
    const size_t src = (size_t)pos_token[pos] * nr + q;
    Zg_pos[i] = own ? zga[src] : from_f<T>(0.f);
    Zu_pos[i] = own ? zua[src] : from_f<T>(0.f);
  }
}

// zg_s[pos][c] = s * zga[token][e*r + c] for c < r, zero up to the padded width rp (same for zu_s)
template <typename T>
__global__ void zcompact_kernel(const T* __restrict__ zga, const T* __restrict__ zua, const int* __restrict__ pos_token,
                                const int* __restrict__ pos_expert, T* __restrict__ zg_s, T* __restrict__ zu_s,
                                int slots, int N, int r, int rp, float s) {
  const long long n = (long long)slots * rp;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / rp), cidx = (int)(i % rp);
    float vg = 0.f, vu = 0.f;
    if (cidx < r) {
      const size_t src = ((size_t)pos_token[pos] * N + pos_expert[pos]) * r + cidx;
      vg = s * to_f(zga[src]);
      vu = s * to_f(zua[src]);
    }
    zg_s[i] = from_f<T>(vg);
    zu_s[i] = from_f<T>(vu);
  }
}

// out[row][c] = in[row][c] for c < r, zero up to rp columns
template <typename T>
__global__ void pad_cols_kernel(const T* __restrict__ in, T* __restrict__ out, long long rows, int r, int rp) {
  const long long n = rows * rp;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long row = i / rp;
    const int cidx = (int)(i % rp);
    out[i] = cidx < r ? in[row * r + cidx] : from_f<T>(0.f);
  }
}

// out[e][rr][c] = in[e][rr][c] for rr < r, zero rows up to rp per expert (A_d is [N, r, f])
template <typename T>
__global__ void pad_rows_kernel(const T* __restrict__ in, T* __restrict__ out, int N, int r, int rp, int f) {
  const long long n = (long long)N * rp * f;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int col = (int)(i % f);
    const int rr = (int)((i / f) % rp);
    const int e = (int)(i / ((long long)f * rp));
    out[i] = rr < r ? in[((long long)e * r + rr) * f + col] : from_f<T>(0.f);
  }
}

// dgate[slot] = sum over column tiles of the partial <Dt, h> (fixed order)
__global__ void dgate_reduce_kernel(const float* __restrict__ part, const int* __restrict__ perm,
                                    float* __restrict__ dgate, int slots, int col_tiles) {
  const int pos = blockIdx.x * blockDim.x + threadIdx.x;
  if (pos >= slots) return;
  float s = 0.f;
  for (int ct = 0; ct < col_tiles; ++ct) s += part[(size_t)ct * slots + pos];
  dgate[perm[pos]] = s;
}

// dabar_t = sum_j da_tj, dbbar_t = sum_j db_tj ; dZg / dZu = dzg / dzu scattered to the expert block
// With `dz_part` (the grouped backward kernel's per-column-group partial sums [groups, slots, 2, r] of the slot's
// own expert) dzg / dzu are those partials added up in group order; else they are read from dzg_sorted / dzu_sorted.
template <typename T>
__global__ void __launch_bounds__(ENT)
combine_bwd_kernel(const T* __restrict__ da_sorted, const T* __restrict__ db_sorted, const T* __restrict__ dzg_sorted,
                   const T* __restrict__ dzu_sorted, const float* __restrict__ dz_part,
                   const int* __restrict__ dz_groups, int slots, const int* __restrict__ inv,
                   const int* __restrict__ expert_idx, T* __restrict__ dabar, T* __restrict__ dbbar,
                   T* __restrict__ dZg, T* __restrict__ dZu, int f, int N, int r, int k, int want_dx) {
  const int t = blockIdx.x;
  __shared__ int pos[MIXLORA_MAX_TOP_K], ex[MIXLORA_MAX_TOP_K];
  __shared__ float dzs[MIXLORA_MAX_TOP_K * 2 * 32];    // fold mode (r <= 32): [slot of the token][dzg, dzu][r]
  if (threadIdx.x < k) {
    pos[threadIdx.x] = inv[(size_t)t * k + threadIdx.x];
    ex[threadIdx.x] = expert_idx[(size_t)t * k + threadIdx.x];
  }
  __syncthreads();
  if (dz_part) {
    // one thread per value of the token's slots; a warp's loads of one group are contiguous
    const int groups = *dz_groups;
    const size_t gstride = (size_t)slots * 2 * r;
    for (int i = threadIdx.x; i < k * 2 * r; i += blockDim.x) {
      const int j = i / (2 * r);
      const float* src = dz_part + (size_t)pos[j] * 2 * r + (i - j * 2 * r);
      float sum = 0.f;
      int g = 0;
      for (; g + 8 <= groups; g += 8) {                // eight groups' loads in flight; the sum keeps group order
        float tv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) tv[u] = __ldg(src + (size_t)(g + u) * gstride);
#pragma unroll
        for (int u = 0; u < 8; ++u) sum += tv[u];
      }
      for (; g < groups; ++g) sum += __ldg(src + (size_t)g * gstride);
      dzs[i] = sum;
    }
    __syncthreads();
  }
  for (int c = threadIdx.x; want_dx && c < f; c += ENT) {
    float sa = 0.f, sb = 0.f;
    for (int j = 0; j < k; ++j) {
      sa += to_f(da_sorted[(size_t)pos[j] * f + c]);
      sb += to_f(db_sorted[(size_t)pos[j] * f + c]);
    }
    dabar[(size_t)t * f + c] = from_f<T>(sa);
    dbbar[(size_t)t * f + c] = from_f<T>(sb);
  }
  const int nr = N * r;
  for (int q = threadIdx.x; q < nr; q += blockDim.x) {
    const int e = q / r, rr = q % r;
    T vg = from_f<T>(0.f), vu = from_f<T>(0.f);
    for (int j = 0; j < k; ++j)
      if (ex[j] == e) {
        if (dz_part) {
          vg = from_f<T>(dzs[j * 2 * r + rr]);
          vu = from_f<T>(dzs[j * 2 * r + r + rr]);
        } else {
          vg = dzg_sorted[(size_t)pos[j] * nr + q];
          vu = dzu_sorted[(size_t)pos[j] * nr + q];
        }
      }
    dZg[(size_t)t * nr + q] = vg;
    dZu[(size_t)t * nr + q] = vu;
  }
}

// Router backward, one thread per token: gate re-normalisation, auxiliary-loss term
// (F_i is piecewise constant, so only P_i carries gradient), softmax.
template <typename T>
__global__ void router_bwd_kernel(const float* __restrict__ probs, const float* __restrict__ gates,
                                  const int* __restrict__ expert_idx, const float* __restrict__ dgate,
                                  const float* __restrict__ F, float* __restrict__ dlogits, T* __restrict__ dl_act,
                                  int tokens, int N, int NP, int k, int renorm, float aux_coef,
                                  const long long* __restrict__ batch_tokens) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= tokens) return;
  // d L_aux / d p_ti = coef N F_i / T with T the tokens of the whole batch (Eq. 8-9): this call's, unless the
  // auxiliary loss was evaluated over data-parallel shards, which leaves the batch's count (and F) in the workspace
  const long long bt = *batch_tokens;
  const float aux_scale = aux_coef * (float)N / (float)(bt > 0 ? bt : (long long)tokens);
  float dp[MIXLORA_MAX_EXPERTS];
#pragma unroll
  for (int e = 0; e < MIXLORA_MAX_EXPERTS; ++e) dp[e] = (e < N) ? aux_scale * F[e] : 0.f;
  float q = 0.f, inner = 0.f;
  for (int j = 0; j < k; ++j) {
    const int e = expert_idx[(size_t)t * k + j];
    q += probs[(size_t)t * N + e];
    inner = fmaf(gates[(size_t)t * k + j], dgate[(size_t)t * k + j], inner);
  }
  for (int j = 0; j < k; ++j) {
    const int e = expert_idx[(size_t)t * k + j];
    const float dg = dgate[(size_t)t * k + j];
    const float v = renorm ? (dg - inner) / q : dg;
#pragma unroll
    for (int ee = 0; ee < MIXLORA_MAX_EXPERTS; ++ee)
      if (ee == e) dp[ee] += v;
  }
  float dot = 0.f;
#pragma unroll
  for (int e = 0; e < MIXLORA_MAX_EXPERTS; ++e)
    if (e < N) dot = fmaf(probs[(size_t)t * N + e], dp[e], dot);
#pragma unroll
  for (int e = 0; e < MIXLORA_MAX_EXPERTS; ++e) {
    if (e < NP) {
      float v = (e < N) ? probs[(size_t)t * N + e] * (dp[e] - dot) : 0.f;
      if (e < N) dlogits[(size_t)t * N + e] = v;
      if (dl_act) dl_act[(size_t)t * NP + e] = from_f<T>(v);
    }
  }
}

// out[e] = sum_t dl[t, e], one block per expert, fixed order.
__global__ void __launch_bounds__(256)
colsum_kernel(const float* __restrict__ dl, float* __restrict__ out, int tokens, int N, int accumulate) {
  __shared__ float sp[256];
  const int e = blockIdx.x;
  float s = 0.f;
  for (int t = threadIdx.x; t < tokens; t += 256) s += dl[(size_t)t * N + e];
  sp[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sp[threadIdx.x] += sp[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[e] = accumulate ? out[e] + sp[0] : sp[0];
}

// router weight in the activation type, rows padded to NP with zeros
template <typename T>
__global__ void wr_act_kernel(const float* __restrict__ w_router, T* __restrict__ wr_act, int N, int NP, int d) {
  const long long n = (long long)NP * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    int e = (int)(i / d);
    wr_act[i] = from_f<T>(e < N ? w_router[i] : 0.f);
  }
}

inline int grid_for(long long n, int block) {
  long long g = (n + block - 1) / block;
  return (int)(g < 1 ? 1 : (g > 148 * 16 ? 148 * 16 : g));
}

template <typename T>
cudaError_t bd_cat_t(const Ctx& c) {
  const long long n = (long long)c.s.d_model * c.s.n_experts * c.s.rank;
  bd_cat_kernel<T><<<grid_for(n, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.b_down), c.at<T>(c.L.bd_cat),
                                                      c.s.d_model, c.s.n_experts, c.s.rank, c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t bgu_cat_t(const Ctx& c) {
  const long long n = (long long)c.s.d_ff * c.s.n_experts * c.s.rank;
  bd_cat_kernel<T><<<grid_for(n, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.b_gate), c.at<T>(c.L.bg_cat),
                                                      c.s.d_ff, c.s.n_experts, c.s.rank, c.scale);
  bd_cat_kernel<T><<<grid_for(n, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.b_up), c.at<T>(c.L.bu_cat),
                                                      c.s.d_ff, c.s.n_experts, c.s.rank, c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t zpos_t(const Ctx& c) {
  const int slots = c.s.tokens * c.s.top_k;
  zpos_kernel<T><<<grid_for((long long)slots * c.s.rank * c.s.n_experts, 256), 256, 0, c.st>>>(
      c.at<T>(c.L.zga), c.at<T>(c.L.zua), c.at<int>(c.L.pos_token), c.at<int>(c.L.pos_expert), c.at<T>(c.L.Zg_pos),
      c.at<T>(c.L.Zu_pos), slots, c.s.n_experts, c.s.rank);
  return cudaGetLastError();
}

template <typename T>
cudaError_t zcompact_t(const Ctx& c) {
  const int slots = c.s.tokens * c.s.top_k, r = c.s.rank, rp = pad_rank(r);
  zcompact_kernel<T><<<grid_for((long long)slots * rp, 256), 256, 0, c.st>>>(
      c.at<T>(c.L.zga), c.at<T>(c.L.zua), c.at<int>(c.L.pos_token), c.at<int>(c.L.pos_expert), c.at<T>(c.L.zg_s),
      c.at<T>(c.L.zu_s), slots, c.s.n_experts, r, rp, c.scale);
  if (rp != r) {   // parameter-only repacks for the grouped kernels; the backward pass finds them in the workspace
    const long long rows = (long long)c.s.n_experts * c.s.d_ff;
    pad_cols_kernel<T><<<grid_for(rows * rp, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.b_gate),
                                                                  c.at<T>(c.L.bgp), rows, r, rp);
    pad_cols_kernel<T><<<grid_for(rows * rp, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.b_up),
                                                                  c.at<T>(c.L.bup), rows, r, rp);
    pad_rows_kernel<T><<<grid_for(rows * rp, 256), 256, 0, c.st>>>(reinterpret_cast<const T*>(c.p.a_down),
                                                                  c.at<T>(c.L.adp), c.s.n_experts, r, rp, c.s.d_ff);
  }
  return cudaGetLastError();
}

template <typename T>
cudaError_t lora_b_swiglu_t(const Ctx& c) {
  const int slots = c.s.tokens * c.s.top_k;
  const int blocks = (slots + SL - 1) / SL;
  const size_t smem = 2 * SL * c.s.rank * sizeof(float);
  lora_b_swiglu_kernel<T><<<blocks, ENT, smem, c.st>>>(
      c.at<T>(c.L.G), c.at<T>(c.L.U), c.at<T>(c.L.zga), c.at<T>(c.L.zua), reinterpret_cast<const T*>(c.p.b_gate),
      reinterpret_cast<const T*>(c.p.b_up), c.at<int>(c.L.pos_token), c.at<int>(c.L.pos_expert), c.at<T>(c.L.h_sorted),
      slots, c.s.d_ff, c.s.n_experts, c.s.rank, c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t combine_h_t(const Ctx& c) {
  // with bf16 activations the f-wide sum runs in its own vectorised kernel; this one then only scatters Zs
  constexpr bool vec = sizeof(T) == 2;
  combine_h_kernel<T><<<c.s.tokens, vec ? 128 : ENT, 0, c.st>>>(
      c.at<T>(c.L.h_sorted), c.at<T>(c.L.zd_all), ctx_folds_zd(c) ? c.at<float>(c.L.zd_part) : nullptr,
      c.at<int>(c.L.work_count) + 4, c.s.tokens * c.s.top_k, c.at<float>(c.L.gates), c.at<int>(c.L.inv),
      c.at<int>(c.L.expert_idx),
      c.at<T>(c.L.hbar), c.at<T>(c.L.Zs), c.s.d_ff, c.s.n_experts, c.s.rank, c.s.top_k, vec ? 0 : 1);
  return cudaGetLastError();
}

template <typename T>
cudaError_t swiglu_bwd_t(const Ctx& c) {
  const int slots = c.s.tokens * c.s.top_k;
  const int blocks = (slots + SL - 1) / SL;
  const size_t smem = 3 * SL * c.s.rank * sizeof(float);
  swiglu_bwd_kernel<T><<<blocks, ENT, smem, c.st>>>(
      c.at<T>(c.L.G), c.at<T>(c.L.U), c.at<T>(c.L.D), c.at<T>(c.L.zga), c.at<T>(c.L.zua), c.at<T>(c.L.spd),
      reinterpret_cast<const T*>(c.p.b_gate), reinterpret_cast<const T*>(c.p.b_up),
      reinterpret_cast<const T*>(c.p.a_down), c.at<float>(c.L.gates), c.at<int>(c.L.perm), c.at<int>(c.L.pos_token),
      c.at<int>(c.L.pos_expert), c.at<T>(c.L.h_sorted), c.at<T>(c.L.da_sorted), c.at<T>(c.L.db_sorted),
      c.at<float>(c.L.dgate), slots, c.s.d_ff, c.s.n_experts, c.s.rank,
      c.scale);
  return cudaGetLastError();
}

template <typename T>
cudaError_t slot_prep_bwd_t(const Ctx& c) {
  const int slots = c.s.tokens * c.s.top_k;
  slot_prep_bwd_kernel<T><<<grid_for((long long)slots * c.s.rank * c.s.n_experts, 256), 256, 0, c.st>>>(
      c.at<T>(c.L.spd), c.at<float>(c.L.gates), c.at<int>(c.L.perm), c.at<int>(c.L.pos_token),
      c.at<int>(c.L.pos_expert), c.at<T>(c.L.dZd_pos), c.at<T>(c.L.p_s), slots, c.s.n_experts,
      c.s.rank, pad_rank(c.s.rank));
  return cudaGetLastError();
}

template <typename T>
cudaError_t combine_bwd_t(const Ctx& c, int want_dx) {
  constexpr bool vec = sizeof(T) == 2;
  combine_bwd_kernel<T><<<c.s.tokens, vec ? 128 : ENT, 0, c.st>>>(
      c.at<T>(c.L.da_sorted), c.at<T>(c.L.db_sorted), c.at<T>(c.L.dzg_all), c.at<T>(c.L.dzu_all),
      ctx_folds_dz(c) ? c.at<float>(c.L.dz_part) : nullptr, c.at<int>(c.L.work_count) + 3,
      c.s.tokens * c.s.top_k, c.at<int>(c.L.inv), c.at<int>(c.L.expert_idx), c.at<T>(c.L.dabar), c.at<T>(c.L.dbbar), c.at<T>(c.L.dZg),
      c.at<T>(c.L.dZu), c.s.d_ff, c.s.n_experts, c.s.rank, c.s.top_k, vec ? 0 : want_dx);
  return cudaGetLastError();
}

template <typename T>
cudaError_t router_bwd_t(const Ctx& c, float aux_coef, float* d_bias, int accumulate, int want_dx) {
  const int T_ = c.s.tokens, N = c.s.n_experts, NP = round_up8(N);
  router_bwd_kernel<T><<<(T_ + 127) / 128, 128, 0, c.st>>>(
      c.at<float>(c.L.probs), c.at<float>(c.L.gates), c.at<int>(c.L.expert_idx), c.at<float>(c.L.dgate),
      c.at<float>(c.L.stat_F), c.at<float>(c.L.dlogits), c.at<T>(c.L.dl_act), T_, N, NP, c.s.top_k,
      c.s.renormalize, aux_coef, reinterpret_cast<const long long*>(c.ws + c.L.status + 8));
  if (d_bias) colsum_kernel<<<N, 256, 0, c.st>>>(c.at<float>(c.L.dlogits), d_bias, T_, N, accumulate);
  if (want_dx)
    wr_act_kernel<T><<<grid_for((long long)NP * c.s.d_model, 256), 256, 0, c.st>>>(c.p.w_router, c.at<T>(c.L.wr_act), N,
                                                                                 NP, c.s.d_model);
  return cudaGetLastError();
}


// ---- the block inside its layer (Eq. 5 / Eq. 6): RMS normalisation in front, its Jacobian behind -------------
// One block per token, 16-byte loads and stores; a thread keeps its chunks of the row in registers between the
// reduction and the write, so the row is read once.  kNormChunks * kNormThreads 16-byte chunks bound the width.
constexpr int kNormThreads = 256;
constexpr int kNormChunks = 4;

template <typename T> struct Vec16 { static constexpr int n = 16 / sizeof(T); };
template <typename T>
__device__ __forceinline__ void load16(const T* p, float* o) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int j = 0; j < Vec16<T>::n; ++j) o[j] = to_f(e[j]);
}
template <typename T>
__device__ __forceinline__ void store16(T* p, const float* v) {
  uint4 raw;
  T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
  for (int j = 0; j < Vec16<T>::n; ++j) e[j] = from_f<T>(v[j]);
  *reinterpret_cast<uint4*>(p) = raw;
}

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < kNormThreads / 32; ++w) t += red[w];   // fixed order: the same bits in every thread and run
  return t;
}

// xn = w_norm * z * inv_rms (one rounding), inv_rms = 1 / sqrt(mean(z^2) + eps)
template <typename T>
__global__ void __launch_bounds__(kNormThreads) rmsnorm_fwd_kernel(const T* __restrict__ z, const T* __restrict__ w_norm,
                                                                  float eps, T* __restrict__ xn,
                                                                  float* __restrict__ inv_rms, int d) {
  constexpr int V = Vec16<T>::n;
  __shared__ float red[kNormThreads / 32];
  const size_t row = (size_t)blockIdx.x * d;
  float v[kNormChunks][V];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < kNormChunks; ++i) {
    const int c = (threadIdx.x + i * kNormThreads) * V;
    if (c < d) {
      load16(z + row + c, v[i]);
#pragma unroll
      for (int j = 0; j < V; ++j) ss = fmaf(v[i][j], v[i][j], ss);
    }
  }
  const float inv = rsqrtf(block_sum(ss, red) / (float)d + eps);
  if (threadIdx.x == 0) inv_rms[blockIdx.x] = inv;
#pragma unroll
  for (int i = 0; i < kNormChunks; ++i) {
    const int c = (threadIdx.x + i * kNormThreads) * V;
    if (c < d) {
      float w[V];
      load16(w_norm + c, w);
#pragma unroll
      for (int j = 0; j < V; ++j) w[j] = w[j] * v[i][j] * inv;
      store16(xn + row + c, w);
    }
  }
}

// dz = dh + inv_rms * (u - xh * mean(u * xh)),  u = dxn * w_norm,  xh = z * inv_rms.  dxn and dz may be the same
// buffer: every element is read before the block writes it.
template <typename T>
__global__ void __launch_bounds__(kNormThreads) rmsnorm_bwd_kernel(const T* __restrict__ z, const T* __restrict__ w_norm,
                                                                  const float* __restrict__ inv_rms, const T* dxn,
                                                                  const T* __restrict__ dh, T* dz, int d) {
  constexpr int V = Vec16<T>::n;
  __shared__ float red[kNormThreads / 32];
  const size_t row = (size_t)blockIdx.x * d;
  const float inv = inv_rms[blockIdx.x];
  float u[kNormChunks][V], xh[kNormChunks][V];
  float dot = 0.f;
#pragma unroll
  for (int i = 0; i < kNormChunks; ++i) {
    const int c = (threadIdx.x + i * kNormThreads) * V;
    if (c < d) {
      float w[V];
      load16(dxn + row + c, u[i]);
      load16(w_norm + c, w);
      load16(z + row + c, xh[i]);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        u[i][j] *= w[j];
        xh[i][j] *= inv;
        dot = fmaf(u[i][j], xh[i][j], dot);
      }
    }
  }
  const float m = block_sum(dot, red) / (float)d;
#pragma unroll
  for (int i = 0; i < kNormChunks; ++i) {
    const int c = (threadIdx.x + i * kNormThreads) * V;
    if (c < d) {
      float g[V];
      load16(dh + row + c, g);
#pragma unroll
      for (int j = 0; j < V; ++j) g[j] += inv * (u[i][j] - xh[i][j] * m);
      store16(dz + row + c, g);
    }
  }
}

// C[m][n] += R[m][n] (fp32 check mode; the tensor-core path adds the residual in its epilogue)
template <typename T>
__global__ void residual_add_kernel(T* __restrict__ C, long long ldc, const T* __restrict__ R, long long ldr, int M, int N) {
  const long long n = (long long)M * N;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long m = i / N, col = i % N;
    C[m * ldc + col] = from_f<T>(to_f(C[m * ldc + col]) + to_f(R[m * ldr + col]));
  }
}

}  // namespace

cudaError_t launch_bd_cat(const Ctx& c) { return c.bf16 ? bd_cat_t<bf16>(c) : bd_cat_t<float>(c); }
cudaError_t launch_lora_b_swiglu(const Ctx& c) { return c.bf16 ? lora_b_swiglu_t<bf16>(c) : lora_b_swiglu_t<float>(c); }
cudaError_t launch_combine_h(const Ctx& c) {
  if (!c.bf16) return combine_h_t<float>(c);
#define MIXLORA_COMBINE_H(KK)                                                                                      \
  combine_h_vec_kernel<KK><<<c.s.tokens, ENT, 0, c.st>>>(c.at<bf16>(c.L.h_sorted), c.at<float>(c.L.gates),          \
                                                        c.at<int>(c.L.inv), c.at<bf16>(c.L.hbar), c.s.d_ff, c.s.top_k)
  switch (c.s.top_k) {
    case 1: MIXLORA_COMBINE_H(1); break;
    case 2: MIXLORA_COMBINE_H(2); break;
    case 3: MIXLORA_COMBINE_H(3); break;
    case 4: MIXLORA_COMBINE_H(4); break;
    default: MIXLORA_COMBINE_H(0); break;
  }
#undef MIXLORA_COMBINE_H
  return combine_h_t<bf16>(c);
}
cudaError_t launch_swiglu_bwd(const Ctx& c) { return c.bf16 ? swiglu_bwd_t<bf16>(c) : swiglu_bwd_t<float>(c); }
cudaError_t launch_slot_prep_bwd(const Ctx& c) { return c.bf16 ? slot_prep_bwd_t<bf16>(c) : slot_prep_bwd_t<float>(c); }
cudaError_t launch_combine_bwd(const Ctx& c, int want_dx) {
  if (!c.bf16) return combine_bwd_t<float>(c, want_dx);
  if (want_dx)
    combine_bwd_vec_kernel<<<c.s.tokens, ENT, 0, c.st>>>(c.at<bf16>(c.L.da_sorted), c.at<bf16>(c.L.db_sorted),
                                                        c.at<int>(c.L.inv), c.at<bf16>(c.L.dabar),
                                                        c.at<bf16>(c.L.dbbar), c.s.d_ff, c.s.top_k);
  return combine_bwd_t<bf16>(c, want_dx);
}
cudaError_t launch_zcompact(const Ctx& c) { return c.bf16 ? zcompact_t<bf16>(c) : zcompact_t<float>(c); }
cudaError_t launch_zpos(const Ctx& c) { return c.bf16 ? zpos_t<bf16>(c) : zpos_t<float>(c); }
cudaError_t launch_dgate_reduce(const Ctx& c, int col_tiles) {
  const int slots = c.s.tokens * c.s.top_k;
  dgate_reduce_kernel<<<(slots + 255) / 256, 256, 0, c.st>>>(c.at<float>(c.L.dgate_part), c.at<int>(c.L.perm),
                                                            c.at<float>(c.L.dgate), slots, col_tiles);
  return cudaGetLastError();
}
cudaError_t launch_bgu_cat(const Ctx& c) { return c.bf16 ? bgu_cat_t<bf16>(c) : bgu_cat_t<float>(c); }
cudaError_t launch_router_bwd(const Ctx& c, float aux_coef, float* d_bias, int accumulate, int want_dx) {
  return c.bf16 ? router_bwd_t<bf16>(c, aux_coef, d_bias, accumulate, want_dx)
                : router_bwd_t<float>(c, aux_coef, d_bias, accumulate, want_dx);
}

int rmsnorm_max_width(int bf16_mode) { return kNormThreads * kNormChunks * (bf16_mode ? 8 : 4); }
cudaError_t launch_rmsnorm_fwd(const Ctx& c, const void* z, const void* w_norm, float eps, void* xn, float* inv_rms) {
  if (c.s.tokens == 0) return cudaSuccess;
  if (c.bf16)
    rmsnorm_fwd_kernel<bf16><<<c.s.tokens, kNormThreads, 0, c.st>>>(
        reinterpret_cast<const bf16*>(z), reinterpret_cast<const bf16*>(w_norm), eps, reinterpret_cast<bf16*>(xn), inv_rms,
        c.s.d_model);
  else
    rmsnorm_fwd_kernel<float><<<c.s.tokens, kNormThreads, 0, c.st>>>(
        reinterpret_cast<const float*>(z), reinterpret_cast<const float*>(w_norm), eps, reinterpret_cast<float*>(xn),
        inv_rms, c.s.d_model);
  return cudaGetLastError();
}
cudaError_t launch_rmsnorm_bwd(const Ctx& c, const void* z, const void* w_norm, const float* inv_rms, const void* dxn,
                               const void* dh, void* dz) {
  if (c.s.tokens == 0) return cudaSuccess;
  if (c.bf16)
    rmsnorm_bwd_kernel<bf16><<<c.s.tokens, kNormThreads, 0, c.st>>>(
        reinterpret_cast<const bf16*>(z), reinterpret_cast<const bf16*>(w_norm), inv_rms,
        reinterpret_cast<const bf16*>(dxn), reinterpret_cast<const bf16*>(dh), reinterpret_cast<bf16*>(dz), c.s.d_model);
  else
    rmsnorm_bwd_kernel<float><<<c.s.tokens, kNormThreads, 0, c.st>>>(
        reinterpret_cast<const float*>(z), reinterpret_cast<const float*>(w_norm), inv_rms,
        reinterpret_cast<const float*>(dxn), reinterpret_cast<const float*>(dh), reinterpret_cast<float*>(dz),
        c.s.d_model);
  return cudaGetLastError();
}
cudaError_t launch_residual_add(const Ctx& c, void* C, long long ldc, const void* R, long long ldr, int M, int N) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  const int grid = grid_for((long long)M * N, 256);
  if (c.bf16)
    residual_add_kernel<bf16><<<grid, 256, 0, c.st>>>(reinterpret_cast<bf16*>(C), ldc, reinterpret_cast<const bf16*>(R),
                                                      ldr, M, N);
  else
    residual_add_kernel<float><<<grid, 256, 0, c.st>>>(reinterpret_cast<float*>(C), ldc,
                                                       reinterpret_cast<const float*>(R), ldr, M, N);
  return cudaGetLastError();
}

}  // namespace mixlora
