// Generic SIMT product with fp32 accumulation (see SGemm in common.cuh).
// It serves the fp32 check mode, the skinny LoRA products and every shape the tensor-core
// kernel does not take.  64 x 64 output tile, 16-deep reduction step, 4 x 4 values per thread.
#include "common.cuh"

namespace mixlora {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

__device__ __forceinline__ float ld_elem(const void* p, long long idx, int is_bf16) {
  return is_bf16 ? __bfloat162float(reinterpret_cast<const bf16*>(p)[idx]) : reinterpret_cast<const float*>(p)[idx];
}

// Loads a [rows x BK] tile of one operand into smem as tile[k][row].
__device__ __forceinline__ void load_tile(float (*tile)[BM + 1], const SOperand& o, long long gbase, int row0, int row_end,
                                          int k0, int k_end, int tid) {
  // the thread -> element map follows the unit stride, for coalescing
  const bool k_fast = (o.sk == 1 && o.gk == nullptr);
#pragma unroll
  for (int it = 0; it < (BM * BK) / NT; ++it) {
    int e = tid + it * NT;
    int r, k;
    if (k_fast) { k = e % BK; r = e / BK; } else { r = e % BM; k = e / BM; }
    int gr = row0 + r, gk = k0 + k;
    float v = 0.f;
    if (gr < row_end && gk < k_end) {
      long long ri = o.gi ? (long long)o.gi[gr] : (long long)gr;
      long long ki = o.gk ? (long long)o.gk[gk] : (long long)gk;
      v = ld_elem(o.p, gbase + ri * o.si + ki * o.sk, o.is_bf16);
    }
    tile[k][r] = v;
  }
}

__global__ void __launch_bounds__(NT) simt_gemm_kernel(const SGemm g) {
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int tid = threadIdx.x;
  const int grp = blockIdx.z;
  int m_begin = 0, m_end = g.M;
  int kseg0_begin = 0, kseg0_end = g.K[0];
  if (g.group_mode == 1) { m_begin = g.seg_off[grp]; m_end = g.seg_off[grp + 1]; }
  if (g.group_mode == 2) { kseg0_begin = g.seg_off[grp]; kseg0_end = g.seg_off[grp + 1]; }
  const int m0 = m_begin + blockIdx.y * BM;
  const int n0 = blockIdx.x * BN;
  if (m0 >= m_end || n0 >= g.N) return;

  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int sgi = 0; sgi < g.nseg; ++sgi) {
    const SOperand& A = g.A[sgi];
    const SOperand& B = g.B[sgi];
    int kb = (sgi == 0) ? kseg0_begin : 0;
    int ke = (sgi == 0) ? kseg0_end : g.K[sgi];
    const long long abase = (long long)grp * A.sg, bbase = (long long)grp * B.sg;
    for (int k0 = kb; k0 < ke; k0 += BK) {
      load_tile(As, A, abase, m0, m_end, k0, ke, tid);
      load_tile(Bs, B, bbase, n0, g.N, k0, ke, tid);
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
      __syncthreads();
    }
  }

  const long long cbase = (long long)grp * g.c_sg;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= m_end) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      long long idx = cbase + (long long)m * g.c_sm +
                      (g.c_nb > 0 ? (long long)(n / g.c_nb) * g.c_sblk + (long long)(n % g.c_nb) * g.c_sn
                                  : (long long)n * g.c_sn);
      float v = g.alpha * acc[i][j];
      if (g.c_is_bf16) {
        bf16* C = reinterpret_cast<bf16*>(g.C);
        if (g.accumulate) v += __bfloat162float(C[idx]);
        C[idx] = __float2bfloat16(v);
      } else {
        float* C = reinterpret_cast<float*>(g.C);
        if (g.accumulate) v += C[idx];
        C[idx] = v;
      }
    }
  }
}

}  // namespace

cudaError_t launch_simt_gemm(const SGemm& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.groups <= 0) return cudaSuccess;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.groups);
  if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidConfiguration;
  simt_gemm_kernel<<<grid, NT, 0, st>>>(g);
  return cudaGetLastError();
}

}  // namespace mixlora
