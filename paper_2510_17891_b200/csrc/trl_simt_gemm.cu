// fp32 CUDA-core GEMM with generic strides: the TRL_F32 path of the library (small
// problems and a second opinion for the tensor-core path).  64x64x16 tiles, 256 threads,
// 4x4 register micro-tiles.
#include "trl_internal.h"

namespace trl {

constexpr int BM = 64, BN = 64, BK = 16;

__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtGemm p) {
  int M = p.M, K = p.K;
  if (p.live_from_blocks) {
    const int live = max(0, min(p.nblk[0] - p.blk_off, p.blk_cap)) * kRowBlock;
    if (p.live_from_blocks == 1) M = min(M, live); else K = min(K, live);
  }
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  const bool a_kfast = p.sak == 1, b_nfast = p.sbn == 1;
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int m, k;
      if (a_kfast) { m = idx >> 4; k = idx & 15; } else { m = idx & 63; k = idx >> 6; }
      const int gm = m0 + m, gk = k0 + k;
      As[k][m] = (gm < M && gk < K) ? p.A[(long)gm * p.sam + (long)gk * p.sak] : 0.f;
      int n, kb;
      if (b_nfast) { n = idx & 63; kb = idx >> 6; } else { n = idx >> 4; kb = idx & 15; }
      const int gn = n0 + n, gkb = k0 + kb;
      Bs[kb][n] = (gn < p.N && gkb < K) ? p.B[(long)gkb * p.sbk + (long)gn * p.sbn] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= p.N) continue;
      float* c = p.C + (long)gm * p.ldc + gn;
      *c = p.accumulate ? *c + acc[i][j] : acc[i][j];
    }
  }
}

void launch_simt_gemm(const SimtGemm& p, cudaStream_t s) {
  dim3 grid(cdiv(p.N, BN), cdiv(p.M, BM));
  simt_gemm_kernel<<<grid, 256, 0, s>>>(p);
  note_launch();
}

}  // namespace trl
