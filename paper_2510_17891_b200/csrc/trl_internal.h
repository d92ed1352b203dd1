// Internal declarations shared by the translation units of libtrl (host side only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "trl.h"

namespace trl {

constexpr int kRowBlock = 128;   // rows per row block = TMEM lanes of one accumulator tile

// process-wide count of kernels this library has enqueued (statistics only)
void note_launch(int n = 1);
unsigned long long launches_so_far();

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Bounds-checked debug build (-DTRL_DEBUG_BOUNDS): stores whose index comes out of the row packing
// (a packed row, a global row looked up in rowmap) are checked against the extent of their buffer;
// a violation sets TRL_ERR_BOUNDS in the status word and the store is skipped.  In the normal build
// the check is the constant true.
#ifdef __CUDACC__
#ifdef TRL_DEBUG_BOUNDS
__device__ __forceinline__ bool trl_bounds_violation(int32_t* status) {
  if (status) atomicOr(status, 1 << TRL_ERR_BOUNDS);
  return false;
}
#define TRL_IN_BOUNDS(idx, extent, status) \
  (((unsigned long long)(idx) < (unsigned long long)(extent)) ? true : trl::trl_bounds_violation(status))
#else
#define TRL_IN_BOUNDS(idx, extent, status) true
#endif
#endif
inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// Row packing: the valid rows of all rollouts, in order, get consecutive packed indices
// q = row_first[b] + t (t < len[b]); 128 consecutive packed rows form one row block (one
// accumulator tile).  Built on the device from `len` (no host round trip).
struct RowPack {
  int* nblk;       // [1]     ceil(n_rows / 128)
  int* n_rows;     // [1]     number of valid rows
  int* row_first;  // [B+1]   packed index of each rollout's first row (exclusive prefix sum of len)
  int* rowmap;     // [cap*128] packed row -> global row b*T + t (defined for q < n_rows)
  int cap;         // ceil(B*T / 128): upper bound on nblk
  long n_total;    // B*T: number of global rows
};
size_t row_pack_bytes(int B, int T);
RowPack carve_row_pack(void* base, int B, int T);

// ---- small kernels (trl_small_kernels.cu) ------------------------------------------
void launch_build_row_pack(const int32_t* len, int B, int T, RowPack rb, int32_t* status, cudaStream_t s);
void launch_hrd_advantages(const float* r_plan, const float* r_code, const int32_t* len, const int32_t* bnd,
                           int P, int G, int T, int adv_mode, float* A_plan, float* A_code, uint8_t* seg,
                           float* adv, int32_t* n_plan, int32_t* n_code, int64_t* n_valid, int32_t* status,
                           cudaStream_t s);
// n_rows > max_rows (a multiple of 128): flag TRL_ERR_ROWS_BOUND and drop the excess rows
void launch_clamp_rows(RowPack rb, int max_rows, int32_t* status, cudaStream_t s);
int  pg_loss_tiles(int T);
// ids may be null; when given, tokens whose id is outside [0, V) are left out like padding
void launch_pg_loss(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                    const int32_t* len, int P, int G, int T, trl_pg_config cfg, float* loss, float* g,
                    float* stats, float* partials, const int32_t* ids, int V, cudaStream_t s);
// merge per-vocabulary-tile (max, sumexp) partials into lse / logp and scatter to global rows
void launch_merge_lse(const float2* partials, const float* tgt, int n_tiles, int rows_cap, RowPack rb,
                      const int32_t* ids, const int32_t* len, int B, int T, int V, float* logp, float* lse,
                      int32_t* status, cudaStream_t s);
// out[r, :] = src[row, :] (times row_scale[r] when given) for r < R, where the packed row is
// q = q_off + r and row = rowmap[q] (from_packed = 0: src is the caller's [N,H] tensor) or
// row = q (from_packed = 1: src is already packed); rows q >= n_rows are written as zeros.
void launch_pack_rows_bf16(const __nv_bfloat16* src, __nv_bfloat16* out, int H, int R, RowPack rb, int q_off,
                           int from_packed, const float* row_scale, cudaStream_t s);
// Chunk-local finish of the fused step: lse = c + log(sum_k psum), logp, g = d loss/d logp,
// the per-row factor -g exp(c - lse) for the gradient GEMMs, and the one-hot fix of E / E^T.
struct FusedMergeArgs {
  const float* psum; const float* tgt; int n_tiles; int R; RowPack rb; int blk_off;
  const int32_t* ids; const int32_t* len; const float* hint; const float* old_logp; const float* adv;
  const uint8_t* seg; int P, G, T, V; trl_pg_config cfg;
  float* logp; float* lse; float* g; float* neg_alpha;
  int* blk_active;                  // [R/128] 1 if any row of the block has a non-zero factor
  __nv_bfloat16* E;
  int32_t* status;
  int R_live;                       // rows of the chunk that exist (0: R); R stays the stride of psum
};
void launch_fused_merge(const FusedMergeArgs& a, cudaStream_t s);
// blk_active[i] = 1 if any of the 128 packed rows of row block i has g != 0 (i < nblk)
void launch_flag_active_blocks(const float* g, RowPack rb, int* blk_active, cudaStream_t s);
// fp32 path helpers
void launch_pack_rows_f32(const float* hidden, float* Xp, int H, int R, RowPack rb, int blk_off, cudaStream_t s);
void launch_row_lse_f32(const float* S, int V, int R, RowPack rb, int blk_off, const int32_t* ids,
                        float* logp, float* lse, int32_t* status, cudaStream_t s);
void launch_ds_inplace_f32(float* S, int V, int R, RowPack rb, int blk_off, const int32_t* ids,
                           const float* lse, const float* g, cudaStream_t s);
void launch_scatter_rows_f32(const float* dHp, float* dHidden, int H, int R, RowPack rb, int blk_off, cudaStream_t s);
void launch_zero_padded_f32(float* a, float* b, const int32_t* len, int B, int T, cudaStream_t s);

// ---- fp32 CUDA-core GEMM (trl_simt_gemm.cu) ----------------------------------------
// C[m,n] (+)= sum_k A(m,k) B(k,n); A(m,k) = A[m*sam + k*sak], B(k,n) = B[k*sbk + n*sbn].
// If live_from_blocks != 0 the extent named by it (1: M, 2: K) is
// 128 * clamp(*nblk - blk_off, 0, blk_cap) instead of the host value.
struct SimtGemm {
  const float* A; long sam, sak;
  const float* B; long sbk, sbn;
  float* C; long ldc;
  int M, N, K;
  int accumulate;
  int live_from_blocks; const int* nblk; int blk_off, blk_cap;
};
void launch_simt_gemm(const SimtGemm& p, cudaStream_t s);

// ---- tcgen05 GEMM family (trl_tc_gemm.cu) ------------------------------------------
enum TcEpilogue { TC_EPI_LSE = 0, TC_EPI_DS = 1, TC_EPI_DH = 2, TC_EPI_DW = 3, TC_EPI_E = 4 };
struct TcGemm {
  int epi;
  // operands, bf16.  a_rows / b_rows = extent of the M / N dimension, K = extent of the
  // contraction.  K-major operand (forward; A of DH): stored [rows, K], pitch ld.  MN-major
  // operand (B of DH; A and B of DW): stored [K, rows], pitch ld.
  const void* A; long a_rows; long a_ld;
  const void* B; long b_rows; long b_ld;
  long b_k;                                  // K extent of B's storage if it differs from K (0: same)
  int K;                                     // host K extent (TC_EPI_DW: K = 128 * live blocks of the chunk)
  int N;                                     // GEMM N extent = b_rows that are meaningful
  int m_blocks;                              // TC_EPI_DW: fixed number of 128-row blocks of A; others: from row blocks
  RowPack rb; int blk_off, blk_cap;        // chunk of row blocks
  // all but TC_EPI_DW: this launch works on M positions [pos_off, pos_off + pos_cap) of the chunk only (pos_cap 0:
  // all of them); a position is an entry of the list of active row blocks when blk_active is given, else a row block
  int pos_off, pos_cap;
  unsigned* pace_ctr; int pace_every;         // soft pacing of the CTAs every pace_every k-blocks (null: off); zero the counter before the launch
  int raster_band_blocks;                    // 128-row blocks rasterised together (0: default)
  int cta_group;                             // CTAs per MMA: 1, 2 (cluster pairs), 0: the build's default
  // epilogue arguments
  const int32_t* ids; const float* lse; const float* g;
  float2* partials; float* tgt; int rows_cap;          // LSE
  __nv_bfloat16* dS; long ds_ld;                       // DS, E
  __nv_bfloat16* dHidden; long dh_ld; long dh_rows;    // DH (dh_rows: rows of dHidden, for the debug build's checks)
  float* dW; long dw_ld; int V;                        // DW
  float* psum;                                         // E: row sums per vocabulary tile [n_tiles, rows_cap]
  const float* row_scale;                              // DH: optional per-scratch-row factor
  const int* blk_active;                               // DS, DH, DW: optional per-row-block activity flags of the chunk
  int32_t* status;
};
// returns cudaSuccess or the error of tensor-map creation / launch
cudaError_t launch_tc_gemm(const TcGemm& p, cudaStream_t s);
int tc_num_sms();
int tc_default_cta_group(int fwd);   // CTAs per MMA in effect for the forward (1) / gradient (0) GEMMs
int tc_wave_aligned_blocks(int n_cols);   // M positions (128-row blocks) per launch of a gradient GEMM that fill whole waves of CTAs
int tc_raster_band_override(int epi);   // raster band in 128-row blocks from TRL_RASTER_BAND_<LSE|DS|DH|DW|E>, 0: none

}  // namespace trl
