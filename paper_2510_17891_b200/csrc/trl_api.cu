// extern "C" entry points of libtrl: argument checks, workspace carving, kernel sequencing.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "trl_internal.h"

using namespace trl;

namespace {

constexpr int kRecommendedChunkRowsBf16 = 32768;
constexpr int kRecommendedChunkRowsF32 = 2048;
// 128-row blocks whose tiles are rasterised together (their A rows stay in L2 while B streams)
constexpr int kRasterBandFwd = 32;
constexpr int kRasterBandFwdE = 32;   // forward tiles that also store E / dS
constexpr int kRasterBandBwd = 8;

int check_device() {      // the current device must be compute capability 10.x (cached per device)
  static std::atomic<int> cached[64];      // 0: not looked up yet; otherwise status + 1
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TRL_ERR_CUDA;
  const int c = cached[dev].load(std::memory_order_relaxed);
  if (c) return c - 1;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TRL_ERR_CUDA;
  const int st = (major == 10) ? TRL_OK : TRL_ERR_ARCH;
  cached[dev].store(st + 1, std::memory_order_relaxed);
  return st;
}

// Alignment contract of the boundary: tensors the kernels touch with 16-byte accesses or through
// TMA must start on a 16-byte boundary; everything else on the boundary of its element type.
bool al16(const void* p) { return ((uintptr_t)p & 15) == 0; }
bool al4(const void* p) { return ((uintptr_t)p & 3) == 0; }
bool al8(const void* p) { return ((uintptr_t)p & 7) == 0; }

bool shapes_ok(int B, int T, int H, int V) {
  return B > 0 && T > 0 && H > 0 && V > 0 && (long)B * T < (1L << 31) - 256 && (long)V * H < (1L << 40);
}

struct Carver {
  char* base; size_t off = 0;
  explicit Carver(void* p) : base((char*)p) {}
  template <class Tp> Tp* take(size_t n) {
    Tp* r = (Tp*)(base + off);
    off += align_up(n * sizeof(Tp), 256);
    return r;
  }
};

int rows_cap_of(int B, int T) { return cdiv(B * T, kRowBlock) * kRowBlock; }
size_t xp_bytes(int B, int T, int H) { return align_up((size_t)rows_cap_of(B, T) * H * 2, 256); }   // packed hidden rows
size_t fwd_extra_bf16(int B, int T, int V) {     // target logits + (max, sum-exp) partials per vocabulary tile
  const size_t rows_cap = rows_cap_of(B, T);
  return align_up(rows_cap * 4, 256) + align_up((size_t)cdiv(V, 256) * rows_cap * 8, 256);
}
size_t fwd_bytes_bf16(int B, int T, int H, int V) { return row_pack_bytes(B, T) + xp_bytes(B, T, H) + fwd_extra_bf16(B, T, V); }
size_t fwd_bytes_f32(int B, int T, int H, int V, int R) {
  return row_pack_bytes(B, T) + align_up((size_t)R * H * 4, 256) + align_up((size_t)R * V * 4, 256);
}
size_t bwd_fixed_bf16(int B, int T, int H, int V) {     // row packing, packed hidden, row-block activity flags, pacing counters
  (void)V;
  return row_pack_bytes(B, T) + xp_bytes(B, T, H) + 2 * align_up((size_t)cdiv(B * T, kRowBlock) * 4, 256);
}
size_t bwd_per_rows_bf16(int H, int V, int R) { (void)H; return align_up((size_t)R * V * 2, 256); }   // dS chunk
size_t bwd_bytes_f32(int B, int T, int H, int V, int R) {
  return row_pack_bytes(B, T) + 2 * align_up((size_t)R * H * 4, 256) + align_up((size_t)R * V * 4, 256);
}
size_t loss_bytes(int B, int T) { return align_up((size_t)B * pg_loss_tiles(T) * 4 * sizeof(float), 256); }
// fused step: fixed part (row packing, packed hidden, loss partials) and per-chunk part for R rows
// (scaled hidden rows, E, row sums per vocabulary tile, target logits, row factors)
size_t fused_fixed_bf16(int B, int T, int H, int V) { return bwd_fixed_bf16(B, T, H, V) + loss_bytes(B, T); }
size_t fused_per_rows_bf16(int H, int V, int R) {
  return align_up((size_t)H * R * 2, 256) + align_up((size_t)R * V * 2, 256) + align_up((size_t)cdiv(V, 256) * R * 4, 256) +
         2 * align_up((size_t)R * 4, 256) + align_up((size_t)(R / kRowBlock) * 4, 256);
}

// banded schedule: E, the scaled hidden rows, the row factors and the activity flags are kept for all
// RB rows (RB = the caller's bound on the number of valid rows, rounded up to 128); row sums and
// target logits are per chunk of Rc rows
int banded_rows(int B, int T, int rows_bound) {
  const int cap = rows_cap_of(B, T);
  if (rows_bound <= 0 || rows_bound > B * T) return cap;
  return cdiv(rows_bound, kRowBlock) * kRowBlock;
}
size_t fused_banded_bytes(int B, int T, int H, int V, int rows_bound, bool with_fwd_extra) {
  const size_t RB = banded_rows(B, T, rows_bound);
  const size_t Rc = RB < (size_t)kRecommendedChunkRowsBf16 ? RB : (size_t)kRecommendedChunkRowsBf16;
  return fused_fixed_bf16(B, T, H, V) + align_up(RB * H * 2, 256) + align_up(RB * V * 2, 256) +
         align_up((size_t)cdiv(V, 256) * Rc * 4, 256) + align_up(Rc * 4, 256) + align_up(RB * 4, 256) +
         align_up((RB / kRowBlock) * 4, 256) + (with_fwd_extra ? fwd_extra_bf16(B, T, V) : 0);
}

// largest multiple of 128 rows (<= cap) whose scratch fits into `avail` bytes
template <class F>
int fit_rows(size_t avail, int cap, F bytes_of) {
  int lo = 0, hi = cap / kRowBlock;
  while (lo < hi) {
    int mid = (lo + hi + 1) / 2;
    if (bytes_of(mid * kRowBlock) <= avail) lo = mid; else hi = mid - 1;
  }
  return lo * kRowBlock;
}

size_t ws_bytes(int which, int B, int T, int H, int V, trl_dtype dt, bool minimum) {
  if (!shapes_ok(B, T, H, V)) return 0;
  if (dt != TRL_F32 && dt != TRL_BF16) return 0;
  const int cap = rows_cap_of(B, T);
  switch (which) {
    case TRL_CALL_TOKEN_LOGPROBS:
      if (dt == TRL_BF16) return fwd_bytes_bf16(B, T, H, V);
      return fwd_bytes_f32(B, T, H, V, minimum ? kRowBlock : (cap < kRecommendedChunkRowsF32 ? cap : kRecommendedChunkRowsF32));
    case TRL_CALL_PG_LOSS_FWD:
      return align_up((size_t)B * pg_loss_tiles(T) * 4 * sizeof(float), 256);
    case TRL_CALL_PG_LOSS_BWD:
      if (dt == TRL_BF16) {
        const int R = minimum ? kRowBlock : (cap < kRecommendedChunkRowsBf16 ? cap : kRecommendedChunkRowsBf16);
        return bwd_fixed_bf16(B, T, H, V) + bwd_per_rows_bf16(H, V, R);
      }
      return bwd_bytes_f32(B, T, H, V, minimum ? kRowBlock : (cap < kRecommendedChunkRowsF32 ? cap : kRecommendedChunkRowsF32));
    case TRL_CALL_PG_STEP_FUSED: {
      if (dt == TRL_BF16) {
        const int R = minimum ? kRowBlock : (cap < kRecommendedChunkRowsBf16 ? cap : kRecommendedChunkRowsBf16);
        // the forward workspace is appended for the lse_hint == NULL case
        return fused_fixed_bf16(B, T, H, V) + fused_per_rows_bf16(H, V, R) + fwd_extra_bf16(B, T, V);
      }
      size_t a = ws_bytes(TRL_CALL_TOKEN_LOGPROBS, B, T, H, V, dt, minimum);
      size_t b = ws_bytes(TRL_CALL_PG_LOSS_BWD, B, T, H, V, dt, minimum);
      size_t c = loss_bytes(B, T);
      return (a > b ? a : b) > c ? (a > b ? a : b) : c;
    }
  }
  return 0;
}

#define TRL_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return TRL_ERR_CUDA; } while (0)

// The gradient GEMMs are issued as several launches whose tiles fill whole waves of CTAs.  Every
// launch starts its CTAs together again: CTAs that move through K in step find the operands their
// neighbours stream in L2, CTAs that have drifted apart fetch them from DRAM a second time.
constexpr int kDwBands = 16;        // launches of the dW GEMM per chunk (rounded to whole waves)

// k-blocks between two points at which the CTAs of the dHidden GEMM wait for one another (its
// tiles run through K = V, thousands of k-blocks, and drift apart otherwise)
constexpr int kPaceEvery = 64;

// dHidden of one chunk: windows of the chunk's (active) row blocks.  `pace` points at zeroed
// counters, one per launch (one per row block of the chunk is always enough).
cudaError_t launch_dh_in_windows(TcGemm dh, unsigned* pace, cudaStream_t s) {
  const int win = tc_wave_aligned_blocks(dh.N);
  dh.pace_ctr = pace; dh.pace_every = kPaceEvery;
  if (win <= 0 || win >= dh.blk_cap) return launch_tc_gemm(dh, s);
  for (int po = 0; po < dh.blk_cap; po += win) {
    dh.pos_off = po; dh.pos_cap = win;
    if (cudaError_t e = launch_tc_gemm(dh, s)) return e;
    if (dh.pace_ctr) ++dh.pace_ctr;
  }
  return cudaSuccess;
}

// dW of one chunk: bands of vocabulary rows.  `dw` describes the whole GEMM (A = E or dS [K, V],
// m_blocks, dW, V for all V rows).
int dw_band_plan(int V, int H, int n_bands_wanted, int32_t* band_begin);
cudaError_t launch_dw_in_bands(TcGemm dw, int V, int H, cudaStream_t s) {
  int32_t begin[kDwBands + 1];
  // no band shorter than four waves of tiles: a small GEMM stays one launch
  const long waves = (long)cdiv(V, 256) * cdiv(H, 256) / tc_num_sms();
  const int wanted = (int)(waves / 4 < kDwBands ? waves / 4 : kDwBands);
  const int nb = wanted >= 2 ? dw_band_plan(V, H, wanted, begin) : 1;
  if (nb <= 1) return launch_tc_gemm(dw, s);
  const __nv_bfloat16* A = (const __nv_bfloat16*)dw.A;
  float* out = dw.dW;
  for (int j = 0; j < nb; ++j) {
    const int v0 = begin[j], vn = begin[j + 1] - v0;
    dw.A = A + v0; dw.a_rows = vn; dw.m_blocks = cdiv(vn, kRowBlock); dw.dW = out + (size_t)v0 * H; dw.V = vn;
    if (cudaError_t e = launch_tc_gemm(dw, s)) return e;
  }
  return cudaSuccess;
}

}  // namespace

extern "C" {

size_t trl_workspace_bytes(int which_call, int B, int T, int H, int V, trl_dtype dt) {
  return ws_bytes(which_call, B, T, H, V, dt, false);
}
size_t trl_workspace_bytes_min(int which_call, int B, int T, int H, int V, trl_dtype dt) {
  return ws_bytes(which_call, B, T, H, V, dt, true);
}

unsigned long long trl_kernel_launches(void) { return launches_so_far(); }

const char* trl_config_string(void) {
  static char buf[160];
  static std::once_flag once;
  std::call_once(once, [] {
    auto band = [](int epi, int own) { const int o = tc_raster_band_override(epi); return o ? o : own; };
    snprintf(buf, sizeof(buf), "cta_group_fwd=%d cta_group_bwd=%d raster_band_lse=%d raster_band_e=%d raster_band_dh=%d raster_band_dw=%d",
             tc_default_cta_group(1), tc_default_cta_group(0), band(TC_EPI_LSE, kRasterBandFwd), band(TC_EPI_E, kRasterBandFwdE),
             band(TC_EPI_DH, kRasterBandBwd), band(TC_EPI_DW, kRasterBandBwd));
  });
  return buf;
}

const char* trl_status_string(int status) {
  switch (status) {
    case TRL_OK: return "ok";
    case TRL_ERR_INVALID_ARG: return "invalid argument";
    case TRL_ERR_SHAPE: return "invalid shape";
    case TRL_ERR_DTYPE: return "unsupported dtype";
    case TRL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case TRL_ERR_ARCH: return "device is not sm_100";
    case TRL_ERR_CUDA: return "CUDA error";
    case TRL_ERR_BAD_INDEX: return "index out of range (device)";
    case TRL_ERR_TIMEOUT: return "pipeline wait timed out (device)";
    case TRL_ERR_BAD_HINT: return "lse_hint out of range (device)";
    case TRL_ERR_ROWS_BOUND: return "more valid rows than rows_bound (device)";
    case TRL_ERR_BOUNDS: return "store index outside its buffer (device, debug build)";
  }
  return "unknown status";
}

int trl_token_logprobs(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                       int B, int T, int H, int V, trl_dtype dt, float* logp, float* lse,
                       void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (!hidden || !W || !ids || !len || !logp || !lse || !workspace) return TRL_ERR_INVALID_ARG;
  if (dt != TRL_F32 && dt != TRL_BF16) return TRL_ERR_DTYPE;
  if (!shapes_ok(B, T, H, V)) return TRL_ERR_SHAPE;
  if (dt == TRL_BF16 && ((H % 8) || (V % 8))) return TRL_ERR_SHAPE;
  if (((uintptr_t)workspace & 255) != 0) return TRL_ERR_INVALID_ARG;
  if (!al16(hidden) || !al16(W) || !al16(ids) || !al4(len) || !al16(logp) || !al16(lse) || (status_dev && !al4(status_dev)))
    return TRL_ERR_INVALID_ARG;
  if (workspace_bytes < trl_workspace_bytes_min(TRL_CALL_TOKEN_LOGPROBS, B, T, H, V, dt)) return TRL_ERR_WORKSPACE_TOO_SMALL;
  if (int e = check_device()) return e;
  cudaStream_t s = (cudaStream_t)stream;
  const int cap_rows = rows_cap_of(B, T);

  Carver cv(workspace);
  RowPack rb = carve_row_pack(cv.take<char>(row_pack_bytes(B, T)), B, T);
  launch_build_row_pack(len, B, T, rb, status_dev, s);

  if (dt == TRL_BF16) {
    const int nt = cdiv(V, 256);
    __nv_bfloat16* Xp = cv.take<__nv_bfloat16>((size_t)cap_rows * H);
    float* tgt = cv.take<float>(cap_rows);
    float2* partials = cv.take<float2>((size_t)nt * cap_rows);
    launch_pack_rows_bf16((const __nv_bfloat16*)hidden, Xp, H, cap_rows, rb, 0, 0, nullptr, s);
    TcGemm g;
    memset(&g, 0, sizeof(g));
    g.epi = TC_EPI_LSE;
    g.A = Xp; g.a_rows = cap_rows; g.a_ld = H;
    g.B = W; g.b_rows = V; g.b_ld = H;
    g.K = H; g.N = V;
    g.rb = rb; g.blk_off = 0; g.blk_cap = rb.cap; g.raster_band_blocks = kRasterBandFwd;
    g.ids = ids; g.partials = partials; g.tgt = tgt; g.rows_cap = cap_rows; g.status = status_dev;
    TRL_CUDA_OK(launch_tc_gemm(g, s));
    launch_merge_lse(partials, tgt, nt, cap_rows, rb, ids, len, B, T, V, logp, lse, status_dev, s);
  } else {
    const size_t avail = workspace_bytes - row_pack_bytes(B, T);
    const int R = fit_rows(avail, cap_rows < kRecommendedChunkRowsF32 ? cap_rows : kRecommendedChunkRowsF32,
                           [&](int r) { return align_up((size_t)r * H * 4, 256) + align_up((size_t)r * V * 4, 256); });
    if (R < kRowBlock) return TRL_ERR_WORKSPACE_TOO_SMALL;
    float* Xp = cv.take<float>((size_t)R * H);
    float* S = cv.take<float>((size_t)R * V);
    const int CB = R / kRowBlock;
    launch_zero_padded_f32(logp, lse, len, B, T, s);
    for (int blk_off = 0; blk_off < rb.cap; blk_off += CB) {
      launch_pack_rows_f32((const float*)hidden, Xp, H, R, rb, blk_off, s);
      SimtGemm sg{Xp, H, 1, (const float*)W, 1, H, S, V, R, V, H, 0, 1, rb.nblk, blk_off, CB};
      launch_simt_gemm(sg, s);
      launch_row_lse_f32(S, V, R, rb, blk_off, ids, logp, lse, status_dev, s);
    }
  }
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}

int trl_hrd_advantages(const float* r_plan, const float* r_code, const int32_t* len, const int32_t* bnd,
                       int P, int G, int T, int adv_mode, float* A_plan, float* A_code, uint8_t* seg, float* adv,
                       int32_t* n_plan, int32_t* n_code, int64_t* n_valid, int32_t* status_dev, void* stream) {
  if (!r_plan || !r_code || !len || !bnd || !A_plan || !A_code || !seg || !adv || !n_plan || !n_code || !n_valid)
    return TRL_ERR_INVALID_ARG;
  if (P <= 0 || G <= 0 || T <= 0 || (long)P * G > 65535 || (long)P * G * T >= (1L << 31)) return TRL_ERR_SHAPE;
  if (adv_mode != 0 && adv_mode != 1) return TRL_ERR_INVALID_ARG;
  if (!al4(r_plan) || !al4(r_code) || !al4(len) || !al4(bnd) || !al4(A_plan) || !al4(A_code) || !al16(seg) || !al16(adv) ||
      !al4(n_plan) || !al4(n_code) || !al8(n_valid) || (status_dev && !al4(status_dev)))
    return TRL_ERR_INVALID_ARG;
  if (int e = check_device()) return e;
  launch_hrd_advantages(r_plan, r_code, len, bnd, P, G, T, adv_mode, A_plan, A_code, seg, adv, n_plan, n_code,
                        n_valid, status_dev, (cudaStream_t)stream);
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}

int trl_pg_loss_fwd(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                    const int32_t* len, int P, int G, int T, trl_pg_config cfg, float* loss, float* g, float* stats,
                    void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  (void)status_dev;
  if (!logp || !old_logp || !adv || !seg || !len || !loss || !g || !workspace) return TRL_ERR_INVALID_ARG;
  if (P <= 0 || G <= 0 || T <= 0 || (long)P * G > 65535 || (long)P * G * T >= (1L << 31)) return TRL_ERR_SHAPE;
  if (!(cfg.eps_lo >= 0.f) || !(cfg.eps_hi >= 0.f) || !(cfg.alpha >= 0.f) || (cfg.clip_form & ~1) || (cfg.agg_mode & ~1))
    return TRL_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) != 0) return TRL_ERR_INVALID_ARG;
  if (!al16(logp) || !al16(old_logp) || !al16(adv) || !al16(seg) || !al16(g) || !al4(len) || !al4(loss) || (stats && !al4(stats)))
    return TRL_ERR_INVALID_ARG;
  if (workspace_bytes < trl_workspace_bytes(TRL_CALL_PG_LOSS_FWD, P * G, T, 1, 1, TRL_F32)) return TRL_ERR_WORKSPACE_TOO_SMALL;
  if (int e = check_device()) return e;
  launch_pg_loss(logp, old_logp, adv, seg, len, P, G, T, cfg, loss, g, stats, (float*)workspace, nullptr, 0,
                 (cudaStream_t)stream);
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}

int trl_pg_loss_bwd(const void* hidden, const void* W, const int32_t* ids, const int32_t* len, const float* lse,
                    const float* g, int B, int T, int H, int V, trl_dtype dt, void* dHidden, float* dW,
                    void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (!hidden || !W || !ids || !len || !lse || !g || !dHidden || !dW || !workspace) return TRL_ERR_INVALID_ARG;
  if (dt != TRL_F32 && dt != TRL_BF16) return TRL_ERR_DTYPE;
  if (!shapes_ok(B, T, H, V)) return TRL_ERR_SHAPE;
  if (dt == TRL_BF16 && ((H % 8) || (V % 8))) return TRL_ERR_SHAPE;
  if (((uintptr_t)workspace & 255) != 0) return TRL_ERR_INVALID_ARG;
  if (!al16(hidden) || !al16(W) || !al16(dHidden) || !al16(dW) || !al16(ids) || !al4(len) || !al16(lse) || !al16(g) ||
      (status_dev && !al4(status_dev)))
    return TRL_ERR_INVALID_ARG;
  if (workspace_bytes < trl_workspace_bytes_min(TRL_CALL_PG_LOSS_BWD, B, T, H, V, dt)) return TRL_ERR_WORKSPACE_TOO_SMALL;
  if (int e = check_device()) return e;
  cudaStream_t s = (cudaStream_t)stream;
  const int cap_rows = rows_cap_of(B, T);
  const size_t N = (size_t)B * T;
  // rows per chunk that the workspace allows; decided before anything is enqueued
  int R = 0;
  if (dt == TRL_BF16) {
    R = fit_rows(workspace_bytes - bwd_fixed_bf16(B, T, H, V), cap_rows < kRecommendedChunkRowsBf16 ? cap_rows : kRecommendedChunkRowsBf16,
                 [&](int r) { return bwd_per_rows_bf16(H, V, r); });
  } else {
    R = fit_rows(workspace_bytes - row_pack_bytes(B, T), cap_rows < kRecommendedChunkRowsF32 ? cap_rows : kRecommendedChunkRowsF32,
                 [&](int r) { return 2 * align_up((size_t)r * H * 4, 256) + align_up((size_t)r * V * 4, 256); });
  }
  if (R < kRowBlock) return TRL_ERR_WORKSPACE_TOO_SMALL;

  Carver cv(workspace);
  RowPack rb = carve_row_pack(cv.take<char>(row_pack_bytes(B, T)), B, T);
  launch_build_row_pack(len, B, T, rb, status_dev, s);
  TRL_CUDA_OK(cudaMemsetAsync(dW, 0, (size_t)V * H * sizeof(float), s));

  if (dt == TRL_BF16) {
    TRL_CUDA_OK(cudaMemsetAsync(dHidden, 0, N * H * 2, s));
    __nv_bfloat16* Xp = cv.take<__nv_bfloat16>((size_t)cap_rows * H);
    int* blk_active = cv.take<int>(rb.cap);
    unsigned* pace = cv.take<unsigned>(rb.cap);
    TRL_CUDA_OK(cudaMemsetAsync(pace, 0, (size_t)rb.cap * sizeof(unsigned), s));
    __nv_bfloat16* dS = cv.take<__nv_bfloat16>((size_t)R * V);
    launch_pack_rows_bf16((const __nv_bfloat16*)hidden, Xp, H, cap_rows, rb, 0, 0, nullptr, s);
    launch_flag_active_blocks(g, rb, blk_active, s);     // row blocks with g == 0 everywhere are skipped below
    const int CB = R / kRowBlock;
    for (int blk_off = 0; blk_off < rb.cap; blk_off += CB) {
      TcGemm a;
      memset(&a, 0, sizeof(a));
      a.rb = rb; a.blk_off = blk_off; a.blk_cap = CB; a.status = status_dev; a.blk_active = blk_active + blk_off;
      // dS chunk = g (onehot - softmax), from a recomputed logits tile
      TcGemm ds = a;
      ds.epi = TC_EPI_DS; ds.raster_band_blocks = kRasterBandFwdE;
      ds.A = Xp; ds.a_rows = cap_rows; ds.a_ld = H; ds.B = W; ds.b_rows = V; ds.b_ld = H; ds.K = H; ds.N = V;
      ds.ids = ids; ds.lse = lse; ds.g = g; ds.dS = dS; ds.ds_ld = V;
      TRL_CUDA_OK(launch_tc_gemm(ds, s));
      // dHidden rows of the chunk = dS W   (W read as an N-contiguous operand)
      TcGemm dh = a;
      dh.epi = TC_EPI_DH; dh.raster_band_blocks = kRasterBandBwd;
      dh.A = dS; dh.a_rows = R; dh.a_ld = V; dh.B = W; dh.b_rows = H; dh.b_ld = H; dh.K = V; dh.N = H;
      dh.dHidden = (__nv_bfloat16*)dHidden; dh.dh_ld = H; dh.dh_rows = (long)N;
      TRL_CUDA_OK(launch_dh_in_windows(dh, pace + blk_off, s));
      // dW += dS^T hidden   (both operands M/N-contiguous: dS [R,V] and the chunk's packed rows [.,H])
      TcGemm dw = a;
      dw.epi = TC_EPI_DW; dw.raster_band_blocks = kRasterBandBwd;
      dw.A = dS; dw.a_rows = V; dw.a_ld = V; dw.K = R; dw.N = H;
      dw.B = Xp + (size_t)blk_off * kRowBlock * H; dw.b_rows = H; dw.b_ld = H;
      dw.b_k = cap_rows - blk_off * kRowBlock < R ? cap_rows - blk_off * kRowBlock : R;
      dw.m_blocks = cdiv(V, kRowBlock); dw.dW = dW; dw.dw_ld = H; dw.V = V;
      TRL_CUDA_OK(launch_dw_in_bands(dw, V, H, s));
    }
  } else {
    TRL_CUDA_OK(cudaMemsetAsync(dHidden, 0, N * H * 4, s));
    float* Xp = cv.take<float>((size_t)R * H);
    float* dHp = cv.take<float>((size_t)R * H);
    float* S = cv.take<float>((size_t)R * V);
    const int CB = R / kRowBlock;
    for (int blk_off = 0; blk_off < rb.cap; blk_off += CB) {
      launch_pack_rows_f32((const float*)hidden, Xp, H, R, rb, blk_off, s);
      SimtGemm fwd{Xp, H, 1, (const float*)W, 1, H, S, V, R, V, H, 0, 1, rb.nblk, blk_off, CB};
      launch_simt_gemm(fwd, s);
      launch_ds_inplace_f32(S, V, R, rb, blk_off, ids, lse, g, s);
      SimtGemm dh{S, V, 1, (const float*)W, H, 1, dHp, H, R, H, V, 0, 1, rb.nblk, blk_off, CB};
      launch_simt_gemm(dh, s);
      launch_scatter_rows_f32(dHp, (float*)dHidden, H, R, rb, blk_off, s);
      SimtGemm dw{S, 1, V, Xp, H, 1, dW, H, V, H, R, 1, 2, rb.nblk, blk_off, CB};
      launch_simt_gemm(dw, s);
    }
  }
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}


}  // extern "C"

namespace {

struct DwBands {            // dW finished band by band (host arrays)
  int n; const int32_t* begin; void* const* events; int rows_bound;
};

int fused_banded(const void* hidden, const void* W, const int32_t* ids, const int32_t* len, const float* old_logp,
                 const float* lse_hint, const float* adv, const uint8_t* seg, int P, int G, int T, int H, int V,
                 trl_pg_config cfg, float* logp, float* lse, float* loss, float* g, float* stats, void* dHidden, float* dW,
                 void* workspace, size_t workspace_bytes, int32_t* status_dev, cudaStream_t s, const DwBands& bands);

int fused_impl(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
               const float* old_logp, const float* lse_hint, const float* adv, const uint8_t* seg,
               int P, int G, int T, int H, int V, trl_dtype dt, trl_pg_config cfg,
               float* logp, float* lse, float* loss, float* g, float* stats, void* dHidden, float* dW,
               void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream, const DwBands* bands) {
  if (!hidden || !W || !ids || !len || !old_logp || !adv || !seg || !logp || !lse || !loss || !g || !dHidden || !dW ||
      !workspace)
    return TRL_ERR_INVALID_ARG;
  if (dt != TRL_F32 && dt != TRL_BF16) return TRL_ERR_DTYPE;
  if (P <= 0 || G <= 0 || (long)P * G > 65535) return TRL_ERR_SHAPE;
  const int B = P * G;
  if (!shapes_ok(B, T, H, V)) return TRL_ERR_SHAPE;
  if (dt == TRL_BF16 && ((H % 8) || (V % 8))) return TRL_ERR_SHAPE;
  if (!(cfg.eps_lo >= 0.f) || !(cfg.eps_hi >= 0.f) || !(cfg.alpha >= 0.f) || (cfg.clip_form & ~1) || (cfg.agg_mode & ~1))
    return TRL_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) != 0) return TRL_ERR_INVALID_ARG;
  if (!al16(hidden) || !al16(W) || !al16(dHidden) || !al16(dW) || !al16(ids) || !al4(len) || !al16(old_logp) || !al16(adv) ||
      !al16(seg) || !al16(logp) || !al16(lse) || !al16(g) || !al4(loss) || (lse_hint && !al16(lse_hint)) || (stats && !al4(stats)) ||
      (status_dev && !al4(status_dev)))
    return TRL_ERR_INVALID_ARG;
  if (bands) {
    if (dt != TRL_BF16) return TRL_ERR_DTYPE;
    if (bands->n < 1 || !bands->begin || bands->begin[0] != 0 || bands->begin[bands->n] != V) return TRL_ERR_INVALID_ARG;
    for (int j = 0; j < bands->n; ++j)      // bands are whole 256-row tiles of dW, in order
      if (bands->begin[j + 1] <= bands->begin[j] || (bands->begin[j] % 256) != 0) return TRL_ERR_INVALID_ARG;
    if (workspace_bytes < fused_banded_bytes(B, T, H, V, bands->rows_bound, lse_hint == nullptr)) return TRL_ERR_WORKSPACE_TOO_SMALL;
    if (int e = check_device()) return e;
    return fused_banded(hidden, W, ids, len, old_logp, lse_hint, adv, seg, P, G, T, H, V, cfg, logp, lse, loss, g, stats,
                        dHidden, dW, workspace, workspace_bytes, status_dev, (cudaStream_t)stream, *bands);
  }
  if (workspace_bytes < trl_workspace_bytes_min(TRL_CALL_PG_STEP_FUSED, B, T, H, V, dt)) return TRL_ERR_WORKSPACE_TOO_SMALL;
  if (int e = check_device()) return e;

  if (dt == TRL_F32) {   // the fp32 path has no fused schedule: run the three calls in order
    if (int e = trl_token_logprobs(hidden, W, ids, len, B, T, H, V, dt, logp, lse, workspace, workspace_bytes, status_dev, stream)) return e;
    if (int e = trl_pg_loss_fwd(logp, old_logp, adv, seg, len, P, G, T, cfg, loss, g, stats, workspace, workspace_bytes, status_dev, stream)) return e;
    return trl_pg_loss_bwd(hidden, W, ids, len, lse, g, B, T, H, V, dt, dHidden, dW, workspace, workspace_bytes, status_dev, stream);
  }

  cudaStream_t s = (cudaStream_t)stream;
  const int cap_rows = rows_cap_of(B, T);
  const size_t N = (size_t)B * T;
  const int nt = cdiv(V, 256);
  const size_t fwd_extra = lse_hint ? 0 : fwd_extra_bf16(B, T, V);
  if (workspace_bytes < fused_fixed_bf16(B, T, H, V) + fwd_extra + fused_per_rows_bf16(H, V, kRowBlock))
    return TRL_ERR_WORKSPACE_TOO_SMALL;
  const size_t avail = workspace_bytes - fused_fixed_bf16(B, T, H, V) - fwd_extra;
  const int R = fit_rows(avail, cap_rows < kRecommendedChunkRowsBf16 ? cap_rows : kRecommendedChunkRowsBf16,
                         [&](int r) { return fused_per_rows_bf16(H, V, r); });
  if (R < kRowBlock) return TRL_ERR_WORKSPACE_TOO_SMALL;

  Carver cv(workspace);
  RowPack rb = carve_row_pack(cv.take<char>(row_pack_bytes(B, T)), B, T);
  __nv_bfloat16* Xp = cv.take<__nv_bfloat16>((size_t)cap_rows * H);
  cv.take<int>(rb.cap);                              // (the four-call backward keeps its activity flags here)
  unsigned* pace = cv.take<unsigned>(rb.cap);
  float* loss_partials = cv.take<float>((size_t)B * pg_loss_tiles(T) * 4);
  __nv_bfloat16* Xs = cv.take<__nv_bfloat16>((size_t)H * R);
  __nv_bfloat16* E = cv.take<__nv_bfloat16>((size_t)R * V);
  float* psum = cv.take<float>((size_t)nt * R);
  float* tgt = cv.take<float>(R);
  float* neg_alpha = cv.take<float>(R);
  int* blk_active = cv.take<int>(R / kRowBlock);

  launch_build_row_pack(len, B, T, rb, status_dev, s);
  TRL_CUDA_OK(cudaMemsetAsync(dW, 0, (size_t)V * H * sizeof(float), s));
  TRL_CUDA_OK(cudaMemsetAsync(dHidden, 0, N * H * 2, s));
  TRL_CUDA_OK(cudaMemsetAsync(pace, 0, (size_t)rb.cap * sizeof(unsigned), s));
  launch_zero_padded_f32(logp, lse, len, B, T, s);
  launch_pack_rows_bf16((const __nv_bfloat16*)hidden, Xp, H, cap_rows, rb, 0, 0, nullptr, s);

  TcGemm base;
  memset(&base, 0, sizeof(base));
  base.rb = rb; base.status = status_dev;

  const float* hint = lse_hint;
  if (!hint) {   // exact log-partition first; it then serves as the shift, so E is the softmax itself
    float* tgt_all = cv.take<float>(cap_rows);
    float2* partials = cv.take<float2>((size_t)nt * cap_rows);
    TcGemm f = base;
    f.epi = TC_EPI_LSE; f.raster_band_blocks = kRasterBandFwd;
    f.A = Xp; f.a_rows = cap_rows; f.a_ld = H; f.B = W; f.b_rows = V; f.b_ld = H; f.K = H; f.N = V;
    f.blk_off = 0; f.blk_cap = rb.cap; f.ids = ids; f.partials = partials; f.tgt = tgt_all; f.rows_cap = cap_rows;
    TRL_CUDA_OK(launch_tc_gemm(f, s));
    launch_merge_lse(partials, tgt_all, nt, cap_rows, rb, ids, len, B, T, V, logp, lse, status_dev, s);
    hint = lse;
  }

  const int CB = R / kRowBlock;
  for (int blk_off = 0; blk_off < rb.cap; blk_off += CB) {
    TcGemm a = base;
    a.blk_off = blk_off; a.blk_cap = CB;
    // forward tile -> E = exp(z - c), row sums, sampled token's logit
    TcGemm e = a;
    e.epi = TC_EPI_E; e.raster_band_blocks = kRasterBandFwdE;
    e.A = Xp; e.a_rows = cap_rows; e.a_ld = H; e.B = W; e.b_rows = V; e.b_ld = H; e.K = H; e.N = V;
    e.ids = ids; e.lse = hint; e.dS = E; e.ds_ld = V; e.psum = psum; e.tgt = tgt; e.rows_cap = R;
    TRL_CUDA_OK(launch_tc_gemm(e, s));
    FusedMergeArgs m{psum, tgt, nt, R, rb, blk_off, ids, len, hint, old_logp, adv, seg, P, G, T, V, cfg,
                     logp, lse, g, neg_alpha, blk_active, E, status_dev};
    launch_fused_merge(m, s);
    launch_pack_rows_bf16(Xp, Xs, H, R, rb, blk_off * kRowBlock, 1, neg_alpha, s);
    // dHidden rows = neg_alpha * (E' W)
    TcGemm dh = a;
    dh.epi = TC_EPI_DH; dh.raster_band_blocks = kRasterBandBwd;
    dh.A = E; dh.a_rows = R; dh.a_ld = V; dh.B = W; dh.b_rows = H; dh.b_ld = H; dh.K = V; dh.N = H;
    dh.dHidden = (__nv_bfloat16*)dHidden; dh.dh_ld = H; dh.dh_rows = (long)N; dh.row_scale = neg_alpha; dh.blk_active = blk_active;
    TRL_CUDA_OK(launch_dh_in_windows(dh, pace + blk_off, s));
    // dW += E'^T (neg_alpha * hidden)
    TcGemm dw = a;
    dw.epi = TC_EPI_DW; dw.raster_band_blocks = kRasterBandBwd;
    dw.A = E; dw.a_rows = V; dw.a_ld = V; dw.B = Xs; dw.b_rows = H; dw.b_ld = H; dw.K = R; dw.N = H;
    dw.m_blocks = cdiv(V, kRowBlock); dw.dW = dW; dw.dw_ld = H; dw.V = V; dw.blk_active = blk_active;
    TRL_CUDA_OK(launch_dw_in_bands(dw, V, H, s));
  }
  // loss, statistics (and g once more, identically) over all rows now that logp is complete; rows
  // whose token id is out of range stay out of it, as they stayed out of the gradients
  launch_pg_loss(logp, old_logp, adv, seg, len, P, G, T, cfg, loss, g, stats, loss_partials, ids, V, s);
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}

// The same step with E kept for all rows, so that the dW GEMM can run vocabulary band by vocabulary
// band over all row chunks: a band of dW is final as soon as its launches are done, and an event
// recorded there lets the caller start reducing it across ranks while later bands are computed.
// Every 256-row tile of dW receives the same per-chunk contributions in the same order as in the
// chunk-by-chunk schedule above, so the results are bit-identical to it.
int fused_banded(const void* hidden, const void* W, const int32_t* ids, const int32_t* len, const float* old_logp,
                 const float* lse_hint, const float* adv, const uint8_t* seg, int P, int G, int T, int H, int V,
                 trl_pg_config cfg, float* logp, float* lse, float* loss, float* g, float* stats, void* dHidden, float* dW,
                 void* workspace, size_t workspace_bytes, int32_t* status_dev, cudaStream_t s, const DwBands& bands) {
  (void)workspace_bytes;
  const int B = P * G;
  const int cap_rows = rows_cap_of(B, T);
  const size_t N = (size_t)B * T;
  const int nt = cdiv(V, 256);
  const int RB = banded_rows(B, T, bands.rows_bound);
  const int Rc = RB < kRecommendedChunkRowsBf16 ? RB : kRecommendedChunkRowsBf16;

  Carver cv(workspace);
  RowPack rb = carve_row_pack(cv.take<char>(row_pack_bytes(B, T)), B, T);
  __nv_bfloat16* Xp = cv.take<__nv_bfloat16>((size_t)cap_rows * H);
  cv.take<int>(rb.cap);                                // keeps the fixed part laid out as fused_fixed_bf16 counts it
  unsigned* pace = cv.take<unsigned>(rb.cap);
  float* loss_partials = cv.take<float>((size_t)B * pg_loss_tiles(T) * 4);
  __nv_bfloat16* Xs = cv.take<__nv_bfloat16>((size_t)RB * H);
  __nv_bfloat16* E = cv.take<__nv_bfloat16>((size_t)RB * V);
  float* psum = cv.take<float>((size_t)nt * Rc);
  float* tgt = cv.take<float>(Rc);
  float* neg_alpha = cv.take<float>(RB);
  int* blk_active = cv.take<int>(RB / kRowBlock);

  launch_build_row_pack(len, B, T, rb, status_dev, s);
  launch_clamp_rows(rb, RB, status_dev, s);            // more valid rows than the caller's bound: flagged, the excess is dropped
  TRL_CUDA_OK(cudaMemsetAsync(pace, 0, (size_t)rb.cap * sizeof(unsigned), s));
  TRL_CUDA_OK(cudaMemsetAsync(dW, 0, (size_t)V * H * sizeof(float), s));
  TRL_CUDA_OK(cudaMemsetAsync(dHidden, 0, N * H * 2, s));
  launch_zero_padded_f32(logp, lse, len, B, T, s);
  launch_pack_rows_bf16((const __nv_bfloat16*)hidden, Xp, H, cap_rows, rb, 0, 0, nullptr, s);

  TcGemm base;
  memset(&base, 0, sizeof(base));
  base.rb = rb; base.status = status_dev;

  const float* hint = lse_hint;
  if (!hint) {
    float* tgt_all = cv.take<float>(cap_rows);
    float2* partials = cv.take<float2>((size_t)nt * cap_rows);
    TcGemm f = base;
    f.epi = TC_EPI_LSE; f.raster_band_blocks = kRasterBandFwd;
    f.A = Xp; f.a_rows = cap_rows; f.a_ld = H; f.B = W; f.b_rows = V; f.b_ld = H; f.K = H; f.N = V;
    f.blk_off = 0; f.blk_cap = rb.cap; f.ids = ids; f.partials = partials; f.tgt = tgt_all; f.rows_cap = cap_rows;
    TRL_CUDA_OK(launch_tc_gemm(f, s));
    launch_merge_lse(partials, tgt_all, nt, cap_rows, rb, ids, len, B, T, V, logp, lse, status_dev, s);
    hint = lse;
  }

  const int CB = Rc / kRowBlock, NB = RB / kRowBlock;
  for (int blk_off = 0; blk_off < NB; blk_off += CB) {
    const int cb = NB - blk_off < CB ? NB - blk_off : CB;          // blocks of this chunk
    __nv_bfloat16* Ec = E + (size_t)blk_off * kRowBlock * V;
    TcGemm a = base;
    a.blk_off = blk_off; a.blk_cap = cb;
    TcGemm e = a;
    e.epi = TC_EPI_E; e.raster_band_blocks = kRasterBandFwdE;
    e.A = Xp; e.a_rows = cap_rows; e.a_ld = H; e.B = W; e.b_rows = V; e.b_ld = H; e.K = H; e.N = V;
    e.ids = ids; e.lse = hint; e.dS = Ec; e.ds_ld = V; e.psum = psum; e.tgt = tgt; e.rows_cap = Rc;
    TRL_CUDA_OK(launch_tc_gemm(e, s));
    FusedMergeArgs m{psum, tgt, nt, Rc, rb, blk_off, ids, len, hint, old_logp, adv, seg, P, G, T, V, cfg,
                     logp, lse, g, neg_alpha + (size_t)blk_off * kRowBlock, blk_active + blk_off, Ec, status_dev};
    m.R_live = cb * kRowBlock;
    launch_fused_merge(m, s);
    launch_pack_rows_bf16(Xp, Xs + (size_t)blk_off * kRowBlock * H, H, cb * kRowBlock, rb, blk_off * kRowBlock, 1,
                          neg_alpha + (size_t)blk_off * kRowBlock, s);
    TcGemm dh = a;
    dh.epi = TC_EPI_DH; dh.raster_band_blocks = kRasterBandBwd;
    dh.A = Ec; dh.a_rows = cb * kRowBlock; dh.a_ld = V; dh.B = W; dh.b_rows = H; dh.b_ld = H; dh.K = V; dh.N = H;
    dh.dHidden = (__nv_bfloat16*)dHidden; dh.dh_ld = H; dh.dh_rows = (long)N; dh.row_scale = neg_alpha + (size_t)blk_off * kRowBlock;
    dh.blk_active = blk_active + blk_off;
    TRL_CUDA_OK(launch_dh_in_windows(dh, pace + blk_off, s));
  }
  for (int j = 0; j < bands.n; ++j) {
    const int v0 = bands.begin[j], vn = bands.begin[j + 1] - v0;
    for (int blk_off = 0; blk_off < NB; blk_off += CB) {
      const int cb = NB - blk_off < CB ? NB - blk_off : CB;
      TcGemm dw = base;
      dw.blk_off = blk_off; dw.blk_cap = cb;
      dw.epi = TC_EPI_DW; dw.raster_band_blocks = kRasterBandBwd;
      dw.A = E + (size_t)blk_off * kRowBlock * V + v0; dw.a_rows = vn; dw.a_ld = V;
      dw.B = Xs + (size_t)blk_off * kRowBlock * H; dw.b_rows = H; dw.b_ld = H; dw.K = cb * kRowBlock; dw.N = H;
      dw.m_blocks = cdiv(vn, kRowBlock); dw.dW = dW + (size_t)v0 * H; dw.dw_ld = H; dw.V = vn;
      dw.blk_active = blk_active + blk_off;
      TRL_CUDA_OK(launch_tc_gemm(dw, s));
    }
    if (bands.events && bands.events[j]) TRL_CUDA_OK(cudaEventRecord((cudaEvent_t)bands.events[j], s));
  }
  launch_pg_loss(logp, old_logp, adv, seg, len, P, G, T, cfg, loss, g, stats, loss_partials, ids, V, s);
  TRL_CUDA_OK(cudaGetLastError());
  return TRL_OK;
}

}  // namespace

extern "C" {

int trl_pg_step_fused(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                      const float* old_logp, const float* lse_hint, const float* adv, const uint8_t* seg,
                      int P, int G, int T, int H, int V, trl_dtype dt, trl_pg_config cfg,
                      float* logp, float* lse, float* loss, float* g, float* stats, void* dHidden, float* dW,
                      void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  return fused_impl(hidden, W, ids, len, old_logp, lse_hint, adv, seg, P, G, T, H, V, dt, cfg, logp, lse, loss, g, stats,
                    dHidden, dW, workspace, workspace_bytes, status_dev, stream, nullptr);
}

int trl_pg_step_fused_banded(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                             const float* old_logp, const float* lse_hint, const float* adv, const uint8_t* seg,
                             int P, int G, int T, int H, int V, trl_dtype dt, trl_pg_config cfg,
                             float* logp, float* lse, float* loss, float* g, float* stats, void* dHidden, float* dW,
                             int n_bands, const int32_t* band_begin, void* const* band_events, int rows_bound,
                             void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  DwBands b{n_bands, band_begin, band_events, rows_bound};
  return fused_impl(hidden, W, ids, len, old_logp, lse_hint, adv, seg, P, G, T, H, V, dt, cfg, logp, lse, loss, g, stats,
                    dHidden, dW, workspace, workspace_bytes, status_dev, stream, &b);
}

size_t trl_pg_step_fused_banded_workspace_bytes(int B, int T, int H, int V, int rows_bound) {
  if (!shapes_ok(B, T, H, V)) return 0;
  return fused_banded_bytes(B, T, H, V, rows_bound, true);
}

int trl_dw_band_plan(int V, int H, int n_bands_wanted, int32_t* band_begin) {
  return dw_band_plan(V, H, n_bands_wanted, band_begin);
}

}  // extern "C"

namespace {

int dw_band_plan(int V, int H, int n_bands_wanted, int32_t* band_begin) {
  if (V <= 0 || H <= 0 || n_bands_wanted < 1 || !band_begin) return 0;
  // Whole 256-row tiles of dW per band, as equal as possible.  A band's launch has (tiles of the
  // band) x (tiles along H) CTA tiles; the tile count per band is rounded up to the smallest count
  // that fills whole waves of a B200's 148 CTAs, so that no band ends in a nearly empty wave.
  const int m_tiles = cdiv(V, 256), n_tiles = cdiv(H, 256);
  int a = 148, b = n_tiles;
  while (b) { const int t = a % b; a = b; b = t; }        // a = gcd(148, n_tiles)
  const int q = 148 / a;
  int per = cdiv(m_tiles, n_bands_wanted);
  if (per > q) per = ((per + q / 2) / q) * q;             // nearest multiple of q
  int n;
  for (;;) {
    n = cdiv(m_tiles, per);
    if (n > 1 && (m_tiles - (n - 1) * per) * 4 < per) --n;  // a short last band joins the one before it
    if (n <= n_bands_wanted) break;
    per += (per >= q) ? q : 1;
  }
  for (int j = 0; j < n; ++j) band_begin[j] = j * per * 256;
  band_begin[n] = V;
  return n;
}

}  // namespace
