// Memory-bound kernels of the HRD policy-gradient path: row-block construction, HRD
// advantages (Section 2.3, Eq. 2), the clipped surrogate and its derivative, the merge of
// per-vocabulary-tile log-sum-exp partials, and layout helpers.
#include <atomic>

#include "trl_internal.h"

namespace trl {

static std::atomic<unsigned long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

__device__ __forceinline__ void flag_status(int32_t* status, int code) {
  if (status) atomicOr(status, 1 << code);
}

size_t row_pack_bytes(int B, int T) {
  const size_t cap_rows = (size_t)cdiv(B * T, kRowBlock) * kRowBlock;
  return align_up((2 + (size_t)B + 1 + cap_rows) * sizeof(int), 256);
}

RowPack carve_row_pack(void* base, int B, int T) {
  RowPack rb;
  int* p = (int*)base;
  rb.cap = cdiv(B * T, kRowBlock);
  rb.n_total = (long)B * T;
  rb.nblk = p;
  rb.n_rows = p + 1;
  rb.row_first = p + 2;
  rb.rowmap = p + 2 + (B + 1);
  return rb;
}

__device__ __forceinline__ long packed_to_global(const RowPack& rb, int q) {
  return q < rb.n_rows[0] ? (long)rb.rowmap[q] : -1;
}

// One CTA: exclusive prefix sum of the (clamped) lengths.
__global__ void build_row_pack_kernel(const int32_t* __restrict__ len, int B, int T, RowPack rb, int32_t* status) {
  __shared__ int s_sum[1024];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int per = (B + nt - 1) / nt;
  const int b0 = min(tid * per, B), b1 = min(b0 + per, B);
  int cnt = 0;
  bool bad = false;
  for (int b = b0; b < b1; ++b) {
    int L = len[b];
    if (L < 0 || L > T) { bad = true; L = max(0, min(L, T)); }
    cnt += L;
  }
  if (bad) flag_status(status, TRL_ERR_BAD_INDEX);
  s_sum[tid] = cnt;
  __syncthreads();
  for (int off = 1; off < nt; off <<= 1) {      // inclusive Hillis-Steele scan
    int v = (tid >= off) ? s_sum[tid - off] : 0;
    __syncthreads();
    s_sum[tid] += v;
    __syncthreads();
  }
  int first = s_sum[tid] - cnt;
  if (tid == nt - 1) {
    rb.n_rows[0] = s_sum[tid];
    rb.nblk[0] = (s_sum[tid] + kRowBlock - 1) / kRowBlock;
    rb.row_first[B] = s_sum[tid];
  }
  for (int b = b0; b < b1; ++b) {
    rb.row_first[b] = first;
    first += max(0, min(len[b], T));
  }
}

__global__ void __launch_bounds__(256) fill_rowmap_kernel(const int32_t* __restrict__ len, int B, int T, RowPack rb,
                                                          int32_t* status) {
  const size_t n = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (n >= (size_t)B * T) return;
  const int b = (int)(n / T), t = (int)(n % T);
  if (t < max(0, min(len[b], T))) {
    const long q = (long)rb.row_first[b] + t;
    if (TRL_IN_BOUNDS(q, (long)rb.cap * kRowBlock, status)) rb.rowmap[q] = (int)n;
  }
}

void launch_build_row_pack(const int32_t* len, int B, int T, RowPack rb, int32_t* status, cudaStream_t s) {
  build_row_pack_kernel<<<1, 1024, 0, s>>>(len, B, T, rb, status);
  note_launch();
  const size_t N = (size_t)B * T;
  fill_rowmap_kernel<<<(unsigned)((N + 255) / 256), 256, 0, s>>>(len, B, T, rb, status);
  note_launch();
}

__global__ void clamp_rows_kernel(RowPack rb, int max_rows, int32_t* status) {
  if (rb.n_rows[0] > max_rows) {
    flag_status(status, TRL_ERR_ROWS_BOUND);
    rb.n_rows[0] = max_rows;
    rb.nblk[0] = max_rows / kRowBlock;
  }
}
void launch_clamp_rows(RowPack rb, int max_rows, int32_t* status, cudaStream_t s) {
  clamp_rows_kernel<<<1, 1, 0, s>>>(rb, max_rows, status);
  note_launch();
}

// ------------------------------------------------------------------------------------
// HRD advantages.  grid = (token tiles, B).  Each CTA re-derives its group's means with a
// warp-shuffle reduction over the G rewards of the prompt (fp64), then streams out the
// segment labels and per-token advantages of its token tile with 16-byte stores.
// ------------------------------------------------------------------------------------
constexpr int kAdvTile = 8192;   // tokens per CTA

__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(256) hrd_adv_kernel(
    const float* __restrict__ r_plan, const float* __restrict__ r_code, const int32_t* __restrict__ len,
    const int32_t* __restrict__ bnd, int P, int G, int T, int adv_mode, float* __restrict__ A_plan,
    float* __restrict__ A_code, uint8_t* __restrict__ seg, float* __restrict__ adv, int32_t* __restrict__ n_plan,
    int32_t* __restrict__ n_code, int64_t* __restrict__ n_valid, int32_t* status) {
  __shared__ float s_A[2];
  __shared__ int s_lb[2];
  const int b = blockIdx.y, i = b / G;
  const int tid = threadIdx.x;
  if (tid < 32) {
    double sp = 0, sc = 0;
    for (int j = tid; j < G; j += 32) { sp += (double)r_plan[i * G + j]; sc += (double)r_code[i * G + j]; }
    sp = warp_sum(sp); sc = warp_sum(sc);
    const double mp = sp / G, mc = sc / G;
    double ap = (double)r_plan[b] - mp, ac = (double)r_code[b] - mc;
    if (adv_mode == 1) {
      double vp = 0, vc = 0;
      for (int j = tid; j < G; j += 32) {
        double dp = (double)r_plan[i * G + j] - mp, dc = (double)r_code[i * G + j] - mc;
        vp += dp * dp; vc += dc * dc;
      }
      vp = warp_sum(vp); vc = warp_sum(vc);
      ap /= (sqrt(vp / G) + 1e-6); ac /= (sqrt(vc / G) + 1e-6);
    }
    if (tid == 0) {
      int L = len[b], Bd = bnd[b];
      bool bad = (L < 0 || L > T);
      L = max(0, min(L, T));
      bad |= (Bd < 0 || Bd > L);
      Bd = max(0, min(Bd, L));
      if (bad) flag_status(status, TRL_ERR_BAD_INDEX);
      s_A[0] = (float)ap; s_A[1] = (float)ac; s_lb[0] = L; s_lb[1] = Bd;
      if (blockIdx.x == 0) {
        A_plan[b] = (float)ap; A_code[b] = (float)ac; n_plan[b] = Bd; n_code[b] = L - Bd;
      }
    }
    if (blockIdx.x == 0 && b == 0) {          // sum of lengths: one warp, fixed order, integers
      long long tot = 0;
      for (int k = tid; k < P * G; k += 32) tot += max(0, min(len[k], T));
      for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
      if (tid == 0) n_valid[0] = tot;
    }
  }
  __syncthreads();
  const float ap = s_A[0], ac = s_A[1];
  const int L = s_lb[0], Bd = s_lb[1];
  const int t_begin = blockIdx.x * kAdvTile, t_end = min(T, t_begin + kAdvTile);
  const size_t base = (size_t)b * T;
  // A warp covers 512 consecutive tokens per iteration when rows are 16-aligned.  Every store
  // instruction of the warp writes 512 contiguous bytes: lane i writes the 16 segment bytes of
  // tokens [16i, 16i+16), and for q = 0..3 the four advantages of tokens [128q + 4i, 128q + 4i + 4).
  if ((T & 15) == 0) {
    const int lane = tid & 31, wid = tid >> 5;
    for (int t0 = t_begin + wid * 512; t0 < t_end; t0 += 8 * 512) {
      uint32_t w[4];
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const int tt = t0 + lane * 16 + q;
        const int sg = tt < Bd ? 1 : (tt < L ? 2 : 0);
        if ((q & 3) == 0) w[q >> 2] = 0;
        w[q >> 2] |= (uint32_t)sg << (8 * (q & 3));
      }
      if (t0 + lane * 16 < t_end) *reinterpret_cast<uint4*>(seg + base + t0 + lane * 16) = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int tt = t0 + 128 * q + 4 * lane;
        float a[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) a[k] = (tt + k) < Bd ? ap : ((tt + k) < L ? ac : 0.f);
        if (tt < t_end) *reinterpret_cast<float4*>(adv + base + tt) = make_float4(a[0], a[1], a[2], a[3]);
      }
    }
  } else {
    for (int t = t_begin + tid; t < t_end; t += 256) {
      const int sg = t < Bd ? 1 : (t < L ? 2 : 0);
      seg[base + t] = (uint8_t)sg;
      adv[base + t] = sg == 1 ? ap : (sg == 2 ? ac : 0.f);
    }
  }
}

void launch_hrd_advantages(const float* r_plan, const float* r_code, const int32_t* len, const int32_t* bnd,
                           int P, int G, int T, int adv_mode, float* A_plan, float* A_code, uint8_t* seg,
                           float* adv, int32_t* n_plan, int32_t* n_code, int64_t* n_valid, int32_t* status,
                           cudaStream_t s) {
  dim3 grid(cdiv(T, kAdvTile), P * G);
  hrd_adv_kernel<<<grid, 256, 0, s>>>(r_plan, r_code, len, bnd, P, G, T, adv_mode, A_plan, A_code, seg, adv,
                                      n_plan, n_code, n_valid, status);
  note_launch();
}

// ------------------------------------------------------------------------------------
// Clipped surrogate.  Stage 1: grid = (tiles, B), each CTA reduces its token tile of one
// rollout in a fixed order and writes 4 partial sums; also writes g.  Stage 2: one CTA
// combines the partials in index order in fp64 -> bit-reproducible loss.
// ------------------------------------------------------------------------------------
constexpr int kLossTile = 16384;
int pg_loss_tiles(int T) { return cdiv(T, kLossTile); }

// One token of the surrogate: returns w*u and writes s and g (before the 1/normaliser factor
// `inv` is applied to g by the caller's choice of inv).  Shared by the stand-alone loss kernel and
// the fused step so both take the same decisions in the same arithmetic.
struct TokenTerm { float wu, g, s; };
__device__ __forceinline__ TokenTerm surrogate_token(float logp, float old_logp, float A, int sg,
                                                    const trl_pg_config& cfg, float inv) {
  const float lo = 1.0f - cfg.eps_lo, hi = 1.0f + cfg.eps_hi;
  const float s = expf(logp - old_logp);
  const float w = sg == 1 ? cfg.alpha : (sg == 2 ? 1.0f : 0.f);
  const float unclipped = A * s;
  TokenTerm t;
  t.s = s;
  if (cfg.clip_form == 0) {
    const float clipped = A * fminf(fmaxf(s, lo), hi);
    t.wu = w * fminf(unclipped, clipped);
    t.g = (unclipped <= clipped) ? -w * A * s * inv : 0.f;
  } else {                       // A * min{s, clip(s)} = A * min(s, 1 + eps_hi)
    t.wu = w * A * fminf(s, hi);
    t.g = (s <= hi) ? -w * A * s * inv : 0.f;
  }
  return t;
}

__device__ __forceinline__ long long total_valid_tokens(const int32_t* len, int B, int T, long long* sh) {
  long long tot = 0;
  for (int k = threadIdx.x; k < B; k += blockDim.x) tot += max(0, min(len[k], T));
  for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = tot;
  __syncthreads();
  long long r = 0;
  for (int k = 0; k < (int)(blockDim.x >> 5); ++k) r += sh[k];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(256) pg_loss_stage1_kernel(
    const float* __restrict__ logp, const float* __restrict__ old_logp, const float* __restrict__ adv,
    const uint8_t* __restrict__ seg, const int32_t* __restrict__ len, int P, int G, int T, trl_pg_config cfg,
    float* __restrict__ g, float* __restrict__ partials, const int32_t* __restrict__ ids, int V) {
  // ids (may be null): tokens whose id is outside [0, V) are skipped like padding
  const int b = blockIdx.y, tid = threadIdx.x;
  const int L = max(0, min(len[b], T));
  const int t_begin = blockIdx.x * kLossTile, t_end = min(T, t_begin + kLossTile);
  const size_t base = (size_t)b * T;
  __shared__ long long sh_tot[8];
  float inv = L > 0 ? 1.0f / ((float)P * (float)G * (float)L) : 0.f;
  if (cfg.agg_mode == 1) {
    const long long ntok = total_valid_tokens(len, P * G, T, sh_tot);
    inv = ntok > 0 ? 1.0f / (float)ntok : 0.f;
  }
  const float lo = 1.0f - cfg.eps_lo, hi = 1.0f + cfg.eps_hi;
  float acc = 0.f, n_hi = 0.f, n_lo = 0.f, sum_s = 0.f;
  if ((T & 3) == 0) {          // 4 tokens per thread: 16-byte loads and stores
    for (int t = t_begin + tid * 4; t < t_end; t += 256 * 4) {
      float gq[4] = {0.f, 0.f, 0.f, 0.f};
      if (t < L) {
        const size_t n = base + t;
        const float4 lp = *reinterpret_cast<const float4*>(logp + n);
        const float4 ol = *reinterpret_cast<const float4*>(old_logp + n);
        const float4 ad = *reinterpret_cast<const float4*>(adv + n);
        const uchar4 sg = *reinterpret_cast<const uchar4*>(seg + n);
        const float lpa[4] = {lp.x, lp.y, lp.z, lp.w}, ola[4] = {ol.x, ol.y, ol.z, ol.w}, ada[4] = {ad.x, ad.y, ad.z, ad.w};
        const int sga[4] = {sg.x, sg.y, sg.z, sg.w};
        int4 idq = make_int4(0, 0, 0, 0);
        if (ids) idq = *reinterpret_cast<const int4*>(ids + n);
        const int ida[4] = {idq.x, idq.y, idq.z, idq.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (t + k < L && (!ids || (unsigned)ida[k] < (unsigned)V)) {
            const TokenTerm tt = surrogate_token(lpa[k], ola[k], ada[k], sga[k], cfg, inv);
            acc += tt.wu;
            gq[k] = tt.g;
            n_hi += tt.s > hi ? 1.f : 0.f;
            n_lo += tt.s < lo ? 1.f : 0.f;
            sum_s += tt.s;
          }
        }
      }
      *reinterpret_cast<float4*>(g + base + t) = make_float4(gq[0], gq[1], gq[2], gq[3]);
    }
  } else {
    for (int t = t_begin + tid; t < t_end; t += 256) {
      float gn = 0.f;
      if (t < L && (!ids || (unsigned)ids[base + t] < (unsigned)V)) {
        const size_t n = base + t;
        const TokenTerm tt = surrogate_token(logp[n], old_logp[n], adv[n], seg[n], cfg, inv);
        acc += tt.wu;
        gn = tt.g;
        n_hi += tt.s > hi ? 1.f : 0.f;
        n_lo += tt.s < lo ? 1.f : 0.f;
        sum_s += tt.s;
      }
      g[base + t] = gn;
    }
  }
  __shared__ float red[4][8];
  float v[4] = {acc, n_hi, n_lo, sum_s};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    for (int o = 16; o > 0; o >>= 1) v[q] += __shfl_xor_sync(0xffffffffu, v[q], o);
    if ((tid & 31) == 0) red[q][tid >> 5] = v[q];
  }
  __syncthreads();
  if (tid < 4) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += red[tid][w];
    partials[((size_t)b * gridDim.x + blockIdx.x) * 4 + tid] = s;
  }
}

// One CTA.  Thread b adds its rollouts' tile partials in tile order (independent loads),
// divides by the length, and the block combines the per-thread fp64 sums in a fixed tree.
__global__ void __launch_bounds__(256) pg_loss_stage2_kernel(const float* __restrict__ partials,
                                                             const int32_t* __restrict__ len, int P, int G, int T,
                                                             int tiles, int agg_mode, float* __restrict__ loss,
                                                             float* __restrict__ stats) {
  __shared__ double red[5][8];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, B = P * G;
  double v[5] = {0, 0, 0, 0, 0};          // J, n_hi, n_lo, sum_s, tokens
  for (int b = tid; b < B; b += 256) {
    const int L = max(0, min(len[b], T));
    const float4* p4 = reinterpret_cast<const float4*>(partials) + (size_t)b * tiles;
    double a = 0;
#pragma unroll 8
    for (int k = 0; k < tiles; ++k) {
      const float4 p = p4[k];
      a += p.x; v[1] += p.y; v[2] += p.z; v[3] += p.w;
    }
    if (L > 0) v[0] += agg_mode == 1 ? a : a / L;
    v[4] += L;
  }
#pragma unroll
  for (int q = 0; q < 5; ++q) {
    for (int o = 16; o > 0; o >>= 1) v[q] += __shfl_xor_sync(0xffffffffu, v[q], o);
    if (lane == 0) red[q][wid] = v[q];
  }
  __syncthreads();
  if (tid == 0) {
    double t[5] = {0, 0, 0, 0, 0};
    for (int q = 0; q < 5; ++q)
      for (int k = 0; k < 8; ++k) t[q] += red[q][k];
    loss[0] = agg_mode == 1 ? (float)(t[4] > 0 ? -t[0] / t[4] : 0.0) : (float)(-t[0] / ((double)P * (double)G));
    if (stats) {
      const double d = t[4] > 0 ? t[4] : 1.0;
      stats[0] = (float)(t[1] / d); stats[1] = (float)(t[2] / d); stats[2] = (float)(t[3] / d);
      stats[3] = (float)t[4];
    }
  }
}

void launch_pg_loss(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                    const int32_t* len, int P, int G, int T, trl_pg_config cfg, float* loss, float* g,
                    float* stats, float* partials, const int32_t* ids, int V, cudaStream_t s) {
  const int tiles = pg_loss_tiles(T);
  dim3 grid(tiles, P * G);
  pg_loss_stage1_kernel<<<grid, 256, 0, s>>>(logp, old_logp, adv, seg, len, P, G, T, cfg, g, partials, ids, V);
  note_launch();
  pg_loss_stage2_kernel<<<1, 256, 0, s>>>(partials, len, P, G, T, tiles, cfg.agg_mode, loss, stats);
  note_launch();
}

// ------------------------------------------------------------------------------------
// Merge of per-vocabulary-tile partials: lse = M + log sum_k l_k exp(m_k - M).
// One thread per global row; padded rows get 0.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) merge_lse_kernel(const float2* __restrict__ partials,
                                                        const float* __restrict__ tgt, int n_tiles, int rows_cap,
                                                        RowPack rb, const int32_t* __restrict__ ids,
                                                        const int32_t* __restrict__ len, int B, int T, int V,
                                                        float* __restrict__ logp, float* __restrict__ lse,
                                                        int32_t* status) {
  const size_t n = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (n >= (size_t)B * T) return;
  const int b = (int)(n / T), t = (int)(n % T);
  const int L = max(0, min(len[b], T));
  float out_lp = 0.f, out_lse = 0.f;
  if (t < L) {
    const size_t prow = (size_t)rb.row_first[b] + t;
    float M = -INFINITY;
    for (int k = 0; k < n_tiles; ++k) M = fmaxf(M, partials[(size_t)k * rows_cap + prow].x);
    float l = 0.f;
    for (int k = 0; k < n_tiles; ++k) {
      const float2 p = partials[(size_t)k * rows_cap + prow];
      l += p.y * __expf(p.x - M);
    }
    out_lse = M + __logf(l);
    const int id = ids[n];
    if ((unsigned)id < (unsigned)V) out_lp = tgt[prow] - out_lse;
    else flag_status(status, TRL_ERR_BAD_INDEX);
  }
  logp[n] = out_lp;
  lse[n] = out_lse;
}

void launch_merge_lse(const float2* partials, const float* tgt, int n_tiles, int rows_cap, RowPack rb,
                      const int32_t* ids, const int32_t* len, int B, int T, int V, float* logp, float* lse,
                      int32_t* status, cudaStream_t s) {
  const size_t N = (size_t)B * T;
  merge_lse_kernel<<<(unsigned)((N + 255) / 256), 256, 0, s>>>(partials, tgt, n_tiles, rows_cap, rb, ids, len, B, T,
                                                               V, logp, lse, status);
  note_launch();
}

// ------------------------------------------------------------------------------------
// Row packing / gathering in bf16 (one CTA per output row, 16-byte loads and stores): the
// packed copy of hidden that the forward GEMMs read, and the scaled chunk rows that are the
// B operand of dW = dS^T hidden in the fused step.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) pack_rows_bf16_kernel(const __nv_bfloat16* __restrict__ src,
                                                             __nv_bfloat16* __restrict__ out, int H, int R, RowPack rb,
                                                             int q_off, int from_packed,
                                                             const float* __restrict__ row_scale) {
  const int r = blockIdx.x;
  const int q = q_off + r;
  const int n_rows = rb.n_rows[0];
  if (q >= rb.nblk[0] * kRowBlock) return;          // beyond the last live block: never read
  uint4* dst = reinterpret_cast<uint4*>(out + (size_t)r * H);
  if (q >= n_rows) {
    for (int i = threadIdx.x; i < H / 8; i += 128) dst[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  const size_t row = from_packed ? (size_t)q : (size_t)rb.rowmap[q];
  const uint4* s4 = reinterpret_cast<const uint4*>(src + row * H);
  const float sc = row_scale ? row_scale[r] : 1.0f;
  for (int i = threadIdx.x; i < H / 8; i += 128) {
    uint4 x = s4[i];
    if (row_scale) {
      __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&x);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float2 f = __bfloat1622float2(h2[k]);
        h2[k] = __floats2bfloat162_rn(f.x * sc, f.y * sc);
      }
    }
    dst[i] = x;
  }
}

void launch_pack_rows_bf16(const __nv_bfloat16* src, __nv_bfloat16* out, int H, int R, RowPack rb, int q_off,
                           int from_packed, const float* row_scale, cudaStream_t s) {
  pack_rows_bf16_kernel<<<R, 128, 0, s>>>(src, out, H, R, rb, q_off, from_packed, row_scale);
  note_launch();
}

// ------------------------------------------------------------------------------------
// Fused step, per chunk: one thread per scratch row.  The GEMM stored E = exp(z - c), the sampled
// token's logit z_t, and per vocabulary tile the row sum of E over every column except the sampled
// token's.  With S' = sum_{v != t} E_v and E_t = exp(z_t - c):
//   lse = c + log(S' + E_t),  logp = z_t - lse,  g = d loss / d logp (same formula as
//   pg_loss_stage1_kernel),  dS = g onehot - g exp(c - lse) E = neg_alpha (E - exp(lse - c) onehot),
// so the kernel stores neg_alpha = -g exp(c - lse) and replaces the sampled token's entry of E by
// E_t - exp(lse - c) = -S'.  Formed this way the entry has no cancellation however close the
// token's probability is to 1 (E_t and exp(lse - c) then agree to many digits).
// A row whose token id is out of range is flagged and treated as padding (g = 0).
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) fused_merge_kernel(FusedMergeArgs a) {
  // one CTA = one 128-row block of the chunk
  const int r = blockIdx.x * 128 + threadIdx.x;
  const int q = a.blk_off * kRowBlock + r;
  const int R_live = a.R_live > 0 ? a.R_live : a.R;
  if (blockIdx.x * 128 >= R_live || a.blk_off + (int)blockIdx.x >= a.rb.nblk[0]) return;   // whole block not live
  float gn = 0.f;
  if (r < R_live && q < a.rb.n_rows[0]) {
    const size_t n = (size_t)a.rb.rowmap[q];
    const int b = (int)(n / a.T);
    float s_excl = 0.f;
    for (int k = 0; k < a.n_tiles; ++k) s_excl += a.psum[(size_t)k * a.R + r];
    const float c = a.hint[n];
    const int id = a.ids[n];
    const bool id_ok = (unsigned)id < (unsigned)a.V;
    if (!id_ok) flag_status(a.status, TRL_ERR_BAD_INDEX);
    const float zt = id_ok ? a.tgt[r] : 0.f;
    const float sum = s_excl + (id_ok ? expf(zt - c) : 0.f);
    if (!(sum > 0.f) || !isfinite(sum)) flag_status(a.status, TRL_ERR_BAD_HINT);
    const float lse = c + logf(sum);
    const float lp = id_ok ? zt - lse : 0.f;
    const bool n_ok = TRL_IN_BOUNDS(n, a.rb.n_total, a.status);
    if (n_ok) { a.logp[n] = lp; a.lse[n] = lse; }
    const int L = max(0, min(a.len[b], a.T));
    const float inv = a.cfg.agg_mode == 1 ? 1.0f / (float)a.rb.n_rows[0] : 1.0f / ((float)a.P * (float)a.G * (float)L);
    const TokenTerm tt = surrogate_token(lp, a.old_logp[n], a.adv[n], a.seg[n], a.cfg, inv);
    gn = id_ok ? tt.g : 0.f;
    if (n_ok) a.g[n] = gn;
    if (gn != 0.f) a.E[(size_t)r * a.V + id] = __float2bfloat16_rn(-s_excl);
    gn = -gn * expf(c - lse);
  }
  if (r < R_live) a.neg_alpha[r] = gn;
  const int any = __syncthreads_or(gn != 0.f);
  if (threadIdx.x == 0) a.blk_active[blockIdx.x] = any;
}

__global__ void __launch_bounds__(128) flag_active_blocks_kernel(const float* __restrict__ g, RowPack rb,
                                                                 int* __restrict__ blk_active) {
  if ((int)blockIdx.x >= rb.nblk[0]) return;
  const int q = blockIdx.x * kRowBlock + threadIdx.x;
  const bool on = q < rb.n_rows[0] && g[rb.rowmap[q]] != 0.f;
  const int any = __syncthreads_or(on);
  if (threadIdx.x == 0) blk_active[blockIdx.x] = any;
}

void launch_flag_active_blocks(const float* g, RowPack rb, int* blk_active, cudaStream_t s) {
  flag_active_blocks_kernel<<<rb.cap, 128, 0, s>>>(g, rb, blk_active);
  note_launch();
}

void launch_fused_merge(const FusedMergeArgs& a, cudaStream_t s) {
  fused_merge_kernel<<<cdiv(a.R_live > 0 ? a.R_live : a.R, 128), 128, 0, s>>>(a);
  note_launch();
}

// ------------------------------------------------------------------------------------
// fp32 path helpers.  Scratch row r of a chunk is (block blk_off + r/128, lane r%128).
// ------------------------------------------------------------------------------------
__device__ __forceinline__ long scratch_row_to_global(const RowPack& rb, int blk_off, int r) {
  return packed_to_global(rb, blk_off * kRowBlock + r);
}

__global__ void pack_rows_f32_kernel(const float* __restrict__ hidden, float* __restrict__ Xp, int H, int R,
                                     RowPack rb, int blk_off) {
  const int r = blockIdx.x;
  const long n = scratch_row_to_global(rb, blk_off, r);
  for (int h = threadIdx.x; h < H; h += blockDim.x) Xp[(size_t)r * H + h] = n >= 0 ? hidden[(size_t)n * H + h] : 0.f;
}
void launch_pack_rows_f32(const float* hidden, float* Xp, int H, int R, RowPack rb, int blk_off, cudaStream_t s) {
  pack_rows_f32_kernel<<<R, 128, 0, s>>>(hidden, Xp, H, R, rb, blk_off);
  note_launch();
}

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* sh) {
  for (int o = 16; o > 0; o >>= 1) {
    float u = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, u) : v + u;
  }
  const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[w] = v;
  __syncthreads();
  float r = sh[0];
  for (int k = 1; k < nw; ++k) r = is_max ? fmaxf(r, sh[k]) : r + sh[k];
  return r;
}

__global__ void __launch_bounds__(256) row_lse_f32_kernel(const float* __restrict__ S, int V, int R, RowPack rb,
                                                          int blk_off, const int32_t* __restrict__ ids,
                                                          float* __restrict__ logp, float* __restrict__ lse,
                                                          int32_t* status) {
  __shared__ float sh[8];
  const int r = blockIdx.x;
  const long n = scratch_row_to_global(rb, blk_off, r);
  if (n < 0) return;
  const float* row = S + (size_t)r * V;
  float m = -INFINITY;
  for (int v = threadIdx.x; v < V; v += 256) m = fmaxf(m, row[v]);
  m = block_reduce(m, true, sh);
  float l = 0.f;
  for (int v = threadIdx.x; v < V; v += 256) l += expf(row[v] - m);
  l = block_reduce(l, false, sh);
  if (threadIdx.x == 0 && TRL_IN_BOUNDS(n, rb.n_total, status)) {
    const float L = m + logf(l);
    lse[n] = L;
    const int id = ids[n];
    if ((unsigned)id < (unsigned)V) logp[n] = row[id] - L;
    else { logp[n] = 0.f; flag_status(status, TRL_ERR_BAD_INDEX); }
  }
}
void launch_row_lse_f32(const float* S, int V, int R, RowPack rb, int blk_off, const int32_t* ids, float* logp,
                        float* lse, int32_t* status, cudaStream_t s) {
  row_lse_f32_kernel<<<R, 256, 0, s>>>(S, V, R, rb, blk_off, ids, logp, lse, status);
  note_launch();
}

__global__ void __launch_bounds__(256) ds_inplace_f32_kernel(float* __restrict__ S, int V, int R, RowPack rb,
                                                             int blk_off, const int32_t* __restrict__ ids,
                                                             const float* __restrict__ lse,
                                                             const float* __restrict__ g) {
  const int r = blockIdx.x;
  const long n = scratch_row_to_global(rb, blk_off, r);
  float* row = S + (size_t)r * V;
  if (n < 0) {
    for (int v = threadIdx.x; v < V; v += 256) row[v] = 0.f;
    return;
  }
  const int id = ids[n];
  const float gn = (unsigned)id < (unsigned)V ? g[n] : 0.f, L = lse[n];     // a row with a bad id adds nothing
  for (int v = threadIdx.x; v < V; v += 256) row[v] = gn * ((v == id ? 1.f : 0.f) - expf(row[v] - L));
}
void launch_ds_inplace_f32(float* S, int V, int R, RowPack rb, int blk_off, const int32_t* ids, const float* lse,
                           const float* g, cudaStream_t s) {
  ds_inplace_f32_kernel<<<R, 256, 0, s>>>(S, V, R, rb, blk_off, ids, lse, g);
  note_launch();
}

__global__ void scatter_rows_f32_kernel(const float* __restrict__ dHp, float* __restrict__ dHidden, int H, int R,
                                        RowPack rb, int blk_off) {
  const int r = blockIdx.x;
  const long n = scratch_row_to_global(rb, blk_off, r);
  if (n < 0 || !TRL_IN_BOUNDS(n, rb.n_total, (int32_t*)nullptr)) return;
  for (int h = threadIdx.x; h < H; h += blockDim.x) dHidden[(size_t)n * H + h] = dHp[(size_t)r * H + h];
}
void launch_scatter_rows_f32(const float* dHp, float* dHidden, int H, int R, RowPack rb, int blk_off,
                             cudaStream_t s) {
  scatter_rows_f32_kernel<<<R, 128, 0, s>>>(dHp, dHidden, H, R, rb, blk_off);
  note_launch();
}

__global__ void zero_padded_f32_kernel(float* __restrict__ a, float* __restrict__ b, const int32_t* __restrict__ len,
                                       int B, int T) {
  const size_t n = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (n >= (size_t)B * T) return;
  const int bb = (int)(n / T), t = (int)(n % T);
  if (t >= max(0, min(len[bb], T))) { a[n] = 0.f; b[n] = 0.f; }
}
void launch_zero_padded_f32(float* a, float* b, const int32_t* len, int B, int T, cudaStream_t s) {
  const size_t N = (size_t)B * T;
  zero_padded_f32_kernel<<<(unsigned)((N + 255) / 256), 256, 0, s>>>(a, b, len, B, T);
  note_launch();
}

}  // namespace trl
