// tcgen05 / TMEM bf16 GEMM family for sm_100a.
//
// One persistent, warp-specialised kernel computes C[m,n] = sum_k A[m,k] B[n,k] (bf16
// operands, fp32 accumulation in tensor memory) on 128x256 accumulator tiles.  Each operand is read in
// the layout it already has in memory: K-contiguous ("K-major": hidden and W in the forward,
// dS / E in dHidden = dS W) or M/N-contiguous ("MN-major": W in dHidden = dS W, dS / E and the
// gathered hidden rows in dW = dS^T hidden), so no operand is ever transposed in memory.
// One of five epilogues is applied straight from TMEM:
//   LSE : per-row (max, sum-exp) of the tile's logits + pick-up of the sampled token's
//         logit                                       (token scoring, Section 2.3 ratio s)
//   DS  : dS = g (onehot - exp(z - lse)) as bf16
//   DH  : dHidden rows (bf16), scattered to the caller's row positions
//   DW  : dW += tile (fp32, TMA reduce-add from shared memory)
//   E   : E = exp(z - c) for a per-row shift c (a stale log-partition), as bf16, plus the row
//         sums of E over every column but the sampled token's, and the sampled token's logit.  The softmax is p = E exp(c - lse), a
//         per-row factor the gradient GEMMs fold into their other operand / their epilogue,
//         so the forward GEMM is not repeated in the backward.
//
// Roles: warp 0 = TMA producer (one elected lane), warp 1 = MMA issuer (one elected lane)
// and TMEM owner, warps 2.. = epilogue (groups of four warps, one TMEM lane quadrant each).  Shared-memory
// stages are guarded by full/empty mbarriers; the 512 TMEM columns hold two 128x256 fp32
// accumulators: in the scoring GEMM the epilogue of tile i overlaps the mainloop of tile
// i+1, in the other GEMMs both belong to one 256x256 CTA tile that shares its B operand.
// The dS / E / dW epilogues stage 32-row x 128-byte units in swizzled shared memory and hand
// them to the TMA (bulk tensor store / reduce-add), so global memory sees whole 128 B lines.
// Every wait is bounded: on expiry the CTA raises TRL_ERR_TIMEOUT in the status word,
// all roles leave their loops, TMEM is freed and the kernel returns.
#include <cuda.h>

#include <atomic>
#include <cstdlib>

#include "trl_internal.h"

namespace trl {

int tc_raster_band_override(int epi);

namespace {

// CTAs per MMA for the forward GEMMs (LSE, dS, E) and the gradient GEMMs (dHidden, dW): 1, or 2
// for cluster pairs (tcgen05 cta_group::2)
#ifndef TRL_CTA_GROUP_FWD
#define TRL_CTA_GROUP_FWD 1
#endif
#ifndef TRL_CTA_GROUP_BWD
#define TRL_CTA_GROUP_BWD 1
#endif

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
constexpr int RING_BYTES = 4 * (A_BYTES + B_BYTES);   // 192 KB of operand stages, cut into 3 to 6 stages
constexpr int MAX_STAGES = 6;
constexpr int OUT_STAGE_BYTES = 4 * 2 * 4096;   // 4 epilogue warps x 2 buffers x (32 rows x 128 B)
constexpr int MAX_LIST_BLOCKS = 512;               // longest list of active row blocks a CTA keeps in shared memory
constexpr int SMEM_BYTES = RING_BYTES + OUT_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                           2 * MAX_LIST_BLOCKS /*active row blocks*/;
constexpr uint32_t TMEM_COLS = 512;
constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
constexpr long long WAIT_CYCLES = 4000000000LL;   // ~2-3 s at B200 clocks

struct TcArgs {
  int N, K, m_blocks_fixed, blk_off, blk_cap, raster_band, rows_cap, V;
  int pos_off, pos_cap;      // window of M positions this launch works on (pos_cap 0: all)
  unsigned* pace_ctr; int pace_every;   // soft pacing of the TMA producers (null: off); counter zeroed before the launch
  const int* nblk; const int* n_rows; const int* rowmap;
  const int32_t* ids; const float* lse; const float* g;
  float2* partials; float* tgt;
  __nv_bfloat16* dS; long ds_ld;
  __nv_bfloat16* dHidden; long dh_ld; long dh_rows;
  float* dW; long dw_ld;
  float* psum; const float* row_scale;
  const int* blk_active;     // per row block of the chunk: 0 = every row has a zero gradient factor (may be null)
  int32_t* status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait.  Returns false if the CTA is aborting (own timeout or another role's).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_CYCLES) {
        *abort_flag = 1;
        if (status) atomicOr(status, 1 << TRL_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// ---- CTA pairs (cta_group::2).  The two CTAs of a cluster share one MMA: each holds its own 128
// rows of A and half of the B tile in its own shared memory, the even CTA ("leader") issues the
// instruction, and each CTA's tensor memory receives its own 128 accumulator rows.  Every copy is a
// plain TMA load into the issuing CTA's own shared memory; only its completion is signalled on the
// leader's barrier.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// load into this CTA's shared memory; the bytes are counted on `cluster_bar`, a barrier of the pair's leader
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(cluster_bar), "r"(x), "r"(y)
      : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair once all earlier MMAs are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows are 128 B
// apart inside an 8-row group, groups are 1024 B apart (stride byte offset); the leading
// byte offset is not used for swizzled K-major layouts (set to 1); descriptor version 1.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// MN-major operand, 128-byte swizzle.  The tile is stored as groups of 64 M/N-elements:
// inside a group every k-row is 128 contiguous bytes, 8 k-rows form a 1024 B swizzle atom
// (stride byte offset = distance between 8-row atoms along K = 1024 B), and groups follow
// each other every 64 k-rows x 128 B = 8192 B (leading byte offset).
__device__ __forceinline__ uint64_t make_mnmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)(8192 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor, kind::f16: D = fp32, A = B = bf16, M x N tile; bit 15 / 16 select
// an MN-major A / B operand.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__host__ __device__ constexpr bool a_is_mn(int epi) { return epi == TC_EPI_DW; }
__host__ __device__ constexpr bool b_is_mn(int epi) { return epi == TC_EPI_DW || epi == TC_EPI_DH; }

__device__ __forceinline__ void tile_coords(int tile, int MB, int NT, int band_rows, int& mb, int& nt) {
  const int per_band = band_rows * NT;
  const int band = tile / per_band, within = tile - band * per_band;
  const int rows = min(band_rows, MB - band * band_rows);
  nt = within / rows;
  mb = band * band_rows + (within - nt * rows);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Per-warp staged output: each lane owns one 128-byte row of a 32-row unit.  Rows are
// written with the 128-byte swizzle (16-byte chunk index XOR row%8) the tensor map expects,
// then one lane issues the bulk tensor store (or fp32 reduce-add).  With 4 epilogue warps each
// warp alternates between two 4 KB buffers, with 8 warps each has one.
struct WarpOut {
  uint32_t smem;            // this warp's 4 KB buffer(s), 1024-byte aligned
  const CUtensorMap* tm;
  int lane;
  int n;
  int nbuf;                 // buffers in use: 2 (alternating) or 1
  template <bool REDUCE>
  __device__ __forceinline__ void put(const uint4 (&w)[8], int x, int y) {
    const uint32_t buf = smem + (uint32_t)(nbuf == 2 ? (n & 1) : 0) * 4096u;
    if (lane == 0) {          // the store that last used this buffer must have read it
      if (nbuf == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    __syncwarp();
    const uint32_t row = buf + (uint32_t)lane * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (uint32_t)((j ^ (lane & 7)) << 4)), "r"(w[j].x),
                   "r"(w[j].y), "r"(w[j].z), "r"(w[j].w)
                   : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
      if constexpr (REDUCE)
        asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm),
                     "r"(buf), "r"(x), "r"(y)
                     : "memory");
      else
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm), "r"(buf),
                     "r"(x), "r"(y)
                     : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    ++n;
  }
  __device__ __forceinline__ void drain() {
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
  }
};

// ---------------------------------------------------------------- epilogues
// Each epilogue thread owns one accumulator row (TMEM lane) of the 128x256 tile.
template <int EPI>
__device__ __forceinline__ void epilogue_tile(const TcArgs& p, uint32_t tmem_acc, int quad, int lane, int mb, int nt,
                                              WarpOut& wo) {
  const int r = quad * 32 + lane;           // row within the tile
  const int n0 = nt * BN;
  const uint32_t taddr = tmem_acc + ((uint32_t)(quad * 32) << 16);
  uint32_t v[32];

  if constexpr (EPI == TC_EPI_LSE) {
    const int prow_i = (p.blk_off + mb) * BM + r;          // packed row
    const bool valid = prow_i < p.n_rows[0];
    const long grow = valid ? (long)p.rowmap[prow_i] : 0;
    const int id = valid ? p.ids[grow] : -1;
    float m2 = -INFINITY, l = 0.f, tg = 0.f;
    bool has = false;
    for (int c0 = 0; c0 < BN; c0 += 32) {
      const int ncl = p.N - (n0 + c0);
      if (ncl <= 0) break;
      tc_ld32(taddr + c0, v);
      tc_wait_ld();
      float t[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) t[j] = __uint_as_float(v[j]) * LOG2E;
      if (ncl < 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j) if (j >= ncl) t[j] = -INFINITY;
      }
      float gm = t[0];
#pragma unroll
      for (int j = 1; j < 32; ++j) gm = fmaxf(gm, t[j]);
      const float mnew = fmaxf(m2, gm);
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) s += ex2(t[j] - mnew);
      l = l * ex2(m2 - mnew) + s;
      m2 = mnew;
      const int lc = id - (n0 + c0);
      if (lc >= 0 && lc < 32 && lc < ncl) {
#pragma unroll
        for (int j = 0; j < 32; ++j) if (j == lc) tg = __uint_as_float(v[j]);
        has = true;
      }
    }
    const size_t prow = (size_t)prow_i;
    if (TRL_IN_BOUNDS(prow, p.rows_cap, p.status)) {
      p.partials[(size_t)nt * p.rows_cap + prow] = make_float2(m2 * LN2, l);
      if (has) p.tgt[prow] = tg;
    }
  } else if constexpr (EPI == TC_EPI_DS) {
    const int prow_i = (p.blk_off + mb) * BM + r;          // packed row
    const bool valid = prow_i < p.n_rows[0];
    const long grow = valid ? (long)p.rowmap[prow_i] : 0;
    const int id = valid ? p.ids[grow] : -1;
    const float gg = valid ? p.g[grow] : 0.f;
    const float L2 = valid ? p.lse[grow] * LOG2E : 0.f;
    const bool live = valid && gg != 0.f && (unsigned)id < (unsigned)p.N;   // a row with a bad id adds nothing
    for (int c0 = 0; c0 < BN; c0 += 64) {
      if (p.N - (n0 + c0) <= 0) break;
      uint4 w[8];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        tc_ld32(taddr + c0 + 32 * h, v);
        tc_wait_ld();
        const int lc = id - (n0 + c0 + 32 * h);
        float d[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float pr = ex2(fmaf(__uint_as_float(v[j]), LOG2E, -L2));
          d[j] = live ? gg * ((j == lc ? 1.f : 0.f) - pr) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
          w[4 * h + q] = make_uint4(pack_bf16x2(d[q * 8 + 0], d[q * 8 + 1]), pack_bf16x2(d[q * 8 + 2], d[q * 8 + 3]),
                                    pack_bf16x2(d[q * 8 + 4], d[q * 8 + 5]), pack_bf16x2(d[q * 8 + 6], d[q * 8 + 7]));
      }
      wo.put<false>(w, n0 + c0, mb * BM + quad * 32);     // columns >= V are clipped by the TMA
    }
  } else if constexpr (EPI == TC_EPI_E) {
    const int prow_i = (p.blk_off + mb) * BM + r;          // packed row
    const bool valid = prow_i < p.n_rows[0];
    const long grow = valid ? (long)p.rowmap[prow_i] : 0;
    const int id = valid ? p.ids[grow] : -1;
    const float C2 = valid ? p.lse[grow] * LOG2E : 0.f;      // p.lse holds the shift c here
    const size_t srow = (size_t)mb * BM + r;
    float sum = 0.f, tg = 0.f;
    bool has = false;
    for (int c0 = 0; c0 < BN; c0 += 64) {
      if (p.N - (n0 + c0) <= 0) break;
      uint4 w[8];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int ncl = p.N - (n0 + c0 + 32 * h);           // may be <= 0 for the second half
        tc_ld32(taddr + c0 + 32 * h, v);
        tc_wait_ld();
        float d[32];
        float gs = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float e = ex2(fmaf(__uint_as_float(v[j]), LOG2E, -C2));
          d[j] = (valid && j < ncl) ? e : 0.f;
          gs += d[j];
        }
        const int lc = id - (n0 + c0 + 32 * h);
        if (lc >= 0 && lc < 32 && lc < ncl) {      // the sampled token's column: keep it out of the row sum
          gs = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (j == lc) tg = __uint_as_float(v[j]); else gs += d[j];
          }
          has = true;
        }
        sum += gs;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          w[4 * h + q] = make_uint4(pack_bf16x2(d[q * 8 + 0], d[q * 8 + 1]), pack_bf16x2(d[q * 8 + 2], d[q * 8 + 3]),
                                    pack_bf16x2(d[q * 8 + 4], d[q * 8 + 5]), pack_bf16x2(d[q * 8 + 6], d[q * 8 + 7]));
      }
      wo.put<false>(w, n0 + c0, mb * BM + quad * 32);
    }
    if (TRL_IN_BOUNDS(srow, p.rows_cap, p.status)) {
      p.psum[(size_t)nt * p.rows_cap + srow] = sum;
      if (has) p.tgt[srow] = tg;
    }
  } else if constexpr (EPI == TC_EPI_DH) {
    const int prow_i = (p.blk_off + mb) * BM + r;          // packed row
    const bool valid = prow_i < p.n_rows[0];
    const long grow = valid ? (long)p.rowmap[prow_i] : 0;
    const float rs = p.row_scale ? p.row_scale[(size_t)mb * BM + r] : 1.0f;
    const bool row_ok = TRL_IN_BOUNDS(grow, p.dh_rows, p.status);     // constant true outside the debug build
    __nv_bfloat16* out = p.dHidden + (size_t)grow * p.dh_ld;
    for (int c0 = 0; c0 < BN; c0 += 32) {
      const int ncl = p.N - (n0 + c0);
      if (ncl <= 0) break;
      tc_ld32(taddr + c0, v);
      tc_wait_ld();
      if (valid && row_ok) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (q * 8 < ncl) {
            uint4 w;
            w.x = pack_bf16x2(rs * __uint_as_float(v[q * 8 + 0]), rs * __uint_as_float(v[q * 8 + 1]));
            w.y = pack_bf16x2(rs * __uint_as_float(v[q * 8 + 2]), rs * __uint_as_float(v[q * 8 + 3]));
            w.z = pack_bf16x2(rs * __uint_as_float(v[q * 8 + 4]), rs * __uint_as_float(v[q * 8 + 5]));
            w.w = pack_bf16x2(rs * __uint_as_float(v[q * 8 + 6]), rs * __uint_as_float(v[q * 8 + 7]));
            *reinterpret_cast<uint4*>(out + n0 + c0 + q * 8) = w;
          }
        }
      }
    }
  } else {  // TC_EPI_DW: rows >= V and columns >= H are clipped by the TMA
    for (int c0 = 0; c0 < BN; c0 += 32) {
      if (p.N - (n0 + c0) <= 0) break;
      tc_ld32(taddr + c0, v);
      tc_wait_ld();
      uint4 w[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) w[q] = make_uint4(v[q * 4 + 0], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
      wo.put<true>(w, n0 + c0, mb * BM + quad * 32);
    }
  }
}

// ---------------------------------------------------------------- the kernel
// CG = CTAs that share one MMA (tcgen05 cta_group): 1, or 2 for a cluster pair.
// MT = accumulators (128-row M blocks) per CTA and tile.
//   CG = 1: the scoring GEMM (LSE) uses MT = 1 and alternates between two TMEM accumulators so
//     the epilogue overlaps the next mainloop; all other GEMMs use MT = 2, one B tile in shared
//     memory feeding both accumulators, with the epilogue exposed (two epilogue warp groups drain
//     the two accumulators of the forward GEMMs that store dS / E).
//   CG = 2: a pair works on 256 x 256 (forward GEMMs, MT = 1, two alternating accumulators per
//     CTA) or 512 x 256 (gradient GEMMs, MT = 2) and each CTA stages only its own A rows and half
//     of the B tile: a third to a half less shared-memory traffic per FLOP than CG = 1.
// M block of accumulator j of tile ms in the CTA of rank r: (ms * MT + j) * CG + r.
template <int EPI, int CG> struct TileCfg {
  static constexpr bool FWD = (EPI == TC_EPI_LSE || EPI == TC_EPI_E || EPI == TC_EPI_DS);
  static constexpr int MT = (CG == 2) ? (FWD ? 1 : 2) : ((EPI == TC_EPI_LSE) ? 1 : 2);
  // epilogue warp groups (4 warps each) working in parallel, one accumulator each
  static constexpr int EG = (CG == 1 && (EPI == TC_EPI_E || EPI == TC_EPI_DS)) ? 2 : 1;
  static constexpr int THREADS = 64 + 128 * EG;
  static constexpr int NACC = 2 / MT;                       // accumulator sets in the 512 TMEM columns
  static constexpr int BN_CTA = BN / CG;                    // rows of the B tile this CTA stages
  static constexpr int STG_BYTES = MT * A_BYTES + B_BYTES / CG;   // 48 / 64 KB (CG 1), 32 / 48 KB (CG 2)
  static constexpr int NSTAGE = RING_BYTES / STG_BYTES;           // 4 / 3, 6 / 4
  static_assert(NSTAGE <= MAX_STAGES && NSTAGE >= 2, "stage count");
};

template <int EPI, int CG>
__global__ void __launch_bounds__(TileCfg<EPI, CG>::THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmOut, const TcArgs p) {
  using Cfg = TileCfg<EPI, CG>;
  constexpr int MT = Cfg::MT, NACC = Cfg::NACC, NSTAGE = Cfg::NSTAGE, STG = Cfg::STG_BYTES, EG = Cfg::EG;
  constexpr int BN_CTA = Cfg::BN_CTA;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t out_base = smem_base + RING_BYTES;                    // 1024-aligned
  const uint32_t bar_base = out_base + OUT_STAGE_BYTES;
  // barrier layout (8 B each): full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2]; then tmem slot, abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + RING_BYTES + OUT_STAGE_BYTES + 8 * (2 * MAX_STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + RING_BYTES + OUT_STAGE_BYTES + 8 * (2 * MAX_STAGES + 4) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (CG == 2) ? (int)cluster_ctarank() : 0;        // 0 = the CTA that issues the MMAs
  const int worker = (int)blockIdx.x / CG, n_workers = (int)gridDim.x / CG;   // CTAs (CG 1) or pairs (CG 2)

  // ---- problem extents (identical in every thread, and in both CTAs of a pair)
  int live = p.blk_cap;
  if (p.nblk) live = max(0, min(p.nblk[0] - p.blk_off, p.blk_cap));
  // Row blocks whose rows all have a zero gradient factor (p.blk_active) are left out.  For dW they
  // are k-blocks, which every tile skips alike.  For dS / dHidden they are M blocks: the tiles are
  // formed over the list of active blocks (kept in shared memory), not over all blocks with holes,
  // so that every tile costs the same and the CTAs keep moving through K together, which is
  // what lets them share the streamed operands in L2.
  constexpr bool LISTED = (EPI == TC_EPI_DH || EPI == TC_EPI_DS);
  const bool use_list = LISTED && p.blk_active != nullptr && live <= MAX_LIST_BLOCKS;
  int n_act = live;
  if ((EPI == TC_EPI_DW || LISTED) && p.blk_active) {
    n_act = 0;
    for (int i = 0; i < live; ++i) n_act += p.blk_active[i] != 0;
  }
  // M extent in 128-row blocks: positions in the list of active blocks when one is used.  A launch
  // may be given a window [pos_off, pos_off + pos_cap) of those positions.
  int MB = (EPI == TC_EPI_DW) ? p.m_blocks_fixed : (use_list ? n_act : live);
  const int pos_off = (EPI == TC_EPI_DW || p.pos_cap <= 0) ? 0 : p.pos_off;
  if (EPI != TC_EPI_DW && p.pos_cap > 0) MB = max(0, min(MB - pos_off, p.pos_cap));
  const int MS = (MB + MT * CG - 1) / (MT * CG);                   // tiles along M
  const int K = (EPI == TC_EPI_DW) ? live * BM : p.K;
  const int NT = (p.N + BN - 1) / BN;
  const int nkb = (K + BK - 1) / BK;
  int total = (nkb > 0) ? MS * NT : 0;
  if (n_act == 0 || MB == 0) total = 0;
  if (total == 0 || worker >= total) return;        // the same decision in both CTAs of a pair
  uint16_t* act_list = reinterpret_cast<uint16_t*>(gen_base + RING_BYTES + OUT_STAGE_BYTES + 256);
  if (use_list && warp == 2) {                      // order-preserving list of the active blocks
    int n = 0;
    for (int i0 = 0; i0 < live; i0 += 32) {
      const bool on = i0 + lane < live && p.blk_active[i0 + lane] != 0;
      const unsigned m = __ballot_sync(0xffffffffu, on);
      if (on) act_list[n + __popc(m & ((1u << lane) - 1u))] = (uint16_t)(i0 + lane);
      n += __popc(m);
    }
  }
  // M position i (accumulator j of tile ms in the CTA of rank r: i = (ms * MT + j) * CG + r) -> row block;
  // valid after the __syncthreads below
  auto blk_of = [&](int i) { return use_list ? (int)act_list[pos_off + i] : pos_off + i; };
  // Is M position i (of this launch's window) worked on at all: present, and (without a list) not
  // marked inactive.
  auto pos_on = [&](int i) {
    return i < MB && (use_list || !(LISTED && p.blk_active) || p.blk_active[pos_off + i] != 0);
  };
  // Which accumulators of a tile take part (identical decision in every role and in both CTAs): an
  // accumulator spans the M blocks of all CG CTAs and runs if any of them is worked on.  Which
  // k-blocks take part: for dW, those of active row blocks.
  auto tile_mask = [&](int ms) {
    int m = 0;
    for (int j = 0; j < MT; ++j)
      for (int r = 0; r < CG; ++r)
        if (pos_on((ms * MT + j) * CG + r)) m |= 1 << j;
    return m;
  };
  auto kb_on = [&](int kb) { return !(EPI == TC_EPI_DW && p.blk_active) || p.blk_active[kb >> 1] != 0; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128 * EG * CG); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {           // with CG = 2 the same warp of both CTAs allocates, at the same shared-memory offset
    __syncwarp();
    if constexpr (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (CG == 2) cluster_sync_all();     // the partner's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  auto a_row_of = [&](int mb) {
    // forward GEMMs read the packed hidden rows of the block; the gradient GEMMs read chunk scratch
    return Cfg::FWD ? (p.blk_off + mb) * BM : mb * BM;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one per CTA)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      // Soft pacing: every pace_every k-blocks the producers of all CTAs count themselves in, and a
      // little later each waits (bounded, falling through on expiry) until the others of its wave have
      // reached the same point.  It keeps the CTAs within a few k-blocks of one another, so that an
      // operand tile streamed for one of them is still in L2 when its neighbours ask for it.  No
      // data depends on it: a producer that gives up waiting just goes on, and stops pacing.
      bool pace = (CG == 1) && p.pace_ctr != nullptr && p.pace_every > 0 && (use_list || !(LISTED && p.blk_active));
      const int pace_per_tile = pace ? (nkb + p.pace_every - 1) / p.pace_every : 0;
      for (int tile = worker; tile < total && ok; tile += n_workers) {
        int ms, nt;
        tile_coords(tile, MS, NT, p.raster_band, ms, nt);
        const int mask = tile_mask(ms);                        // accumulators of this tile that take part
        if (mask == 0) continue;
        const int b_row = nt * BN + rank * BN_CTA;
        const int wave = (tile - worker) / n_workers;          // every wave before the last one is full
        const unsigned in_wave = (unsigned)min(n_workers, total - wave * n_workers);
        const unsigned before = (unsigned)wave * (unsigned)n_workers * (unsigned)pace_per_tile;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!kb_on(kb)) continue;
          if (pace) {
            const int ph = kb % p.pace_every;
            if (ph == 0) atomicAdd(p.pace_ctr, 1u);
            if (ph == 2 || (ph < 2 && kb == nkb - 1)) {
              const unsigned target = before + in_wave * (unsigned)(kb / p.pace_every + 1);
              const long long t0 = clock64();
              while (*(volatile unsigned*)p.pace_ctr < target) {
                if (clock64() - t0 > 60000) { pace = false; break; }      // ~40 us
                __nanosleep(200);
              }
            }
          }
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status))) break;
          // bytes of this stage over all CTAs of the pair, expected on the leader's barrier
          if (rank == 0) mbar_expect_tx(full_bar(stage), (uint32_t)(CG * (__popc(mask) * A_BYTES + B_BYTES / CG)));
          const uint32_t fb = (CG == 2) ? map_to_cta(full_bar(stage), 0) : full_bar(stage);
          auto load = [&](uint32_t dst, const CUtensorMap* tm, int x, int y) {
            if constexpr (CG == 2) tma_load_2d_pair(dst, tm, x, y, fb); else tma_load_2d(dst, tm, x, y, fb);
          };
          const uint32_t sa = smem_base + stage * STG;
#pragma unroll
          for (int j = 0; j < MT; ++j) {
            if (mask & (1 << j)) {
              const int pos = (ms * MT + j) * CG + rank;            // beyond the last block: any row, the result is not used
              const int a_row = a_row_of(pos < MB ? blk_of(pos) : 0);
              if constexpr (a_is_mn(EPI)) {       // two 64(M) x 64(K) boxes
                load(sa + j * A_BYTES, &tmA, a_row, kb * BK);
                load(sa + j * A_BYTES + 8192, &tmA, a_row + 64, kb * BK);
              } else {
                load(sa + j * A_BYTES, &tmA, kb * BK, a_row);
              }
            }
          }
          const uint32_t sb = sa + MT * A_BYTES;
          if constexpr (b_is_mn(EPI)) {       // 64(N) x 64(K) boxes
#pragma unroll
            for (int j = 0; j < BN_CTA / 64; ++j) load(sb + j * 8192, &tmB, b_row + 64 * j, kb * BK);
          } else {
            load(sb, &tmB, kb * BK, b_row);
          }
          if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {   // give copies already in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (the leader's, for a pair)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM * CG, BN, a_is_mn(EPI), b_is_mn(EPI));
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      auto commit = [&](uint32_t bar) { if constexpr (CG == 2) tc_commit_pair(bar); else tc_commit(bar); };
      for (int tile = worker; tile < total && ok; tile += n_workers) {
        int ms, nt;
        tile_coords(tile, MS, NT, p.raster_band, ms, nt);
        const int mask = tile_mask(ms);
        if (mask == 0) continue;
        if (!(ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * MT * BN);
        bool first_kb = true;                                  // the first k-block that runs overwrites the accumulator
        for (int kb = 0; kb < nkb; ++kb) {
          if (!kb_on(kb)) continue;
          if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STG;
          const uint32_t sb = sa + MT * A_BYTES;
          const uint64_t db = b_is_mn(EPI) ? make_mnmajor_sw128_desc(sb) : make_kmajor_sw128_desc(sb);
          // one MMA consumes 16 k.  K-major: 32 B further along the 128 B swizzle row (+2 in the
          // >>4 address field).  MN-major: two 8-row atoms of 1024 B further (+128).
          constexpr uint64_t ka = a_is_mn(EPI) ? 128 : 2, kbs = b_is_mn(EPI) ? 128 : 2;
#pragma unroll
          for (int j = 0; j < MT; ++j) {
            if (mask & (1 << j)) {
              const uint64_t da = a_is_mn(EPI) ? make_mnmajor_sw128_desc(sa + j * A_BYTES) : make_kmajor_sw128_desc(sa + j * A_BYTES);
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) {
                const uint32_t accum = (uint32_t)(!(first_kb && k == 0));
                if constexpr (CG == 2) tc_mma_bf16_pair(d_tmem + (uint32_t)(j * BN), da + ka * k, db + kbs * k, idesc, accum);
                else tc_mma_bf16(d_tmem + (uint32_t)(j * BN), da + ka * k, db + kbs * k, idesc, accum);
              }
            }
          }
          first_kb = false;
          commit(empty_bar(stage));
          if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        commit(tfull_bar(acc));
        if (++acc == NACC) { acc = 0; acc_phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue warps: EG groups of 4
    const int quad = warp & 3;           // TMEM lane quadrant this warp may read
    const int grp = (warp - 2) / 4;      // group g drains the accumulators j with j % EG == g
    WarpOut wo{out_base + (uint32_t)(warp - 2) * (8192u / EG), &tmOut, lane, 0, 2 / EG};
    int acc = 0; uint32_t acc_phase = 0;
    for (int tile = worker; tile < total; tile += n_workers) {
      int ms, nt;
      tile_coords(tile, MS, NT, p.raster_band, ms, nt);
      const int mask = tile_mask(ms);
      if (mask == 0) continue;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int j = 0; j < MT; ++j) {
        const int pos = (ms * MT + j) * CG + rank;      // this CTA's M position of accumulator j
        if ((mask & (1 << j)) && (j % EG) == grp && pos_on(pos))
          epilogue_tile<EPI>(p, tmem_base + (uint32_t)((acc * MT + j) * BN), quad, lane, blk_of(pos), nt, wo);
      }
      tc_fence_before();
      if constexpr (CG == 2) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));    // the leader's MMA issuer waits on it
      else mbar_arrive(tempty_bar(acc));
      if (++acc == NACC) { acc = 0; acc_phase ^= 1u; }
    }
    wo.drain();      // staged stores must have left shared memory before the CTA exits
  }

  tc_fence_before();
  __syncthreads();
  // a pair leaves together: the leader's MMAs read the partner's shared memory and the partner's
  // epilogue signals the leader's barriers
  if constexpr (CG == 2) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if constexpr (CG == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode_fn() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    return (EncodeTiledFn)ptr;
  return nullptr;
}
EncodeTiledFn get_encode_fn() {
  static const EncodeTiledFn fn = lookup_encode_fn();   // initialised once, also under concurrent first calls
  return fn;
}

// 2-D bf16 tensor [rows, K] with row pitch `ld` elements; box = [box_rows, 64] elements, 128 B swizzle.
// (MN-major operand: stored [K, mn] with mn contiguous; box = 64 (mn) x 64 (k).)
bool make_tmap(CUtensorMap* tm, const void* base, long rows, long K, long ld, int box_rows, bool mn_major) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)(mn_major ? rows : K), (cuuint64_t)(mn_major ? K : rows)};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)64, (cuuint32_t)(mn_major ? BK : box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Output tile map for the staged stores: [outer, inner] elements, box = 32 rows x 128 bytes.
bool make_out_tmap(CUtensorMap* tm, void* base, long inner, long outer, long ld, bool f32) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const int esz = f32 ? 4 : 2;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
  cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32u};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int EPI, int CG>
cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmOut, const TcArgs& a, int workers,
                       cudaStream_t s) {
  static std::atomic<bool> attr_set[64];   // the attribute is per device; setting it twice is harmless
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<EPI, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(workers * CG));
  cfg.blockDim = dim3((unsigned)TileCfg<EPI, CG>::THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (CG > 1) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tc_gemm_kernel<EPI, CG>, tmA, tmB, tmOut, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int CG>
cudaError_t launch_cg(const TcGemm& g, cudaStream_t s) {
  CUtensorMap tmA, tmB;
  if (!make_tmap(&tmA, g.A, g.a_rows, g.K, g.a_ld, BM, a_is_mn(g.epi))) return cudaErrorInvalidValue;
  if (!make_tmap(&tmB, g.B, g.b_rows, g.b_k > 0 ? g.b_k : g.K, g.b_ld, BN / CG, b_is_mn(g.epi))) return cudaErrorInvalidValue;
  CUtensorMap tmOut = tmA;      // unused by the LSE and DH epilogues
  if (g.epi == TC_EPI_DS || g.epi == TC_EPI_E) {
    if (!make_out_tmap(&tmOut, g.dS, g.N, (long)g.blk_cap * BM, g.ds_ld, false)) return cudaErrorInvalidValue;
  } else if (g.epi == TC_EPI_DW) {
    if (!make_out_tmap(&tmOut, g.dW, g.N, g.V, g.dw_ld, true)) return cudaErrorInvalidValue;
  }
  TcArgs a;
  a.N = g.N; a.K = g.K; a.m_blocks_fixed = g.m_blocks; a.blk_off = g.blk_off; a.blk_cap = g.blk_cap;
  a.rows_cap = g.rows_cap; a.V = g.V; a.pos_off = g.pos_off; a.pos_cap = g.pos_cap;
  a.pace_ctr = g.pace_ctr; a.pace_every = g.pace_every;
  a.nblk = g.rb.nblk; a.n_rows = g.rb.n_rows; a.rowmap = g.rb.rowmap;
  a.ids = g.ids; a.lse = g.lse; a.g = g.g; a.partials = g.partials; a.tgt = g.tgt;
  a.dS = g.dS; a.ds_ld = g.ds_ld;
  a.dHidden = g.dHidden; a.dh_ld = g.dh_ld; a.dh_rows = g.dh_rows; a.dW = g.dW; a.dw_ld = g.dw_ld; a.status = g.status;
  a.psum = g.psum; a.row_scale = g.row_scale; a.blk_active = g.blk_active;
  const bool fwd = (g.epi == TC_EPI_LSE || g.epi == TC_EPI_E || g.epi == TC_EPI_DS);
  const int mt = (CG == 2) ? (fwd ? 1 : 2) : (g.epi == TC_EPI_LSE ? 1 : 2);     // as TileCfg
  // rows of M tiles rasterised together, so that their A rows stay in L2 while B streams: the
  // caller gives it in 128-row blocks
  int band_blocks = g.raster_band_blocks > 0 ? g.raster_band_blocks : 32;
  if (const int env_band = tc_raster_band_override(g.epi)) band_blocks = env_band;
  a.raster_band = band_blocks / (mt * CG);
  if (a.raster_band < 1) a.raster_band = 1;
  const int NT = cdiv(g.N, BN);
  const int m_extent = g.epi == TC_EPI_DW ? g.m_blocks : (g.pos_cap > 0 && g.pos_cap < g.blk_cap ? g.pos_cap : g.blk_cap);
  const long max_tiles = (long)cdiv(m_extent, mt * CG) * NT;
  const int slots = tc_num_sms() / CG;
  const int workers = (int)(max_tiles < (long)slots ? (max_tiles > 0 ? max_tiles : 1) : slots);
  switch (g.epi) {
    case TC_EPI_LSE: return launch_one<TC_EPI_LSE, CG>(tmA, tmB, tmOut, a, workers, s);
    case TC_EPI_DS: return launch_one<TC_EPI_DS, CG>(tmA, tmB, tmOut, a, workers, s);
    case TC_EPI_DH: return launch_one<TC_EPI_DH, CG>(tmA, tmB, tmOut, a, workers, s);
    case TC_EPI_DW: return launch_one<TC_EPI_DW, CG>(tmA, tmB, tmOut, a, workers, s);
    case TC_EPI_E: return launch_one<TC_EPI_E, CG>(tmA, tmB, tmOut, a, workers, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

int tc_num_sms() {
  static std::atomic<int> n[64];
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return 1;
  int v = n[dev].load(std::memory_order_relaxed);
  if (!v) {
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    n[dev].store(v, std::memory_order_relaxed);
  }
  return v > 0 ? v : 1;
}

// CTAs per MMA when the caller leaves it open: the build's default, or TRL_CTA_GROUP=1|2 from the
// environment (read once).  Pairs do a few % more work per clock (less shared-memory traffic), but
// on a power-capped B200 they draw more power per FLOP and end up slower, so 1 is the default.
static int default_cta_group(bool fwd) {
  static const int env = [] {
    const char* e = getenv("TRL_CTA_GROUP");
    return (e && (e[0] == '1' || e[0] == '2') && e[1] == 0) ? e[0] - '0' : 0;
  }();
  return env ? env : (fwd ? TRL_CTA_GROUP_FWD : TRL_CTA_GROUP_BWD);
}

int tc_default_cta_group(int fwd) { return default_cta_group(fwd != 0); }

// Number of 128-row M positions whose tiles (over the N extent `n_cols`) fill whole waves of the
// persistent grid, for a gradient-type GEMM (256-row CTA tiles; 512-row pair tiles with cluster pairs).
int tc_wave_aligned_blocks(int n_cols) {
  const int cg = default_cta_group(false);
  const int slots = tc_num_sms() / cg;
  const int nt = cdiv(n_cols, BN);
  int a = slots, b = nt;
  while (b) { const int t = a % b; a = b; b = t; }      // a = gcd(slots, nt)
  return (slots / a) * 2 * cg;
}

// Raster band (in 128-row blocks) per GEMM from the environment, for sweeps: TRL_RASTER_BAND_LSE,
// _DS, _DH, _DW, _E (read once; 0 = the library's own choice).
int tc_raster_band_override(int epi) {
  static const struct Bands {
    int v[5];
    Bands() {
      const char* names[5] = {"TRL_RASTER_BAND_LSE", "TRL_RASTER_BAND_DS", "TRL_RASTER_BAND_DH", "TRL_RASTER_BAND_DW",
                              "TRL_RASTER_BAND_E"};
      for (int i = 0; i < 5; ++i) {
        const char* e = getenv(names[i]);
        const int x = e ? atoi(e) : 0;
        v[i] = (x > 0 && x <= 4096) ? x : 0;
      }
    }
  } bands;
  return (epi >= 0 && epi < 5) ? bands.v[epi] : 0;
}

cudaError_t launch_tc_gemm(const TcGemm& g, cudaStream_t s) {
  const int cg = g.cta_group > 0 ? g.cta_group : default_cta_group(!(g.epi == TC_EPI_DH || g.epi == TC_EPI_DW));
  return cg == 2 ? launch_cg<2>(g, s) : launch_cg<1>(g, s);
}

}  // namespace trl
