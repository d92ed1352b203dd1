/*
 * libtrl — HRD policy-gradient scoring path for sm_100a (B200), C ABI.
 *
 * The calls follow the statement of the objective in Section 2.3 of the TritonRL paper
 * ("Policy Optimization with Hierarchical Reward Decomposition"):
 *
 *   J(theta)   = E_i [ alpha J^plan_i + J^code_i ]
 *   J^c_i      = (1/G) sum_j (1/|o_ij|) sum_{t in T^c_ij} min[ A^c_ij s_ijt , A^c_ij clip(s_ijt, 1-eps, 1+eps) ]
 *   s_ijt      = pi_theta(o_ijt | .) / pi_theta_old(o_ijt | .)
 *   A^c_ij     = r^c_ij - (1/G) sum_j r^c_ij ,   r^plan = R^speedup, r^code = R^correct   (Eq. 2)
 *
 * Shapes.  P prompts, G rollouts per prompt, B = P*G rollouts, each right-padded to T
 * response tokens; N = B*T rows, row n = b*T + t.  len[b] in [0,T] is |o_ij|, bnd[b] in
 * [0,len[b]] is the index of the first code token (t < bnd: plan segment; bnd <= t < len:
 * code segment).  hidden[n,:] (H values) is the final hidden state that predicts token
 * ids[n]; W is the LM head, [V,H] row-major, no bias, temperature 1.
 *
 * Conventions.
 *  - Every pointer is a DEVICE pointer owned by the caller unless a comment says "host".
 *    The library allocates no device memory and keeps no state that affects results; scratch
 *    comes from a caller-provided workspace of at least trl_workspace_bytes(...) bytes,
 *    256-byte aligned.  Workspaces may be reused between calls on the same stream.
 *  - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default
 *    stream).  Calls return without synchronising.
 *  - Return value: TRL_OK or an error found on the host (bad argument, shape, workspace,
 *    CUDA launch error).  Errors found on the device (token id outside [0,V), len outside
 *    [0,T], bnd outside [0,len], a pipeline wait that ran out) are OR-ed as bit
 *    (1 << code) into *status_dev (int32, caller zero-initialises it; may be NULL).  Lengths
 *    and boundaries are clamped; a row whose token id is out of range gets logp = 0 from the call
 *    that scores it and adds nothing to dHidden / dW (trl_pg_step_fused also leaves it out of
 *    the loss and of g; trl_pg_loss_fwd never sees ids and evaluates it with logp = 0).  No
 *    out-of-bounds access happens.
 *  - Outputs for padded rows (t >= len[b]) are defined: 0.
 *  - Row-major everywhere.  bf16 tensors need H % 8 == 0 and V % 8 == 0 (16-byte rows).
 *  - Alignment.  Every [B*T] and every matrix argument (hidden, W, dHidden, dW, ids, logp,
 *    old_logp, lse, adv, seg, g) must start on a 16-byte boundary: the kernels use 16-byte
 *    accesses and TMA on them.  Per-rollout arrays and scalars (len, bnd, rewards, A_*, n_*,
 *    loss, stats, status_dev) need the alignment of their element type (n_valid: 8 bytes).  A
 *    call given a pointer that breaks this returns TRL_ERR_INVALID_ARG before anything is
 *    launched.  (Allocations from cudaMalloc or a framework's allocator are 256-byte aligned;
 *    the rule matters for offset views into them.)
 */
#ifndef TRL_H_
#define TRL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TRL_OK = 0,
  TRL_ERR_INVALID_ARG = 1,
  TRL_ERR_SHAPE = 2,
  TRL_ERR_DTYPE = 3,
  TRL_ERR_WORKSPACE_TOO_SMALL = 4,
  TRL_ERR_ARCH = 5,       /* device is not compute capability 10.x */
  TRL_ERR_CUDA = 6,       /* a CUDA runtime / driver call failed   */
  TRL_ERR_BAD_INDEX = 7,  /* device-detected: id, len or bnd out of range */
  TRL_ERR_TIMEOUT = 8,    /* device-detected: a bounded pipeline wait expired */
  TRL_ERR_BAD_HINT = 9,   /* device-detected: lse_hint so far off that exp(z - hint) left the fp32 range */
  TRL_ERR_ROWS_BOUND = 10, /* device-detected: more valid rows than the caller's rows_bound (trl_pg_step_fused_banded) */
  TRL_ERR_BOUNDS = 11     /* device-detected, bounds-checked debug build only: a store whose index was computed from the
                             row packing fell outside its buffer (the store is skipped) */
} trl_status;

/* Storage type of hidden / W / dHidden.  TRL_BF16 runs on the tcgen05 tensor cores with
 * fp32 accumulation; TRL_F32 runs fp32 CUDA-core kernels (small problems, second opinion). */
typedef enum { TRL_F32 = 0, TRL_BF16 = 1 } trl_dtype;

typedef enum {
  TRL_CALL_TOKEN_LOGPROBS = 0,
  TRL_CALL_PG_LOSS_FWD = 1,
  TRL_CALL_PG_LOSS_BWD = 2,
  TRL_CALL_PG_STEP_FUSED = 3
} trl_call;

/* Hyper-parameters of the surrogate.  The paper uses eps_lo = eps_hi = 0.2 (training
 * details appendix) and alpha = 0.1 (Section 3.1); alpha weights the plan term. */
typedef struct {
  float eps_lo;   /* lower clip: ratio clipped at 1 - eps_lo */
  float eps_hi;   /* upper clip: ratio clipped at 1 + eps_hi */
  float alpha;    /* weight of J^plan; J^code has weight 1   */
  int clip_form;  /* 0: min[A s, A clip(s)], the HRD objective of Section 2.3.
                     1: A min{s, clip(s)}, the form printed in the uniform-reward appendix; it
                        differs for A < 0 (there s > 1+eps_hi saturates and s < 1-eps_lo does not) */
  int agg_mode;   /* 0: (1/P) sum_i (1/G) sum_j (1/|o_ij|) sum_t, as in the paper.
                     1: mean over all valid tokens of the call (not in the paper)              */
} trl_pg_config;

/* Bytes of workspace the given call wants for these shapes (recommended size).
 * trl_pg_loss_bwd accepts any workspace >= trl_workspace_bytes_min(...) and processes rows
 * in as many chunks as the workspace allows; larger is faster up to the recommended size.
 * Returns 0 for an unknown call or invalid shape. */
size_t trl_workspace_bytes(int which_call, int B, int T, int H, int V, trl_dtype dt);
size_t trl_workspace_bytes_min(int which_call, int B, int T, int H, int V, trl_dtype dt);

/*
 * Token scoring: log pi(o_t | .) of the sampled tokens under one model (Section 2.3, the
 * token probabilities in the ratio s_ijt).  Call once with the current policy's
 * (hidden, W) and once with the old policy's ("reference model" in the uniform-reward
 * appendix) to obtain logp and old_logp.
 *
 *   z[n,v] = sum_k hidden[n,k] W[v,k];  lse[n] = log sum_v exp z[n,v];  logp[n] = z[n,ids[n]] - lse[n]
 *
 * The [N,V] logits are never written to memory (bf16 path: vocabulary tiles are reduced
 * to a running (max, sum-exp) pair in the GEMM epilogue).  The workspace holds a packed copy
 * of the valid rows of `hidden` and the per-tile partials.
 *
 * in : hidden [B*T,H] dt; W [V,H] dt; ids [B*T] int32; len [B] int32
 * out: logp [B*T] f32; lse [B*T] f32 (save lse for trl_pg_loss_bwd)
 */
int trl_token_logprobs(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                       int B, int T, int H, int V, trl_dtype dt,
                       float* logp, float* lse,
                       void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Hierarchical Reward Decomposition (Section 2.3, Eq. 2 and the sentence before it):
 * per-class group-relative advantages, segment labels and per-token advantages.
 *
 *   A_plan[b] = r_plan[b] - mean over the G rollouts of the same prompt (same for A_code)
 *   seg[n] = 1 (plan) if t < bnd[b]; 2 (code) if bnd[b] <= t < len[b]; 0 (padding)
 *   adv[n] = A_plan[b] / A_code[b] / 0 accordingly
 *   n_plan[b] = bnd[b]; n_code[b] = len[b] - bnd[b]; *n_valid = sum_b len[b]
 *
 * adv_mode 0: A = r - mean (the paper).  adv_mode 1: A = (r - mean) / (population std + 1e-6)
 * (not in the paper; the common GRPO normalisation).  Group means are taken in fp64, so a
 * group of identical rewards gives exactly 0.
 *
 * in : r_plan, r_code [P*G] f32; len, bnd [P*G] int32
 * out: A_plan, A_code [P*G] f32; seg [P*G*T] u8; adv [P*G*T] f32; n_plan, n_code [P*G] int32;
 *      n_valid [1] int64.  Needs no workspace.
 */
int trl_hrd_advantages(const float* r_plan, const float* r_code,
                       const int32_t* len, const int32_t* bnd, int P, int G, int T, int adv_mode,
                       float* A_plan, float* A_code, uint8_t* seg, float* adv,
                       int32_t* n_plan, int32_t* n_code, int64_t* n_valid,
                       int32_t* status_dev, void* stream);

/*
 * Clipped surrogate (Section 2.3, the two displayed equations for J and J^c):
 *
 *   s = exp(logp - old_logp);  u = min(adv*s, adv*clip(s, 1-eps_lo, 1+eps_hi))
 *   loss = -(1/P) sum_i (1/G) sum_j (1/len_ij) sum_{t<len_ij} w_t u_t,  w = alpha (plan), 1 (code)
 *   g[n] = d loss / d logp[n] = -w adv s / (P G len) where the unclipped branch is the min, else 0
 *
 * cfg.clip_form / cfg.agg_mode select the two documented variants.  Uniform-reward GRPO (the
 * paper's baseline, one advantage for all tokens of a rollout) is this call with
 * r_plan = r_code = beta R^correct + (1 - beta) R^speedup in trl_hrd_advantages and alpha = 1.
 *
 * Both classes are divided by the whole response length |o_ij| = len.  The sum is taken in
 * a fixed order (bit-reproducible).
 *
 * in : logp, old_logp, adv [P*G*T] f32; seg [P*G*T] u8; len [P*G] int32
 * out: loss [1] f32; g [P*G*T] f32 (0 on padding);
 *      stats [4] f32 or NULL: fraction of valid tokens with s > 1+eps_hi, fraction with
 *      s < 1-eps_lo, mean s, number of valid tokens.
 */
int trl_pg_loss_fwd(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                    const int32_t* len, int P, int G, int T, trl_pg_config cfg,
                    float* loss, float* g, float* stats,
                    void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Backward of the loss to the LM-head inputs (the paper differentiates the objective of
 * Section 2.3 automatically; this is the chain rule through logp = z[ids] - lse):
 *
 *   dS[n,v] = g[n] (1[v = ids[n]] - exp(z[n,v] - lse[n]))      (softmax recomputed from lse)
 *   dHidden = dS W        dW = dS^T hidden
 *
 * dS exists only for one chunk of rows at a time inside the workspace.
 *
 * in : hidden, W, ids, len as in trl_token_logprobs; lse [B*T] f32 from it; g [B*T] f32
 * out: dHidden [B*T,H] dt (padded rows 0); dW [V,H] f32 (overwritten)
 */
int trl_pg_loss_bwd(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                    const float* lse, const float* g,
                    int B, int T, int H, int V, trl_dtype dt,
                    void* dHidden, float* dW,
                    void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Fused schedule of trl_token_logprobs (current policy) + trl_pg_loss_fwd + trl_pg_loss_bwd:
 * same inputs, same outputs, same definitions (Section 2.3 objective and its chain rule), but
 * the forward GEMM is not repeated in the backward.  Per chunk of rows the forward GEMM stores
 * E = exp(z - c) (bf16, chunk-bounded scratch) for a per-row shift c = lse_hint[n]; then
 * lse = c + log sum_v E, logp, g follow per row, and because softmax = E exp(c - lse) the
 * gradient GEMMs run on E directly with the per-row factor folded into their other operand.
 * Results do not depend on c beyond rounding.
 *
 * lse_hint [B*T] f32: any value within ~80 of the row's true log-partition, e.g. the old
 * policy's lse from trl_token_logprobs.  NULL: the exact lse is computed first by an extra
 * forward pass (then this call costs what the three separate calls cost).  A hint so wrong that
 * exp(z - hint) overflows sets TRL_ERR_BAD_HINT in *status_dev.
 *
 * in : hidden, W, ids, len as in trl_token_logprobs; old_logp, adv [B*T] f32, seg [B*T] u8
 *      (from trl_hrd_advantages); lse_hint or NULL
 * out: logp, lse, g [B*T] f32 (0 on padding); loss [1]; stats [4] or NULL;
 *      dHidden [B*T,H] dt (padded rows 0); dW [V,H] f32 (overwritten)
 * TRL_F32 runs the three separate calls internally.
 */
int trl_pg_step_fused(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                      const float* old_logp, const float* lse_hint, const float* adv, const uint8_t* seg,
                      int P, int G, int T, int H, int V, trl_dtype dt, trl_pg_config cfg,
                      float* logp, float* lse, float* loss, float* g, float* stats,
                      void* dHidden, float* dW,
                      void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * trl_pg_step_fused for data-parallel training: same inputs, outputs and results (bit for bit),
 * but dW becomes final band by band, so that its reduction across ranks can overlap the rest of
 * the dW GEMM.  The paper trains on 8 GPUs (training-details appendix) without describing how; the
 * path shards by prompt group, and the LM-head gradient is the one tensor the ranks must sum.
 *
 * E = exp(z - c) is kept for all rows instead of one chunk (workspace:
 * trl_pg_step_fused_banded_workspace_bytes, about rows_bound * V * 2 bytes more), the forward and
 * the dHidden GEMM run chunk by chunk as before, and then the dW GEMM runs once per band of
 * vocabulary rows [band_begin[j], band_begin[j+1]) over all chunks.  After the last launch of
 * band j the event band_events[j] is recorded on `stream`: rows band_begin[j] .. band_begin[j+1]
 * of dW are final from that point of the stream on.  The caller makes a second stream wait for
 * the event and starts the band's all-reduce there (NCCL or its own kernel); nothing in this
 * library communicates.
 *
 * n_bands, band_begin [n_bands + 1] (host): band_begin[0] = 0, band_begin[n_bands] = V, increasing,
 *   every band_begin[j] a multiple of 256 (trl_dw_band_plan makes such a split).
 * band_events [n_bands] (host array of cudaEvent_t, or NULL; single entries may be NULL).
 * rows_bound: an upper bound on sum_b len[b] known on the host, or 0 for B*T.  It sizes the
 *   workspace; if the batch has more valid rows, TRL_ERR_ROWS_BOUND is set in *status_dev and the
 *   excess rows are dropped.
 * TRL_BF16 only.
 */
int trl_pg_step_fused_banded(const void* hidden, const void* W, const int32_t* ids, const int32_t* len,
                             const float* old_logp, const float* lse_hint, const float* adv, const uint8_t* seg,
                             int P, int G, int T, int H, int V, trl_dtype dt, trl_pg_config cfg,
                             float* logp, float* lse, float* loss, float* g, float* stats,
                             void* dHidden, float* dW,
                             int n_bands, const int32_t* band_begin, void* const* band_events, int rows_bound,
                             void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);
size_t trl_pg_step_fused_banded_workspace_bytes(int B, int T, int H, int V, int rows_bound);
/* Splits the V rows of dW into at most n_bands_wanted bands of whole 256-row tiles, sized so that
 * each band's launch fills whole waves of CTAs.  Writes band_begin [returned count + 1] (host; give
 * it n_bands_wanted + 1 entries) and returns the number of bands (0 on bad arguments). */
int trl_dw_band_plan(int V, int H, int n_bands_wanted, int32_t* band_begin);

/*
 * Same computation and outputs as trl_pg_loss_fwd, for callers that cannot allocate device
 * memory and so cannot supply its workspace: a trainer whose memory arena already owns the
 * whole device (a further cudaMalloc fails or fragments it), or a step loop that cannot
 * afford the device-wide synchronisation cudaMalloc / cudaFree imply.  (The paper has no
 * counterpart to this call; it exists for such callers only.)
 *
 * The partial sums live in a fixed 1 MiB array inside the library image (every GPU that
 * loads the library holds it until the process exits).  Limit: P*G*ceil(T/16384) <= 65536,
 * otherwise TRL_ERR_WORKSPACE_TOO_SMALL is returned and nothing is launched.  The call
 * performs no cudaMalloc / cudaFree and calls no allocating routine; inputs and outputs are
 * still the caller's device buffers.
 *
 * The first call on each device looks up the array's device address (the device must be
 * current); make that first call before starting any stream capture.  All calls on a
 * device share the one array: two calls whose kernels may overlap on the GPU (different
 * streams without an ordering between them) race on it and give wrong sums; calls on one
 * stream, or otherwise ordered, are fine.  The array keeps whatever the last call left in
 * it; every value a call reads it has written itself first, so nothing needs clearing.
 */
int trl_pg_loss_fwd_static(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                           const int32_t* len, int P, int G, int T, trl_pg_config cfg,
                           float* loss, float* g, float* stats, int32_t* status_dev, void* stream);

/* Number of kernels this library has enqueued so far in this process (all streams, all
 * calls; memsets are not counted).  Host-side statistic used by the benchmark; there is no
 * counterpart in the paper. */
unsigned long long trl_kernel_launches(void);

/* Host string naming the tuning settings in effect,
 * "cta_group_fwd=<n> cta_group_bwd=<n> raster_band_lse=<n> raster_band_e=<n> raster_band_dh=<n> raster_band_dw=<n>":
 * how many CTAs share one tensor-core instruction in the forward and in the gradient GEMMs (1, or 2
 * for cluster pairs), and how many 128-row blocks of tiles each GEMM rasterises together (the rows
 * that stay in L2 while the other operand streams).  Environment variables, read at the first call,
 * override the library's choices: TRL_CTA_GROUP=1|2 and TRL_RASTER_BAND_LSE / _E / _DH / _DW / _DS=<blocks>.
 * Results are the same whatever the settings.  No counterpart in the paper. */
const char* trl_config_string(void);

/* Host string for a status code (static storage). */
const char* trl_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* TRL_H_ */
