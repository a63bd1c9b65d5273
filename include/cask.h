/*
 * cask.h -- C-ABI boundary of the B200 compression-event library (libcask.so).
 *
 * One "unit" is one (sequence, layer, KV head): a cache of T rows of head_dim
 * elements for keys and for values, rows [0,P) the prompt prefix and rows
 * [P,T) the decode trace, plus the last W ("window") queries of the g query
 * heads that share the KV head.  A compression event reduces every unit to at
 * most B rows.  Units are independent; a batch is a ragged list of units.
 *
 * Conventions that hold for every call unless a parameter says otherwise:
 *   - DEVICE pointers: k, v, q, lse_in, every output array, the workspace.
 *     They are owned by the caller; the library allocates no device memory.
 *   - HOST pointers: the cask_batch struct itself and its per-unit integer
 *     arrays (T, P, B, reserve, k_off, v_off, tok_off); they are read during
 *     the call and may be freed when it returns.
 *   - Calls are asynchronous on the context's stream.  The int returned is 0
 *     or a negative CASK_ERR_* found on the host BEFORE any launch; nothing
 *     on the device traps.  Per-unit outcomes are CASK_ST_* bits.
 *   - Inputs are never modified; outputs must not alias inputs.
 *   - Per-row arrays ("[sumT]") are indexed by tok_off[u] + i.
 *   - Per-slot arrays are [n_units, Bmax]; Bmax >= max_u B[u].
 */
#ifndef CASK_H
#define CASK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes ------------------------------------------------------- */
#define CASK_OK                 0
#define CASK_ERR_NULL          -1   /* a required pointer is NULL                     */
#define CASK_ERR_SHAPE         -2   /* head_dim/group/window/T/P/B/reserve out of range */
#define CASK_ERR_ALIGN         -3   /* a base pointer, offset or row stride breaks the 16-byte rule */
#define CASK_ERR_WORKSPACE     -4   /* workspace NULL or smaller than cask_workspace_bytes */
#define CASK_ERR_UNSUPPORTED   -5   /* a documented but unbuilt combination (paged cache through
                                       the host-buffer or the no-allocation entry point, the
                                       no-allocation entry point on a stream that is being captured) */
#define CASK_ERR_CUDA          -6   /* a CUDA runtime call failed (see cask_last_cuda_error) */
#define CASK_ERR_PARAM         -7   /* gamma/tau/eps/causal out of range              */
#define CASK_ERR_TOO_LARGE     -8   /* batch exceeds a fixed capacity (cask_score_noalloc) */

/* ---- per-unit status bits (plan[6], unit_status[u]) --------------------- */
#define CASK_ST_NOOP_UNDER_BUDGET        1   /* T <= B: every row kept                        */
#define CASK_ST_PREFIX_EVICTED           2   /* stage 1 removed prefix rows                   */
#define CASK_ST_DECODE_CONSOLIDATED      4   /* stage 2 ran core protection + consolidation   */
#define CASK_ST_PREFIX_BUDGET_EXHAUSTED  8   /* decode share cannot hold window + core + rep  */
#define CASK_ST_MERGE_INACTIVE          16   /* stage 2 ran but no row joined any seed        */
#define CASK_ST_TIMEOUT                 32   /* a bounded device wait gave up                 */
#define CASK_ST_BOUNDS                  64   /* a device-side index check failed              */

/* ---- row kinds (kind[i], slot_kind[t]) ---------------------------------- */
#define CASK_KIND_DROPPED  0
#define CASK_KIND_PREFIX   1   /* kept prefix row                          */
#define CASK_KIND_RECENT   2   /* one of the last r decode rows            */
#define CASK_KIND_CORE     3   /* protected core chosen by score           */
#define CASK_KIND_SEED     4   /* anchor of a representative               */
#define CASK_KIND_MERGED   5   /* scratch row folded into a representative */

/* ---- plan[u][0..7] ------------------------------------------------------ */
#define CASK_PLAN_BP     0   /* prefix share B_p = B - reserve            */
#define CASK_PLAN_PKEEP  1   /* prefix rows kept = min(P, B_p)            */
#define CASK_PLAN_BD     2   /* decode share B_d = B - P_keep             */
#define CASK_PLAN_R      3   /* recent rows r                             */
#define CASK_PLAN_C      4   /* core rows chosen by score c               */
#define CASK_PLAN_M      5   /* representatives m                         */
#define CASK_PLAN_FLAGS  6   /* structural CASK_ST_* bits                 */
#define CASK_PLAN_NOUT   7   /* rows after the event                      */

#define CASK_DTYPE_BF16 0
#define CASK_DTYPE_FP32 1

typedef struct cask_ctx cask_ctx;

/*
 * A ragged batch of independent units (Sec. 2.3 of the paper constrains one
 * cache at a time: |R| <= B, C subset of R; nothing couples units).
 * Layout, contiguous (page_size == 0): row i of unit u starts at element
 *   k + k_off[u] + i*row_stride            (same for v with v_off)
 * Layout, paged (page_size > 0): k and v are page pools of n_pages pages of
 * page_size rows; row i of unit u starts at element
 *   k + (block_table[bt_off[u] + i/page_size]*page_size + i%page_size)*row_stride
 * (same page ids for v); k_off and v_off are ignored.  The block table is read
 * on the device; a page id outside [0, n_pages) raises CASK_ST_BOUNDS for the
 * call and is treated as page 0, so nothing is read out of bounds.  The
 * tensor-core kernels serve page sizes 8, 16, 32, 64 and multiples of 128;
 * other page sizes run on the SIMT kernels.  The compacted cache is always
 * written dense ([n_units, Bmax, d]).
 * row_stride >= head_dim; base pointers, offsets*elem and row_stride*elem must
 * be multiples of 16 bytes.  q is [n_units, group, window, head_dim], dense;
 * window query j of a unit belongs to cache row T-window+j.
 */
typedef struct {
    int32_t n_units;
    int32_t head_dim;        /* d: multiple of 8, 8..256                        */
    int32_t group;           /* g: query heads per KV head, >= 1                */
    int32_t window;          /* W: 1 <= W <= T[u] for every unit               */
    int32_t dtype;           /* CASK_DTYPE_BF16 | CASK_DTYPE_FP32 (k, v, q, outputs) */
    int32_t page_size;       /* 0 = contiguous rows; > 0 = rows per page of a paged cache */
    const void* k;           /* DEVICE */
    const void* v;           /* DEVICE */
    const int64_t* k_off;    /* HOST [n_units], elements                        */
    const int64_t* v_off;    /* HOST [n_units], elements                        */
    int64_t row_stride;      /* elements                                        */
    const void* q;           /* DEVICE [n_units, g, W, d]                       */
    const float* lse_in;     /* DEVICE [n_units, g, W] natural-log normalisers of the
                                window queries, or NULL to have them computed   */
    const int32_t* T;        /* HOST [n_units] rows in the cache                */
    const int32_t* P;        /* HOST [n_units] prefix rows, 0 <= P <= T         */
    const int32_t* B;        /* HOST [n_units] budget, >= 1                     */
    const int32_t* reserve;  /* HOST [n_units] slots held back for decode, 0..B */
    const int64_t* tok_off;  /* HOST [n_units+1] offsets into per-row arrays; tok_off[u+1]-tok_off[u] >= T[u] */
    /* paged cache only (page_size > 0) */
    const int32_t* block_table; /* DEVICE physical page id of every logical page, unit after unit */
    const int64_t* bt_off;   /* HOST [n_units+1] first entry of each unit; bt_off[u+1]-bt_off[u] >= ceil(T[u]/page_size) */
    int64_t n_pages;         /* pages in the k and v pools                      */
    /* optional: mass already carried by a row (a representative of an earlier event brings the
       slot_mass it was given then, every other row 0).  Merge weights become
       a_i = s_i + eps + mass_in[i] (Sec. 2.4: the fold preserves group mass); NULL = all zero. */
    const float* mass_in;    /* DEVICE [sumT] or NULL                           */
    /* optional: non-negative channel weights of the merge similarity (Sec. 2.5: frequency bands of
       more future relevance count more; w_c = |kappa(omega_f)| on the channels of band f):
       sim(j,u) = sum_c w_c k_jc k_uc / (|k_j|_w |k_u|_w), |k|_w^2 = sum_c w_c k_c^2.  NULL = cosine. */
    const float* chan_w;     /* DEVICE [head_dim] or NULL                       */
    /* optional, instead of chan_w: the merge distance of Sec. 2.5 in its own, un-squared form,
       d_kappa(k_i,k_j) = sum_f w_f ||k_if - k_jf||_2 over the rotary bands f (pairs of channels), w_f =
       |kappa(omega_f)| >= 0 from the caller.  The paper gives no decision rule for it; the library uses the
       scale-free similarity 1 - d_kappa(k_j,k_u) / (D_j + D_u), D_x = sum_f w_f ||k_xf||_2 (in [0,1]; a row with
       D = 0 has similarity 0) exactly where it uses the cosine: argmax over the seeds, threshold tau.
       band_layout 0: band f = channels (f, f + head_dim/2); 1: channels (2f, 2f + 1).  head_dim must be even.
       This form runs on the SIMT path (one square root per row, seed and band).  NULL = not used. */
    const float* band_w;     /* DEVICE [head_dim/2] or NULL                     */
    int32_t band_layout;     /* 0 | 1; ignored when band_w is NULL              */
} cask_batch;

/*
 * Policy parameters.  The paper gives no values for them (it names a "reserve
 * schedule" and leaves a_i open, Sec. 2.4 / 7.2); defaults in parentheses.
 */
typedef struct {
    float gamma;        /* (0.5) share of the non-recent decode slots given to the core, 0..1 */
    float tau;          /* (0.9) minimum cosine similarity for a scratch row to join a seed   */
    float eps;          /* (1e-9) a_i = s_i + eps keeps every group mass positive, > 0        */
    int32_t causal;     /* (1) window query j sees rows i <= T-W+j; 0: every query sees all rows */
    int32_t score_path; /* (0) 0: tensor-core scoring when the shape allows; 1: always the SIMT kernels */
} cask_params;

/* Outputs of a whole event.  DEVICE pointers; "optional" ones may be NULL. */
typedef struct {
    void* k_out;           /* [n_units, Bmax, d] cache dtype; rows >= n_out[u] are not written */
    void* v_out;           /* [n_units, Bmax, d]                                             */
    int32_t Bmax;
    int32_t* n_out;        /* [n_units] rows kept (== plan[7])                                */
    int32_t* slot_src;     /* [n_units, Bmax] cache row each slot is anchored at, -1 beyond n_out */
    uint8_t* slot_kind;    /* [n_units, Bmax] CASK_KIND_*, 0 beyond n_out                     */
    float* slot_mass;      /* [n_units, Bmax] m_G = sum of a_i over the slot's members        */
    int32_t* assign;       /* [sumT] slot a row went to, -1 if dropped                        */
    float* weight;         /* [sumT] 1 kept singleton, w_i = a_i/m_G group member, 0 dropped  */
    uint8_t* kind;         /* [sumT] CASK_KIND_*                                              */
    int32_t* seed_of;      /* [sumT] cache row of the group's seed (seeds point at themselves), else -1 */
    int32_t* plan;         /* [n_units, 8] CASK_PLAN_*                                        */
    int32_t* unit_status;  /* [n_units] CASK_ST_* bits                                        */
    float* lost_mass;      /* [n_units] sum of a_j over scratch rows that joined nobody       */
    float* s;              /* optional [sumT] scores                                          */
    float* lse;            /* optional [n_units, g, W] natural-log normalisers used           */
    float* sim;            /* optional [sumT] best cosine similarity of non-seed scratch rows, -2 elsewhere */
    /* optional mass diagnostics of Sec. 2.6, [n_units] each: share of the mass of the B best rows of the
       cache that the protected core (recent + core rows) holds, and that the output slots carry */
    float* rho_core;
    float* rho_rep;
    /* optional, [n_units]: within-group dispersion, the first term of the perturbation bound of Sec. 2.6:
       sum over the rows of kind 4/5 of a_i * ||k_i - k~_G||, k~_G the representative as written to k_out, in the
       norm of the merge geometry in use (Euclidean; sqrt(sum_c w_c x_c^2) with chan_w; sum_f w_f ||x_f||_2 with
       band_w).  The second term of that bound is lost_mass. */
    float* dispersion;
} cask_outputs;

/* ---- context ------------------------------------------------------------ */

/* Creates a context bound to `device` and `cuda_stream` (a cudaStream_t, NULL =
 * default stream).  Owns a small pinned staging buffer for per-unit descriptors. */
int cask_create(cask_ctx** out, int device, void* cuda_stream);
int cask_destroy(cask_ctx* ctx);
int cask_set_stream(cask_ctx* ctx, void* cuda_stream);
const char* cask_strerror(int code);
/* Name of the last CUDA error seen by this context ("" if none). */
const char* cask_last_cuda_error(const cask_ctx* ctx);
/* Kernels launched by this context since creation (every call adds its own). */
int64_t cask_launch_count(const cask_ctx* ctx);
/*
 * Optional per-kernel timing.  While enabled, every kernel launch of this context is
 * bracketed by a CUDA event pair on the context's stream.  cask_profile_read waits for
 * the recorded events, adds up the elapsed milliseconds and launch counts per kernel id
 * (arrays of cask_kernel_count() entries, HOST) and forgets them.
 */
int cask_profile_enable(cask_ctx* ctx, int on);
int cask_profile_read(cask_ctx* ctx, float* ms, int64_t* launches);
int cask_kernel_count(void);
const char* cask_kernel_name(int id);
/* 1 if the last cask_score / cask_compress_event used the tensor-core kernels. */
int cask_last_score_path_tensor(const cask_ctx* ctx);
/* Device-side flags (CASK_ST_TIMEOUT, CASK_ST_BOUNDS) raised by the kernels of the last call of this
 * context; waits for the context's stream.  cask_consolidate_scratch ORs the flags raised up to the
 * end of that call into unit_status; cask_compress_event and cask_compress_event_host do so once more
 * as the last step of the event, so there unit_status also carries flags raised by the compaction.
 * The staged cask_compact and cask_writeback_paged write no unit_status: their flags are read here. */
int cask_last_device_flags(cask_ctx* ctx, int32_t* flags_host);

/*
 * SM clock, in kHz, at which the two tensor-core scoring passes of the context's last cask_score /
 * cask_compress_event ran (no counterpart in the paper): one CTA of each pass divides the SM cycles it
 * spent by the wall time they took.  khz_host: HOST, two words (normaliser pass, score pass; 0 for a
 * pass that did not run, both 0 after a call that used the SIMT kernels or the host-buffer entry point).
 * A pass that keeps the exponential, FMA and tensor pipes busy together runs under the board's power
 * limit, below the maximum clock; its rate per clock is judged against this figure.  Waits for the stream.
 */
int cask_last_score_clock_khz(cask_ctx* ctx, int32_t* khz_host);

/*
 * Self-test of the bounded device waits (no counterpart in the paper).  Every wait of the kernels on a
 * hardware barrier gives up after a wall-time limit and makes the kernel end with CASK_ST_TIMEOUT
 * instead of hanging; in a healthy run that path never executes.  This call runs it once: one small
 * CTA waits for `limit_ns` (1,000 .. 100,000,000) on a barrier nobody arrives at, gives up, raises
 * the flag and returns.  Nothing faults and the context stays usable.  ws: DEVICE, at least 64 bytes,
 * 16-byte aligned.  Waits for the stream.  flags_host receives the device flags of the call (also
 * readable through cask_last_device_flags until the next call); waited_ns_host, optional, two words:
 * the time the waiting warp spent before it gave up, and the time two more warps of the CTA, waiting
 * with the default limit (one with each of the two forms of the wait the kernels use: the abort flag
 * read after every probe, or only together with the clock), spent before they saw the first one give
 * up and followed it: the later of the two, 0 if either did not follow.
 */
int cask_selftest_wait_timeout(cask_ctx* ctx, uint64_t limit_ns, void* ws, size_t ws_bytes,
                               int32_t* flags_host, uint64_t* waited_ns_host);

/*
 * Measures what the special-function unit of this GPU sustains (no counterpart in the paper): one CTA of
 * 16 warps per SM runs `iters` (16 .. 2^20) rounds of eight independent chains of the scoring epilogue's
 * per-element mix (FFMA, ex2.approx, FADD, FMUL) and times itself with the SM clock; rate_host receives
 * the median over the SMs of exponentials per clock per SM.  The scoring passes evaluate one exponential
 * per (query row, key), so this rate x SMs x clock is the roof the benchmark holds them against.
 * ws: DEVICE, at least 16 + 8 x SMs bytes, 16-byte aligned.  Waits for the stream.
 */
int cask_selftest_exp_rate(cask_ctx* ctx, int32_t iters, void* ws, size_t ws_bytes, double* rate_host);

/* Bytes of workspace that any call below needs for this batch (host-only arithmetic). */
size_t cask_workspace_bytes(const cask_batch* batch, const cask_params* params);

/*
 * Budget split on the host (Sec. 2.2 slack for the decode stage, Sec. 2.3 |R| <= B
 * with C subset of R, Sec. 5.2 collapse of the available slots).  The paper
 * gives no numbers; the rule used is
 *   B_p = B - reserve;  P_keep = min(P, B_p);  B_d = B - P_keep;  N_d = T - P;
 *   T <= B       -> NOOP_UNDER_BUDGET, all rows kept;
 *   r = min(W, N_d);
 *   N_d <= B_d   -> every decode row kept (c = N_d - r, m = 0);
 *   B_d < r + 2  -> PREFIX_BUDGET_EXHAUSTED: r = min(r, B_d), c = B_d - r, m = 0;
 *   else DECODE_CONSOLIDATED: c = min(ceil(gamma (B_d - r)), B_d - r - 1), m = B_d - r - c.
 * Fills plan[n_units*8] (HOST).  The device calls use the same rule.
 */
int cask_plan_host(const cask_batch* batch, const cask_params* params, int32_t* plan_host);

/* ---- the staged hot path -------------------------------------------------- */

/*
 * Score (Sec. 1: scalar importance per token; the deployed scorer has no
 * formula in the paper, this library uses windowed attention mass):
 *   x_hji = <q_hj, k_i>/sqrt(d);  p = softmax over visible i;  s_i = mean_{h,j} p_hji.
 * s [sumT] fp32 out; lse_out optional [n_units, g, W].
 */
int cask_score(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
               float* s, float* lse_out, void* ws, size_t ws_bytes);

/*
 * A second scorer, from the query-statistics family of the paper's Phase-1 archive (App. B): the horizon kernel
 *     kappa_{pi_h}(omega) = E_{delta ~ pi_h}[e^{i omega delta}] = sum_n pi_h[n] e^{i omega delta_n}
 * of a discrete horizon distribution pi_h over the offsets delta_n, and the horizon-averaged mean score
 *     S_h(k, Delta) = Re sum_f mu_{h,f} conj(k_f) kappa_{pi_h}(omega_f) e^{i omega_f Delta},
 * band f of a vector read as the complex number x[c0] + i x[c1] (channel pairs as for band_w: band_layout 0 =
 * (f, f + head_dim/2), 1 = (2f, 2f + 1)).  The paper gives the two formulas and none of mu, pi, omega, Delta; all
 * come from the caller.  s_i = mean over the g query heads of S_h(k_i, Delta_i), Delta_i = delta[i] or, without
 * `delta`, T - 1 - i (distance to the newest cached row).  No window queries are read and no exponentials taken:
 * one pass over the keys, bound by HBM.  The score is real and can be negative; the merge weights of Sec. 2.4 need
 * a_i > 0, so a caller that feeds these scores to the later stages must shift or clamp them first.
 */
typedef struct {
    const float* mu;          /* DEVICE [n_units, group, head_dim/2, 2] (re, im): mean query per head and band */
    const float* pi;          /* DEVICE [n_units, group, n_delta]: horizon distribution of each head           */
    const float* delta_grid;  /* DEVICE [n_delta]: the offsets pi is defined on                                */
    int32_t n_delta;          /* 1 .. 4096                                                                      */
    const float* omega;       /* DEVICE [head_dim/2]: band frequencies                                          */
    int32_t band_layout;      /* 0 | 1                                                                          */
    const float* delta;       /* DEVICE [sumT] per-row offsets Delta_i, or NULL                                 */
} cask_query_stats;

/* s [sumT] fp32 out.  Uses batch->k, the row layout (contiguous or paged), T, tok_off, group and head_dim (even). */
int cask_score_stats(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                     const cask_query_stats* stats, float* s, void* ws, size_t ws_bytes);

/*
 * Stage 1, prefix eviction (Sec. 2.2): writes plan[n_units,8] and kind for the
 * prefix rows [0,P): the P_keep rows greatest under (score descending, row
 * ascending) get CASK_KIND_PREFIX, the others 0; all P rows if P <= B_p.
 * Decode rows of `kind` are set to 0.
 */
int cask_prefix_evict(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                      const float* s, uint8_t* kind, int32_t* plan, void* ws, size_t ws_bytes);

/*
 * Protected core (Sec. 2.1, 2.3): last r decode rows -> CASK_KIND_RECENT, the c
 * greatest of rows [P, T-r) -> CASK_KIND_CORE; other decode rows stay 0.
 * `plan` is the array cask_prefix_evict wrote.
 */
int cask_select_core(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                     const float* s, const int32_t* plan, uint8_t* kind, void* ws, size_t ws_bytes);

/*
 * Scratch consolidation (Sec. 2.1, 2.4, 2.5): among decode rows of kind 0 the m
 * greatest become seeds (4); every other one joins the seed of highest cosine
 * similarity if that is >= tau (5) or is dropped (0).  Writes seed_of, weight
 * (w_i = a_i/m_G for group members, 0 for dropped scratch), optional sim,
 * unit_status (plan flags | MERGE_INACTIVE) and lost_mass.
 */
int cask_consolidate_scratch(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                             const float* s, const int32_t* plan, uint8_t* kind, int32_t* seed_of,
                             float* weight, float* sim, int32_t* unit_status, float* lost_mass,
                             void* ws, size_t ws_bytes);

/*
 * Compaction (Sec. 2.3 |R| <= B; Sec. 2.4 merge rule): slots are the rows of
 * kind 1..4 in ascending row order; a slot of kind 4 holds sum_i w_i k_i and
 * sum_i w_i v_i over its group (members in ascending row order, fp32
 * accumulation, rounded once to the cache dtype; a group of one is a byte
 * copy); every other slot is a byte copy of its row.  `weight` is read for
 * kinds 4/5 and finalised (1 for kinds 1..3, 0 for kind 0).  Uses out->k_out,
 * v_out, Bmax, n_out, slot_src, slot_kind, slot_mass, assign and, when given,
 * rho_core / rho_rep / dispersion; other fields of `out` are ignored.
 */
int cask_compact(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                 const float* s, const uint8_t* kind, const int32_t* seed_of, float* weight,
                 const cask_outputs* out, void* ws, size_t ws_bytes);

/* The five steps above in order on one stream; results are bit-identical to
 * calling them one by one. */
int cask_compress_event(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                        const cask_outputs* out, void* ws, size_t ws_bytes);

/*
 * Paged cache only: writes the compacted rows back into each unit's own pages (Sec. 2.3: the
 * cache is replaced by its representative set R), slot t of `out` at logical row t, i.e. into
 * the unit's first ceil(n_out/page_size) pages; the other pages of the unit are left as they
 * are and can be returned to the pool by the caller, the block table is not changed.  Call it
 * after the event on the same context (it is ordered on the context's stream); k_pool / v_pool
 * are the pools batch->k / batch->v point to, passed again as writable DEVICE pointers.  Uses
 * out->k_out, v_out, n_out, Bmax.  A contiguous batch is refused with CASK_ERR_SHAPE.
 */
int cask_writeback_paged(cask_ctx* ctx, const cask_batch* batch, const cask_params* params,
                         const cask_outputs* out, void* k_pool, void* v_pool, void* ws, size_t ws_bytes);

/*
 * The same event for callers whose cache lives in HOST memory: batch->k, v,
 * q, lse_in, mass_in, chan_w, band_w and every pointer in `out` are HOST
 * pointers here.  dev_buf is a DEVICE buffer of at least
 * cask_host_event_device_bytes() that holds the staged inputs, outputs and the
 * workspace.  Copies the keys and queries in, decides every row's fate, copies
 * in only the value rows that are kept or merged (gathered through a pinned
 * staging buffer the context owns and grows as needed), compacts, copies out
 * and returns when everything has arrived.
 *
 * A batch with more than 16 MB of keys is cut into up to about ten slices of
 * consecutive units, each a batch of its own inside dev_buf, on streams the
 * context owns (ordered after the work already queued on the context's
 * stream: one for every copy to the device, four the slices take turns on),
 * so that one slice's upload runs while the slice before it is decided,
 * packed, compacted and read back.  For that overlap every HOST
 * array, inputs and outputs, has to be page-locked: a copy to or from pageable
 * memory holds the calling thread until the copy is done.  Units are
 * independent, so the results are those of cask_compress_event on the same
 * units; against one call on the whole batch the last bits of the scores can
 * differ, because the scoring kernel divides a unit's tiles between its CTAs
 * according to what else is in the batch (a batch of one slice gives the same
 * bytes).  cask_last_device_flags() afterwards gives the flags of all slices.
 *
 * Rows of a unit must be dense (row_stride == head_dim) and units laid out at
 * k_off[u] == v_off[u] == tok_off[u]*head_dim; a paged batch is refused with
 * CASK_ERR_UNSUPPORTED, a dev_buf that is too small or not 256-byte aligned
 * with CASK_ERR_WORKSPACE.
 */
size_t cask_host_event_device_bytes(const cask_batch* batch, const cask_params* params, int32_t Bmax);
int cask_compress_event_host(cask_ctx* ctx, const cask_batch* host_batch, const cask_params* params,
                             const cask_outputs* host_out, void* dev_buf, size_t dev_bytes);

/*
 * cask_score for callers that cannot allocate device memory (no counterpart in the paper: it
 * describes no memory management at all).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving engine that has
 * given the whole device to its own memory pool, in a plugin loaded after the memory budget was
 * fixed, or anywhere a workspace cannot be obtained -- and that therefore cannot provide the
 * workspace cask_score asks for.  Here the scratch (unit descriptors, normaliser partials, row
 * tables) sits in one fixed array of CASK_NOALLOC_SCRATCH_BYTES inside the library image; every GPU
 * that loads the library holds that much memory until the process exits.  The call takes no
 * context and makes no cudaMalloc / cudaFree / cudaMallocHost or other allocating call.
 *
 * Same inputs and outputs as cask_score (s [sumT] DEVICE out, lse_out optional DEVICE out), on
 * `device` and `cuda_stream`; it always uses the SIMT scoring kernels, so the scores equal those of
 * cask_score with score_path = 1 and agree with the tensor-core path to rounding.
 * Limits: n_units <= CASK_NOALLOC_MAX_UNITS and
 *   256-byte-rounded sizes of 2 * n_units*g*W*4 + 2 * (sum_u ceil(T[u]/2048))*g*W*4 bytes
 *   + the descriptor table  <=  CASK_NOALLOC_SCRATCH_BYTES;
 * beyond either, CASK_ERR_TOO_LARGE is returned before anything is launched.
 * The first call on a device looks the array's device address up (cudaGetSymbolAddress, once per
 * device); make that first call before any stream capture begins.  A call whose stream is being
 * captured is refused with CASK_ERR_UNSUPPORTED before anything is launched or copied (the unit
 * descriptors go up from a host array that lives only for the duration of the call).  The calling
 * thread's current device is the same after the call as before it.  All calls on a device share
 * the one array: two calls whose kernels may overlap on the GPU (different streams, or different
 * host threads without ordering) race on it and must be serialised by the caller.  Nothing in the
 * array needs clearing between calls: each call writes every word it later reads.
 */
#define CASK_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
#define CASK_NOALLOC_MAX_UNITS 64
int cask_score_noalloc(int device, void* cuda_stream, const cask_batch* batch, const cask_params* params,
                       float* s, float* lse_out);

#ifdef __cplusplus
}
#endif
#endif /* CASK_H */
