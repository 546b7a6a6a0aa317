/*
 * kvc.h -- C ABI of the low-rank KV-cache correction library (B200 / sm_100a).
 *
 * The library turns one agent's shared-context KV cache into the next agent's
 * cache without running the model: it re-aligns cached keys to their new
 * positions (RoPE re-rotation), adds a stored rank-r correction
 * coeff x basis per (layer, KV head), and chains agent to agent with the first
 * agent's cache left exact.  It also builds that rank-r state from an observed
 * pair of caches.
 *
 * Conventions for every entry point
 *   - plain C types only; every pointer says whether it is HOST or DEVICE memory;
 *   - all device work is enqueued on `stream` (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream); no entry point synchronises, and none
 *     allocates device memory: every buffer, scratch included, is the caller's
 *     (kvc_state_update_noalloc alone uses scratch built into the library);
 *   - the return value is KVC_OK (0) or a negative KVC_E_* code; nothing is
 *     launched when an argument check fails;
 *   - bf16 means the upper 16 bits of an IEEE float32, rounded to nearest-even
 *     wherever the library produces one;
 *   - the CUDA device that is current at the call is the one used.
 */
#ifndef KVC_H_
#define KVC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------- */
#define KVC_OK              0
#define KVC_E_INVALID_ARG  (-1)  /* null pointer, negative size, bad enum          */
#define KVC_E_SHAPE        (-2)  /* geometries of the arguments do not agree       */
#define KVC_E_UNSUPPORTED  (-3)  /* valid but not built (head_dim, page size ...)  */
#define KVC_E_ALIAS        (-4)  /* dst overlaps src without being the same cache  */
#define KVC_E_CUDA         (-5)  /* a CUDA runtime / driver call failed            */
#define KVC_E_WORKSPACE    (-6)  /* workspace missing, misaligned or too small     */
#define KVC_E_DEVICE_FLAG  (-7)  /* a kernel recorded an anomaly (see status_poll) */
#define KVC_E_TOO_LARGE    (-8)  /* problem needs more than the built-in scratch   */

/* ---- layouts, dtypes, modes --------------------------------------------- */
#define KVC_CONTIG 0   /* k, v: bf16 [L, H, T, d]                                  */
#define KVC_PAGED  1   /* k, v: bf16 pool [L, n_phys_pages, H, page_size, d]       */

#define KVC_F32  0
#define KVC_BF16 1

#define KVC_ROPE_HALF        0   /* channel c pairs with c + d/2                   */
#define KVC_ROPE_INTERLEAVED 1   /* channel 2c pairs with 2c + 1                   */

#define KVC_PROJECT 0  /* bases given, compute coefficients                        */
#define KVC_FIT     1  /* compute bases (truncated SVD), then coefficients         */
#define KVC_FIT_FAST 2 /* as KVC_FIT, top-r subspace solver where the spectrum allows */

#define KVC_PATH_AUTO    0  /* pick the fastest kernel that supports the arguments */
#define KVC_PATH_GENERIC 1  /* CUDA-core kernels (any supported shape)             */
#define KVC_PATH_TC      2  /* TMA + tcgen05 kernels (d = 128, r <= 64 ...)        */
#define KVC_PATH_MIXED   3  /* kvc_last_path only: a batch split between the two   */

/*
 * One agent's cache of the shared context (the paper's C_{i,seg}, Sec. 2.1 /
 * Eq. 2, held per layer and per KV head).  Caller-owned DEVICE memory.
 *
 * KVC_CONTIG: element (l, h, t, c) at  l*s_layer + h*s_head + t*s_tok + c.
 * KVC_PAGED : logical token t lives in physical page p = page_table[t / page_size]
 *             at row t % page_size: element at
 *             l*s_layer + p*s_page + h*s_head + (t % page_size)*s_tok + c.
 *             One table serves all layers and heads (the serving engine's block
 *             table).  The last page may be partial; rows >= T are never touched,
 *             nor are physical pages the table does not name.
 * Strides are in elements; 0 selects the dense default for the layout.
 * Every row start must be 16-byte aligned (strides multiples of 8 elements).
 */
typedef struct kvc_cache {
  void *k;                    /* DEVICE bf16                                       */
  void *v;                    /* DEVICE bf16                                       */
  int32_t layout;             /* KVC_CONTIG | KVC_PAGED                            */
  int32_t L, H, T, d;         /* layers, KV heads, shared tokens, head dim         */
  int32_t page_size;          /* KVC_PAGED: tokens per page (power of two, >= 8)   */
  int32_t n_phys_pages;       /* KVC_PAGED: pages in the pool; bound for page ids  */
  const int32_t *page_table;  /* DEVICE int32 [ceil(T / page_size)]                */
  int64_t s_layer, s_page, s_head, s_tok;
} kvc_cache;

/*
 * Rank-r state of one workflow edge (Eq. 7: Z ~= A_Z B_Z with A = U_r Sigma_r,
 * B = R_r^T), one independent state per (layer, KV head), keys and values
 * separately.  Caller-owned DEVICE memory.
 *   coeff_*: float32 [L, H, n_cov, r]   (the paper's A)
 *   basis_*: [L, H, r, d] in basis_dtype (the paper's B; rows orthonormal when fitted)
 * n_cov is the covered prefix (App. A.3 "Variable Segment Lengths"): rows
 * t >= n_cov of a cache receive the alignment only.  r == 0 or n_cov == 0 is
 * the empty state (pointers may be NULL).
 */
typedef struct kvc_state {
  float *coeff_k;
  float *coeff_v;
  void *basis_k;
  void *basis_v;
  int32_t r;
  int32_t n_cov;
  int32_t basis_dtype;        /* KVC_F32 | KVC_BF16                                */
  int32_t grouping;           /* KVC_GROUP_HEAD (0) | KVC_GROUP_LAYER              */
} kvc_state;

/*
 * Feature grouping of a state (Sec. 3.1 factorises with B in R^{r x D}, D being the width of the cached
 * features).
 *   KVC_GROUP_HEAD   one state per (layer, KV head), D = d:
 *                    coeff [L, H, n_cov, r], basis [L, H, r, d]                    (the default)
 *   KVC_GROUP_LAYER  one state per layer over all KV heads, D = H d: the coefficients of a token are
 *                    shared by the heads of a layer,
 *                    coeff [L, n_cov, r], basis [L, r, H d]  (head h uses columns h d .. (h+1) d - 1)
 *                    K_dst[l,h,t,:] = bf16( Rot(K_src[l,h,t,:]) + coeff_k[l,t,:] . basis_k[l][:, h d : (h+1) d] )
 * Grouping by layer is served by kvc_apply, kvc_chain, kvc_apply_batch and by kvc_state_update: in
 * KVC_PROJECT mode the projection sums over the heads (coeff[l,t,:] = sum_h Delta[l,h,t,:] . basis[l][:, h]^T);
 * in the FIT modes (r <= 32) the basis rows are the r leading right singular vectors of the layer's
 * concatenated deviation [n_cov, H d], see kvc_state_update.  The gate, the token weights and
 * kvc_apply_multi take grouped states as well (per anchor: pools may mix the two groupings).
 */
#define KVC_GROUP_HEAD  0
#define KVC_GROUP_LAYER 1

/*
 * Rotary position embedding used for the key re-alignment that precedes every
 * cross-agent reuse (Sec. 2.2; App. A.3).  A key cached at position p and
 * reused at position p + s is rotated, pair by pair, by the angle s * f_k with
 * f_k = theta^(-2k/d), k = 0..d/2-1, unless inv_freq overrides the table
 * (scaled-RoPE models).  Values are never rotated.
 * inv_freq is a HOST float64 table on purpose: cos and sin of shift * f_k are formed in float64 on the
 * host and rounded once to float32 (a float32 angle at |shift| ~ 500 already costs 1e-3 on keys of
 * magnitude 40), d/2 values per call that travel in the launch parameters.
 */
typedef struct kvc_rope {
  double theta;
  int32_t pairing;            /* KVC_ROPE_HALF | KVC_ROPE_INTERLEAVED              */
  int32_t reserved;
  const double *inv_freq;     /* HOST float64 [d/2] or NULL                        */
} kvc_rope;

/*
 * kvc_apply -- one hop (Eq. 8 with a single anchor; Sec. 3.3):
 *     K_dst[l,h,t,:] = bf16( Rot_shift(K_src[l,h,t,:]) + coeff_k[l,h,t,:] . basis_k[l,h] )
 *     V_dst[l,h,t,:] = bf16(           V_src[l,h,t,:]  + coeff_v[l,h,t,:] . basis_v[l,h] )
 * for t < n_cov; rows t >= n_cov (and every row of an empty state) keep the
 * re-aligned source: V bit for bit, K bit for bit when shift == 0.
 * Products and sums are accumulated in float32; one rounding to bf16.
 *   src   HOST struct, DEVICE buffers, read only.
 *   st    HOST struct, DEVICE buffers, read only.
 *   shift target position minus source position of the shared context
 *         (difference of the two agents' prefix lengths), any sign.
 *   dst   HOST struct, DEVICE buffers, written.  Same L, H, T, d as src; layout,
 *         strides and page table may differ.  dst may be the very same cache as src
 *         (same pointers, strides and table: in place); any other overlap is
 *         KVC_E_ALIAS when it can be detected from the pointers.
 * Errors: KVC_E_INVALID_ARG, KVC_E_SHAPE, KVC_E_UNSUPPORTED (d not in {64,128},
 * r > 256), KVC_E_ALIAS, KVC_E_CUDA.
 */
int kvc_apply(const kvc_cache *src, const kvc_state *st, int32_t shift, const kvc_rope *rope,
              kvc_cache *dst, void *stream);

/*
 * kvc_chain -- corrections chained along the workflow (Sec. 3.2; App. A.3 "Cache
 * Materialization"): agent 0's cache is exact and only read; for a = 1..n_agents-1
 *     outs[a-1] = kvc_apply(a == 1 ? agent0 : outs[a-2], states[a-1],
 *                           prefix_len[a] - prefix_len[a-1])
 * Each materialised cache is rounded to bf16 before it becomes the next source.
 *   prefix_len HOST int32 [n_agents]; states HOST array [n_agents-1]; outs HOST
 *   array [n_agents-1] of caller-owned destination caches (distinct from one
 *   another and from agent0).
 */
int kvc_chain(const kvc_cache *agent0, int32_t n_agents, const int32_t *prefix_len,
              const kvc_state *states, const kvc_rope *rope, kvc_cache *outs, void *stream);

/*
 * kvc_state_update -- build the rank-r state of the edge src -> tgt (Eq. 12 then
 * Eq. 7), for every (layer, KV head), keys and values:
 *     Delta_K = K_tgt - Rot_shift(K_src),  Delta_V = V_tgt - V_src   (rows t < st->n_cov)
 *   KVC_PROJECT: st->basis_* are inputs; coeff = Delta . basis^T is written (float32).
 *   KVC_FIT    : G = Delta^T Delta (d x d), its top-r eigenvectors become the rows
 *                of st->basis_* (float32; right singular vectors of Delta, largest
 *                singular values first, each row's largest-magnitude entry made
 *                positive; rows beyond min(r, d, n_cov) are zero, and so is a row whose
 *                eigenvalue lies below what float32 resolves beside the largest one,
 *                2.4e-7 of it: a deviation of rank < r gives that many zero rows), then
 *                coeff as above (= U_r Sigma_r).  The eigenvalues and vectors come from a
 *                float32 tridiagonal reduction: accurate to about d * 6e-8 of the largest
 *                eigenvalue; where eigenvalues lie closer than that, the rows span their
 *                common subspace.  st->basis_dtype must be KVC_F32 and r <= 64 (else
 *                KVC_E_UNSUPPORTED).
 *   KVC_FIT_FAST: the same state (Eq. 7 asks for the r largest singular values only), but each
 *                matrix is first tried with a block subspace iteration on its r leading
 *                eigenvectors (r <= 32), which converges in a few steps when the spectrum has a
 *                gap behind the r-th eigenvalue -- a deviation of rank r over a noise floor.  The
 *                result is accepted only when, in float32, every row satisfies
 *                |G b_j - lambda_j b_j| <= 3e-5 lambda_1 and the residual of the whole block is at most
 *                2^-13 of the distance between lambda_r and a bound on every eigenvalue outside the
 *                block (trace(G) minus the sum of the block's eigenvalues: G is positive
 *                semi-definite); any other matrix is solved by KVC_FIT's full eigensolver in the same
 *                call.  Bases, coefficients and the r leading eigenvalues meet KVC_FIT's accuracy.
 *                Difference: for a matrix the subspace solver served, the d - r trailing eigenvalues in
 *                the workspace all hold their MEAN (their exact sum divided by d - r), so the trace is
 *                exact and kvc_effective_rank is exact whenever it does not exceed r.  Which solver
 *                served which matrix is left in the workspace, see kvc_fit_solver.
 *   Layer-grouped states (KVC_GROUP_LAYER, D = H d), both FIT modes, r <= 32: the D x D Gram matrix is
 *                never formed.  The r trial vectors live in the state's bases and are driven to the leading
 *                eigenvectors of G = Delta^T Delta by three applications of G, each one the grouped
 *                projection pass Z = Delta Q^T followed by a back-projection pass Y = Z^T Delta, with an
 *                orthonormalisation of the r rows in between and a Rayleigh-Ritz step at the end
 *                (6 streaming passes over the two caches; the final coefficients are the last projection's
 *                times the Rayleigh-Ritz rotation, a pass over the coefficients only).  A block that the
 *                step finds merely slow (its hashed start was unlucky) gets up to two further rounds of
 *                orthonormalisation, application and Rayleigh-Ritz; their kernels are always launched and
 *                return at once when the round is not needed (nothing is read back to the host).
 *                Rows, coefficients and the r leading eigenvalues are as in KVC_FIT_FAST; the acceptance
 *                test likewise, with the rows' residual limit at 5e-5 lambda_1 and the block's at 1/4096 of
 *                the gap (the projection pass contracts in split bf16 precision, which bounds what can be
 *                measured).  There is no second solver behind it: a matrix that still fails the test (no
 *                gap behind the r-th eigenvalue) gets its Ritz rows all the same, its code in
 *                kvc_group_fit_solver says why, and KVC_FLAG_NOT_CONVERGED is raised.  Workspace layout: the
 *                eigenvalues [L, 2, H d] first (kvc_group_fit_eigenvalues; the r leading ones, then the
 *                mean of the rest), the codes [L, 2] (kvc_group_fit_solver), then scratch.
 *   src == NULL factorises tgt itself (the anchor's base representation, Sec. 3.3).
 *   workspace  DEVICE scratch of at least kvc_workspace_bytes(...) bytes, 256-byte
 *              aligned.  May be NULL when 0 is needed.  After a KVC_FIT / KVC_FIT_FAST call it
 *              holds, as float32: the Gram matrices [L, H, 2, d, d] (2 = K, V), then scratch of the
 *              same size, then the eigenvalues [L, H, 2, d] in descending order.
 * Errors as kvc_apply, plus KVC_E_WORKSPACE.
 */
int kvc_state_update(const kvc_cache *src, const kvc_cache *tgt, int32_t shift, const kvc_rope *rope,
                     kvc_state *st, int32_t mode, void *workspace, size_t workspace_bytes, void *stream);

/* Scratch kvc_state_update needs for this geometry and mode (0 for KVC_PROJECT). */
size_t kvc_workspace_bytes(const kvc_cache *tgt, const kvc_state *st, int32_t mode);

/*
 * After a KVC_FIT_FAST update: DEVICE int32 [L, H, 2] inside its workspace, one entry per matrix
 * (layer, head, K|V): KVC_SOLVER_SUBSPACE (0) when the subspace solver's result was accepted, otherwise
 * the reason the full eigensolver ran instead.  NULL on bad arguments.
 */
#define KVC_SOLVER_SUBSPACE        0
#define KVC_SOLVER_FULL_RANK     (-1)  /* min(r, d, n_cov) > 32: not tried                           */
#define KVC_SOLVER_FULL_DEPENDENT  2   /* zero matrix, or block columns dependent at float32         */
#define KVC_SOLVER_FULL_SLOW       3   /* block residual not at rounding level after five products   */
#define KVC_SOLVER_FULL_NO_GAP     4   /* a-posteriori test failed: no gap behind the r-th eigenvalue */
#define KVC_SOLVER_FULL_SWEEPS     5   /* Jacobi sweep limit                                         */
const int32_t *kvc_fit_solver(const kvc_cache *tgt, const void *workspace);
/* The same two accessors for the workspace of a layer-grouped FIT: float32 [L, 2, H d] and int32 [L, 2]. */
const float *kvc_group_fit_eigenvalues(const kvc_cache *tgt, const void *workspace);
const int32_t *kvc_group_fit_solver(const kvc_cache *tgt, const void *workspace);

/* The argument checks of kvc_state_update (everything but the workspace), launching nothing. */
int kvc_state_update_check(const kvc_cache *src, const kvc_cache *tgt, int32_t shift, const kvc_rope *rope,
                           const kvc_state *st, int32_t mode);

/*
 * kvc_state_update_chain -- the states of every edge of a workflow in one call (the counterpart of
 * kvc_chain for profiling, Sec. 3.2: a calibration trajectory yields every agent's true cache at once):
 * for a = 1..n_agents-1
 *     states[a-1] = kvc_state_update(src = agents[a-1], tgt = agents[a],
 *                                    shift = prefix_len[a] - prefix_len[a-1], mode)
 * with the same results as those n_agents-1 calls.  What differs is the schedule: the Gram passes of all
 * edges run first, then ONE launch solves the eigenproblems of all edges (when the edges share geometry,
 * r and n_cov; a single edge's 2 L H matrices fill the GPU's resident blocks unevenly and leave most SMs
 * idle while the slowest matrices finish), then the projection passes.
 *   agents     HOST array [n_agents] of caches (DEVICE data); prefix_len HOST int32 [n_agents];
 *   states     HOST array [n_agents-1]; n_agents <= 16 (else KVC_E_TOO_LARGE).
 *   workspace  DEVICE scratch of kvc_chain_update_workspace_bytes(...) bytes, 256-byte aligned: edge e
 *              (0-based) owns the kvc_chain_update_edge_stride(...) bytes starting at the sum of the
 *              strides of the edges before it, laid out as kvc_state_update's workspace
 *              (kvc_fit_eigenvalues / kvc_fit_solver / kvc_effective_rank take that address).
 * Errors as kvc_state_update; nothing is launched when any edge fails its checks.
 */
int kvc_state_update_chain(const kvc_cache *agents, int32_t n_agents, const int32_t *prefix_len, const kvc_rope *rope,
                           kvc_state *states, int32_t mode, void *workspace, size_t workspace_bytes, void *stream);
size_t kvc_chain_update_workspace_bytes(const kvc_cache *agents, int32_t n_agents, const kvc_state *states, int32_t mode);
size_t kvc_chain_update_edge_stride(const kvc_cache *tgt, const kvc_state *st, int32_t mode);

/*
 * Multi-segment contexts (Eq. 1; App. A.2).  A trajectory interleaves agent-specific pieces with the
 * shared ones, so between two agents the shared tokens are displaced by an amount that is constant
 * inside a segment and changes from one segment to the next.  A segment list gives every token range
 * its own shift; one call then serves the whole context (no splitting into one call, and for paged
 * caches one page-aligned table slice, per segment).  Segment boundaries need not fall on pages or tiles.
 *   n        1 .. KVC_MAX_SEGMENTS
 *   t_begin  HOST int32 [n], ascending, t_begin[0] == 0: segment j covers tokens t_begin[j] .. t_begin[j+1]-1,
 *            the last one runs to T
 *   shift    HOST int32 [n]
 *   coords   where the low-rank correction lives:
 *            KVC_COORDS_TARGET  at the target's positions, as Eq. 12 measures it:
 *                               K_dst = Rot_s(K_src) + c . B ,   Delta = K_tgt - Rot_s(K_src)
 *            KVC_COORDS_SOURCE  at the source's positions (the canonical-coordinate form of App. A.2: the
 *                               correction is stored once and moves with the token it corrects):
 *                               K_dst = Rot_s(K_src + c . B) ,   Delta = Rot_{-s}(K_tgt) - K_src
 *            With one shift for all tokens, SOURCE coordinates equal TARGET coordinates with the key basis
 *            rotated by kvc_state_realign; with several shifts only SOURCE coordinates keep one basis.
 *            Values are never rotated: the two agree for them.
 * The lists are host arrays on purpose: the cos / sin tables of every segment are formed in float64 on the
 * host, exactly like the single shift's, and travel in the launch parameters (a device position array would
 * need sincos per token and frequency inside the kernels).  kvc_apply_segmented runs on the tensor-core
 * kernel where kvc_apply does (every row picks its segment's table in the epilogue), and so do the passes
 * of kvc_state_update_segmented over the caches where kvc_state_update's do: the Gram pass picks every
 * row's table while it forms the deviation, the projection runs as one launch per segment over that
 * segment's token window (it rotates the basis, not the tokens; on a paged cache a window starts with its
 * page, and the segments run from the last to the first so that every row is last written by its own).
 * Only a layer-grouped state on a paged cache whose segment boundaries are off the page grid has its
 * projection served by the CUDA-core kernel (KVC_PATH_TC forced: KVC_E_UNSUPPORTED).  Everything else is as in kvc_apply / kvc_state_update, including layer-grouped
 * states (whose back-projection pass picks the rows' tables like the Gram pass) and the FIT modes.
 */
#define KVC_MAX_SEGMENTS   16
#define KVC_COORDS_TARGET  0
#define KVC_COORDS_SOURCE  1
typedef struct kvc_segments {
  int32_t n;
  const int32_t *t_begin;
  const int32_t *shift;
  int32_t coords;
} kvc_segments;
int kvc_apply_segmented(const kvc_cache *src, const kvc_state *st, const kvc_segments *segs, const kvc_rope *rope,
                        kvc_cache *dst, void *stream);
int kvc_state_update_segmented(const kvc_cache *src, const kvc_cache *tgt, const kvc_segments *segs, const kvc_rope *rope,
                               kvc_state *st, int32_t mode, void *workspace, size_t workspace_bytes, void *stream);

/*
 * kvc_state_update_noalloc -- kvc_state_update without a workspace argument.
 * (No counterpart in the paper: this exists for integration only.)
 *
 * Some callers cannot obtain device memory at the point where they need a state
 * update: code that runs inside a serving engine whose memory pool was sized and handed
 * out at start-up, plugins that are forbidden to call cudaMalloc because an allocation
 * synchronises the device and would stall the engine's other streams, and processes
 * whose GPU memory is already fully committed to the KV pool.  For them the FIT-mode
 * scratch lives in a fixed array inside the library image (KVC_STATIC_SCRATCH_BYTES on
 * every GPU that loads the library, held until the process exits).  The call performs no
 * cudaMalloc / cudaFree and uses no allocating library routine; inputs and outputs are
 * still the caller's buffers, with the same meaning as in kvc_state_update.
 *
 *  - The arguments are checked first, exactly as kvc_state_update checks them, and a call that
 *    fails a check returns that error and launches nothing.
 *  - Capacity: kvc_workspace_bytes(tgt, st, mode) must not exceed
 *    KVC_STATIC_SCRATCH_BYTES, i.e. L*H <= 64 at d = 128 (L*H <= 255 at d = 64) in the FIT
 *    modes; larger problems return KVC_E_TOO_LARGE and launch nothing (split them by
 *    layer, or use kvc_state_update with your own workspace).  KVC_PROJECT needs no
 *    scratch and is never rejected for size.
 *  - The first call on each device, in ANY mode (a KVC_PROJECT call or a call with an empty state
 *    will do), looks up the array's device address with that device current.  The library's
 *    modules load lazily, so this first call is also the moment the driver sets the array's
 *    bytes aside on that GPU: make it at start-up, before the rest of the GPU's memory is handed to
 *    a pool, and before any stream capture begins.  Later calls take no device memory.
 *  - All calls on one device share the one array, and it keeps the previous call's
 *    contents.  Nothing needs clearing: every kernel of the update writes its part of the
 *    scratch before anything reads it.  Two calls whose device work can overlap (different
 *    streams, or different host threads on different streams) race on the array: serialise them.
 */
#define KVC_STATIC_SCRATCH_BYTES (128 * (2 * 128 * 128 + 128) * 4 + 1024)
int kvc_state_update_noalloc(const kvc_cache *src, const kvc_cache *tgt, int32_t shift, const kvc_rope *rope,
                             kvc_state *st, int32_t mode, void *stream);

/*
 * kvc_apply_batch -- many independent hops in ONE launch (concurrent serving: each
 * item is one request's next hop, with its own length, rank, shift and tables).
 * The computation per item is exactly kvc_apply's.
 *   items      HOST array [n_items]; every item's caches must share d.
 *              Items the tensor-core kernels serve (head_dim 128, 0 < r <= 64 a multiple of 4, ...) run
 *              there, the others (empty states, odd ranks) on the CUDA-core kernel in a launch of
 *              their own: one such request does not slow the rest of the batch down
 *              (kvc_last_path: KVC_PATH_MIXED).
 *   workspace  DEVICE scratch >= kvc_batch_workspace_bytes(n_items), 256-byte aligned;
 *              receives the launch's work table and must stay untouched until the
 *              launch has finished.
 *   staging    HOST buffer of the same size (pinned memory recommended); the work
 *              table is built here and copied to `workspace` on `stream`; it must stay
 *              untouched until that copy has executed.
 * Why the items are a host array and the call makes one host-to-device copy: the work table carries
 * tensor maps, which only the host can encode, and the per-CTA ranges of equal estimated time; building
 * them is this call's job, and one copy of a few hundred KB per launch replaces a second API for it.
 * An item works on the token range [t_begin, t_end) of its caches (0, 0: all rows), so a context made of
 * several shared pieces at different offsets (Eq. 1) is one item per piece over the same caches, each with
 * its own shift: rows outside the range stay untouched in dst, row t of the state's coefficients corrects
 * token t (absolute), covered are the rows t < st.n_cov.  Errors: KVC_E_INVALID_ARG unless
 * 0 <= t_begin < t_end <= T of both caches; KVC_E_UNSUPPORTED when a paged cache's range does not start
 * on a page boundary (kvc_apply_segmented takes boundaries anywhere, for one request at a time).
 * Ranges of two items of one launch must not overlap in dst.
 */
typedef struct kvc_item {
  kvc_cache src;
  kvc_cache dst;
  kvc_state st;
  int32_t shift;
  int32_t t_begin, t_end;   /* token range of the item; both 0: the whole cache */
  int32_t reserved;
} kvc_item;

int kvc_apply_batch(const kvc_item *items, int32_t n_items, const kvc_rope *rope,
                    void *workspace, size_t workspace_bytes, void *staging, void *stream);
size_t kvc_batch_workspace_bytes(int32_t n_items);

/*
 * kvc_chain_fused -- kvc_chain in one pass over agent 0's cache (Sec. 3.2, Eq. 6): every tile of
 * agent 0 is loaded once, carried through all hops in shared memory and stored after every hop, so
 * no intermediate cache is read back.  Same arguments, same results bit for bit as kvc_chain (each
 * hop rounds to bf16 before it feeds the next); per token, layer and head the chain moves
 * 4d + (n_agents - 1)(8r + 4d) bytes instead of (n_agents - 1)(8d + 8r).
 *   workspace  DEVICE, kvc_chain_workspace_bytes(agent0, n_agents) bytes, 128-byte aligned: the hops'
 *              bases rewritten as tensor-core operands (rebuilt by every call)
 * Served fused: head_dim 128, 3 <= n_agents <= KVC_CHAIN_MAX_HOPS + 1, every live state with r <= 64,
 * r a multiple of 4, grouped by head.  Anything else runs hop by hop exactly like kvc_chain (with
 * kvc_set_path(KVC_PATH_TC): KVC_E_UNSUPPORTED instead).
 */
#define KVC_CHAIN_MAX_HOPS 7
int kvc_chain_fused(const kvc_cache *agent0, int32_t n_agents, const int32_t *prefix_len, const kvc_state *states,
                    const kvc_rope *rope, kvc_cache *outs, void *workspace, size_t workspace_bytes, void *stream);
size_t kvc_chain_workspace_bytes(const kvc_cache *agent0, int32_t n_agents);

/*
 * Multi-anchor apply (Eq. 8 with the token-wise weights of App. A.3 "Correction Weighting"):
 *     K_dst[l,h,t,:] = bf16( Rot_shift(K_src[l,h,t,:]) + sum_v w_k[v][t] * coeff_k(v)[l,h,t,:] . basis_k(v)[l,h] )
 *     V_dst[l,h,t,:] = bf16( V_src[l,h,t,:]            + sum_v w_v[v][t] * coeff_v(v)[l,h,t,:] . basis_v(v)[l,h] )
 * anchor v contributing on its covered rows t < deltas[v].n_cov; rows no anchor covers keep the
 * aligned source exactly as in kvc_apply.  This is kvc_apply at the stacked rank sum_v r_v with the
 * weights folded into the coefficients, computed without building the stacked state.
 *   deltas     host array [n_anchors] of the anchors' transition corrections (device factors);
 *              anchors with r = 0 or n_cov = 0 contribute nothing
 *   w_k, w_v   DEVICE float32 [n_anchors][t_pad], t_pad = KVC_MULTI_TPAD(src->T) (T rounded up to a
 *              multiple of 128; the padding must hold finite numbers), 16-byte aligned; NULL = all ones
 *   workspace  DEVICE, kvc_multi_workspace_bytes(...) bytes, 128-byte aligned: the bases rewritten as
 *              tensor-core operands (rebuilt by every call)
 * Limits: head_dim 128; every r_v a multiple of 4, at most 64; at most KVC_MULTI_MAX_BLOCKS rank
 * blocks of 32 in total (sum over anchors of ceil(r_v / 32)), i.e. an effective rank of up to 320.
 * Arguments outside these limits return KVC_E_UNSUPPORTED: this entry point has no CUDA-core variant.
 * dst may be src itself (in place).  Precision as kvc_apply.
 */
#define KVC_MAX_ANCHORS 16
#define KVC_MULTI_MAX_BLOCKS 10
#define KVC_MULTI_TPAD(T) ((((int64_t)(T)) + 127) / 128 * 128)
int kvc_apply_multi(const kvc_cache *src, const kvc_state *deltas, int32_t n_anchors, const float *w_k,
                    const float *w_v, int32_t shift, const kvc_rope *rope, kvc_cache *dst, void *workspace,
                    size_t workspace_bytes, void *stream);
size_t kvc_multi_workspace_bytes(const kvc_cache *src, const kvc_state *deltas, int32_t n_anchors);

/*
 * Effective rank (the diagnostic of Sec. 3.1: the smallest rank whose singular values carry a given
 * share, there 90 %, of the summed squared singular values), from the
 * eigenvalues a KVC_FIT update leaves in its workspace (squared singular values of the factorised
 * deviation or cache).  For every matrix m of n_matrices:
 *     rank[m] = min { k : sum_{i<k} max(evals[m][i], 0) >= energy * sum_i max(evals[m][i], 0) }   (0 if the sum is 0)
 *   evals   DEVICE float32 [n_matrices][d], each row descending (kvc_fit_eigenvalues(...) points at
 *           them inside a FIT workspace: n_matrices = L*H*2, ordered (layer, head, K|V))
 *   energy  in (0, 1], e.g. 0.9
 *   rank    DEVICE int32 [n_matrices]
 * Sums in float64.
 */
int kvc_effective_rank(const float *evals, int32_t n_matrices, int32_t d, double energy, int32_t *rank, void *stream);
/* Address of the eigenvalues inside a KVC_FIT workspace of kvc_state_update for `tgt` (NULL on bad arguments). */
const float *kvc_fit_eigenvalues(const kvc_cache *tgt, const void *workspace);

/*
 * Positional re-alignment of a stored correction (App. A.2: the correction of a prefix relation that
 * recurs is learned a single time, kept as its low-rank factors, and moved to the positions of each reuse).
 * A rotation is linear in the channels, Rot_s(c . B) = c . Rot_s(B), so re-aligning a stored key
 * correction by `shift` positions is rotating every row of its key basis by `shift`:
 *     basis_k_out[l,h,q,:] = Rot_shift(basis_k_in[l,h,q,:]) ,
 * coefficients and value factors are not touched.  Uses: a state fitted at target position p and
 * re-aligned by -p is the same correction in canonical coordinates; re-aligned by p' it applies at
 * position p' through kvc_apply / kvc_apply_multi, whose own `shift` aligns the source cache.
 *   L, H, d      geometry of the basis [L, H, st->r, d], d in {64, 128}
 *   st           the state whose basis_k (device, basis_dtype) is read
 *   basis_k_out  DEVICE, same shape and dtype; may be st->basis_k itself (in place)
 * float32 rotation with the angles' cos / sin computed in float64 on the host, like kvc_apply.
 */
int kvc_state_realign(const kvc_state *st, int32_t L, int32_t H, int32_t d, int32_t shift, const kvc_rope *rope,
                      void *basis_k_out, void *stream);

/*
 * Token-wise interpolation weights (App. A.3 "Correction Weighting and Positional Alignment"):
 * for token t and anchor v the score is the mean over layers, heads and channels of
 *     | C_src[l,h,t,c] - coeff(v)[l,h,t,:] . basis(v)[l,h][:,c] | ,
 * the distance between the source cache and the base cache anchor v reconstructs from its
 * low-rank factors; keys and values are scored separately, keys after both sides were rotated into
 * canonical positional coordinates (the source back by src_pos, anchor v's reconstruction back by
 * anchor_pos[v]).  The weights are the softmax over anchors of -score / temperature:
 *     w_k[v][t], w_v[v][t] , DEVICE float32 [n_anchors][KVC_MULTI_TPAD(src->T)] ,
 * the layout kvc_apply_multi consumes.  A token beyond anchor v's coverage (t >= anchors[v].n_cov)
 * gets weight zero for v and the softmax runs over the anchors that cover it; the padding is zero.
 *   anchors     host array [n_anchors] of the anchors' BASE factorisations (key and value factors)
 *   anchor_pos  host int32 [n_anchors]
 *   workspace   DEVICE, kvc_token_weights_workspace_bytes(src, n_anchors) bytes (the scores:
 *               float32 [n_anchors][2][t_pad], left readable after the call)
 * Limits: head_dim 128, 0 < r <= 64 and a multiple of 4, n_anchors <= KVC_MAX_ANCHORS, half-split RoPE
 * pairing; otherwise KVC_E_UNSUPPORTED (no CUDA-core variant).  Scores are summed with float32
 * atomics: their last bits depend on the order of the additions.
 */
int kvc_token_weights(const kvc_cache *src, int32_t src_pos, const kvc_state *anchors, const int32_t *anchor_pos,
                      int32_t n_anchors, const kvc_rope *rope, double temperature, float *w_k, float *w_v,
                      void *workspace, size_t workspace_bytes, void *stream);
size_t kvc_token_weights_workspace_bytes(const kvc_cache *src, int32_t n_anchors);

/*
 * Reliability gate of the anchor pool (App. A.3 "Reliability Gate", Eqs. 9-11).
 *
 * kvc_gate_distance (Eq. 9): for every anchor v of a pool,
 *     dist_sq[v] = sum over layers l, heads h, tokens t < k of
 *                  || V_src[l,h,t,:] - coeff_v[l,h,t,:] . basis_v[l,h] ||^2 ,
 * the squared Frobenius distance between the source cache's VALUE states and the value states
 * anchor v reconstructs from the low-rank factors of its base cache (a state fitted with
 * kvc_state_update(src = NULL, tgt = the anchor's cache)).  The gate distance of Eq. 9 is
 * sqrt(dist_sq[v]).  Only coeff_v / basis_v of each state are read; the key factors may be NULL.
 *   src       source cache (host descriptor, device data), read only
 *   anchors   host array [n_anchors]; every anchor needs n_cov >= k (anchors whose stored length is
 *             below the comparison length are not compatible: KVC_E_SHAPE), 0 < r <= 256
 *   k         comparison prefix length, 0 <= k <= src->T
 *   dist_sq   DEVICE float64 [n_anchors], overwritten (cleared, then accumulated: the sum's order
 *             over CTAs is not fixed, which moves the result by float64 rounding only)
 * Products run in split bf16 with float32 accumulation like kvc_apply; squares are summed in
 * float32 per 32-channel row segment and in float64 beyond.
 *
 * kvc_gate_weights (Eqs. 10-11), on the device so that no host round trip is needed:
 *     g[v] = softmax_v( -sqrt(dist_sq[v]) / temperature ),   entropy[0] = -sum_v g log2 g / log2 n
 * in float64 (0 log 0 = 0).  n_anchors < 2 returns KVC_E_INVALID_ARG: the method has no gate value
 * then and falls back to dense prefill.  dist_sq, g [n_anchors], entropy [1]: DEVICE float64.
 * The caller accepts the correction when entropy[0] <= tau.
 */
int kvc_gate_distance(const kvc_cache *src, const kvc_state *anchors, int32_t n_anchors, int32_t k,
                      double *dist_sq, void *stream);
int kvc_gate_weights(const double *dist_sq, int32_t n_anchors, double temperature, double *g,
                     double *entropy, void *stream);

/*
 * Device-side anomalies never trap or hang: a kernel that meets a page id outside
 * [0, n_phys_pages) or whose bounded wait on an asynchronous copy runs out skips
 * that tile and ORs a bit into a per-device status word.
 * kvc_status_poll copies the word to *flags and returns KVC_OK when it is zero,
 * KVC_E_DEVICE_FLAG otherwise.  The copy is a device-to-host read of one word, so this call
 * SYNCHRONISES the device: a caller that must not stall its streams polls at a point where it
 * synchronises anyway (end of a batch, after an event wait).  kvc_status_reset clears the word.
 */
#define KVC_FLAG_BAD_PAGE     1u
#define KVC_FLAG_WAIT_EXPIRED 2u
#define KVC_FLAG_NOT_CONVERGED 4u   /* eigensolver hit its sweep limit             */
int kvc_status_poll(uint32_t *flags);
int kvc_status_reset(void);

/*
 * kvc_selftest_wait_expiry -- run the give-up branch of the library's bounded waits once, safely.
 * One CTA waits, through the same bounded wait the streaming kernels use but with a limit of
 * limit_ms milliseconds (0 < limit_ms <= 100), on an mbarrier that nothing arrives on.  Every thread's
 * wait must return "gave up", the CTA's abort flag must be raised and KVC_FLAG_WAIT_EXPIRED must
 * appear in the status word; the context stays usable (nothing traps, faults or loops without bound).
 *   result  HOST int32 [3]: threads whose wait claimed success (expected 0), the abort flag
 *           (expected 1), SM cycles thread 0 spent waiting.
 * Synchronises `stream`.  The caller clears the flag afterwards with kvc_status_reset.
 */
int kvc_selftest_wait_expiry(double limit_ms, int32_t *result, void *stream);

/* Force a kernel family (testing / benchmarking); KVC_PATH_TC returns
 * KVC_E_UNSUPPORTED from later calls whose arguments it cannot serve. */
int kvc_set_path(int32_t path);
/* Which family the last successful launch on this thread used (KVC_PATH_*). */
int kvc_last_path(void);

/* Algorithmic HBM bytes one hop moves (reads + writes of caches, coefficients and
 * bases), the figure the roofline is reported against.  For the FIT modes: two passes over
 * the source and target rows (one for the Gram matrix, one for the projection), however many
 * the implementation makes (the layer-grouped fit makes six). */
int64_t kvc_apply_bytes(const kvc_cache *src, const kvc_state *st);
int64_t kvc_update_bytes(const kvc_cache *tgt, const kvc_state *st, int32_t mode, int32_t has_src);

const char *kvc_strerror(int code);
const char *kvc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVC_H_ */
