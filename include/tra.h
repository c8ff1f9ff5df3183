/*
 * tra.h — C ABI of the Token Radius Attention hot path for NVIDIA B200 (sm_100a).
 *
 * One GPU, one stream per call.  The library allocates device memory only inside
 * tra_plan_create (plan-owned tables, freed by tra_plan_destroy); every tensor is
 * owned by the caller.  Unless stated otherwise a pointer is a DEVICE pointer to
 * contiguous memory, 16-byte aligned.  All calls are asynchronous on `stream`
 * (a cudaStream_t passed as void*, NULL = default stream) and return a status
 * code; none of them synchronises the device or throws.
 *
 * Token order.  N = T*H*W video tokens.  Every token-indexed array handed to the
 * four hot calls is in TILE-MAJOR order (Section 3.3, "Flash Radius Mask Kernel":
 * each H x W frame is cut into tile_h x tile_w tiles, edge tiles clipped; tokens
 * are listed frame by frame, tile by tile, row-major inside a tile).  A block is
 * `block` consecutive tile-major positions (Algorithm 1: q = u*b + i, q < N);
 * NB = ceil(N / block).  tra_tile_major_gather / _scatter move tensors between
 * raster order (n = (t*H + y)*W + x) and tile-major order.  A plan created with
 * TRA_ORDER_RASTER takes Q, K, V and O in raster order instead and needs no such pass
 * (TRA_ORDER_RASTER_QO: Q and O only).
 *
 * Joint text-video attention (Section 3.2, last paragraph; Algorithm 1).  With cfg.n_text > 0 a
 * sequence is the N video tokens followed by n_text text tokens, S = N + n_text; S takes the place
 * of N in every shape below and NB = ceil(S / block).  The first B_v = floor(N / block) blocks, made
 * of video tokens only, are the video blocks; a block pair with u >= B_v or v >= B_v is always kept
 * (this includes the block that holds both the last video and the first text tokens, so that every
 * text key stays visible to every query and a text query sees every key), the gather/scatter leaves
 * text tokens where they are, and text positions get budget S, radius +inf and the last candidate
 * index.  Without text the ragged last block is a video block like any other.
 *
 * Shapes.  Q, K, V, O: bf16 [B, heads, N, head_dim].  entropy, budget, radius,
 * ridx: [B, heads, N].  block_mask: uint8 [B, heads, NB, NB].  row_ptr: int32
 * [B*heads*NB + 1]; col_idx: int32 [nnz], key blocks ascending inside a row.
 */
#ifndef TRA_H_
#define TRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define TRA_OK 0
#define TRA_ERR_INVALID_ARG (-1) /* NULL / misaligned pointer, non-positive size, bad flag     */
#define TRA_ERR_UNSUPPORTED (-2) /* head_dim, block or grid size outside what the kernels take */
#define TRA_ERR_CAPACITY (-3)    /* col_idx capacity too small (reported by tra_plan_status)   */
#define TRA_ERR_CUDA (-4)        /* a CUDA runtime / driver call failed                        */
#define TRA_ERR_TIMEOUT (-5)     /* a bounded device-side wait expired (reported by tra_plan_status) */
#define TRA_ERR_BOUNDS (-6)      /* debug build (-DTRA_DEBUG) only: a kernel computed an index outside its   */
                                 /* array, or its roles disagree on the work they walked; the access was    */
                                 /* skipped (reported by tra_plan_status)                                    */

/* plan flags */
#define TRA_KEEP_DIAGONAL 1u /* force block_mask[u][u] = 1 (a token always sees itself, Eq. 15) */
#define TRA_ORDER_RASTER 2u  /* Q, K, V and O of the attention calls (and of tra_hot_path_host) are in RASTER   */
                             /* order, n = (t*H + y)*W + x: the kernels fetch every run of 16 tile-major     */
                             /* positions, which is 16 consecutive raster rows, with a TMA box of its own and */
                             /* write O rows where they belong, so no gather / scatter pass is needed         */
                             /* (Section 3.3 reorders explicitly).  entropy, lse, budget, radius, ridx and    */
                             /* the mask stay in tile-major order: they only travel between this library's    */
                             /* calls.  Needs W, tile_w and block to be multiples of 16 (else                  */
                             /* tra_plan_create returns TRA_ERR_UNSUPPORTED).                                 */
#define TRA_ORDER_RASTER_QO 4u /* only Q and O are in raster order; K and V are tile-major (gathered by the     */
                               /* caller).  Q is loaded once per thread block and O rows are stored one by one */
                               /* anyway, so this costs nothing in the launches and saves the gather of Q and  */
                               /* the scatter of O; the many K / V tile loads keep their two large boxes.      */
                               /* Same conditions as TRA_ORDER_RASTER, which takes precedence.                 */

/* entropy-to-budget maps */
#define TRA_BUDGET_UNIFORM 0   /* K = ceil(tau exp(H)): the uniform-support map of Eq. 8 (the paper's choice) */
#define TRA_BUDGET_LOGNORMAL 1 /* K = ceil(N Phibar(sqrt(2 (log N - H)) - Phi^-1(tau))): Appendix,           */
                               /* "Entropy-identified Lognormal mapping"                                    */

/* candidate-radius policies for the set R of Eq. 14 when cfg.radii == NULL */
#define TRA_RADII_EXTENDED 0 /* 0..D (D = ceil(frame diagonal)), then D*exp(gamma*m), m = 1..T-1 */
#define TRA_RADII_LITERAL 1  /* 0..D and +infinity as the full-support radius                    */

typedef struct tra_plan tra_plan_t; /* opaque: grid geometry, thresholds, count table, block boxes */

typedef struct {
  int T, H, W;         /* latent grid (Section 2.1); 1 <= T,H,W <= 1023                          */
  int head_dim;        /* d: 64 or 128                                                          */
  int block;           /* b of Algorithm 1: 16..128 for the budget/radius/mask calls; the        */
                       /* attention calls take 33..128; the token mask inside blocks (ridx)     */
                       /* needs 64 or 128                                                       */
  int tile_h, tile_w;  /* tile shape of the tile-major order (Section 3.3)                       */
  double tau;          /* target attention mass of Eq. 4, in (0, 1]                              */
  double gamma;        /* temporal decay rate of Eq. 10, >= 0                                    */
  const double* radii; /* HOST pointer: optional strictly ascending candidate radii; the last    */
                       /* one must reach full support (may be +inf).  NULL = radius_policy       */
  int n_radii;
  int radius_policy;   /* TRA_RADII_* (used when radii == NULL)                                  */
  unsigned flags;      /* TRA_KEEP_DIAGONAL | TRA_ORDER_RASTER | TRA_ORDER_RASTER_QO             */
  int budget_map;      /* TRA_BUDGET_* used by tra_budget_radius                                 */
  int n_text;          /* text tokens that follow the video tokens in every sequence (>= 0)     */
} tra_config_t;

/* ---- plan ---------------------------------------------------------------------------- */

/* Builds the plan for one grid / gamma / candidate set on the current device: tile-major
 * coordinates, the squared-distance thresholds floor(r^2 exp(-2 gamma delta)) of Eq. 15, the
 * boundary-aware count table C_grid of Eq. 13 for every (token coordinate, candidate) — the
 * lookup table of Section 3.2 — and per-block bounding boxes (Section 3.3).  Work is enqueued
 * on `stream`; the call returns after the tables are built (it synchronises that stream).
 * *out is owned by the caller and released with tra_plan_destroy. */
int tra_plan_create(tra_plan_t** out, const tra_config_t* cfg, void* stream);
int tra_plan_destroy(tra_plan_t* plan);

/* Geometry queries (host). */
int tra_plan_num_tokens(const tra_plan_t* plan);   /* S = N + n_text: tokens per sequence */
int tra_plan_num_video_tokens(const tra_plan_t* plan); /* N = T*H*W */
int tra_plan_num_blocks(const tra_plan_t* plan);   /* NB */
int tra_plan_num_radii(const tra_plan_t* plan);    /* |R| */
int tra_plan_num_tile_pairs(const tra_plan_t* plan); /* entries per (batch, head) of the tile-pair table of
                                                        tra_build_block_mask: ceil(NT / 2); 0 for blocks <= 32 */
/* Copies plan tables to HOST buffers (synchronises): radii[|R|] (double), theta[|R|*T]
 * (int32, theta[k*T + delta]), coord[N*3] (int32 t,y,x per tile-major position).  Any may be NULL. */
int tra_plan_tables(const tra_plan_t* plan, double* radii, int32_t* theta, int32_t* coord);
/* Copies the count table to a HOST buffer uint32 [T*H*W*|R|], indexed ((t*H+y)*W+x)*|R| + k. */
int tra_plan_count_table(const tra_plan_t* plan, uint32_t* counts);

/* Reads and clears the plan's device status word (synchronises `stream`): TRA_OK, or the
 * first TRA_ERR_CAPACITY / TRA_ERR_TIMEOUT / TRA_ERR_BOUNDS a kernel of this plan recorded since the
 * last call. */
int tra_plan_status(tra_plan_t* plan, void* stream);

const char* tra_status_string(int status);

/* Self-test of the device-side error path (the paper has no counterpart): launches one warp that
 * waits, with the same bounded wait the attention kernels use, on a barrier nothing arrives on.
 * After limit_ms (1..1000) the wait gives up and records TRA_ERR_TIMEOUT in the plan status; the
 * kernel then returns normally and the context stays usable.  Asynchronous on `stream`. */
int tra_selftest_wait_timeout(tra_plan_t* plan, int limit_ms, void* stream);

/* ---- layout (Section 3.3: Q, K, V are reordered before attention, O restored after) -- */

/* dst[bh, p, :] = src[bh, raster(p), :] for every tile-major position p.  row_bytes = bytes of
 * one token row (multiple of 16); n_bh = B*heads.  src and dst must not overlap. */
int tra_tile_major_gather(const tra_plan_t* plan, const void* src_raster, void* dst_tile_major,
                          int n_bh, int row_bytes, void* stream);
/* dst[bh, raster(p), :] = src[bh, p, :] — the inverse. */
int tra_tile_major_scatter(const tra_plan_t* plan, const void* src_tile_major, void* dst_raster,
                           int n_bh, int row_bytes, void* stream);

/* ---- the four hot calls ------------------------------------------------------------- */

/* Dense attention of Eq. 1 fused with the attention entropy of Eq. 2, accumulated from the
 * online-softmax state as in Algorithm 2 (H = m + log l - a/l, nats).
 *   Q, K, V : bf16 [B, heads, N, head_dim], 128-byte aligned.
 *   O       : bf16, same shape (written).
 *   entropy : fp32 [B, heads, N] or NULL (NULL = plain dense attention, no entropy work).
 *   lse     : fp32 [B, heads, N] or NULL; log sum_j exp(s_ij), exact to fp32 rounding (the row sum
 *             of the unrounded probabilities is kept next to the bf16-rounded one that normalises O).
 *   sm_scale: multiplies q.k; pass 1/sqrt(head_dim) for Eq. 1. */
int tra_entropy_attn(const tra_plan_t* plan, const void* Q, const void* K, const void* V, void* O,
                     float* entropy, float* lse, int B, int heads, float sm_scale, void* stream);

/* Entropy -> token budget -> radius (Eq. 8 and Eq. 14; Appendix "Entropy-to-budget-to-radius
 * lookup"): budget = clamp(ceil(tau * exp(entropy)), 1, N) evaluated in fp64 (or the lognormal
 * map of the appendix when the plan was created with TRA_BUDGET_LOGNORMAL); ridx = index of
 * the smallest candidate radius whose C_grid at the token's coordinate reaches the budget;
 * radius = that candidate as fp32 (+inf for an infinite full-support radius).
 *   entropy: fp32 [B, heads, N];  budget: int32 or NULL;  radius: fp32 or NULL;  ridx: uint16. */
int tra_budget_radius(const tra_plan_t* plan, const float* entropy, int32_t* budget, float* radius,
                      uint16_t* ridx, int B, int heads, void* stream);

/* Algorithm 1: block mask from per-query radii.  For every (head, query block u, key block v):
 * c_j = number of valid queries of u whose disk (Eq. 15) holds key column j; keep the pair iff
 * some c_j > 0 and 10*#{c_j > b/3} > 6*#{c_j > 0}.  Block bounding boxes only skip pairs whose
 * vote is already decided; the result equals the unpruned vote bit for bit.
 *   ridx      : uint16 [B, heads, N] from tra_budget_radius.
 *   block_mask: uint8 [B, heads, NB, NB] (written, 0/1).
 *   row_ptr   : int32 [B*heads*NB + 1] (written); col_idx: int32 [col_idx_capacity] (written,
 *               ascending inside a row).  If nnz exceeds the capacity, TRA_ERR_CAPACITY is recorded
 *               in the plan status, col_idx holds the first `capacity` entries and every row_ptr
 *               offset is clamped to the capacity, so that a later tra_sparse_attn stays inside
 *               col_idx (its result is then incomplete; read the status).
 *   nnz_out   : device int64 or NULL; total retained blocks.
 *   tile_pairs: int32 [B*heads, ceil(NT/2), 2] or NULL, NT = ceil(NB / G) query tiles, G = 2 blocks
 *               per tile for blocks of up to 64 tokens, else 1 (written).  The paper has
 *               no counterpart: tra_sparse_attn gives each thread block two query tiles (128 rows of
 *               tensor-core work each, of which the first G * block hold queries) that
 *               share the key/value tiles they both retain, and this table pairs tiles whose block
 *               lists are similar (entry -1 = no second tile).  Pass it to tra_sparse_attn together
 *               with row_ptr / col_idx; it changes the speed of that call, never its result.
 *               Blocks of 32 tokens or fewer have no attention launch and no query tiles:
 *               with such a plan a non-NULL tile_pairs returns TRA_ERR_UNSUPPORTED (nothing is run).
 *               The pairing kernel runs beside the list kernels on a stream the plan owns, forked from and
 *               joined to `stream` by two plan-owned events (this also works inside a stream capture):
 *               everything the call writes is complete for later work on `stream`, but calls with
 *               tile_pairs on ONE plan must not be issued from several host threads at once. */
int tra_build_block_mask(const tra_plan_t* plan, const uint16_t* ridx, uint8_t* block_mask,
                         int32_t* row_ptr, int32_t* col_idx, int64_t col_idx_capacity,
                         int64_t* nnz_out, int32_t* tile_pairs, int B, int heads, void* stream);

/* The active-block list for callers that cannot allocate (the paper has no counterpart: this is
 * about how the library is embedded, not about the method).  Some users of this library may not
 * call cudaMalloc, or any allocator, at the point where the mask is rebuilt: code that runs as a
 * plugin inside another framework's memory pool, a server that hands out all device memory at
 * start-up, a latency-critical thread that must stay out of the allocator's lock.  Such a caller
 * needs row_ptr / col_idx / tile_pairs for tra_sparse_attn and has no use for the Boolean mask, which
 * is then scratch; this call keeps that scratch in a fixed array of TRA_STATIC_BLOCK_MASK_BYTES
 * (16 MiB) inside the library's device image.  Every GPU on which the library is loaded holds those
 * 16 MiB until the process exits.
 *   Arguments and results as tra_build_block_mask without `block_mask`: the same row_ptr, col_idx,
 *   nnz_out and tile_pairs, bit for bit; the same recorded errors.
 *   Limit: B * heads * NB * NB <= TRA_STATIC_BLOCK_MASK_BYTES, else TRA_ERR_CAPACITY is returned and
 *   nothing runs (the 75.6K-token, 40-head shape with 128-token blocks needs 13.97 MB).
 *   The call itself allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *   The first call on a device looks up the array's device address (once per device, with that device
 *   current); make that first call before starting any stream capture.
 *   All calls on a device share the one array, which keeps the last call's mask: two calls whose
 *   kernels can overlap on the GPU (different streams without an ordering between them) race; order
 *   them.  Nothing needs clearing between calls: a call writes every mask entry it later reads.
 * Errors: TRA_ERR_INVALID_ARG (NULL pointer, non-positive count, a current device other than the
 * plan's), TRA_ERR_CAPACITY (mask larger than the array, see above; or, recorded in the plan status,
 * col_idx too small), TRA_ERR_UNSUPPORTED / TRA_ERR_CUDA as for tra_build_block_mask. */
#define TRA_STATIC_BLOCK_MASK_BYTES (16u << 20)
int tra_build_block_list_static(const tra_plan_t* plan, const uint16_t* ridx, int32_t* row_ptr,
                                int32_t* col_idx, int64_t col_idx_capacity, int64_t* nnz_out,
                                int32_t* tile_pairs, int B, int heads, void* stream);

/* Block-sparse attention (Eq. 16 as executed: Section 3.2, last paragraph, and "Limitations"):
 * softmax attention of each query over the valid keys of the retained key blocks of its block row.
 *   ridx == NULL: retained blocks are evaluated in full, no token mask inside them (what the
 *                 paper's block-sparse execution does);
 *   ridx != NULL: uint16 [B, heads, N] from tra_budget_radius; inside the retained blocks a video
 *                 query additionally sees only the video keys inside its disk (the token mask of
 *                 Eq. 15 on top of the block list); text keys and text queries are not masked.
 *   row_ptr == NULL and col_idx == NULL (only with ridx != NULL): Eq. 16 itself, no block list — a
 *                 video query sees exactly the video keys inside its disk, text keys and text
 *                 queries are not masked.  The kernel finds the key blocks a query block can reach
 *                 from the plan's block boxes; no [heads, NB, NB] mask is needed.
 * A query that is left with no visible key gets O = 0 and lse = -inf.
 *   row_ptr, col_idx: the CSR list written by tra_build_block_mask (reusable across calls:
 *   Section 3.3, warm-up reuse).  tile_pairs: the table the same call wrote, or NULL (consecutive
 *   tiles share a thread block); any table in which every tile 0 .. NT-1 of a (batch, head) appears
 *   exactly once gives the same result.  Q, K, V, O as in tra_entropy_attn.  lse: fp32 or NULL, exact
 *   to fp32 rounding. */
int tra_sparse_attn(const tra_plan_t* plan, const void* Q, const void* K, const void* V,
                    const int32_t* row_ptr, const int32_t* col_idx, const uint16_t* ridx,
                    const int32_t* tile_pairs, void* O, float* lse, int B, int heads, float sm_scale,
                    void* stream);

/* ---- the whole pass over HOST tensors (the paper has no counterpart: plumbing around the calls
 * above for callers whose Q, K, V and O live in host memory) ----------------------------- */

/* One pass of the hot path — tile-major layout, dense attention + entropy, budget / radius, block
 * mask, block-sparse attention (retained blocks in full), layout back — over
 *   Q_host, K_host, V_host : HOST pointers, bf16 [heads, S, head_dim], RASTER token order (read),
 *   O_host                 : HOST pointer, same shape and order (written): the block-sparse output.
 * Heads are independent problems, so the pass runs in groups of at most `group` heads (the first
 * group holds `first_group` <= group heads, so that the kernels start early, the following ones
 * twice as many as the one before until `group` is reached, and the last group is split so that
 * little output is left to copy after the last kernel); the host-to-device copy of
 * the next group and the device-to-host copy of the previous one run on two copy streams owned by
 * the plan while the kernels of the current group run on `stream`.  Pinned (page-locked) host
 * memory is needed for the copies to overlap; pageable memory works but serialises.
 *   workspace : DEVICE memory, 256-byte aligned, at least tra_hot_path_host_workspace_bytes(plan,
 *               group) bytes; owned by the caller, free to reuse once `stream` has passed the call.
 * The call allocates no device memory (on its first uses it creates the plan's two copy streams and
 * a pool of events, which later calls reuse).  The current device must be the one the plan was
 * created on.  It returns after enqueueing; `stream` completes after the last copy in
 * either direction, so synchronising `stream` (or an event recorded on it) makes O_host valid.
 * Calls that share a plan or a workspace must be ordered on `stream`.
 * Errors: TRA_ERR_INVALID_ARG (NULL / misaligned pointer, non-positive count or scale, another
 * current device), TRA_ERR_CAPACITY (workspace too small), TRA_ERR_CUDA; kernel-side errors as for
 * the four calls.  After a non-OK return part of the pass may already be enqueued, with the copy
 * streams and `stream` waiting on one another: synchronise `stream` before the workspace or the
 * host buffers are reused. */
size_t tra_hot_path_host_workspace_bytes(const tra_plan_t* plan, int group);
int tra_hot_path_host(tra_plan_t* plan, const void* Q_host, const void* K_host, const void* V_host,
                      void* O_host, void* workspace, size_t workspace_bytes, int heads, int group,
                      int first_group, float sm_scale, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TRA_H_ */
