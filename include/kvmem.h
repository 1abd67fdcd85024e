/* kvmem.h - C ABI of the KVMem recall step on one NVIDIA B200 (sm_100a).
 *
 * One recall step (paper Sec. 4.1, Sec. 5.2): score every historical paged-KV block of a
 * session against the current query through the Mean-K attention-space index, select the
 * top blocks under the active-context budget, assemble the query-dependent execution
 * view from the block table, and run GQA decode attention over that view.
 *
 * Conventions
 *   - Every pointer is marked HOST or DEVICE.  Device buffers, including the pool's backing
 *     storage, views, outputs and workspaces, are owned by the caller; the library owns only
 *     the opaque handle and its host-side metadata and never allocates device memory.
 *   - All device work is enqueued on the given stream (a cudaStream_t passed as void*) and is
 *     asynchronous unless a call says otherwise.  A pool is not thread-safe.  The pool's device must be the calling
 *     thread's current device in every call that enqueues work (KVMEM_E_STATE otherwise).
 *   - Every call returns a kvmem_status_t.  Argument, state and capacity errors are detected
 *     on the host before anything is enqueued and leave the pool unchanged; kvmem_last_error()
 *     then describes the failure.  Anomalies seen on the device (a block id out of range, a
 *     bounded wait that expired) set a sticky status word read by kvmem_device_status().
 *   - Element type of K, V, q and the index is bf16 (2 bytes).  Scores, attention outputs
 *     and log-sum-exp values are fp32.
 *   - Logical block ids are the append order within a session, i.e. chronological order
 *     (Sec. 5.2, block records).  Only whole blocks of block_tokens tokens exist: the Mean-K
 *     index covers completed blocks only (Sec. 5.2).
 *   - Keys and queries are taken to be position-independent already (Sec. 4.3, "Mean-K
 *     Retrieval-Index Construction"); K is copied into the view unchanged.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 */
#ifndef KVMEM_H_
#define KVMEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvmem_pool kvmem_pool_t; /* opaque; created and destroyed by the library */

typedef enum {
    KVMEM_OK = 0,
    KVMEM_E_INVALID = -1,     /* bad argument (null, out of range, misaligned, partial block)   */
    KVMEM_E_CAPACITY = -2,    /* pool, session or caller buffer too small                       */
    KVMEM_E_STATE = -3,       /* page already in use, session empty, stale handle               */
    KVMEM_E_CUDA = -4,        /* a CUDA runtime or driver call failed                           */
    KVMEM_E_TIMEOUT = -5,     /* device status: a bounded wait inside a kernel gave up          */
    KVMEM_E_UNSUPPORTED = -6, /* shape outside what the kernels were built for                  */
    KVMEM_E_DEVICE_RANGE = -7 /* device status: a block or page id was out of range and skipped */
} kvmem_status_t;

/* Geometry of the paged KV repository (Sec. 3.1: logical blocks of B_blk tokens; Sec. 5.2:
 * blocks aligned with physical pages). */
typedef struct {
    int32_t n_layers;               /* scored attention layers L (1 in the benchmark configurations)   */
    int32_t n_q_heads;              /* H                                                               */
    int32_t n_kv_heads;             /* G; H % G == 0                                                   */
    int32_t head_dim;               /* d; 128 is what the kernels are built for                        */
    int32_t block_tokens;           /* B_blk; a multiple of 16, at most 256                            */
    int32_t max_sessions;           /* independent workspaces sharing the page pool                    */
    int32_t max_blocks;             /* physical pages in the pool                                      */
    int32_t max_blocks_per_session; /* rows of one session's block table and index                     */
    int32_t device;                 /* CUDA device ordinal                                             */
    int32_t rope_max_positions;     /* 0: no rotary support.  Else the pool holds a cos/sin table for
                                       positions [0, rope_max_positions): the native window, since every
                                       token is encoded and re-encoded inside an execution view (8 bytes x
                                       head_dim / 2 per position)                                      */
    float rope_theta;               /* rotary base (e.g. 1e6); used when rope_max_positions > 0        */
    int32_t rope_in_block_keys;     /* 0: the pages hold raw (position-free) keys.  1 (needs rotary support with
                                       rope_max_positions >= block_tokens; the fused materialise+attend pass on this
                                       layout needs 64-token blocks): a page holds k' = RoPE(k, t), t the token's offset inside its
                                       block, so that a block placed at compact position p0 needs the rotation
                                       of p0 alone: the position-consistent view rotates by one angle set per
                                       block, and the copy-free attention rotates the QUERY back by p0 once per
                                       block instead of every key forward (q . R(p0 + t) k = (R(-p0) q) . R(t) k).
                                       The Mean-K index is built from the raw keys either way              */
    int32_t fp8_pages;              /* 0: pages hold bf16.  1 (head_dim 128, 64-token blocks; rotary support only together
                                       with rope_in_block_keys, in which case the codes are those of RoPE(k, t) and
                                       kvmem_paged_attend_fp8_rope is the position-consistent reader): the
                                       repository itself is FP8 (Sec. 6.1: the KV cache is kept in FP8): a page holds the
                                       E4M3 codes of k / fp8_k_scale ([64 tokens][128] bytes per layer and KV head) and
                                       of v / fp8_v_scale transposed ([128 dims][64 tokens] bytes), i.e. the tiles of the
                                       FP8 execution view; half the memory and half the traffic of every pass over
                                       pages.  kvmem_append_blocks still takes bf16 K and V and builds the bf16 Mean-K
                                       index from them; kvmem_materialize_fp8 and kvmem_paged_attend_fp8 are the calls
                                       that read such pages, the bf16 page readers return KVMEM_E_STATE            */
    float fp8_k_scale;              /* static per-tensor scales of an FP8 repository (positive, finite)              */
    float fp8_v_scale;
} kvmem_pool_config_t;

/* Selection budget (Eq. "active_budget", Eq. "active_capacity" in Sec. 3.1; selector in
 * Sec. 4.3).  The number of blocks kept is
 *     k = min(budget_blocks, floor((max_view_tokens - mandatory_tokens) / block_tokens), NB), k >= 0.
 * The oldest n_sink_blocks and newest n_recent_blocks are kept first (sinks before recents,
 * truncated to k, overlap counted once); remaining slots go to the largest scores, equal
 * scores to the lower block id.  Reserved blocks still take part in the softmax. */
typedef struct {
    int32_t budget_blocks;    /* requested k                                    */
    int32_t max_view_tokens;  /* B_a = min(B_model, B_gpu), in tokens           */
    int32_t mandatory_tokens; /* N(Q_tau): context the view must leave room for */
    int32_t n_sink_blocks;
    int32_t n_recent_blocks;
} kvmem_select_params_t;

/* ---- pure host helpers (no CUDA call) -------------------------------------------------- */

/* Bytes of DEVICE storage kvmem_pool_create needs for this geometry (0 if cfg is invalid).
 * Holds the K/V pages, the Mean-K index, the block tables, a status word and, if enabled, the rotary table. */
size_t kvmem_pool_bytes(const kvmem_pool_config_t* cfg /*HOST*/);

/* The budget clamp above for a session of n_blocks blocks; never negative. */
int32_t kvmem_budget_blocks(const kvmem_select_params_t* params /*HOST*/, int32_t block_tokens, int32_t n_blocks);

/* Bytes of DEVICE workspace kvmem_select needs for n_sessions sessions and n_q_tokens query
 * tokens per session (0 if the arguments are invalid). */
size_t kvmem_select_workspace_bytes(const kvmem_pool_config_t* cfg /*HOST*/, int32_t n_sessions, int32_t n_q_tokens);

/* Bytes of DEVICE workspace kvmem_view_attend needs (split-K partial results). */
size_t kvmem_attend_workspace_bytes(const kvmem_pool_config_t* cfg /*HOST*/, int32_t n_sessions, int32_t n_q_tokens);

/* Description of the calling thread's last failure (static storage, never NULL). */
const char* kvmem_last_error(void);

/* ---- pool lifetime ---------------------------------------------------------------------- */

/* Create a pool inside caller-owned DEVICE storage of at least kvmem_pool_bytes(cfg) bytes,
 * 256-byte aligned.  The storage must outlive the pool.  Clears the tables and the status word
 * (synchronous).  KVMEM_E_UNSUPPORTED if the device is not compute capability 10.x. */
int kvmem_pool_create(const kvmem_pool_config_t* cfg /*HOST*/, void* storage /*DEVICE*/, size_t bytes,
                      kvmem_pool_t** out /*HOST*/);
int kvmem_pool_destroy(kvmem_pool_t* pool);

/* Forget a session's blocks and return its pages to the free list.  The host-side bookkeeping changes at once; the
 * session's block count on the device is cleared on `stream`, so calls enqueued after it on that stream (select, top-k,
 * attention over its pages) see an empty session: n_sel = 0, nothing read.  Work enqueued earlier that still reads
 * the session's pages must have been ordered before any append that reuses them (same stream, or an event). */
int kvmem_session_reset(kvmem_pool_t* pool, int32_t session, void* stream);

/* Blocks appended to a session so far, or a negative status. */
int32_t kvmem_session_blocks(const kvmem_pool_t* pool, int32_t session);

/* ---- repository and index (Sec. 4.3, Eq. "mean_k_index"; Sec. 5.3 "Incremental Indexing") - */

/* Append n_blocks completed blocks to a session: copy their K and V into physical pages,
 * extend the block table and compute the Mean-K entry of each new block,
 *     kbar[l][b][g] = (1/B) * sum_{i in b} k[l][i][g]
 * (fp32 sum in ascending token order, one round-to-nearest-even to bf16).
 *   k, v       DEVICE bf16 [n_blocks * block_tokens][n_layers][n_kv_heads][head_dim], 16-byte aligned;
 *              may be released once the stream has run the call
 *   phys_ids   HOST int32 [n_blocks] page ids to use, or NULL to take free pages in ascending order
 * On a pool created with rope_in_block_keys, k holds raw keys, the index is built from them, and the
 * page receives RoPE(k, t), t = the token's offset inside its block.
 * Errors: KVMEM_E_CAPACITY (session or pool full), KVMEM_E_STATE (page in use), KVMEM_E_INVALID.  The session's block
 * count on the device is raised only after the kernel that writes the new pages and index rows has been enqueued, so
 * a KVMEM_E_CUDA from this call leaves the session as it was, on the host and on the device. */
int kvmem_append_blocks(kvmem_pool_t* pool, int32_t session, const void* k /*DEVICE*/, const void* v /*DEVICE*/,
                        int32_t n_blocks, const int32_t* phys_ids /*HOST*/, void* stream);

/* ---- position-consistent keys (Sec. 4.3: positional encoding removed before indexing and from the
 * query; Sec. 4.4: RoPE applied to raw K at the assigned compact position, V copied unchanged, with
 * precomputed sine/cosine tables).  Needs rope_max_positions > 0.  Rotary variant: pairs (i, i + d/2),
 * frequency theta^(-2i/d), table = fp32 cos/sin of the fp64 angle; a rotated element is four fp32
 * products and two fp32 sums (no fused multiply-add), rounded once to bf16. ------------------------ */

/* kvmem_append_blocks for keys that still carry RoPE: token t of new block i was encoded at position
 * block_pos0[i] + t (its position in the execution window it was computed in).  The encoding is removed,
 * the raw keys are stored in the pages and indexed; block_pos0 is kept in the block record.  (With
 * rope_in_block_keys the raw keys are indexed and the pages receive RoPE(raw, t), t the offset in the block.)
 *   block_pos0  HOST int32 [n_blocks]; every position must lie in [0, rope_max_positions) */
int kvmem_append_blocks_rope(kvmem_pool_t* pool, int32_t session, const void* k_roped /*DEVICE*/, const void* v /*DEVICE*/,
                             int32_t n_blocks, const int32_t* phys_ids /*HOST*/, const int32_t* block_pos0 /*HOST*/,
                             void* stream);

/* Rotate n_rows x n_vec vectors of head_dim elements: y[r][v] = RoPE(x[r][v], positions[r]), or the
 * inverse rotation (inverse != 0), e.g. to bring the current query into the position-independent space
 * the index lives in.  x, y DEVICE bf16 [n_rows][n_vec][head_dim] (may alias); positions DEVICE int32
 * [n_rows].  Rows with a position outside the table are left unwritten and flagged in the status word. */
int kvmem_rope_rotate(kvmem_pool_t* pool, const void* x /*DEVICE*/, void* y /*DEVICE*/, int64_t n_rows, int32_t n_vec,
                      const int32_t* positions /*DEVICE*/, int32_t inverse, void* stream);

/* kvmem_materialize with position-consistent keys: the key of view token j*B + t is the raw key rotated
 * to compact position first_position + j*B + t; values are copied unchanged.  With rope_in_block_keys the
 * stored key already carries the rotation of t and is rotated by first_position + j*B: one set of angles per
 * block (the result differs from the raw-key path by one extra bf16 rounding of the stored key).
 * first_position + budget * B must not exceed rope_max_positions (KVMEM_E_INVALID otherwise). */
int kvmem_materialize_rope(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids /*DEVICE*/,
                           int32_t sel_stride, const int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/,
                           void* view_v /*DEVICE*/, int32_t view_cap_tokens, int32_t first_position, void* stream);

/* ---- the recall step ----------------------------------------------------------------------- */

/* Scores only (Eq. "kvmem-block-score", Sec. 4.3): the first half of kvmem_select, same arguments and
 * definitions; scores (required) receives score_scale * R for every session.  score_scale (0 selects 1) lets a rank
 * that holds 1/N of the heads of a session write its share of the head mean directly (score_scale = 1/N): the sum of
 * the ranks' outputs is then R, with no arithmetic outside the library. */
int kvmem_score(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/, int32_t n_q_tokens,
                float* scores /*DEVICE*/, float score_scale, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Selection alone (Sec. 4.3: reserve sink and recent blocks, fill the budget with the largest R_b, ties to the
 * lower id, chronological output): the second half of kvmem_select, for scores the caller already has (for
 * example from kvmem_score_host_index).  scores DEVICE fp32 [n_sessions][scores_stride], non-negative; the
 * session lengths are the pool's.  sel_ids, sel_stride, n_sel and errors as in kvmem_select. */
int kvmem_topk(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const float* scores /*DEVICE*/,
               int32_t scores_stride, const kvmem_select_params_t* params /*HOST*/, int32_t* sel_ids /*DEVICE*/,
               int32_t sel_stride, int32_t* n_sel /*DEVICE*/, void* stream);

/* Block relevance against an index that lives in HOST memory (Sec. 5.2: the index is streamed to the GPU in
 * tiles and softmax statistics are carried across tiles; Sec. 5.3 "Incremental Indexing" keeps the index small
 * enough for that).  R is the same quantity kvmem_score computes (Eq. "kvmem-block-score"), for one session.
 *   index_host  HOST bf16 [n_layers][n_kv_heads][index_stride_blocks][head_dim], 16-byte aligned; page-locked
 *               memory makes the copies asynchronous and fast, pageable memory works but serialises
 *   n_blocks    blocks to score (<= index_stride_blocks)
 *   q           DEVICE bf16 [n_q_tokens][n_layers][n_q_heads][head_dim], 1..16 query tokens
 *   tile_blocks blocks per head and tile, a multiple of 128
 *   scores      DEVICE fp32 [n_blocks]
 *   staging     DEVICE, kvmem_score_host_staging_bytes(): two tiles, 256-byte aligned
 *   workspace   DEVICE, kvmem_score_host_workspace_bytes(): fp32 logits of all blocks and the per-tile statistics
 * Tile i + 1 is copied (on a stream the pool owns) while tile i is scored on `stream`; the two are ordered by
 * events only.  When the call returns, work is queued on both streams; `stream` alone has to be waited for.
 * index_host must stay valid until then.  Calls on one pool must not overlap.  Errors: KVMEM_E_INVALID,
 * KVMEM_E_CAPACITY, KVMEM_E_CUDA as elsewhere. */
size_t kvmem_score_host_workspace_bytes(const kvmem_pool_t* pool, int32_t n_blocks, int32_t n_q_tokens, int32_t tile_blocks);
size_t kvmem_score_host_staging_bytes(const kvmem_pool_t* pool, int32_t tile_blocks);
int kvmem_score_host_index(kvmem_pool_t* pool, const void* index_host /*HOST*/, int32_t n_blocks, int32_t index_stride_blocks,
                           const void* q /*DEVICE*/, int32_t n_q_tokens, int32_t tile_blocks, float* scores /*DEVICE*/,
                           void* staging /*DEVICE*/, size_t staging_bytes, void* workspace /*DEVICE*/,
                           size_t workspace_bytes, void* stream);

/* Score and select (Sec. 4.3, Eq. "kvmem-block-score"; selector; Sec. 5.2 tiled scoring with the
 * softmax kept global across tiles).  For each session s in [session_first, session_first + n_sessions):
 *     R_b = sum_m (1/(L*H)) sum_{l,h} softmax_{b' in all blocks of s}( q[m][l][h] . kbar[l][b'][g(h)] / sqrt(d) )_b
 * then the selector described at kvmem_select_params_t.
 *   q          DEVICE bf16 [n_sessions][n_q_tokens][n_layers][n_q_heads][head_dim], 16-byte aligned
 *   sel_ids    DEVICE int32 [n_sessions][sel_stride]: ascending logical ids; entries past n_sel untouched
 *   sel_stride >= the clamped budget of every session
 *   n_sel      DEVICE int32 [n_sessions]
 *   scores     DEVICE fp32 [n_sessions][max_blocks_per_session] receives R (first NB entries), or NULL
 *   workspace  DEVICE, kvmem_select_workspace_bytes(), 256-byte aligned; contents undefined afterwards
 * One query chunk gives one score vector and one selection (sum over its tokens). */
int kvmem_select(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                 int32_t n_q_tokens, const kvmem_select_params_t* params /*HOST*/, int32_t* sel_ids /*DEVICE*/,
                 int32_t sel_stride, int32_t* n_sel /*DEVICE*/, float* scores /*DEVICE*/, void* workspace /*DEVICE*/,
                 size_t workspace_bytes, void* stream);

/* Assemble the execution view (Sec. 4.4 "execution view"; Sec. 5.2): view tokens
 * [j*B, (j+1)*B) of session s are block sel_ids[s][j]'s K and V, fetched through the block table.
 *   view_k, view_v  DEVICE bf16 [n_sessions][n_layers][n_kv_heads][view_cap_tokens][head_dim], 16-byte aligned
 *   n_sel is read on the device; blocks that would not fit view_cap_tokens are skipped and flagged.
 * An id outside the session (or a table entry outside the pool) is skipped as well: its view tokens are left
 * untouched and kvmem_device_status reports KVMEM_E_DEVICE_RANGE.  Tokens past n_sel * B are left untouched. */
int kvmem_materialize(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids /*DEVICE*/,
                      int32_t sel_stride, const int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/,
                      void* view_v /*DEVICE*/, int32_t view_cap_tokens, void* stream);

/* Incremental execution view (Eq. "kvmem-working-set-delta", Sec. 4.4: only what changed between two consecutive
 * working sets moves).  view_k / view_v hold the view kvmem_materialize (or this call) built from prev_ids; afterwards
 * they hold the view of sel_ids, bit-identical to kvmem_materialize's.  A slot j whose block stays (prev_ids[s][j] ==
 * sel_ids[s][j], j < n_prev[s]) is neither read nor written; every other slot receives its block from the pages
 * through the block table.  (A retained block that changes its slot is fetched from the repository rather than
 * shifted inside the view: with the whole history in HBM both cost one read and one write, and fetching has no
 * ordering hazard.)  HBM traffic: 2 bytes per byte of the slots that change.
 *   prev_ids  DEVICE int32 [n_sessions][sel_stride], n_prev DEVICE int32 [n_sessions]: the selection the view holds
 *   stats     DEVICE int32 [n_sessions][3] or NULL: slots unchanged, retained blocks that moved, incoming blocks
 * Other arguments and errors as kvmem_materialize.  prev_ids and sel_ids must be different buffers. */
int kvmem_materialize_delta(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const int32_t* prev_ids /*DEVICE*/,
                            const int32_t* n_prev /*DEVICE*/, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                            const int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/, void* view_v /*DEVICE*/,
                            int32_t view_cap_tokens, int32_t* stats /*DEVICE, may be NULL*/, void* stream);

/* GQA decode attention over the view (QW3 attention kernels, Sec. 5.1; decode over the fixed
 * working set, Sec. 5.2).  For every query token m, layer l and head h, over the first
 * T = n_sel[s] * B view tokens of KV head g(h), without mask:
 *     out = softmax(q . K^T * scale) V        lse = ln sum_t exp(q . k_t * scale)
 * lse lets the caller merge attention over the tokens it appends after the view.
 *   q        DEVICE bf16 [n_sessions][n_q_tokens][n_layers][n_q_heads][head_dim]
 *   out      DEVICE fp32 [n_sessions][n_q_tokens][n_layers][n_q_heads][head_dim]
 *   lse      DEVICE fp32 [n_sessions][n_q_tokens][n_layers][n_q_heads]
 *   scale    0 selects 1/sqrt(head_dim)
 *   workspace DEVICE, kvmem_attend_workspace_bytes(), 256-byte aligned
 * T = 0 gives out = 0 and lse = -inf.  n_q_tokens * (H/G) <= 64 query rows per KV head and call (e.g. 1 + 7 draft tokens
 * with 8 query heads per KV head): up to 16 rows the K/V stream bounds the pass, with 32 or 64 rows the same stream
 * is read once and the tensor-core work per byte doubles or quadruples (the position-consistent and FP8 variants
 * take 16 rows).  Any block size the pool accepts (the view is walked in 64-token tiles; a shorter last tile is
 * masked); head_dim 128.  The calls that read pages through the block table (kvmem_materialize_attend,
 * kvmem_paged_attend, kvmem_paged_attend_rope on raw keys, kvmem_view_cache_attend) take block sizes that divide
 * 64 tokens (a tile is then 64 / B selected blocks, the last one possibly partly filled) or are a multiple of it,
 * among them the paper's default of 32 tokens (Sec. 4.3), also on the in-block key layout (kvmem_paged_attend_rope
 * then rotates the query back once per block of a tile); kvmem_materialize_attend_rope on the in-block layout and the
 * FP8 repository are built for 64-token blocks.  Other shapes return KVMEM_E_UNSUPPORTED. */
int kvmem_view_attend(kvmem_pool_t* pool, int32_t n_sessions, const void* q /*DEVICE*/, int32_t n_q_tokens,
                      const void* view_k /*DEVICE*/, const void* view_v /*DEVICE*/, int32_t view_cap_tokens,
                      const int32_t* n_sel /*DEVICE*/, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                      void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* kvmem_materialize followed by kvmem_view_attend as ONE pass over the selected blocks (Sec. 4.4 execution
 * view + Sec. 5.2 decode over it): each selected K/V tile is read once from the page pool through the
 * block table, written to its place in the view, and attended over while it sits in shared memory.
 * Same arguments, results, limits and error behaviour as the two separate calls; the view it leaves
 * behind is bit-identical to kvmem_materialize's, and out/lse are those of kvmem_view_attend on it.
 * HBM traffic per view byte drops from 2 reads + 1 write to 1 read + 1 write.  (The one difference: an id outside
 * the session cannot be skipped by a pass that also attends, so page 0 stands in for it, in the view and in out/lse,
 * and KVMEM_E_DEVICE_RANGE is reported; the results of such a call are to be discarded.) */
int kvmem_materialize_attend(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                             int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                             const int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/, void* view_v /*DEVICE*/,
                             int32_t view_cap_tokens, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                             void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Copy-free execution view (Sec. 4.4: the view as a page table over non-contiguous physical pages;
 * Sec. 5.3 "Copy-free execution-view assembly"): GQA decode attention straight over the selected
 * blocks' pages, in the order of sel_ids, through the block table.  No contiguous view is written.
 * out and lse equal kvmem_view_attend's on the view kvmem_materialize would build from the same ids
 * (same tiles, same order, same arithmetic).  HBM traffic: one read per view byte.
 * Arguments as in kvmem_materialize_attend, without the view buffers. */
int kvmem_paged_attend(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                       int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                       const int32_t* n_sel /*DEVICE*/, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                       void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Copy-free execution view with position-consistent keys (Sec. 4.4: the view is a page table over the
 * physical pages, and RoPE is applied to raw K at the block's assigned compact position): as
 * kvmem_paged_attend, but the warps that attend over a tile rotate their key fragments, between the tile's
 * arrival from the pages and their use, to compact position first_position + j*block_tokens + t (j = index in
 * sel_ids).  The angle of a position p1 + b (p1 the first of a warp's 16 positions, b < 16) is composed from the
 * table rows of p1 and of b: cos and sin within a few fp32 units in the last place of the table's own row, so a
 * rotated key is within one bf16 rounding step of kvmem_rope_rotate's, and out and lse are those of
 * kvmem_view_attend on the view kvmem_materialize_rope would build from the same ids within the attention
 * tolerance (not bit for bit); they equal kvmem_materialize_attend_rope's on a raw-key pool bit for bit.  Nothing is
 * written besides out and lse.  The pool's pages must hold raw keys and q must carry RoPE at its own position.
 * HBM traffic: one read per view byte (the rotary rows are 2 KiB per 64-token tile).
 * On a pool created with rope_in_block_keys (pages hold k' = RoPE(k, t)) no key is rotated: the logit
 * q . R(p0 + t) k equals (R(-p0) q) . k', p0 = first_position + j*block_tokens, so the 16 query rows are rotated
 * back by p0 once per block (arithmetic of kvmem_rope_rotate, inverse; the rotated query is a bf16 vector)
 * and the stored keys feed the tensor cores as they are.  The result is the same mathematics as attention
 * over kvmem_materialize_rope's view, one rounding of the query instead of one of each key apart.
 * Extra errors: KVMEM_E_STATE without a rotary table; KVMEM_E_INVALID if
 * [first_position, first_position + sel_stride*block_tokens) leaves the table. */
int kvmem_paged_attend_rope(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                            int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                            const int32_t* n_sel /*DEVICE*/, int32_t first_position, float scale, float* out /*DEVICE*/,
                            float* lse /*DEVICE*/, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* kvmem_materialize_rope followed by kvmem_view_attend in one call (Sec. 4.4: the execution view with keys
 * encoded at their compact positions, then decode over it).  Same arguments as kvmem_materialize_attend plus
 * first_position and a q that carries RoPE at its own position.  ONE pass, 1 read + 1 write per view byte.
 * On a pool with rope_in_block_keys each K tile is rotated by its block's compact position while it sits in shared
 * memory, then stored and attended over: the view left behind is kvmem_materialize_rope's and out/lse are
 * kvmem_view_attend's on it, bit for bit.
 * On a raw-key pool the warps that attend over a tile rotate its key fragments to their compact positions on the way
 * to the tensor cores and hand them back to the tile, which is then stored.  Their angles are composed from two
 * table rows as in kvmem_paged_attend_rope, so the view's VALUES are kvmem_materialize_rope's bit for bit and its KEYS
 * are within one bf16 rounding step of them (a small fraction of the elements differs at all); out/lse are the
 * attention over the view this call writes.  Callers that need the key bytes of kvmem_materialize_rope exactly use
 * that call and kvmem_view_attend.  (The view's last 64-token tile must lie inside the rotary table: first_position +
 * the view length rounded up to 64.)
 * Extra errors: KVMEM_E_STATE without a rotary table; KVMEM_E_INVALID if the compact positions leave it. */
int kvmem_materialize_attend_rope(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                                  int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                                  const int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/, void* view_v /*DEVICE*/,
                                  int32_t view_cap_tokens, int32_t first_position, float scale, float* out /*DEVICE*/,
                                  float* lse /*DEVICE*/, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Working-set delta between two consecutive steps (Eq. "kvmem-working-set-delta", Sec. 4.4):
 *     retained R = W_next n W_prev,   incoming L = W_next \ W_prev,   outgoing E = W_prev \ W_next.
 * prev_ids / next_ids are the ascending id lists kvmem_select wrote at the two steps, a block's slot is
 * its index in its list (compact position / block_tokens).  All DEVICE int32:
 *   prev_ids, next_ids [n_sessions][stride];  n_prev, n_next [n_sessions]
 *   retained [n_sessions][stride][3] = (id, slot in prev, slot in next)   ascending ids
 *   incoming [n_sessions][stride][2] = (id, slot in next);  outgoing [n_sessions][stride] = id
 *   counts   [n_sessions][3] = (|R|, |L|, |E|)
 * A retained block whose slot moved needs its resident keys re-rotated by (new - old) * block_tokens
 * positions (kvmem_rope_rotate); only incoming blocks have to be fetched. */
int kvmem_working_set_delta(kvmem_pool_t* pool, int32_t n_sessions, const int32_t* prev_ids /*DEVICE*/,
                            const int32_t* n_prev /*DEVICE*/, const int32_t* next_ids /*DEVICE*/,
                            const int32_t* n_next /*DEVICE*/, int32_t stride, int32_t* retained /*DEVICE*/,
                            int32_t* incoming /*DEVICE*/, int32_t* outgoing /*DEVICE*/, int32_t* counts /*DEVICE*/,
                            void* stream);

/* FP8 execution view (the paper's evaluation keeps the KV cache in FP8, Sec. 6.1): kvmem_materialize and
 * kvmem_view_attend for a view that stores one byte per element.
 * Element = E4M3 code (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities, largest value 448) of
 * x * (1 / scale): one fp32 product, round to nearest with ties to even, saturated to +-448; one static scale
 * per tensor (k_scale for keys, v_scale for values), > 0.  (The paper states no scaling rule; static
 * per-tensor scales are how FP8 KV caches are commonly run.)
 *   view_k8   DEVICE uint8 [n_sessions][n_layers][n_kv_heads][view_cap_tokens][head_dim]
 *   view_v8t  DEVICE uint8 [n_sessions][n_layers][n_kv_heads][view_cap_tokens / 64][head_dim][64]: values are
 *             transposed inside every 64-token tile, so that attention reads both operands along the index it
 *             contracts over
 *   both 128-byte aligned; view_cap_tokens a multiple of 64; other arguments as in kvmem_materialize /
 *   kvmem_view_attend.  Built for head_dim 128 and 64-token blocks (KVMEM_E_UNSUPPORTED otherwise).
 * kvmem_materialize_fp8 reads the bf16 pages through the block table and writes the codes (2 bytes read + 1
 * byte written per element).  kvmem_view_attend_fp8 computes out = softmax(q . (k8 * k_scale)^T * scale)
 * (v8 * v_scale) and lse over the first n_sel[s] * 64 view tokens: half the bytes of the bf16 view; the codes
 * are widened to f16 (exactly) in registers and contracted on the tensor cores with fp32 accumulation. */
int kvmem_materialize_fp8(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids /*DEVICE*/,
                          int32_t sel_stride, const int32_t* n_sel /*DEVICE*/, void* view_k8 /*DEVICE*/,
                          void* view_v8t /*DEVICE*/, int32_t view_cap_tokens, float k_scale, float v_scale, void* stream);
int kvmem_view_attend_fp8(kvmem_pool_t* pool, int32_t n_sessions, const void* q /*DEVICE*/, int32_t n_q_tokens,
                          const void* view_k8 /*DEVICE*/, const void* view_v8t /*DEVICE*/, int32_t view_cap_tokens,
                          const int32_t* n_sel /*DEVICE*/, float scale, float k_scale, float v_scale, float* out /*DEVICE*/,
                          float* lse /*DEVICE*/, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Position-consistent FP8 execution view (Sec. 4.4 + Sec. 6.1) from a pool of bf16 pages with a rotary table: as
 * kvmem_materialize_fp8, but the key of view token j*64 + t is first rotated to compact position first_position + j*64 + t
 * (arithmetic of kvmem_rope_rotate, one rounding to bf16; with rope_in_block_keys the stored key is rotated by
 * first_position + j*64) and then quantised: element = E4M3 code of RoPE(k, position)_bf16 / k_scale.  Values as in
 * kvmem_materialize_fp8.  kvmem_view_attend_fp8 then attends over it with a q that carries RoPE at its own position.
 * Extra errors: KVMEM_E_STATE without a rotary table or on an FP8 repository; KVMEM_E_INVALID if the compact positions
 * leave the table. */
int kvmem_materialize_fp8_rope(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids /*DEVICE*/,
                               int32_t sel_stride, const int32_t* n_sel /*DEVICE*/, void* view_k8 /*DEVICE*/,
                               void* view_v8t /*DEVICE*/, int32_t view_cap_tokens, int32_t first_position, float k_scale,
                               float v_scale, void* stream);

/* On a pool created with fp8_pages: kvmem_materialize_fp8 copies the selected blocks' 8 KiB tiles as they are (1 byte
 * read + 1 byte written per element; k_scale and v_scale must be the pool's, KVMEM_E_INVALID otherwise), and
 * kvmem_paged_attend_fp8 is the copy-free execution view over such a repository (Sec. 5.3): attention straight
 * over the selected pages through the block table, nothing written besides out and lse; results are those of
 * kvmem_view_attend_fp8 on the view kvmem_materialize_fp8 would build, with the pool's scales (same tiles, same
 * order, same arithmetic).  HBM traffic: one byte per element of the selected blocks.
 * Arguments as kvmem_paged_attend.  KVMEM_E_STATE on a pool with bf16 pages. */
int kvmem_paged_attend_fp8(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                           int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                           const int32_t* n_sel /*DEVICE*/, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                           void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* kvmem_paged_attend_fp8 with position-consistent keys, for a pool with fp8_pages AND rope_in_block_keys (the
 * paper's three mechanisms together: FP8 KV cache, Sec. 6.1; keys encoded at their compact positions, Sec. 4.4;
 * copy-free view, Sec. 5.3).  The pages hold the codes of RoPE(k, t) / fp8_k_scale, t the offset inside the block;
 * codes cannot be re-encoded without a second quantisation, so no key is touched: the logit q . R(p0 + t) k equals
 * (R(-p0) q) . RoPE(k, t), and the 16 query rows are rotated back by the block's compact position p0 =
 * first_position + j*64 once per block (arithmetic of kvmem_rope_rotate, inverse; the rotated query is rounded to
 * bf16, then widened to f16 for the tensor cores).  q carries RoPE at its own position.
 * Extra errors: KVMEM_E_STATE unless the pool has both options; KVMEM_E_INVALID if the compact positions leave the
 * rotary table. */
int kvmem_paged_attend_fp8_rope(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                                int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                                const int32_t* n_sel /*DEVICE*/, int32_t first_position, float scale, float* out /*DEVICE*/,
                                float* lse /*DEVICE*/, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* kvmem_materialize_fp8 followed by kvmem_view_attend_fp8 as ONE pass: every selected tile is read once from the pages,
 * stored to its place in the FP8 view and attended over while it sits in shared memory.  Over an FP8 repository that is
 * 1 byte read + 1 byte written per element; over a bf16 repository (64-token blocks) the tile is quantised on the way
 * (2 bytes read + 1 byte written per element; arithmetic of kvmem_materialize_fp8) with the pool's fp8_k_scale and
 * fp8_v_scale, 1 where the configuration leaves them at 0.  The view and out/lse are those of the two separate calls
 * with the same scales, bit for bit.  Arguments as kvmem_materialize_attend with the FP8 view buffers. */
int kvmem_materialize_attend_fp8(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q /*DEVICE*/,
                                 int32_t n_q_tokens, const int32_t* sel_ids /*DEVICE*/, int32_t sel_stride,
                                 const int32_t* n_sel /*DEVICE*/, void* view_k8 /*DEVICE*/, void* view_v8t /*DEVICE*/,
                                 int32_t view_cap_tokens, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                                 void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* Execution cache: the execution view kept across steps, with working-set reuse and bounded delta
 * re-RoPE (Sec. 4.4: the two views; "Retrieval-Aware Hierarchical Reuse"; Eq. "kvmem-working-set-delta").
 *
 * The cache is cap_blocks slots ("active GPU pages") in caller-owned DEVICE memory of
 * kvmem_view_cache_bytes() bytes, 256-byte aligned, for ONE session.  A slot holds one block in the
 * pool's page format ([K|V][L][G][block_tokens][d] bf16): K encoded for the block's current compact
 * position, V unchanged.  The pool's pages must hold raw (position-independent) keys and the pool must
 * have a rotary table.  kvmem_view_cache_update moves the cache from the previous working set to
 * sel_ids (ascending, as kvmem_select writes them; *n_sel <= cap_blocks):
 *   - a block that is resident and selected again keeps its slot (no data moves); every other slot is
 *     reclaimed; incoming blocks, in ascending id order, take the free slots in ascending slot order,
 *     their K built from raw K with RoPE at compact position first_position + j*block_tokens + t (j =
 *     index in sel_ids), their V copied;
 *   - a retained block whose index j changed has its keys re-encoded: rotated in place by
 *     (j_new - j_old) * block_tokens positions while fewer than max_delta_ropes such rotations have been
 *     applied since its keys were last built from raw K, otherwise rebuilt from raw K (counter reset).
 *     max_delta_ropes = 0 rebuilds every moved block, i.e. the cache always equals
 *     kvmem_materialize_rope's view.
 * Rotation arithmetic as in kvmem_rope_rotate (fp32 products and sums, no fused multiply-add, one
 * rounding to bf16), so cache contents are reproducible bit for bit.
 * stats (DEVICE int32[4], may be NULL) = (retained and unmoved, delta re-RoPEd, rebuilt, incoming).
 * Records inside the cache, at the byte offsets kvmem_view_cache_layout writes to offsets[6] (HOST):
 *   [0] pages  [1] slot_block int32[cap] (-1 = empty)  [2] slot_pos int32[cap]  [3] slot_cnt int32[cap]
 *   [4] view_slots int32[cap]: slot of the j-th selected block (the view's page table)  [5] n_view int32.
 * kvmem_view_cache_attend: GQA decode attention over the cached view through view_slots (no compaction);
 * q [M][L][H][d] bf16, out/lse/workspace/scale as in kvmem_view_attend with n_sessions = 1.
 * Errors: KVMEM_E_STATE without a rotary table; KVMEM_E_INVALID for bad pointers, cap_blocks outside
 * [1, 32768] or positions outside the table; KVMEM_E_CAPACITY if cache_bytes is too small.  A selection
 * longer than cap_blocks or an id outside the session is clamped / skipped on the device and reported as
 * KVMEM_E_DEVICE_RANGE by kvmem_device_status.  Calls on one cache must be ordered (same stream). */
size_t kvmem_view_cache_bytes(const kvmem_pool_t* pool, int32_t cap_blocks);
int kvmem_view_cache_layout(const kvmem_pool_t* pool, int32_t cap_blocks, size_t* offsets /*HOST [6]*/);
int kvmem_view_cache_reset(kvmem_pool_t* pool, void* cache /*DEVICE*/, size_t cache_bytes, int32_t cap_blocks, void* stream);
int kvmem_view_cache_update(kvmem_pool_t* pool, int32_t session, const int32_t* sel_ids /*DEVICE*/,
                            const int32_t* n_sel /*DEVICE*/, void* cache /*DEVICE*/, size_t cache_bytes,
                            int32_t cap_blocks, int32_t max_delta_ropes, int32_t first_position,
                            int32_t* stats /*DEVICE, may be NULL*/, void* stream);
int kvmem_view_cache_attend(kvmem_pool_t* pool, const void* q /*DEVICE*/, int32_t n_q_tokens, void* cache /*DEVICE*/,
                            size_t cache_bytes, int32_t cap_blocks, float scale, float* out /*DEVICE*/,
                            float* lse /*DEVICE*/, void* workspace /*DEVICE*/, size_t workspace_bytes, void* stream);

/* kvmem_view_attend for callers that cannot allocate device memory.  (The paper has no counterpart.)
 * Who needs it: a serving process that gave all of HBM to its KV pool at start-up and runs with
 * its allocator frozen, a plug-in that only ever sees the buffers of one request, or a latency path
 * where a device-synchronising cudaMalloc is not acceptable.  Same arguments, definitions and
 * results as kvmem_view_attend, except that the split-K workspace is a fixed array inside the
 * library (about 4 MiB, held on every GPU that loads the library until the process exits).
 *   - Limit: n_sessions * n_layers * n_kv_heads <= 8 per call; more returns KVMEM_E_CAPACITY with
 *     a message, and nothing is enqueued.
 *   - The call allocates nothing: no cudaMalloc, cudaFree or allocating library routine.
 *   - The first call on a device looks up the array's device address (the pool's device must be
 *     the current device); make that first call before starting any stream capture.  The address
 *     is remembered for the life of the process: the device's primary context must not be reset
 *     (cudaDeviceReset) while the library is in use.
 *   - All calls in the process share the array and it keeps the previous call's contents.  Nothing
 *     in it needs clearing (every slot that is read is overwritten first), but two calls whose
 *     kernels overlap on the GPU (different streams, or different pools on one device) race on it:
 *     keep them on one stream or order them with events. */
int kvmem_view_attend_static(kvmem_pool_t* pool, int32_t n_sessions, const void* q /*DEVICE*/, int32_t n_q_tokens,
                             const void* view_k /*DEVICE*/, const void* view_v /*DEVICE*/, int32_t view_cap_tokens,
                             const int32_t* n_sel /*DEVICE*/, float scale, float* out /*DEVICE*/, float* lse /*DEVICE*/,
                             void* stream);

/* The whole recall step for callers whose query and results live in HOST memory: copies q to the
 * device, runs kvmem_select and kvmem_materialize_attend, copies out and lse back and waits for the
 * stream (synchronous).  Same definitions and limits as the individual calls.
 *   q_host     HOST bf16 [n_sessions][n_q_tokens][L][H][d]   (pinned memory makes the copies asynchronous)
 *   out_host   HOST fp32 [n_sessions][n_q_tokens][L][H][d];  lse_host HOST fp32 [n_sessions][n_q_tokens][L][H]
 *              (when both are pinned, device-mapped memory the last kernel of the step writes them directly
 *              and no copy is issued; otherwise they are copied from the staging buffer)
 *   staging    DEVICE, kvmem_step_staging_bytes(), 256-byte aligned: device copies of q, out, lse
 * sel_ids, n_sel, views and workspaces are DEVICE buffers as in the individual calls and hold the
 * step's selection and view afterwards. */
size_t kvmem_step_staging_bytes(const kvmem_pool_config_t* cfg /*HOST*/, int32_t n_sessions, int32_t n_q_tokens);
int kvmem_recall_step_host(kvmem_pool_t* pool, int32_t session_first, int32_t n_sessions, const void* q_host /*HOST*/,
                           int32_t n_q_tokens, const kvmem_select_params_t* params /*HOST*/, int32_t* sel_ids /*DEVICE*/,
                           int32_t sel_stride, int32_t* n_sel /*DEVICE*/, void* view_k /*DEVICE*/, void* view_v /*DEVICE*/,
                           int32_t view_cap_tokens, float scale, float* out_host /*HOST*/, float* lse_host /*HOST*/,
                           void* staging /*DEVICE*/, size_t staging_bytes, void* select_workspace /*DEVICE*/,
                           size_t select_workspace_bytes, void* attend_workspace /*DEVICE*/,
                           size_t attend_workspace_bytes, void* stream);

/* ---- inspection ------------------------------------------------------------------------------ */

/* Mean-K index of a session: DEVICE bf16 [n_layers][n_kv_heads][max_blocks_per_session][head_dim]
 * (rows >= *n_blocks undefined).  The pointer aliases pool storage. */
int kvmem_get_index(kvmem_pool_t* pool, int32_t session, const void** index /*HOST, receives DEVICE ptr*/,
                    int32_t* n_blocks /*HOST*/);

/* Block table of a session: DEVICE int32 [max_blocks_per_session], logical id -> physical page. */
int kvmem_get_block_table(kvmem_pool_t* pool, int32_t session, const int32_t** table /*HOST, receives DEVICE ptr*/,
                          int32_t* n_blocks /*HOST*/);

/* Synchronise the stream and fetch (and clear) the sticky device status word: KVMEM_OK,
 * KVMEM_E_TIMEOUT or KVMEM_E_DEVICE_RANGE.  Returns KVMEM_OK if the read itself worked. */
int kvmem_device_status(kvmem_pool_t* pool, int32_t* status /*HOST*/, void* stream);

/* Self-test of the failure path every kernel of this library shares.  (The paper has no counterpart.)  All waits
 * inside the kernels (for a TMA copy, for another warp) are bounded: after a time limit the kernel records
 * KVMEM_E_TIMEOUT in the status word and returns, so that a lost copy cannot hang the GPU.  A healthy run never takes
 * that path; this call does: one warp waits limit_us microseconds (1 .. 100,000) for a barrier nobody arrives at, with
 * the same wait routine, then sets KVMEM_E_TIMEOUT and returns.  The kernel ends by itself and the context and the pool
 * stay usable; kvmem_device_status then reports (and clears) KVMEM_E_TIMEOUT.
 *   waited_ns  DEVICE uint64, may be NULL: receives the time the wait lasted, in nanoseconds */
int kvmem_selftest_wait_timeout(kvmem_pool_t* pool, uint32_t limit_us, uint64_t* waited_ns /*DEVICE*/, void* stream);

/* Process-wide implementation switches used to compare kernel variants; "gather_mode" and "score_mode"
 * never change results, "chunk_poly" moves scores by a few 1e-6 relative.  (No counterpart in the paper.)  "gather_mode": 1 = bulk asynchronous copies through shared memory
 * (default), 0 = 128-bit load/store copy.  "score_mode" (decode-sized queries): 1 = dot products on the
 * tensor cores (default), 0 = fp32 ALU kernel that reduces the query rows with warp shuffles.
 * "chunk_poly" (multi-token chunks): n in 2..5 = every n-th exponential of the two softmax passes is a
 * degree-4 polynomial on the FMA pipe instead of a special-function-unit instruction (default 4), 0 = none.
 * "topk_cluster" (sessions above 16,384 blocks): 1 = selection by a thread-block cluster of 8 CTAs that merge
 * their histograms through distributed shared memory (default), 0 = by one CTA that re-reads the scores per pass.
 * "topk_items" (sessions of at most 16,384 blocks): 0 = the selection kernel holds the fewest scores per thread
 * (1, 2, 4, 8 or 16) that cover the session (default), n = at least n; never changes a result.
 * "attend_splits" (0 = chosen by the library, else forced split-K count), "attend_lookahead" (0 = chosen by the
 * library, else tiles the attention producers may run ahead), "gather_ctas" (0 = chosen by the library, else the
 * number of copy CTAs), "attend_landed" (-1 = chosen by the library, 1 / 0 = the lookahead counts tiles that have not
 * landed in shared memory yet / that have not been consumed yet): the knobs of the bytes-in-flight sweeps; only
 * "attend_splits" can move a result, by the rounding of a different split-K merge order.
 * "pdl": 1 = the kernels of a step are launched with programmatic stream serialization, so that the
 * launch latency of each overlaps the tail of the one before (default), 0 = plain launches.
 * The switches are process-wide (every pool, every thread) and atomic: a call that runs while another thread changes a
 * switch sees either value. */
int kvmem_set_option(const char* name /*HOST*/, int32_t value);

#ifdef __cplusplus
}
#endif
#endif /* KVMEM_H_ */
