// GQA decode attention over the execution view (QW3 attention kernels, Sec. 5.1; decode over the
// fixed working set, Sec. 5.2):  out = softmax(q K^T * scale) V,  lse = ln sum_t exp(s_t), no mask.
//
// Split-K flash decoding.  Grid = (split, layer x KV head, session).  A split owns a contiguous
// range of 64-token view tiles.  Inside a CTA one producer warp streams tiles with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, mbarrier completion) into a ring of 32 KiB stages
// (K tile + V tile); two groups of four consumer warps take tiles alternately, each warp 16 tokens.  The M*(H/G) <= 16 query rows of
// the KV head form one m16 MMA tile: S = Q K^T and O += P V run on bf16 mma.sync with fp32
// accumulators (at 16 flop per view byte the step would otherwise be ALU-bound instead of
// HBM-bound), online softmax in fp32 in the exp2 domain.  Each warp carries its own (m, l, O); the
// CTA merges its warps in shared memory and writes one partial per split; a second kernel merges
// the splits in split order with the usual log-sum-exp rescale, so the result does not depend on
// timing.  Every mbarrier wait is bounded and reports KVMEM_E_TIMEOUT through the status word.
#include <cudaTypedefs.h>
#include <math.h>

#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"
#include "kvmem_rope.cuh"

namespace kvmem {

constexpr int kAttStages = 6;
constexpr int kAttConsumers = 8;
constexpr int kAttGroups = 2;                   // consumer groups; kAttStages % kAttGroups == 0
static_assert(kAttStages % kAttGroups == 0, "each group must own whole stages");
constexpr int kAttThreads = (kAttConsumers + 1) * 32;
constexpr int kAttRopeStages = 6;               // the position-consistent raw-key modes: data stages,
constexpr int kAttRopeGroups = 2;               // consumer groups
constexpr int kAttRopeConsumers = 8;            // and consumer warps (12 warps in 3 groups spill at the 128-register cap: 345 us against 257)
constexpr int kTile = 64;                       // tokens per tile: 64 / B selected blocks, or a 64-token slice of one
constexpr int kD = 128;
// Rotary angles of the raw-key modes.  A consumer warp owns 16 consecutive compact positions p1 .. p1 + 15 of a tile
// (p1 = the tile's first position + 16 x the warp's index in its group).  The angle of pair i at p1 + b is the sum of its
// angles at p1 and at b, so (cos, sin)(p1 + b) = (cos, sin)(p1) composed with (cos, sin)(b): the rows of offsets
// b = 0 .. 15 are loaded once per CTA (8 KiB) and a tile brings only the four rows of its warps' p1 (2 KiB) instead of
// the rows of all its 64 positions (32 KiB per tile and KV head, which made shared memory per tile in flight the bound
// of these modes).  The composed values differ from the table's own row of p1 + b by fp32 rounding (a few units in the
// last place of cos and sin), hence the rotated key by at most one bf16 rounding step on rare elements.
constexpr int kRotRowBytes = (kD / 2) * 8;      // one table row: (cos, sin) fp32 of 64 pairs
constexpr int kRopeShare = 16;                  // compact positions per consumer warp and tile
constexpr int kOffsPitch = kRotRowBytes + 64;   // offset rows 576 B apart: the 128-bit reads of a quarter-warp (two rows) hit 32 different banks
constexpr int kOffsBytes = kRopeShare * kOffsPitch;
constexpr int kBaseBytes = (kTile / kRopeShare) * kRotRowBytes;        // per stage: the rows of p0, p0 + 16, p0 + 32, p0 + 48
static_assert(kAttRopeStages % kAttRopeGroups == 0 && kAttRopeConsumers % kAttRopeGroups == 0, "each group must own whole stages");
constexpr int kHalfBytes = kTile * 128;         // one 64-dim half of a tile: 64 rows x 128 B
constexpr int kStageBytes = 4 * kHalfBytes;     // K lo, K hi, V lo, V hi
constexpr int kMaxSplits = 64;
constexpr int kRowsPad = 16;                    // query rows of one m16 row tile
constexpr int kMaxRows = 64;                    // query rows per KV head and call: up to four row tiles
constexpr int kMergeStride = 136;               // floats per merged row in shared memory
constexpr size_t kAttSmem = (size_t)kAttStages * kStageBytes + 1024;
constexpr size_t kAttSmemRope = (size_t)kAttRopeStages * (kStageBytes + kBaseBytes) + kOffsBytes + 1024;
constexpr int kQrotBytes = kRowsPad * kD * 2;   // one rotated query tile: 16 rows x 256 B
constexpr size_t kAttSmemQrot = kAttSmem + (size_t)kAttStages * kQrotBytes;
constexpr int kQrotWarps = 2;                   // query-rotator warps; they take tiles alternately
constexpr int kKrotWarps = 2;                   // key-tile rotator warps of the position-consistent fused pass; alternate tiles

struct AttendArgs {
    const __nv_bfloat16* q;
    const int32_t* n_sel;
    float* part_o;      // [ns*LG][n_splits][16][128]
    float2* part_ml;    // [ns*LG][n_splits][16]
    int32_t* status;
    int M, L, H, G, r, rows, n_splits, cap_tokens;
    int rows_pad;                // 16 x row tiles: rows of a split's partial result
    float scale_log2e;
    // fused view assembly (attend_split_kernel<true>): tiles come from the page pool through the block table
    const int32_t* sel_ids;      // [n_sessions][sel_stride]
    const int32_t* tables;       // [max_sessions][max_bps]
    const int32_t* nblocks_dev;  // [max_sessions]
    int session_first, sel_stride, max_bps, max_blocks;
    // position-consistent copy-free view (attend_split_kernel<3>): raw keys are rotated in shared memory
    int lookahead;               // tiles the producer may run ahead of the consumers (0: as many as there are stages)
    int landed;                  // 1: the lookahead counts tiles that have not landed yet instead of tiles not yet consumed
    int block_tokens;            // tokens per selected block (view length = n_sel * block_tokens); 64 in the paged modes
    const float2* rope;          // [rope_positions][64] (cos, sin)
    int first_position;          // compact position of view token 0
    int rope_positions;          // rows of the rotary table
};

// query rows per KV head, in m16 MMA row tiles: 1, 2 or 4 (16, 32 or 64 rows)
static int row_tiles_for(int rows) { return rows <= 16 ? 1 : rows <= 32 ? 2 : 4; }

AttendPlan plan_attend(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, int sm_count) {
    (void)sm_count;
    AttendPlan p{};
    p.n_splits = kMaxSplits;
    const int rows = std::max(1, n_q_tokens) * (c.n_q_heads / c.n_kv_heads);
    p.rows_pad = kRowsPad * row_tiles_for(std::min(rows, kMaxRows));
    const size_t heads = (size_t)n_sessions * c.n_layers * c.n_kv_heads;
    p.part_o_bytes = align_up(heads * kMaxSplits * p.rows_pad * kD * sizeof(float), 256);
    p.part_ml_bytes = align_up(heads * kMaxSplits * p.rows_pad * sizeof(float2), 256);
    p.total = p.part_o_bytes + p.part_ml_bytes;
    return p;
}

Option g_attend_landed{-1};     // -1: chosen in launch_attend; 0 / 1: the lookahead counts tiles not yet consumed / not yet landed
Option g_attend_lookahead{0};   // 0: chosen in launch_attend; > 0: forced number of tiles in flight per CTA
Option g_attend_splits{0};   // 0: chosen by the cost model below; > 0: forced (kernel-variant switch)

// splits per head: fewest waves of CTAs over the SMs, counting a fixed per-CTA cost in tiles
static int choose_splits(int heads, int max_tiles, int sms) {
    const int overhead = 6;
    long long best_cost = -1;
    int best = 1;
    for (int s = 1; s <= kMaxSplits && s <= std::max(1, max_tiles); ++s) {
        const long long waves = ((long long)heads * s + sms - 1) / sms;
        const long long cost = waves * ((max_tiles + s - 1) / s + overhead);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

// MODE 0: tiles are read from the materialised view.
// MODE 1: tiles are read from the page pool through the block table (what the gather reads), one
//         extra warp stores every tile into the view with TMA while the consumers attend over it,
//         so the view is assembled and attended in one pass: 1 read + 1 write per view byte
//         instead of 2 reads + 1 write.
// MODE 3: MODE 2 with position-consistent keys (Sec. 4.4: RoPE is applied to raw K at the block's compact
//         position): each consumer warp rotates its key fragments in registers between ldmatrix and the MMAs (one
//         rounding to bf16), with angles composed from two table rows (the warp's first position, which comes with
//         the tile, and the offset inside its 16 positions, loaded once per CTA: see kRopeShare above).  The result
//         is attention over kvmem_materialize_rope's view up to that composition (a key within one bf16 step on rare
//         elements) and no byte is written.
// MODE 4: position-consistent keys over pages that hold k' = RoPE(k, t), t the offset inside the block: the logit
//         q . R(p0 + t) k equals (R(-p0) q) . k', so two extra warps, taking tiles alternately, rotate the 16 query rows back by the tile's
//         compact position p0 (one rotary row per tile instead of 64) into a small shared-memory ring, the
//         consumers fetch their A fragments from it with ldmatrix, and the keys go to the MMAs as stored.
// MODE 5: MODE 1 for pages that hold k' = RoPE(k, t) (offset inside the block), leaving a position-consistent view: two
//         extra warps, taking tiles alternately, rotate every K tile in place in shared memory by its compact
//         position p0 (one set of angles per tile, arithmetic of kvmem_rope_rotate) as soon as it has landed; the
//         consumers and the view writer wait for the rotated tile.  The view equals kvmem_materialize_rope's and
//         out/lse equal kvmem_view_attend's on it, with 1 read + 1 write per view byte.
// MODE 6: MODE 1 with the keys of MODE 3 (raw keys, position-consistent view in one pass): the consumer warps rotate
//         their key fragments as in MODE 3, write each register back to the four bytes of the swizzled tile it came from,
//         and the view writer stores the tile once the four warps that share it have done so.  Values are copied bit for
//         bit; keys are kvmem_materialize_rope's up to the composition of the angles.
// MODE 2: copy-free execution view (Sec. 5.3 "Copy-free execution-view assembly"): tiles are read from
//         the pages through the block table and attended over; no contiguous view is written.
// RT: m16 row tiles of query rows per KV head.  RT = 1 (up to 16 rows): two groups of four consumer warps take the tiles
// alternately.  RT = 2 (up to 32 rows): every consumer warp sees every tile, four warps per row tile, 16 tokens each.
// RT = 4 (up to 64 rows): two warps per row tile, 32 tokens each.  The K/V stream is read once whatever RT is; with
// more row tiles the consumers do more arithmetic per byte and the pass moves from HBM-bound towards issue-bound.
// SUB (MODE 4 only): selected blocks per 64-token tile (64 / B for B < 64); every block of a tile has its own compact
// position, hence its own rotated copy of the query (four data stages then, to make room for the copies).
template <int MODE, int RT = 1, int SUB = 1>
__global__ void __launch_bounds__(MODE == 3 ? (kAttRopeConsumers + 1) * 32 : MODE == 6 ? (kAttRopeConsumers + 2) * 32 : kAttThreads + (MODE == 1 ? 32 : MODE == 4 ? 32 * kQrotWarps : MODE == 5 ? 32 + 32 * kKrotWarps : 0), 1)
attend_split_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_pages, AttendArgs a) {
    constexpr bool FUSED = MODE == 1 || MODE == 5 || MODE == 6;   // a view-writer warp shares every stage with the consumers
    constexpr bool KROT = MODE == 5;       // rotator warps re-encode every K tile in place before anybody else reads it
    constexpr bool PAGED = MODE != 0;      // the producer reads pages through the block table
    constexpr bool ROPE = MODE == 3 || MODE == 6;   // the consumers re-encode their key fragments in registers before the MMAs
    constexpr bool KWB = MODE == 6;        // ... and write them back into the stage, from where the view writer stores the tile
    constexpr bool QROT = MODE == 4;       // a rotator warp re-encodes the query per tile instead
    extern __shared__ unsigned char smem_dyn[];
    static_assert(SUB == 1 || (MODE == 4 && (SUB == 2 || SUB == 4)), "several blocks per tile with their own rotation: the query-rotating mode only");
    constexpr int STAGES = ROPE ? kAttRopeStages : (QROT && SUB > 1) ? 4 : kAttStages;
    constexpr int CONSUMERS = ROPE ? kAttRopeConsumers : kAttConsumers;
    constexpr int GROUPS = ROPE ? kAttRopeGroups : RT > 1 ? 1 : kAttGroups;
    static_assert(RT == 1 || (MODE <= 2 && (RT == 2 || RT == 4)), "several row tiles: the plain modes only");
    constexpr int WPR = RT == 1 ? 4 : CONSUMERS / RT;      // consumer warps that share the tokens of a tile (for one row tile)
    constexpr int SLICES = 4 / WPR;                        // 16-token slices per warp and tile
    __shared__ uint64_t full_bar[kAttStages], empty_bar[kAttStages], tab_full;      // tab_full: the raw-key modes' offset rows are in place
    __shared__ uint64_t q_full[kAttStages];     // MODE 4: rotated query of the stage's tile is in place; MODE 5: its K tile is rotated
    __shared__ float merge_m[kAttRopeConsumers][kRowsPad], merge_l[kAttRopeConsumers][kRowsPad];

    unsigned char* stages = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, lg = blockIdx.y, s = blockIdx.z;
    const int LG = a.L * a.G;
    const int z = s * LG + lg;
    const int l = lg / a.G, g = lg % a.G;

    // what needs no global memory comes first, so that it overlaps the tail of the kernel before this one
    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) {
            ptx::mbar_init(&full_bar[i], 1);
            ptx::mbar_init(&empty_bar[i], CONSUMERS / GROUPS + (FUSED ? 1 : 0));
        }
        ptx::mbar_init(&tab_full, 1);
        for (int i = 0; i < kAttStages; ++i) ptx::mbar_init(&q_full[i], KWB ? CONSUMERS / GROUPS : 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(PAGED ? &map_pages : &map_k);
    }
    __syncthreads();
    pdl_wait();        // everything earlier in the stream is complete and visible from here on

    // view length in tokens; the kernel works in 64-token tiles, whatever the block size of the view (a multiple of
    // 16, so each consumer warp's 16 tokens are all inside or all outside the view)
    const int btok = a.block_tokens;
    // The producer's first page lookup is a chain of dependent reads (count of selected blocks, ids, block table) ahead of
    // the first tile.  When the selection fills its row (the budget binds, the usual case) the ids this CTA starts at are
    // known without the count, so they are requested together with it and used if the count confirms them.
    int spec_j = -1, spec_id = -1;
    if (PAGED && warp == CONSUMERS) {
        const int n_sub = btok < kTile ? kTile / btok : 1, tpb = btok > kTile ? btok / kTile : 1;
        const long long tok_h = min((long long)a.sel_stride * btok, (long long)a.cap_tokens);
        const int blk_h = (int)((tok_h + kTile - 1) / kTile);
        const int t0_h = (int)((long long)blk_h * split / a.n_splits);
        spec_j = (t0_h * n_sub + lane) / tpb;
        if (spec_j < a.sel_stride) spec_id = a.sel_ids[(size_t)s * a.sel_stride + spec_j];
        else spec_j = -1;
    }
    const long long n_tok_ll = min((long long)max(a.n_sel[s], 0) * btok, (long long)a.cap_tokens);
    const int n_tok = (int)n_tok_ll;
    const int n_blk = (n_tok + kTile - 1) / kTile;
    const int t0 = (int)((long long)n_blk * split / a.n_splits);
    const int t1 = (int)((long long)n_blk * (split + 1) / a.n_splits);
    const int n_tiles = t1 - t0;
    const int ahead = a.lookahead > 0 ? min(a.lookahead, STAGES) : STAGES;

    float o[16][4];           // O accumulators: 16 n-tiles of 8 dims
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f; }

    if (warp == CONSUMERS) {
        // ---------------- producer ----------------
        if (!PAGED) {
            if (lane == 0 && n_tiles > 0) {
                ptx::prefetch_tensormap(&map_k);
                ptx::prefetch_tensormap(&map_v);
                for (int it = 0; it < n_tiles; ++it) {
                    const int st = it % STAGES;
                    bool ok = true;
                    if (ahead < STAGES && it >= ahead) {          // at most `ahead` tiles in flight (see the paged producer)
                        const int jt = it - ahead;
                        ok = a.landed ? ptx::mbar_wait(&full_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1))
                                      : ptx::mbar_wait(&empty_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1));
                    }
                    if (ok && it >= STAGES) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / STAGES) & 1) ^ 1));
                    if (!ok) {
                        atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                        break;
                    }
                    unsigned char* dst = stages + (size_t)st * kStageBytes;
                    const int y = (t0 + it) * kTile;
                    ptx::mbar_expect_tx(&full_bar[st], kStageBytes);
                    ptx::tma_load_3d(dst, &map_k, 0, y, z, &full_bar[st]);
                    ptx::tma_load_3d(dst + kHalfBytes, &map_k, 64, y, z, &full_bar[st]);
                    ptx::tma_load_3d(dst + 2 * kHalfBytes, &map_v, 0, y, z, &full_bar[st]);
                    ptx::tma_load_3d(dst + 3 * kHalfBytes, &map_v, 64, y, z, &full_bar[st]);
                }
            }
        } else if (n_tiles > 0) {
            // A 64-token tile is 64 / B selected blocks (B < 64: one page lookup and one set of loads per block) or a
            // 64-token slice of one selected block (B >= 64).  The whole warp looks up pages, 32 slots at a time (a slot
            // is one block of a tile); lane 0 issues the loads.
            if (lane == 0) ptx::prefetch_tensormap(&map_pages);
            unsigned char* const rot_offs = stages + (size_t)STAGES * kStageBytes;       // [16 offsets][64 pairs], rows kOffsPitch apart
            unsigned char* const rot_base = rot_offs + kOffsBytes;                       // [STAGES][4 rows of 64 pairs]
            if (ROPE && lane == 0) {
                // rows of positions 0 .. 15, once per CTA and ahead of the page lookups
                ptx::mbar_expect_tx(&tab_full, (uint32_t)kRopeShare * kRotRowBytes);
                for (int b = 0; b < kRopeShare; ++b)
                    ptx::bulk_g2s(rot_offs + (size_t)b * kOffsPitch, a.rope + (size_t)b * (kD / 2), kRotRowBytes, &tab_full);
            }
            const int NB = a.nblocks_dev[a.session_first + s];
            const int B = btok;
            const int n_sub = B < kTile ? kTile / B : 1;      // selected blocks per tile
            const int tpb = B > kTile ? B / kTile : 1;        // tiles per selected block
            const int box_rows = B < kTile ? B : kTile;
            const int n_sel_blk = n_tok / B;                  // selected blocks inside the view
            int base_slot = 0, my_page = 0;
            auto lookup = [&](int slot) -> int {
                const int j = (t0 * n_sub + slot) / tpb;      // index in sel_ids
                if (slot >= n_tiles * n_sub || j >= n_sel_blk) return -1;          // past this CTA's range or the view's ragged end
                const int id = (slot == lane && j == spec_j) ? spec_id : a.sel_ids[(size_t)s * a.sel_stride + j];
                int pg = -1;
                if (id >= 0 && id < NB) pg = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
                if (pg < 0 || pg >= a.max_blocks) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); pg = 0; }
                return pg;           // a flagged id reads page 0 instead of faulting; the status word reports it
            };
            my_page = lookup(lane);
            bool ok = true;
            if (B == kTile) {
                // One block per tile, the common case, kept as lean as the tile needs (one shuffle, four loads): the
                // producer's own instructions sit on the critical path of a read-only stream.
                for (int it = 0; it < n_tiles; ++it) {
                    if (it >= base_slot + 32) { base_slot = it; my_page = lookup(base_slot + lane); }
                    const int page = __shfl_sync(0xffffffffu, my_page, it - base_slot);
                    if (lane == 0) {
                        const int st = it % STAGES;
                        if (ok && ahead < STAGES && it >= ahead) {
                            const int jt = it - ahead;
                            ok = (KROT || a.landed) ? ptx::mbar_wait(&full_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1))
                                                    : ptx::mbar_wait(&empty_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1));
                        }
                        if (ok && it >= STAGES) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / STAGES) & 1) ^ 1));
                        if (ok) {
                            unsigned char* dst = stages + (size_t)st * kStageBytes;
                            // page layout [K|V][L*G][64 tokens][128]: rows of 256 B
                            const int yk = ((page * 2 + 0) * LG + lg) * kTile, yv = ((page * 2 + 1) * LG + lg) * kTile;
                            ptx::mbar_expect_tx(&full_bar[st], kStageBytes + (ROPE ? kBaseBytes : 0));
                            if (ROPE) {
                                // the rotary rows of the four warps' first positions travel with the tile
                                const float2* rows = a.rope + (size_t)(a.first_position + (t0 + it) * kTile) * (kD / 2);
#pragma unroll
                                for (int w = 0; w < kTile / kRopeShare; ++w)
                                    ptx::bulk_g2s(rot_base + (size_t)st * kBaseBytes + (size_t)w * kRotRowBytes,
                                                  rows + (size_t)w * kRopeShare * (kD / 2), kRotRowBytes, &full_bar[st]);
                            }
                            ptx::tma_load_2d(dst, &map_pages, 0, yk, &full_bar[st]);
                            ptx::tma_load_2d(dst + kHalfBytes, &map_pages, 64, yk, &full_bar[st]);
                            ptx::tma_load_2d(dst + 2 * kHalfBytes, &map_pages, 0, yv, &full_bar[st]);
                            ptx::tma_load_2d(dst + 3 * kHalfBytes, &map_pages, 64, yv, &full_bar[st]);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
                }
            } else
            for (int it = 0; it < n_tiles; ++it) {
                if (it * n_sub >= base_slot + 32) { base_slot = it * n_sub; my_page = lookup(base_slot + lane); }
                int pages[4] = {-1, -1, -1, -1};
                if (n_sub == 1) {
                    pages[0] = __shfl_sync(0xffffffffu, my_page, (it - base_slot) & 31);
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) pages[u] = u < n_sub ? __shfl_sync(0xffffffffu, my_page, (it * n_sub + u - base_slot) & 31) : -1;
                }
                if (lane == 0) {
                    const int st = it % STAGES;
                    // at most `ahead` tiles in flight: tile it - ahead has left its stage (the same phase is waited for
                    // again, and found complete, when that stage is refilled)
                    if (ok && ahead < STAGES && it >= ahead) {
                        const int jt = it - ahead;
                        // KROT: a landed tile waits for its rotation in shared memory, which is no longer an HBM
                        // request in flight; the limit applies to tiles that have not landed yet
                        ok = (KROT || a.landed) ? ptx::mbar_wait(&full_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1))
                                                : ptx::mbar_wait(&empty_bar[jt % STAGES], (uint32_t)((jt / STAGES) & 1));
                    }
                    if (ok && it >= STAGES) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / STAGES) & 1) ^ 1));
                    if (ok) {
                        unsigned char* dst = stages + (size_t)st * kStageBytes;
                        int n_valid = 0;
#pragma unroll
                        for (int u = 0; u < 4; ++u) n_valid += (u < n_sub && pages[u] >= 0) ? 1 : 0;
                        // page layout [K|V][L*G][B tokens][128]: rows of 256 B
                        ptx::mbar_expect_tx(&full_bar[st], (uint32_t)n_valid * 4u * (uint32_t)box_rows * 128u + (ROPE ? (uint32_t)kBaseBytes : 0u));
                        if (ROPE) {
                            const float2* rows = a.rope + (size_t)(a.first_position + (t0 + it) * kTile) * (kD / 2);
#pragma unroll
                            for (int w = 0; w < kTile / kRopeShare; ++w)
                                ptx::bulk_g2s(rot_base + (size_t)st * kBaseBytes + (size_t)w * kRotRowBytes,
                                              rows + (size_t)w * kRopeShare * (kD / 2), kRotRowBytes, &full_bar[st]);
                        }
                        const int row_in_block = ((t0 + it) % tpb) * kTile;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (u < n_sub && pages[u] >= 0) {
                                const int yk = ((pages[u] * 2 + 0) * LG + lg) * B + row_in_block, yv = ((pages[u] * 2 + 1) * LG + lg) * B + row_in_block;
                                unsigned char* d = dst + (size_t)u * B * 128;
                                ptx::tma_load_2d(d, &map_pages, 0, yk, &full_bar[st]);
                                ptx::tma_load_2d(d + kHalfBytes, &map_pages, 64, yk, &full_bar[st]);
                                ptx::tma_load_2d(d + 2 * kHalfBytes, &map_pages, 0, yv, &full_bar[st]);
                                ptx::tma_load_2d(d + 3 * kHalfBytes, &map_pages, 64, yv, &full_bar[st]);
                            }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
            }
        }
    } else if (FUSED && warp == CONSUMERS + 1) {
        // ---------------- view writer: every tile that lands in shared memory is stored to the view ----------------
        if (lane == 0 && n_tiles > 0) {
            ptx::prefetch_tensormap(&map_k);
            ptx::prefetch_tensormap(&map_v);
            bool ok = true;
            for (int it = 0; it < n_tiles; ++it) {
                const int st = it % STAGES;
                ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((it / STAGES) & 1));
                if ((KROT || KWB) && ok) ok = ptx::mbar_wait(&q_full[st], (uint32_t)((it / STAGES) & 1));
                if (!ok) break;
                unsigned char* src = stages + (size_t)st * kStageBytes;
                const int y = (t0 + it) * kTile;
                // the store box is min(B, 64) rows: a ragged last tile stores only the blocks the view has
                const int box_rows = btok < kTile ? btok : kTile;
                const int n_valid = min(kTile, n_tok - y) / box_rows;
                for (int u = 0; u < n_valid; ++u) {
                    const unsigned char* sb = src + (size_t)u * box_rows * 128;
                    ptx::tma_store_3d(&map_k, sb, 0, y + u * box_rows, z);
                    ptx::tma_store_3d(&map_k, sb + kHalfBytes, 64, y + u * box_rows, z);
                    ptx::tma_store_3d(&map_v, sb + 2 * kHalfBytes, 0, y + u * box_rows, z);
                    ptx::tma_store_3d(&map_v, sb + 3 * kHalfBytes, 64, y + u * box_rows, z);
                }
                ptx::bulk_commit();
                if (KWB) {
                    // four stages and a tile that is held until its consumers have rotated it: the stage goes back as soon
                    // as this store has read it, not one tile later
                    ptx::bulk_wait_read<0>();
                    ptx::mbar_arrive(&empty_bar[st]);
                } else if (it > 0) {                       // all but the newest store have left shared memory
                    ptx::bulk_wait_read<1>();
                    ptx::mbar_arrive(&empty_bar[(it - 1) % STAGES]);
                }
            }
            ptx::bulk_wait_read<0>();
            if (ok && !KWB) ptx::mbar_arrive(&empty_bar[(n_tiles - 1) % STAGES]);
            else if (!ok) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
            ptx::bulk_wait<0>();                           // the view is complete before the kernel ends
        }
    } else if (KROT && warp > CONSUMERS + 1) {
        // ---------------- key rotators: K tile <- RoPE(K tile, p0(tile)), in place ----------------
        // Lane -> 16-byte chunk c = lane & 7 of the low half (dims 8c..8c+7, paired with the same chunk of the high
        // half) of tokens (lane >> 3) + 4 i: the lane's 8 (cos, sin) pairs serve its sixteen tokens.  A quarter-warp
        // covers one 128-byte row of the swizzled tile: conflict-free 128-bit accesses.
        if (n_tiles > 0) {
            const int c = lane & 7;
            auto fetch_row = [&](int it, float4 (&t4)[4]) {
                int p0 = a.first_position + (t0 + min(it, n_tiles - 1)) * kTile;
                if (p0 < 0 || p0 >= a.rope_positions) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); p0 = 0; }
                const float4* cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)p0 * (kD / 2) + c * 8);
#pragma unroll
                for (int w = 0; w < 4; ++w) t4[w] = __ldg(cs4 + w);
            };
            const int it_first = warp - CONSUMERS - 2;
            float4 t4[4], t4_next[4];
            fetch_row(it_first, t4_next);
            for (int it = it_first; it < n_tiles; it += kKrotWarps) {
                const int st = it % STAGES;
#pragma unroll
                for (int w = 0; w < 4; ++w) t4[w] = t4_next[w];
                fetch_row(it + kKrotWarps, t4_next);
                const bool ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((it / STAGES) & 1));
                if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
                unsigned char* klo = stages + (size_t)st * kStageBytes;
#pragma unroll 4
                for (int i = 0; i < kTile / 4; ++i) {
                    const int tok = (lane >> 3) + 4 * i;
                    unsigned char* plo = klo + tok * 128 + ((c ^ (tok & 7)) << 4);
                    const uint4 lo = *reinterpret_cast<const uint4*>(plo), hi = *reinterpret_cast<const uint4*>(plo + kHalfBytes);
                    uint4 lo_o, hi_o;
                    rotate8_cs(lo, hi, t4, 1.0f, lo_o, hi_o);
                    *reinterpret_cast<uint4*>(plo) = lo_o;
                    *reinterpret_cast<uint4*>(plo + kHalfBytes) = hi_o;
                }
                ptx::fence_proxy_async_smem();      // the view writer's bulk stores read these bytes through the async proxy
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&q_full[st]);
            }
        }
    } else if (QROT && warp > CONSUMERS) {
        // ---------------- query rotator: Q'(tile) = RoPE^-1(q, p0(tile)) for the 16 query rows ----------------
        // Lane -> 16-byte chunk c = lane & 7 of the low half (dims 8c..8c+7, paired with 64+8c..) of rows
        // (lane >> 3) + 4 i: the lane's 8 (cos, sin) pairs serve its four rows.  Q' is stored [16 rows][256 B] with
        // the 16-byte chunk index XOR-ed with the row's low 3 bits, which keeps the consumers' ldmatrix conflict-free.
        if (n_tiles > 0) {
            const int c = lane & 7;
            uint4 raw_lo[4], raw_hi[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = (lane >> 3) + 4 * i;
                raw_lo[i] = raw_hi[i] = make_uint4(0u, 0u, 0u, 0u);
                if (row < a.rows) {
                    const __nv_bfloat16* qr = a.q + ((((size_t)s * a.M + row / a.r) * a.L + l) * a.H + (size_t)g * a.r + row % a.r) * kD;
                    raw_lo[i] = *reinterpret_cast<const uint4*>(qr + c * 8);
                    raw_hi[i] = *reinterpret_cast<const uint4*>(qr + kD / 2 + c * 8);
                }
            }
            unsigned char* qring = stages + (size_t)STAGES * kStageBytes;
            const int tpb = btok > kTile ? btok / kTile : 1;       // tiles per block (blocks larger than a tile)
            // position of the block that holds sub-block u of tile it: the query is rotated back by it
            auto block_pos = [&](int it, int u) -> int { return a.first_position + (((t0 + it) * SUB + u) / tpb) * btok; };
            auto fetch_row = [&](int p0, float4 (&t4)[4]) {
                if (p0 < 0 || p0 >= a.rope_positions) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); p0 = 0; }
                const float4* cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)p0 * (kD / 2) + c * 8);
#pragma unroll
                for (int w = 0; w < 4; ++w) t4[w] = __ldg(cs4 + w);
            };
            const int it_first = warp - CONSUMERS - 1;
            // SUB == 1: the rotary row of a tile is fetched one of this warp's tiles ahead (an L2 round trip per tile would
            // otherwise sit on the critical path of every tile); SUB > 1: the rows of a tile's blocks are fetched when
            // the tile comes up, before the wait for its stage
            float4 t4[SUB][4], t4_next[4];
            if (SUB == 1) fetch_row(block_pos(min(it_first, n_tiles - 1), 0), t4_next);
            for (int it = it_first; it < n_tiles; it += kQrotWarps) {
                const int st = it % STAGES;
                int n_valid = 1;
                if (SUB == 1) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) t4[0][w] = t4_next[w];
                    fetch_row(block_pos(min(it + kQrotWarps, n_tiles - 1), 0), t4_next);
                } else {
                    n_valid = min(kTile, n_tok - (t0 + it) * kTile) / btok;       // blocks the (possibly ragged) tile holds
#pragma unroll
                    for (int u = 0; u < SUB; ++u)
                        if (u < n_valid) fetch_row(block_pos(it, u), t4[u]);
                }
                bool ok = true;
                if (it >= STAGES) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / STAGES) & 1) ^ 1));
                if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
#pragma unroll
                for (int u = 0; u < SUB; ++u) {
                    if (u >= n_valid) continue;
                    unsigned char* qb = qring + ((size_t)st * SUB + u) * kQrotBytes;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = (lane >> 3) + 4 * i;
                        uint4 lo_o, hi_o;
                        rotate8_cs(raw_lo[i], raw_hi[i], t4[u], -1.0f, lo_o, hi_o);
                        *reinterpret_cast<uint4*>(qb + row * 256 + ((c ^ (row & 7)) << 4)) = lo_o;
                        *reinterpret_cast<uint4*>(qb + row * 256 + (((c + 8) ^ (row & 7)) << 4)) = hi_o;
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&q_full[st]);
            }
        }
    } else {
        // ---------------- consumers ----------------
        // Q fragments (A operand, m16k16 x 8 k-steps).  Row j = m * r + hr  ->  q[s][m][l][g*r + hr].
        uint32_t qf[8][4];
        if (!QROT) {
            const int row_a = (RT == 1 ? 0 : (warp / WPR) * kRowsPad) + (lane >> 2), row_b = row_a + 8;
            const __nv_bfloat16* qa = nullptr;
            const __nv_bfloat16* qb = nullptr;
            if (row_a < a.rows) qa = a.q + ((((size_t)s * a.M + row_a / a.r) * a.L + l) * a.H + (size_t)g * a.r + row_a % a.r) * kD;
            if (row_b < a.rows) qb = a.q + ((((size_t)s * a.M + row_b / a.r) * a.L + l) * a.H + (size_t)g * a.r + row_b % a.r) * kD;
            const int kq = 2 * (lane & 3);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qf[ks][0] = qa ? *reinterpret_cast<const uint32_t*>(qa + ks * 16 + kq) : 0u;
                qf[ks][1] = qb ? *reinterpret_cast<const uint32_t*>(qb + ks * 16 + kq) : 0u;
                qf[ks][2] = qa ? *reinterpret_cast<const uint32_t*>(qa + ks * 16 + kq + 8) : 0u;
                qf[ks][3] = qb ? *reinterpret_cast<const uint32_t*>(qb + ks * 16 + kq + 8) : 0u;
            }
        }
        const uint32_t stage0 = ptx::smem_u32(stages);
        const int mj = lane >> 3, mr = lane & 7;        // ldmatrix: matrix index and row within it
        // Two groups of four warps.  Group grp takes tiles grp, grp + 2, ...; with an even number of
        // stages it therefore meets the phases of "its" stages strictly in order, which an mbarrier
        // parity wait requires.  Inside a tile, warp wq owns tokens [16 wq, 16 wq + 16).
        const int grp = RT == 1 ? warp >> 2 : 0, wq0 = RT == 1 ? (warp & 3) : (warp % WPR) * SLICES;

        for (int it = grp; it < n_tiles; it += GROUPS) {
            const int st = it % STAGES;
            bool arrived = ptx::mbar_wait(&full_bar[st], (uint32_t)((it / STAGES) & 1));
            if (ROPE && it == grp) arrived = arrived && ptx::mbar_wait(&tab_full, 0u);       // the offset rows, once
            if (QROT || KROT) arrived = arrived && ptx::mbar_wait(&q_full[st], (uint32_t)((it / STAGES) & 1));
            if (!__all_sync(0xffffffffu, arrived)) {          // warp-uniform decision
                if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                break;
            }
            bool k_handed_over = false;                      // KWB: this warp's share of the tile is rotated and back in the stage
#pragma unroll
            for (int sl = 0; sl < SLICES; ++sl) {
            const int wq = wq0 + sl;
            if ((t0 + it) * kTile + wq * 16 >= n_tok) continue;      // this warp's 16 tokens lie beyond a ragged view end
            const uint32_t kbase = stage0 + (uint32_t)st * kStageBytes;
            const uint32_t vbase = kbase + 2 * kHalfBytes;
            // QROT: this tile's rotated query; its A fragments are fetched two k-steps at a time, next to their use
            const int qrow = mr + 8 * (mj & 1);
            const uint32_t qaddr = stage0 + (uint32_t)STAGES * kStageBytes + (uint32_t)(st * SUB + (SUB > 1 ? (wq * 16) / btok : 0)) * kQrotBytes + (uint32_t)qrow * 256u;

            // S = Q K^T for this warp's 16 tokens: 2 n-tiles (8 tokens each) x 8 k-steps
            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f; }
            if (!ROPE) {
#pragma unroll
                for (int kp = 0; kp < 4; ++kp) {            // 32 dims = 4 chunks of 16 B = 2 k-steps
                    const int cg = kp * 4 + mj;             // 16-byte chunk along d (0..15)
                    const uint32_t half_off = (uint32_t)(cg >> 3) * kHalfBytes;
                    const int c = cg & 7;
                    if (QROT) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int ks = 2 * kp + h;
                            ptx::ldmatrix_x4(qaddr + (uint32_t)(((ks * 2 + (mj >> 1)) ^ (qrow & 7)) << 4), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
                        }
                    }
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        const int tok = wq * 16 + nt * 8 + mr;
                        const uint32_t addr = kbase + half_off + (uint32_t)tok * 128u + (uint32_t)((c ^ (tok & 7)) << 4);
                        uint32_t b0, b1, b2, b3;
                        ptx::ldmatrix_x4(addr, b0, b1, b2, b3);
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp], b0, b1);
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp + 1], b2, b3);
                    }
                }
            } else {
                // Dimension i pairs with i + 64: the fragment of chunk cg (low half) and the one of chunk cg + 8
                // (high half) sit in the same lane, so a lane rotates what it holds: registers lo[j], hi[j] carry
                // dims 8 (4 kp + j) + 2 (lane & 3) + {0, 1} (+ 64) of token wq*16 + nt*8 + lane/4.
                // (cos, sin) of this lane's pairs at the warp's first position p1 (the row that came with the tile) and at
                // the offsets b of its tokens inside the warp's share (the rows loaded once)
                const unsigned char* rot_offs = stages + (size_t)STAGES * kStageBytes;
                const unsigned char* base_row = rot_offs + kOffsBytes + (size_t)st * kBaseBytes + (size_t)wq * kRotRowBytes;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int tok = wq * 16 + nt * 8 + mr;
                    const int rtok = wq * 16 + nt * 8 + (lane >> 2);              // the token whose elements this lane holds
                    uint32_t lo[2][4], hi[2][4];
#pragma unroll
                    for (int kp = 0; kp < 2; ++kp) {
                        const int c = kp * 4 + mj;
                        const uint32_t addr = kbase + (uint32_t)tok * 128u + (uint32_t)((c ^ (tok & 7)) << 4);
                        ptx::ldmatrix_x4(addr, lo[kp][0], lo[kp][1], lo[kp][2], lo[kp][3]);
                        ptx::ldmatrix_x4(addr + kHalfBytes, hi[kp][0], hi[kp][1], hi[kp][2], hi[kp][3]);
                        const float4* orow = reinterpret_cast<const float4*>(rot_offs + (size_t)(nt * 8 + (lane >> 2)) * kOffsPitch) + (kp * 16 + (lane & 3));
                        const float4* brow = reinterpret_cast<const float4*>(base_row) + (kp * 16 + (lane & 3));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float4 o4 = orow[j * 4], b4 = brow[j * 4];      // pairs 8 (4 kp + j) + 2 (lane & 3) + {0, 1}
                            float4 t;                                             // (cos, sin)(p1 + b) = (cos, sin)(p1) o (cos, sin)(b)
                            t.x = fmaf(b4.x, o4.x, -(b4.y * o4.y)); t.y = fmaf(b4.y, o4.x, b4.x * o4.y);
                            t.z = fmaf(b4.z, o4.z, -(b4.w * o4.w)); t.w = fmaf(b4.w, o4.z, b4.z * o4.w);
                            const float a0 = __uint_as_float(lo[kp][j] << 16), a1 = __uint_as_float(lo[kp][j] & 0xffff0000u);
                            const float b0 = __uint_as_float(hi[kp][j] << 16), b1 = __uint_as_float(hi[kp][j] & 0xffff0000u);
                            const float l0 = fmaf(a0, t.x, -(b0 * t.y)), h0 = fmaf(b0, t.x, a0 * t.y);
                            const float l1 = fmaf(a1, t.z, -(b1 * t.w)), h1 = fmaf(b1, t.z, a1 * t.w);
                            lo[kp][j] = ptx::pack_bf16x2(l0, l1);
                            hi[kp][j] = ptx::pack_bf16x2(h0, h1);
                            if (KWB) {
                                // register j of an ldmatrix x4 holds matrix j = 16-byte chunk 4 kp + j of token rtok, bytes 4 (lane & 3)..
                                unsigned char* pk = stages + (size_t)st * kStageBytes + (size_t)rtok * 128 + ((((kp * 4 + j) ^ (rtok & 7)) << 4) + 4 * (lane & 3));
                                *reinterpret_cast<uint32_t*>(pk) = lo[kp][j];
                                *reinterpret_cast<uint32_t*>(pk + kHalfBytes) = hi[kp][j];
                            }
                        }
                    }
                    // the k-steps in the order of the other modes, so that the logits are the same bits
#pragma unroll
                    for (int kp = 0; kp < 2; ++kp) {
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp], lo[kp][0], lo[kp][1]);
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp + 1], lo[kp][2], lo[kp][3]);
                    }
#pragma unroll
                    for (int kp = 0; kp < 2; ++kp) {
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp + 4], hi[kp][0], hi[kp][1]);
                        ptx::mma_bf16_16816(sc[nt], qf[2 * kp + 5], hi[kp][2], hi[kp][3]);
                    }
                }
                if (KWB) {
                    ptx::fence_proxy_async_smem();      // the view writer's bulk stores read these bytes through the async proxy
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&q_full[st]);
                    k_handed_over = true;
                }
            }
            // online softmax (exp2 domain); this thread holds rows lane/4 (c0,c1) and lane/4 + 8 (c2,c3)
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                sc[nt][0] *= a.scale_log2e; sc[nt][1] *= a.scale_log2e; sc[nt][2] *= a.scale_log2e; sc[nt][3] *= a.scale_log2e;
                mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
                mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const bool grew = (mn0 != m_run[0]) || (mn1 != m_run[1]);
            if (__any_sync(0xffffffffu, grew)) {         // a running maximum moved: rescale what is accumulated
                const float corr0 = exp2f(m_run[0] - mn0), corr1 = exp2f(m_run[1] - mn1);
                l_run[0] *= corr0; l_run[1] *= corr1;
#pragma unroll
                for (int nd = 0; nd < 16; ++nd) { o[nd][0] *= corr0; o[nd][1] *= corr0; o[nd][2] *= corr1; o[nd][3] *= corr1; }
                m_run[0] = mn0; m_run[1] = mn1;
            }
            uint32_t pa[4];
            {
                const float p00 = exp2f(sc[0][0] - mn0), p01 = exp2f(sc[0][1] - mn0);
                const float p02 = exp2f(sc[0][2] - mn1), p03 = exp2f(sc[0][3] - mn1);
                const float p10 = exp2f(sc[1][0] - mn0), p11 = exp2f(sc[1][1] - mn0);
                const float p12 = exp2f(sc[1][2] - mn1), p13 = exp2f(sc[1][3] - mn1);
                l_run[0] += (p00 + p01) + (p10 + p11);
                l_run[1] += (p02 + p03) + (p12 + p13);
                pa[0] = ptx::pack_bf16x2(p00, p01); pa[1] = ptx::pack_bf16x2(p02, p03);
                pa[2] = ptx::pack_bf16x2(p10, p11); pa[3] = ptx::pack_bf16x2(p12, p13);
            }
            // O += P V : one k-step (this warp's 16 tokens) x 16 n-tiles (8 dims)
            {
                const int tok = wq * 16 + (mj & 1) * 8 + mr;
#pragma unroll
                for (int np = 0; np < 8; ++np) {
                    const int cg = np * 2 + (mj >> 1);
                    const uint32_t addr = vbase + (uint32_t)(cg >> 3) * kHalfBytes + (uint32_t)tok * 128u +
                                          (uint32_t)(((cg & 7) ^ (tok & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ptx::ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                    ptx::mma_bf16_16816(o[2 * np], pa, b0, b1);
                    ptx::mma_bf16_16816(o[2 * np + 1], pa, b2, b3);
                }
            }
            }       // slices
            if (KWB && !k_handed_over) {                    // nothing of this tile was this warp's to rotate (ragged view end)
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&q_full[st]);
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&empty_bar[st]);
        }
        // row sums live spread over the 4 lanes of a quad
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1); l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1); l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    }

    // every issued tile has been consumed (or a wait gave up): the ring can be reused for the merge
    __syncthreads();
    float* merge_o = reinterpret_cast<float*>(stages);          // [consumer][16][kMergeStride]
    if (warp < CONSUMERS) {
        const int row_a = lane >> 2, row_b = row_a + 8, col = 2 * (lane & 3);
        float* base = merge_o + (size_t)warp * kRowsPad * kMergeStride;
#pragma unroll
        for (int nd = 0; nd < 16; ++nd) {
            *reinterpret_cast<float2*>(base + row_a * kMergeStride + nd * 8 + col) = make_float2(o[nd][0], o[nd][1]);
            *reinterpret_cast<float2*>(base + row_b * kMergeStride + nd * 8 + col) = make_float2(o[nd][2], o[nd][3]);
        }
        if ((lane & 3) == 0) {
            merge_m[warp][row_a] = m_run[0]; merge_l[warp][row_a] = l_run[0];
            merge_m[warp][row_b] = m_run[1]; merge_l[warp][row_b] = l_run[1];
        }
    }
    __syncthreads();
    if (tid < 256) {
        const int col = tid & 127, r0 = (tid >> 7) * 8;
        const size_t pbase = ((size_t)z * a.n_splits + split) * a.rows_pad;
        constexpr int NW = RT == 1 ? CONSUMERS : WPR;       // warps whose partial results share a query row
#pragma unroll
        for (int rt = 0; rt < RT; ++rt) {
            const int w0 = RT == 1 ? 0 : rt * WPR;
            for (int row = r0; row < r0 + 8; ++row) {
                float mx = -INFINITY;
#pragma unroll
                for (int w = w0; w < w0 + NW; ++w) mx = fmaxf(mx, merge_m[w][row]);
                float acc = 0.0f, lsum = 0.0f;
#pragma unroll
                for (int w = w0; w < w0 + NW; ++w) {
                    const float mw = merge_m[w][row];
                    if (mw > -INFINITY) {
                        const float f = exp2f(mw - mx);
                        acc += f * merge_o[((size_t)w * kRowsPad + row) * kMergeStride + col];
                        lsum += f * merge_l[w][row];
                    }
                }
                a.part_o[(pbase + rt * kRowsPad + row) * kD + col] = acc;
                if (col == 0) a.part_ml[pbase + rt * kRowsPad + row] = make_float2(mx, lsum);
            }
        }
    }
}

// Merge the splits of one query row of one (session, layer, KV head) in split order; write O and LSE.
// U splits are in flight at a time (8, or 24 when there are more than 8 splits: the usual 18 then take one round trip).
template <int U>
__global__ void __launch_bounds__(128)
attend_merge_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml, float* __restrict__ out,
                    float* __restrict__ lse, int M, int L, int H, int G, int r, int n_splits, int rows_pad) {
    pdl_wait();        // everything earlier in the stream is complete and visible from here on
    pdl_trigger();     // the next kernel's CTAs may take their places; they wait in the same way
    const int row = blockIdx.x, z = blockIdx.y, LG = L * G;
    const int s = z / LG, lg = z % LG, l = lg / G, g = lg % G;
    const int col = threadIdx.x;
    const size_t p0 = (size_t)z * n_splits * rows_pad + row;          // split sp lives at p0 + sp * rows_pad
    // U splits at a time: the statistics and the partial outputs of a batch are loaded before any of them is used, and
    // the first batch is requested together with the statistics the maximum needs, so that a merge costs a few memory
    // round trips instead of one per split (same split order, same arithmetic)
    float2 ml[U];
    float po[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t pi = p0 + (size_t)min(u, n_splits - 1) * rows_pad;
        ml[u] = part_ml[pi];
        po[u] = part_o[pi * kD + col];
    }
    float mx = -INFINITY;
#pragma unroll
    for (int u = 0; u < U; ++u) mx = fmaxf(mx, ml[u].x);
    for (int sp = U; sp < n_splits; ++sp) mx = fmaxf(mx, part_ml[p0 + (size_t)sp * rows_pad].x);
    float acc = 0.0f, lsum = 0.0f;
    for (int sp0 = 0; sp0 < n_splits; sp0 += U) {
        if (sp0 > 0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t pi = p0 + (size_t)min(sp0 + u, n_splits - 1) * rows_pad;
                ml[u] = part_ml[pi];
                po[u] = part_o[pi * kD + col];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (sp0 + u < n_splits) {
                const float f = ml[u].x > -INFINITY ? exp2f(ml[u].x - mx) : 0.0f;
                acc += f * po[u];
                lsum += f * ml[u].y;
            }
        }
    }
    const int m = row / r, hr = row % r;
    const size_t orow = (((size_t)s * M + m) * L + l) * H + (size_t)g * r + hr;
    out[orow * kD + col] = lsum > 0.0f ? acc / lsum : 0.0f;
    if (col == 0) lse[orow] = lsum > 0.0f ? (mx + log2f(lsum)) * 0.6931471805599453f : -INFINITY;
}

cudaError_t launch_attend_merge(const float* part_o, const float2* part_ml, float* out, float* lse, int rows, int heads, int M, int L,
                                int H, int G, int r, int n_splits, int rows_pad, cudaStream_t st) {
    if (n_splits <= 8)
        launch_pdl(attend_merge_kernel<8>, dim3((unsigned)rows, (unsigned)heads), dim3(kD), 0, st, part_o, part_ml, out, lse, M, L, H, G, r,
                   n_splits, rows_pad);
    else
        launch_pdl(attend_merge_kernel<24>, dim3((unsigned)rows, (unsigned)heads), dim3(kD), 0, st, part_o, part_ml, out, lse, M, L, H, G, r,
                   n_splits, rows_pad);
    return cudaGetLastError();
}

static PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    }
    return fn;
}

// view [heads][cap_tokens][128] bf16 as a 3-D tensor; box = 64 dims x 64 tokens x 1 head, 128-byte swizzle
static bool make_view_map(CUtensorMap* map, const __nv_bfloat16* view, int heads, int cap_tokens, int box_rows = kTile) {
    PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)cap_tokens, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)cap_tokens * kD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(view), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// page pool [max_blocks * 2 * L*G * 64 rows][128] bf16 as a 2-D tensor; box = 64 dims x 64 tokens, 128-byte swizzle
static bool make_pages_map(CUtensorMap* map, const kvmem_pool& p, const __nv_bfloat16* pages, int n_pages) {
    PFN_cuTensorMapEncodeTiled_v12000 enc = get_encode();
    if (!enc) return false;
    const Geometry& g = p.geo;
    cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)n_pages * 2 * g.L * g.G * g.B};
    cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)std::min(g.B, kTile)};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(pages), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// sel_ids == nullptr: attend over an already materialised view.  Otherwise: assemble the view from the
// pages of sessions [session_first, session_first + n_sessions) and attend over it in the same kernel.
cudaError_t launch_attend(const kvmem_pool& p, int n_sessions, const __nv_bfloat16* q, int M,
                          const __nv_bfloat16* view_k, const __nv_bfloat16* view_v, int view_cap_tokens,
                          const int32_t* n_sel, float scale, float* out, float* lse, void* workspace,
                          cudaStream_t st, const int32_t* sel_ids, int sel_stride, int session_first, const PagedSource* alt,
                          int rope_first_position) {
    const Geometry& g = p.geo;
    const int LG = g.L * g.G, heads = n_sessions * LG;
    const bool fused = sel_ids != nullptr;
    const bool paged_only = fused && view_k == nullptr;     // copy-free: attend straight over the pages
    CUtensorMap map_k, map_v, map_pages;
    // alt: the pages and tables are not the pool's own (attention over an execution cache)
    if (fused && !make_pages_map(&map_pages, p, alt ? alt->pages : p.pages, alt ? alt->n_pages : g.max_blocks)) return cudaErrorInvalidValue;
    if (paged_only) {
        map_k = map_pages; map_v = map_pages;               // unused by this mode
    } else {
        // the fused pass stores blocks (boxes of min(B, 64) rows); attention over a finished view loads whole 64-token tiles
        const int box_rows = fused ? std::min(g.B, kTile) : kTile;
        if (!make_view_map(&map_k, view_k, heads, view_cap_tokens, box_rows) || !make_view_map(&map_v, view_v, heads, view_cap_tokens, box_rows))
            return cudaErrorInvalidValue;
    }
    if (!fused) map_pages = map_k;
    static PerDeviceOnce attr_done;
    if (attr_done.pending(p.cfg.device)) {
        cudaError_t e = cudaFuncSetAttribute(attend_split_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<0, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_split_kernel<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmemRope);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmemQrot);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<4, 1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmemQrot);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<4, 1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmemQrot);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<5>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_split_kernel<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmemRope);
        if (e != cudaSuccess) return e;
        attr_done.mark(p.cfg.device);
    }
    AttendPlan plan = plan_attend(p.cfg, n_sessions, M, p.sm_count);
    AttendArgs a{};
    a.q = q; a.n_sel = n_sel;
    a.part_o = reinterpret_cast<float*>(workspace);
    a.part_ml = reinterpret_cast<float2*>(reinterpret_cast<char*>(workspace) + plan.part_o_bytes);
    a.status = p.status_dev;
    a.M = M; a.L = g.L; a.H = g.H; a.G = g.G; a.r = g.r; a.rows = M * g.r;
    a.rows_pad = plan.rows_pad;
    const int RT = row_tiles_for(a.rows);
    if (a.rows > kMaxRows) return cudaErrorInvalidValue;
    if (RT > 1 && rope_first_position >= 0) return cudaErrorInvalidValue;      // the rotating modes take one row tile
    a.n_splits = g_attend_splits > 0 ? std::min((int)g_attend_splits, kMaxSplits) : choose_splits(heads, (view_cap_tokens + kTile - 1) / kTile, p.sm_count);
    a.cap_tokens = view_cap_tokens;
    const float sc = scale > 0.0f ? scale : 1.0f / sqrtf((float)g.d);
    a.scale_log2e = sc * 1.4426950408889634f;
    a.sel_ids = sel_ids; a.tables = p.tables; a.nblocks_dev = p.nblocks_dev;
    a.session_first = session_first; a.sel_stride = sel_stride; a.max_bps = g.max_bps; a.max_blocks = g.max_blocks;
    if (alt) {
        a.tables = alt->tables; a.nblocks_dev = alt->nblocks_dev; a.max_bps = alt->table_stride; a.max_blocks = alt->n_pages;
    }
    a.rope = p.rope_dev; a.first_position = rope_first_position; a.block_tokens = g.B; a.rope_positions = p.cfg.rope_max_positions;
    // How far the producers run ahead.  Measured on this part: a long single-wave stream is fastest with a bounded number
    // of bytes in flight over all SMs (more outstanding requests than the bandwidth-delay product only lengthen the queues
    // in front of HBM and, where the kernel also writes, mix more reads and writes): about 19 MiB counted up to consumption
    // when the kernel only reads, about 9.5 MiB counted up to arrival in shared memory when it also writes the view (a
    // landed tile that waits for its consumers, its store or its rotation is no longer an HBM request: 338.8 us against
    // 345.1 us with 14 MiB counted up to consumption).  Short streams and multi-wave grids keep every stage in flight.
    a.lookahead = g_attend_lookahead;
    const bool writes_view = fused && !paged_only;
    a.landed = g_attend_landed >= 0 ? g_attend_landed : (writes_view ? 1 : 0);
    if (a.lookahead == 0) {
        const long long ctas = (long long)a.n_splits * heads;
        const int tiles_per_cta = ((view_cap_tokens + kTile - 1) / kTile + a.n_splits - 1) / a.n_splits;
        if (ctas <= p.sm_count && tiles_per_cta >= 64) {
            const double target = (writes_view ? (a.landed ? 9.5 : 14.0) : 19.0) * 1024.0 * 1024.0;
            a.lookahead = std::max(2, std::min(kAttStages, (int)(target / ((double)ctas * kStageBytes) + 0.5)));
        }
    }
    // the copy-free raw-key pass is bound by what its consumer warps issue per tile, not by HBM: every stage in flight
    // (233 us per step at a 1M-token history against 249 with five and 305 with four)
    if (paged_only && rope_first_position >= 0 && !p.cfg.rope_in_block_keys && g_attend_lookahead == 0) a.lookahead = kAttRopeStages;
    dim3 grid((unsigned)a.n_splits, (unsigned)LG, (unsigned)n_sessions);
    if (paged_only && rope_first_position >= 0 && p.cfg.rope_in_block_keys && g.B == 32)
        launch_pdl(attend_split_kernel<4, 1, 2>, dim3(grid), dim3(kAttThreads + 32 * kQrotWarps), kAttSmemQrot, st, map_k, map_v, map_pages, a);
    else if (paged_only && rope_first_position >= 0 && p.cfg.rope_in_block_keys && g.B == 16)
        launch_pdl(attend_split_kernel<4, 1, 4>, dim3(grid), dim3(kAttThreads + 32 * kQrotWarps), kAttSmemQrot, st, map_k, map_v, map_pages, a);
    else if (paged_only && rope_first_position >= 0 && p.cfg.rope_in_block_keys)
        launch_pdl(attend_split_kernel<4>, dim3(grid), dim3(kAttThreads + 32 * kQrotWarps), kAttSmemQrot, st, map_k, map_v, map_pages, a);
    else if (paged_only && rope_first_position >= 0)
        launch_pdl(attend_split_kernel<3>, dim3(grid), dim3((kAttRopeConsumers + 1) * 32), kAttSmemRope, st, map_k, map_v, map_pages, a);
    else if (fused && !paged_only && rope_first_position >= 0 && p.cfg.rope_in_block_keys)
        launch_pdl(attend_split_kernel<5>, dim3(grid), dim3(kAttThreads + 32 + 32 * kKrotWarps), kAttSmem, st, map_k, map_v, map_pages, a);
    else if (fused && !paged_only && rope_first_position >= 0)
        launch_pdl(attend_split_kernel<6>, dim3(grid), dim3((kAttRopeConsumers + 2) * 32), kAttSmemRope, st, map_k, map_v, map_pages, a);
    else {
#define KVMEM_ATTEND_LAUNCH(MODE, THREADS)                                                                              \
    do {                                                                                                                \
        if (RT == 1) launch_pdl(attend_split_kernel<MODE, 1>, dim3(grid), dim3(THREADS), kAttSmem, st, map_k, map_v, map_pages, a);      \
        else if (RT == 2) launch_pdl(attend_split_kernel<MODE, 2>, dim3(grid), dim3(THREADS), kAttSmem, st, map_k, map_v, map_pages, a); \
        else launch_pdl(attend_split_kernel<MODE, 4>, dim3(grid), dim3(THREADS), kAttSmem, st, map_k, map_v, map_pages, a);              \
    } while (0)
        if (paged_only) KVMEM_ATTEND_LAUNCH(2, kAttThreads);
        else if (fused) KVMEM_ATTEND_LAUNCH(1, kAttThreads + 32);
        else KVMEM_ATTEND_LAUNCH(0, kAttThreads);
#undef KVMEM_ATTEND_LAUNCH
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_attend_merge(a.part_o, a.part_ml, out, lse, a.rows, heads, M, g.L, g.H, g.G, g.r, a.n_splits, a.rows_pad, st);
}

}  // namespace kvmem
