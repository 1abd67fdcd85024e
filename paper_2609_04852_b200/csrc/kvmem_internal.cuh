// Internal declarations shared by the translation units of libkvmem_b200 (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <atomic>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "kvmem.h"

namespace kvmem {

constexpr int kSMs = 148;                 // B200: 2 dies x 74 SMs
constexpr uint32_t kSpinLimit = 1u << 24;            // bounded waits: try_wait attempts before a kernel gives up
constexpr uint64_t kWaitLimitNs = 1000ull * 1000 * 1000;  // ... or about one second of wall time

// ---- device-resident layout inside the caller's storage --------------------------------------
//   pages   [max_blocks][2 (K|V)][L][G][B][d] bf16   one (block, K|V, l, g) tile is B*d*2 contiguous bytes
//   index   [max_sessions][L][G][max_blocks_per_session][d] bf16
//   tables  [max_sessions][max_blocks_per_session] int32 (logical -> physical page)
//   nblocks [max_sessions] int32
//   status  int32 (sticky device status word)
//   pos0    [max_sessions][max_blocks_per_session] int32: original position of each block's first token (rotary pools)
//   rope    [rope_max_positions][d/2] float2 (cos, sin)                                         (rotary pools)
struct Layout {
    size_t pages_off, index_off, tables_off, nblocks_off, status_off, pos0_off, rope_off, total;
    size_t page_elems;  // bf16 elements per page
    size_t tile_elems;  // B * d
    size_t index_elems_per_session;
};

struct Geometry {
    int L, H, G, d, B, r;
    int max_sessions, max_blocks, max_bps;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A kernel attribute (cudaFuncSetAttribute) belongs to one device: launchers that opt in to large dynamic shared
// memory do it once per device ordinal, keyed by the pool's device.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    bool done[kMaxDevices] = {};
    bool pending(int device) const { return device < 0 || device >= kMaxDevices || !done[device]; }
    void mark(int device) { if (device >= 0 && device < kMaxDevices) done[device] = true; }
};

bool config_valid(const kvmem_pool_config_t& c, const char** why);
Layout make_layout(const kvmem_pool_config_t& c);

}  // namespace kvmem

struct kvmem_pool {
    uint64_t magic;
    kvmem_pool_config_t cfg;
    kvmem::Geometry geo;
    kvmem::Layout lay;
    char* base;                         // DEVICE storage
    __nv_bfloat16* pages;
    __nv_bfloat16* index;
    int32_t* tables;
    int32_t* nblocks_dev;
    int32_t* status_dev;
    int32_t* pos0_dev;                  // null unless rope_max_positions > 0
    float2* rope_dev;
    std::vector<int32_t> sess_blocks;               // host mirror of nblocks
    std::vector<std::vector<int32_t>> sess_pages;   // host mirror of tables
    std::vector<uint8_t> page_used;
    int32_t free_hint;
    int sm_count;
    // host-resident index scoring: a copy stream and its events, created on first use
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_ready[2] = {nullptr, nullptr}, ev_free[2] = {nullptr, nullptr}, ev_start = nullptr;
};

namespace kvmem {

constexpr uint64_t kMagic = 0x4b564d454d423230ull;  // "KVMEMB20"

void set_error(const char* fmt, ...);

// tuning switches (kvmem_set_option)
// Kernel-variant switches set by kvmem_set_option and read by every launch: process-wide, so they are atomics (relaxed:
// a switch is an independent integer, nothing is published through it).
struct Option {
    std::atomic<int> v;
    explicit constexpr Option(int x) : v(x) {}
    operator int() const { return v.load(std::memory_order_relaxed); }
    Option& operator=(int x) { v.store(x, std::memory_order_relaxed); return *this; }
};
extern Option g_score_mode;    // 1: tensor-core decode scoring (default), 0: fp32 ALU + warp-shuffle kernel
extern Option g_chunk_poly;    // chunked scoring: every n-th exponential on the FMA pipe (0: all on the special-function unit)
extern Option g_gather_mode;   // 1: TMA bulk ring (default), 0: 128-bit ld/st copy
extern Option g_attend_landed;
extern Option g_topk_items;    // 0: the top-k kernel holds the fewest scores per thread that cover the session; 1..16: at least this many
extern Option g_topk_cluster;  // 1: sessions above 16,384 blocks are selected by a cluster of 8 CTAs (default), 0: by one CTA
extern Option g_gather_ctas;
extern Option g_attend_lookahead;
extern Option g_attend_splits; // 0: split count from the cost model (default); > 0: forced
extern Option g_pdl;           // 1: the kernels of a step are launched with programmatic stream serialization (default), 0: plain launches

// Programmatic dependent launch.  A kernel launched through launch_pdl may be scheduled while the previous
// kernel of the stream is still running; its first statement is pdl_wait(), which returns once that
// kernel (and, because every such kernel waits first, everything before it) has completed and its
// writes are visible.  pdl_trigger() lets the next kernel's CTAs take their places early.  What is
// hidden is the launch latency between the short dependent kernels of a step.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- kernel launchers (each defined next to its kernel) ----------------------------------------
// All return cudaGetLastError() after the launch.

cudaError_t launch_append(const kvmem_pool& p, int session, int b_first, int n_blocks, const __nv_bfloat16* k,
                          const __nv_bfloat16* v, cudaStream_t st, bool derope = false);

struct ScoreWorkspace {
    float* logits;     // [ns][L][G][rows_pad][nb_pad]
    float2* partials;  // [ns][L][G][rows_pad][n_parts]: per-CTA (max, sum-exp) of each row
    float* scores;     // [ns][max_bps]  (used when the caller passes no score buffer)
    size_t logits_bytes, partials_bytes, scores_bytes, total;
    int rows, rows_pad, nb_pad, n_chunks;
};
ScoreWorkspace plan_score_workspace(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, char* base);

cudaError_t launch_score_decode(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q,
                                int M, const ScoreWorkspace& ws, float* scores, int scores_stride, float score_scale, cudaStream_t st);

// scoring against a host-resident index, streamed in tiles (kvmem_score.cu)
struct HostScorePlan {
    float* logits;      // [L][G][rows_pad][nb_pad]
    float2* partials;   // [L][G][rows_pad][part_stride]: (max, sum-exp) per row, tile and CTA
    float2* merged;     // [L][G][rows_pad]
    size_t logits_bytes, partials_bytes, merged_bytes, total, staging_bytes;
    int rows, rows_pad, nb_pad, n_tiles, parts_per_tile, part_stride;
};
HostScorePlan plan_host_score(const kvmem_pool_config_t& c, int n_blocks, int n_q_tokens, int tile_blocks, int sm_count, char* base);
cudaError_t launch_score_host_index(kvmem_pool& p, const __nv_bfloat16* index_host, int n_blocks, int stride_blocks,
                                    const __nv_bfloat16* q, int M, int tile_blocks, void* staging, const HostScorePlan& ws,
                                    float* scores, cudaStream_t st);
// FP8 (E4M3) execution view (kvmem_fp8.cu)
cudaError_t launch_gather_fp8(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids, int sel_stride,
                              const int32_t* n_sel, uint8_t* view_k, uint8_t* view_v, int view_cap_tokens, float k_scale,
                              float v_scale, cudaStream_t st, int rope_first_position = -1);
cudaError_t launch_attend_fp8(const kvmem_pool& p, int n_sessions, const __nv_bfloat16* q, int M, const uint8_t* view_k,
                              const uint8_t* view_v, int view_cap_tokens, const int32_t* n_sel, float scale, float k_scale,
                              float v_scale, float* out, float* lse, void* workspace, cudaStream_t st,
                              const int32_t* sel_ids = nullptr, int sel_stride = 0, int session_first = 0,
                              int rope_first_position = -1);
// FP8 repository (pool created with fp8_pages): quantising append
cudaError_t launch_append_fp8(const kvmem_pool& p, int session, int b_first, int n_blocks, const __nv_bfloat16* k,
                              const __nv_bfloat16* v, cudaStream_t st, bool derope = false);

// working-set delta (kvmem_delta.cu)
cudaError_t launch_working_set_delta(const kvmem_pool& p, int n_sessions, const int32_t* prev_ids, const int32_t* n_prev,
                                     const int32_t* next_ids, const int32_t* n_next, int stride, int32_t* retained,
                                     int32_t* incoming, int32_t* outgoing, int32_t* counts, cudaStream_t st);

// rotary position embedding (kvmem_rope.cu)
cudaError_t launch_rope_rotate(const kvmem_pool& p, const __nv_bfloat16* x, __nv_bfloat16* y, long long n_rows, int n_vec,
                               const int32_t* positions, int inverse, cudaStream_t st);
cudaError_t launch_gather_rope(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids,
                               int sel_stride, const int32_t* n_sel, __nv_bfloat16* view_k, __nv_bfloat16* view_v,
                               int view_cap_tokens, int first_position, cudaStream_t st);

// multi-token query chunks: tcgen05 two-pass contraction
struct ChunkWorkspace {
    float2* rowstat;   // [ns][L][G][n_chunks][4][rows_pad] (max, sum-exp) per run of block tiles and slice of the tile columns
    float* shift;      // [ns][L][G][shift_stride]: -(max + log2 Z) of every query row, -inf on padding rows
    float* colsum;     // [ns][L][G][4][nb_pad]: per-head, per-column-slice sums of the softmax weights over the head's query rows
    float* scores;     // [ns][max_bps]
    size_t rowstat_bytes, shift_bytes, colsum_bytes, scores_bytes, total;
    int rows, rows_pad, n_panels, nb_pad, n_chunks, shift_stride;
};
ChunkWorkspace plan_chunk_workspace(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, char* base);
bool chunked_scoring_supported(const kvmem_pool_config_t& c, int n_q_tokens);
constexpr int kMaxDecodeTokens = 16;   // more query tokens than this take the tensor-core path
cudaError_t launch_score_chunked(const kvmem_pool& p, int session_first, int n_sessions, const __nv_bfloat16* q, int M,
                                 const ChunkWorkspace& ws, float* scores, int scores_stride, float score_scale, cudaStream_t st);

// Execution cache (working-set reuse with bounded delta re-RoPE): offsets inside the caller's buffer
struct CacheLayout {
    size_t pages, slot_block, slot_pos, slot_cnt, view_slots, n_view, iota, action, old_pos, free_list, total;
};
CacheLayout cache_layout(size_t page_elems, int cap);
// where paged attention finds its pages and tables when they are not the pool's own
struct PagedSource {
    const __nv_bfloat16* pages;
    int n_pages;
    const int32_t* tables;
    int table_stride;
    const int32_t* nblocks_dev;
    const int32_t* sel_ids;
    const int32_t* n_sel;
};
cudaError_t launch_view_cache_reset(const kvmem_pool& p, void* cache, int cap, cudaStream_t st);
cudaError_t launch_view_cache_update(const kvmem_pool& p, int session, const int32_t* sel_ids, const int32_t* n_sel,
                                     void* cache, int cap, int max_delta, int first_position, int32_t* stats,
                                     cudaStream_t st);
void view_cache_paged_source(const kvmem_pool& p, void* cache, int cap, PagedSource* src);

cudaError_t launch_topk(const kvmem_pool& p, int session_first, int n_sessions, const float* scores,
                        int scores_stride, const kvmem_select_params_t& prm, int32_t* sel_ids, int sel_stride,
                        int32_t* n_sel, cudaStream_t st);

// prev_ids != null: incremental view, slots whose block stays are skipped; delta_stats (may be null) receives the counts
// merges the splits of every (session, layer, KV head) row in split order (defined with the bf16 attention kernel; the FP8
// attention kernels write partials of the same layout and share it)
cudaError_t launch_attend_merge(const float* part_o, const float2* part_ml, float* out, float* lse, int rows, int heads, int M, int L,
                                int H, int G, int r, int n_splits, int rows_pad, cudaStream_t st);
cudaError_t launch_gather(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids,
                          int sel_stride, const int32_t* n_sel, __nv_bfloat16* view_k, __nv_bfloat16* view_v,
                          int view_cap_tokens, cudaStream_t st, const int32_t* prev_ids = nullptr, const int32_t* n_prev = nullptr,
                          int32_t* delta_stats = nullptr);

struct AttendPlan {
    int n_splits;
    int rows_pad;          // 16
    size_t part_o_bytes, part_ml_bytes, total;
};
AttendPlan plan_attend(const kvmem_pool_config_t& c, int n_sessions, int n_q_tokens, int sm_count);

cudaError_t launch_attend(const kvmem_pool& p, int n_sessions, const __nv_bfloat16* q, int M,
                          const __nv_bfloat16* view_k, const __nv_bfloat16* view_v, int view_cap_tokens,
                          const int32_t* n_sel, float scale, float* out, float* lse, void* workspace,
                          cudaStream_t st, const int32_t* sel_ids = nullptr, int sel_stride = 0, int session_first = 0,
                          const PagedSource* alt = nullptr, int rope_first_position = -1);

}  // namespace kvmem
