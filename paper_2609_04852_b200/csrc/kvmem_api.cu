// C ABI of libkvmem_b200: argument checking, pool and session bookkeeping, launch sequencing.
// Every step of the recall path runs in the kernels of the sibling files; nothing here computes.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <cmath>
#include <new>

#include "kvmem_internal.cuh"

namespace kvmem {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

bool config_valid(const kvmem_pool_config_t& c, const char** why) {
    auto bad = [&](const char* w) { *why = w; return false; };
    if (c.n_layers < 1 || c.n_layers > 256) return bad("n_layers must be in [1, 256]");
    if (c.n_kv_heads < 1 || c.n_q_heads < 1 || c.n_q_heads % c.n_kv_heads != 0)
        return bad("n_q_heads must be a positive multiple of n_kv_heads");
    if (c.head_dim < 8 || c.head_dim > 512 || c.head_dim % 8 != 0) return bad("head_dim must be a multiple of 8 in [8, 512]");
    if (c.block_tokens < 16 || c.block_tokens > 256 || c.block_tokens % 16 != 0)
        return bad("block_tokens must be a multiple of 16 in [16, 256]");
    if (c.max_sessions < 1 || c.max_sessions > 65535) return bad("max_sessions must be in [1, 65535]");
    if (c.max_blocks < 1) return bad("max_blocks must be positive");
    if (c.max_blocks_per_session < 1 || c.max_blocks_per_session > c.max_blocks)
        return bad("max_blocks_per_session must be in [1, max_blocks]");
    if (c.device < 0) return bad("device must be a CUDA ordinal");
    if (c.rope_max_positions < 0) return bad("rope_max_positions must be non-negative");
    if (c.rope_max_positions > 0 && !(c.rope_theta > 1.0f)) return bad("rope_theta must exceed 1 when rotary support is on");
    if (c.rope_max_positions > 0 && c.head_dim % 16 != 0) return bad("rotary support needs head_dim to be a multiple of 16");
    if (c.rope_in_block_keys != 0 && c.rope_in_block_keys != 1) return bad("rope_in_block_keys must be 0 or 1");
    if (c.rope_in_block_keys && c.rope_max_positions < c.block_tokens)
        return bad("rope_in_block_keys needs rotary support covering at least one block (rope_max_positions >= block_tokens)");
    if (c.fp8_pages != 0 && c.fp8_pages != 1) return bad("fp8_pages must be 0 or 1");
    if (c.fp8_pages) {
        if (c.head_dim != 128 || c.block_tokens != 64) return bad("an FP8 repository needs head_dim 128 and 64-token blocks");
        if (c.rope_max_positions > 0 && !c.rope_in_block_keys)
            return bad("an FP8 repository with rotary support needs rope_in_block_keys (codes cannot be re-encoded; the query is rotated instead)");
        if (!(c.fp8_k_scale > 0.0f) || !(c.fp8_v_scale > 0.0f) || !std::isfinite(c.fp8_k_scale) || !std::isfinite(c.fp8_v_scale))
            return bad("fp8_k_scale and fp8_v_scale must be positive and finite");
    }
    return true;
}

Layout make_layout(const kvmem_pool_config_t& c) {
    Layout l{};
    l.tile_elems = (size_t)c.block_tokens * c.head_dim;
    l.page_elems = 2 * (size_t)c.n_layers * c.n_kv_heads * l.tile_elems;
    l.index_elems_per_session = (size_t)c.n_layers * c.n_kv_heads * c.max_blocks_per_session * c.head_dim;
    size_t off = 0;
    l.pages_off = off;
    off = align_up(off + (size_t)c.max_blocks * l.page_elems * (c.fp8_pages ? 1 : 2), 256);      // bf16 or E4M3 elements
    l.index_off = off;
    off = align_up(off + (size_t)c.max_sessions * l.index_elems_per_session * 2, 256);
    l.tables_off = off;
    off = align_up(off + (size_t)c.max_sessions * c.max_blocks_per_session * 4, 256);
    l.nblocks_off = off;
    off = align_up(off + (size_t)c.max_sessions * 4, 256);
    l.status_off = off;
    off = align_up(off + 256, 256);
    l.pos0_off = off;
    if (c.rope_max_positions > 0) off = align_up(off + (size_t)c.max_sessions * c.max_blocks_per_session * 4, 256);
    l.rope_off = off;
    if (c.rope_max_positions > 0) off = align_up(off + (size_t)c.rope_max_positions * (c.head_dim / 2) * sizeof(float2), 256);
    l.total = off;
    return l;
}

static bool pool_ok(const kvmem_pool* p) {
    if (!p || p->magic != kMagic) {
        set_error("pool handle is null or stale");
        return false;
    }
    return true;
}

// pool_ok plus: the pool's device is the calling thread's current device.  Every call that enqueues work launches on the
// current device with the pool's pointers, so a mismatch is refused on the host instead of faulting on the wrong GPU.
static bool pool_live(const kvmem_pool* p) {
    if (!pool_ok(p)) return false;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device != p->cfg.device) {
        (void)cudaGetLastError();
        set_error("the pool lives on device %d but device %d is current", p->cfg.device, device);
        return false;
    }
    return true;
}

static bool sessions_ok(const kvmem_pool* p, int first, int n) {
    if (first < 0 || n < 1 || first + n > p->cfg.max_sessions) {
        set_error("sessions [%d, %d) outside [0, %d)", first, first + n, p->cfg.max_sessions);
        return false;
    }
    return true;
}

// the calls that read bf16 pages refuse an FP8 repository (and the other way round) instead of misreading it
static bool pages_are(const kvmem_pool* p, bool fp8, const char* who) {
    if ((p->cfg.fp8_pages != 0) == fp8) return true;
    set_error("%s reads %s pages, the pool holds %s", who, fp8 ? "FP8" : "bf16", fp8 ? "bf16" : "FP8");
    return false;
}

static int cuda_fail(const char* what, cudaError_t e) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return KVMEM_E_CUDA;
}

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

// The passes that read pages through the block table walk the view in 64-token tiles: a tile is 64 / B whole blocks or
// a 64-token slice of one block.  in_block_rotation: the pass rotates by one angle set per tile (in-block key layout),
// which needs tile == block.
static bool paged_block_size_ok(const kvmem_pool* p, bool in_block_rotation, const char* who) {
    const int B = p->cfg.block_tokens;
    if (p->cfg.head_dim != 128 || !(64 % B == 0 || B % 64 == 0)) {
        set_error("%s is built for head_dim 128 and block sizes that divide or are a multiple of 64 tokens", who);
        return false;
    }
    if (in_block_rotation && B != 64) {
        set_error("%s on a pool with rope_in_block_keys rotates once per 64-token tile and needs 64-token blocks", who);
        return false;
    }
    return true;
}

}  // namespace kvmem

using namespace kvmem;

extern "C" {

const char* kvmem_last_error(void) { return g_err; }

size_t kvmem_pool_bytes(const kvmem_pool_config_t* cfg) {
    const char* why = "";
    if (!cfg || !config_valid(*cfg, &why)) {
        set_error("invalid pool configuration: %s", cfg ? why : "null");
        return 0;
    }
    return make_layout(*cfg).total;
}

int32_t kvmem_budget_blocks(const kvmem_select_params_t* prm, int32_t block_tokens, int32_t n_blocks) {
    if (!prm || block_tokens <= 0) return 0;
    int64_t room = (int64_t)prm->max_view_tokens - (int64_t)prm->mandatory_tokens;
    int64_t k = room > 0 ? room / block_tokens : 0;
    k = std::min<int64_t>(k, prm->budget_blocks);
    k = std::min<int64_t>(k, n_blocks);
    return (int32_t)std::max<int64_t>(k, 0);
}

size_t kvmem_select_workspace_bytes(const kvmem_pool_config_t* cfg, int32_t n_sessions, int32_t n_q_tokens) {
    const char* why = "";
    if (!cfg || !config_valid(*cfg, &why) || n_sessions < 1 || n_sessions > cfg->max_sessions || n_q_tokens < 1) {
        set_error("invalid arguments to kvmem_select_workspace_bytes");
        return 0;
    }
    if (n_q_tokens > kMaxDecodeTokens) return plan_chunk_workspace(*cfg, n_sessions, n_q_tokens, nullptr).total;
    return plan_score_workspace(*cfg, n_sessions, n_q_tokens, nullptr).total;
}

size_t kvmem_attend_workspace_bytes(const kvmem_pool_config_t* cfg, int32_t n_sessions, int32_t n_q_tokens) {
    const char* why = "";
    if (!cfg || !config_valid(*cfg, &why) || n_sessions < 1 || n_q_tokens < 1) {
        set_error("invalid arguments to kvmem_attend_workspace_bytes");
        return 0;
    }
    return plan_attend(*cfg, n_sessions, n_q_tokens, kSMs).total;
}

int kvmem_pool_create(const kvmem_pool_config_t* cfg, void* storage, size_t bytes, kvmem_pool_t** out) {
    const char* why = "";
    if (!out) { set_error("out is null"); return KVMEM_E_INVALID; }
    *out = nullptr;
    if (!cfg || !config_valid(*cfg, &why)) {
        set_error("invalid pool configuration: %s", cfg ? why : "null");
        return KVMEM_E_INVALID;
    }
    if (!storage || !aligned(storage, 256)) { set_error("storage must be a 256-byte aligned device pointer"); return KVMEM_E_INVALID; }
    Layout lay = make_layout(*cfg);
    if (bytes < lay.total) {
        set_error("storage holds %zu bytes, the pool needs %zu", bytes, lay.total);
        return KVMEM_E_CAPACITY;
    }
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, cfg->device);
    if (e != cudaSuccess) return cuda_fail("cudaGetDeviceProperties", e);
    if (prop.major != 10) {
        set_error("device %d is compute capability %d.%d; this library is built for sm_100a only", cfg->device,
                  prop.major, prop.minor);
        return KVMEM_E_UNSUPPORTED;
    }
    kvmem_pool* p = new (std::nothrow) kvmem_pool();
    if (!p) { set_error("host allocation failed"); return KVMEM_E_CAPACITY; }
    p->magic = kMagic;
    p->cfg = *cfg;
    p->geo = Geometry{cfg->n_layers, cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim, cfg->block_tokens,
                      cfg->n_q_heads / cfg->n_kv_heads, cfg->max_sessions, cfg->max_blocks, cfg->max_blocks_per_session};
    p->lay = lay;
    p->base = (char*)storage;
    p->pages = (__nv_bfloat16*)(p->base + lay.pages_off);
    p->index = (__nv_bfloat16*)(p->base + lay.index_off);
    p->tables = (int32_t*)(p->base + lay.tables_off);
    p->nblocks_dev = (int32_t*)(p->base + lay.nblocks_off);
    p->status_dev = (int32_t*)(p->base + lay.status_off);
    p->sess_blocks.assign(cfg->max_sessions, 0);
    p->sess_pages.assign(cfg->max_sessions, {});
    p->page_used.assign(cfg->max_blocks, 0);
    p->free_hint = 0;
    p->sm_count = prop.multiProcessorCount;
    p->pos0_dev = cfg->rope_max_positions > 0 ? (int32_t*)(p->base + lay.pos0_off) : nullptr;
    p->rope_dev = cfg->rope_max_positions > 0 ? (float2*)(p->base + lay.rope_off) : nullptr;
    e = cudaMemset(p->base + lay.tables_off, 0, lay.rope_off - lay.tables_off);
    if (e == cudaSuccess && cfg->rope_max_positions > 0) {
        // cos/sin of position * theta^(-2i/d): angle in fp64, one rounding to fp32 (built here, on the host)
        const int half = cfg->head_dim / 2;
        std::vector<double> freq(half);
        for (int i = 0; i < half; ++i) freq[i] = pow((double)cfg->rope_theta, -2.0 * (double)i / (double)cfg->head_dim);
        const int chunk = 4096;
        std::vector<float2> rows((size_t)chunk * half);
        for (int p0 = 0; e == cudaSuccess && p0 < cfg->rope_max_positions; p0 += chunk) {
            const int n = std::min(chunk, cfg->rope_max_positions - p0);
            for (int r = 0; r < n; ++r)
                for (int i = 0; i < half; ++i) {
                    const double ang = (double)(p0 + r) * freq[i];
                    rows[(size_t)r * half + i] = make_float2((float)cos(ang), (float)sin(ang));
                }
            e = cudaMemcpy(p->rope_dev + (size_t)p0 * half, rows.data(), (size_t)n * half * sizeof(float2), cudaMemcpyHostToDevice);
        }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete p; return cuda_fail("clearing pool metadata", e); }
    *out = p;
    return KVMEM_OK;
}

int kvmem_pool_destroy(kvmem_pool_t* pool) {
    if (!pool_ok(pool)) return KVMEM_E_STATE;
    pool->magic = 0;
    if (pool->copy_stream) {            // the copy stream of host-resident index scoring: drain it, then let it go
        cudaStreamSynchronize(pool->copy_stream);
        for (int i = 0; i < 2; ++i) {
            if (pool->ev_ready[i]) cudaEventDestroy(pool->ev_ready[i]);
            if (pool->ev_free[i]) cudaEventDestroy(pool->ev_free[i]);
        }
        if (pool->ev_start) cudaEventDestroy(pool->ev_start);
        cudaStreamDestroy(pool->copy_stream);
    }
    delete pool;
    return KVMEM_OK;
}

int kvmem_session_reset(kvmem_pool_t* p, int32_t session, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    // the device's block count first: kernels that size their work from it see an empty session from here on in stream order
    cudaError_t e = cudaMemsetAsync(p->nblocks_dev + session, 0, 4, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("clearing the session's block count", e);
    for (int32_t pg : p->sess_pages[session]) p->page_used[pg] = 0;
    p->sess_pages[session].clear();
    p->sess_blocks[session] = 0;
    p->free_hint = 0;
    return KVMEM_OK;
}

int32_t kvmem_session_blocks(const kvmem_pool_t* p, int32_t session) {
    if (!pool_ok(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    return p->sess_blocks[session];
}

static int append_impl(kvmem_pool_t* p, int32_t session, const void* k, const void* v, int32_t n_blocks,
                       const int32_t* phys_ids, const int32_t* block_pos0, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    if (n_blocks < 0) { set_error("n_blocks is negative"); return KVMEM_E_INVALID; }
    if (n_blocks == 0) return KVMEM_OK;
    if (!k || !v || !aligned(k, 16) || !aligned(v, 16)) { set_error("k and v must be 16-byte aligned device pointers"); return KVMEM_E_INVALID; }
    const int have = p->sess_blocks[session];
    if ((int64_t)have + n_blocks > p->cfg.max_blocks_per_session) {
        set_error("session %d holds %d blocks; %d more exceed max_blocks_per_session = %d", session, have, n_blocks,
                  p->cfg.max_blocks_per_session);
        return KVMEM_E_CAPACITY;
    }
    // choose pages without touching the pool until every id is known to be usable
    std::vector<int32_t> ids(n_blocks);
    if (phys_ids) {
        std::vector<int32_t> sorted(phys_ids, phys_ids + n_blocks);
        std::sort(sorted.begin(), sorted.end());
        for (int i = 0; i < n_blocks; ++i) {
            int32_t pg = phys_ids[i];
            if (pg < 0 || pg >= p->cfg.max_blocks) { set_error("page id %d outside [0, %d)", pg, p->cfg.max_blocks); return KVMEM_E_INVALID; }
            if (p->page_used[pg]) { set_error("page %d is already in use", pg); return KVMEM_E_STATE; }
            if (i > 0 && sorted[i] == sorted[i - 1]) { set_error("page id %d given twice", sorted[i]); return KVMEM_E_INVALID; }
            ids[i] = pg;
        }
    } else {
        int32_t pg = p->free_hint, got = 0;
        for (; pg < p->cfg.max_blocks && got < n_blocks; ++pg)
            if (!p->page_used[pg]) ids[got++] = pg;
        if (got < n_blocks) { set_error("pool has %d free pages, %d needed", got, n_blocks); return KVMEM_E_CAPACITY; }
    }
    if (block_pos0) {
        if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
        for (int i = 0; i < n_blocks; ++i)
            if (block_pos0[i] < 0 || (int64_t)block_pos0[i] + p->cfg.block_tokens > p->cfg.rope_max_positions) {
                set_error("block %d: positions [%d, %d) outside the rotary table [0, %d)", i, block_pos0[i],
                          block_pos0[i] + p->cfg.block_tokens, p->cfg.rope_max_positions);
                return KVMEM_E_INVALID;
            }
    }
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* table = p->tables + (size_t)session * p->cfg.max_blocks_per_session;
    cudaError_t e = cudaMemcpyAsync(table + have, ids.data(), (size_t)n_blocks * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail("block table upload", e);
    const int32_t total = have + n_blocks;
    if (block_pos0) {
        e = cudaMemcpyAsync(p->pos0_dev + (size_t)session * p->cfg.max_blocks_per_session + have, block_pos0,
                            (size_t)n_blocks * 4, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail("block position upload", e);
    }
    e = p->cfg.fp8_pages ? launch_append_fp8(*p, session, have, n_blocks, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, st, block_pos0 != nullptr)
                         : launch_append(*p, session, have, n_blocks, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, st, block_pos0 != nullptr);
    if (e != cudaSuccess) return cuda_fail("append kernel launch", e);
    // the device's block count last: it never covers index rows whose kernel was not enqueued
    e = cudaMemcpyAsync(p->nblocks_dev + session, &total, 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail("block count upload", e);
    for (int32_t pg : ids) { p->page_used[pg] = 1; p->sess_pages[session].push_back(pg); }
    if (!phys_ids) p->free_hint = ids.back() + 1;
    p->sess_blocks[session] = total;
    return KVMEM_OK;
}

int kvmem_append_blocks(kvmem_pool_t* p, int32_t session, const void* k, const void* v, int32_t n_blocks,
                        const int32_t* phys_ids, void* stream) {
    return append_impl(p, session, k, v, n_blocks, phys_ids, nullptr, stream);
}

int kvmem_append_blocks_rope(kvmem_pool_t* p, int32_t session, const void* k_roped, const void* v, int32_t n_blocks,
                             const int32_t* phys_ids, const int32_t* block_pos0, void* stream) {
    if (!block_pos0) { set_error("block_pos0 is null"); return KVMEM_E_INVALID; }
    return append_impl(p, session, k_roped, v, n_blocks, phys_ids, block_pos0, stream);
}

int kvmem_rope_rotate(kvmem_pool_t* p, const void* x, void* y, int64_t n_rows, int32_t n_vec, const int32_t* positions,
                      int32_t inverse, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
    if (!x || !y || !positions || !aligned(x, 16) || !aligned(y, 16) || n_rows < 0 || n_vec < 1) {
        set_error("kvmem_rope_rotate: null or misaligned pointer, or bad sizes");
        return KVMEM_E_INVALID;
    }
    if (n_rows == 0) return KVMEM_OK;
    cudaError_t e = launch_rope_rotate(*p, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, n_rows, n_vec, positions, inverse,
                                       (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("rotary kernel launch", e);
    return KVMEM_OK;
}

int kvmem_materialize_rope(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids,
                           int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v, int32_t view_cap_tokens,
                           int32_t first_position, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
    if (!sel_ids || !n_sel || !view_k || !view_v || !aligned(view_k, 16) || !aligned(view_v, 16)) {
        set_error("kvmem_materialize_rope: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (sel_stride < 1 || view_cap_tokens < p->cfg.block_tokens || view_cap_tokens % p->cfg.block_tokens != 0) {
        set_error("view_cap_tokens must be a positive multiple of block_tokens and sel_stride positive");
        return KVMEM_E_INVALID;
    }
    const int64_t last = (int64_t)first_position + std::min<int64_t>((int64_t)sel_stride * p->cfg.block_tokens, view_cap_tokens);
    if (first_position < 0 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last,
                  p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_gather_rope(*p, session_first, n_sessions, sel_ids, sel_stride, n_sel, (__nv_bfloat16*)view_k,
                                       (__nv_bfloat16*)view_v, view_cap_tokens, first_position, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("rotary gather kernel launch", e);
    return KVMEM_OK;
}

// scoring stage shared by kvmem_score and kvmem_select; *sc_out receives where the scores were written
static int score_impl(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                      float* scores, float score_scale, void* workspace, size_t workspace_bytes, cudaStream_t st, float** sc_out) {
    if (!q || !aligned(q, 16) || !workspace || !aligned(workspace, 256)) {
        set_error("scoring: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1) { set_error("n_q_tokens must be positive"); return KVMEM_E_INVALID; }
    if (p->cfg.head_dim != 128) { set_error("scoring kernels are built for head_dim 128"); return KVMEM_E_UNSUPPORTED; }
    float* sc = nullptr;
    cudaError_t e;
    if (n_q_tokens > kMaxDecodeTokens) {
        // a multi-token chunk makes scoring a dense contraction: tensor-core path
        if (!chunked_scoring_supported(p->cfg, n_q_tokens)) {
            set_error("chunked scoring needs head_dim 128, H/G dividing 128 and n_q_tokens * H/G <= 4096 "
                      "(scores are additive over query tokens: split a longer chunk and add)");
            return KVMEM_E_UNSUPPORTED;
        }
        ChunkWorkspace cw = plan_chunk_workspace(p->cfg, n_sessions, n_q_tokens, (char*)workspace);
        if (workspace_bytes < cw.total) { set_error("select workspace holds %zu bytes, %zu needed", workspace_bytes, cw.total); return KVMEM_E_CAPACITY; }
        sc = scores ? scores : cw.scores;
        e = launch_score_chunked(*p, session_first, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, cw, sc,
                                 p->cfg.max_blocks_per_session, score_scale, st);
    } else {
        ScoreWorkspace ws = plan_score_workspace(p->cfg, n_sessions, n_q_tokens, (char*)workspace);
        if (workspace_bytes < ws.total) { set_error("select workspace holds %zu bytes, %zu needed", workspace_bytes, ws.total); return KVMEM_E_CAPACITY; }
        sc = scores ? scores : ws.scores;
        e = launch_score_decode(*p, session_first, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, ws, sc,
                                p->cfg.max_blocks_per_session, score_scale, st);
    }
    if (e != cudaSuccess) return cuda_fail("score kernel launch", e);
    *sc_out = sc;
    return KVMEM_OK;
}

int kvmem_score(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens, float* scores,
                float score_scale, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!scores) { set_error("scores is null"); return KVMEM_E_INVALID; }
    if (!(score_scale >= 0.0f) || !std::isfinite(score_scale)) { set_error("score_scale must be non-negative and finite (0 selects 1)"); return KVMEM_E_INVALID; }
    float* sc = nullptr;
    return score_impl(p, session_first, n_sessions, q, n_q_tokens, scores, score_scale > 0.0f ? score_scale : 1.0f, workspace,
                      workspace_bytes, (cudaStream_t)stream, &sc);
}

// ---- index in host memory, streamed in tiles

static bool host_score_args_ok(const kvmem_pool_t* p, int32_t n_blocks, int32_t n_q_tokens, int32_t tile_blocks) {
    if (n_blocks < 1 || n_q_tokens < 1 || n_q_tokens > kMaxDecodeTokens) {
        set_error("host-index scoring takes 1..%d query tokens and at least one block", kMaxDecodeTokens);
        return false;
    }
    if (tile_blocks < 128 || tile_blocks % 128 != 0) { set_error("tile_blocks must be a positive multiple of 128"); return false; }
    if (p->cfg.head_dim != 128) { set_error("scoring kernels are built for head_dim 128"); return false; }
    if ((int64_t)p->cfg.n_layers * p->cfg.n_kv_heads * tile_blocks > 0x7fffffffll) { set_error("tile too large"); return false; }
    return true;
}

size_t kvmem_score_host_workspace_bytes(const kvmem_pool_t* p, int32_t n_blocks, int32_t n_q_tokens, int32_t tile_blocks) {
    if (!p || !host_score_args_ok(p, n_blocks, n_q_tokens, tile_blocks)) return 0;
    return plan_host_score(p->cfg, n_blocks, n_q_tokens, tile_blocks, p->sm_count, nullptr).total;
}

size_t kvmem_score_host_staging_bytes(const kvmem_pool_t* p, int32_t tile_blocks) {
    if (!p || !host_score_args_ok(p, 1, 1, tile_blocks)) return 0;
    return plan_host_score(p->cfg, 1, 1, tile_blocks, p->sm_count, nullptr).staging_bytes;
}

int kvmem_score_host_index(kvmem_pool_t* p, const void* index_host, int32_t n_blocks, int32_t index_stride_blocks, const void* q,
                           int32_t n_q_tokens, int32_t tile_blocks, float* scores, void* staging, size_t staging_bytes,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!host_score_args_ok(p, n_blocks, n_q_tokens, tile_blocks)) return KVMEM_E_INVALID;
    if (!index_host || !q || !scores || !staging || !workspace || !aligned(index_host, 16) || !aligned(q, 16) ||
        !aligned(staging, 256) || !aligned(workspace, 256)) {
        set_error("kvmem_score_host_index: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (index_stride_blocks < n_blocks) { set_error("index_stride_blocks is below n_blocks"); return KVMEM_E_INVALID; }
    HostScorePlan plan = plan_host_score(p->cfg, n_blocks, n_q_tokens, tile_blocks, p->sm_count, (char*)workspace);
    if (workspace_bytes < plan.total) { set_error("workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    if (staging_bytes < plan.staging_bytes) { set_error("staging holds %zu bytes, %zu needed", staging_bytes, plan.staging_bytes); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_score_host_index(*p, (const __nv_bfloat16*)index_host, n_blocks, index_stride_blocks,
                                            (const __nv_bfloat16*)q, n_q_tokens, tile_blocks, staging, plan, scores,
                                            (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("host-index scoring", e);
    return KVMEM_OK;
}

int kvmem_topk(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const float* scores, int32_t scores_stride,
               const kvmem_select_params_t* prm, int32_t* sel_ids, int32_t sel_stride, int32_t* n_sel, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!scores || !prm || !sel_ids || !n_sel) { set_error("kvmem_topk: null pointer"); return KVMEM_E_INVALID; }
    if (prm->n_sink_blocks < 0 || prm->n_recent_blocks < 0) { set_error("sink/recent counts must be non-negative"); return KVMEM_E_INVALID; }
    int max_k = 0, max_nb = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s) {
        max_k = std::max(max_k, kvmem_budget_blocks(prm, p->cfg.block_tokens, p->sess_blocks[s]));
        max_nb = std::max(max_nb, p->sess_blocks[s]);
    }
    if (sel_stride < max_k) { set_error("sel_stride %d is below the clamped budget %d", sel_stride, max_k); return KVMEM_E_CAPACITY; }
    if (scores_stride < max_nb) { set_error("scores_stride %d is below the session length %d", scores_stride, max_nb); return KVMEM_E_INVALID; }
    cudaError_t e = launch_topk(*p, session_first, n_sessions, scores, scores_stride, *prm, sel_ids, sel_stride, n_sel,
                                (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("top-k kernel launch", e);
    return KVMEM_OK;
}

int kvmem_select(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                 const kvmem_select_params_t* prm, int32_t* sel_ids, int32_t sel_stride, int32_t* n_sel, float* scores,
                 void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!prm || !sel_ids || !n_sel) { set_error("kvmem_select: null pointer"); return KVMEM_E_INVALID; }
    if (prm->n_sink_blocks < 0 || prm->n_recent_blocks < 0) { set_error("sink/recent counts must be non-negative"); return KVMEM_E_INVALID; }
    int max_k = 0;
    for (int s = session_first; s < session_first + n_sessions; ++s)
        max_k = std::max(max_k, kvmem_budget_blocks(prm, p->cfg.block_tokens, p->sess_blocks[s]));
    if (sel_stride < max_k) { set_error("sel_stride %d is below the clamped budget %d", sel_stride, max_k); return KVMEM_E_CAPACITY; }
    cudaStream_t st = (cudaStream_t)stream;
    float* sc = nullptr;
    int rc = score_impl(p, session_first, n_sessions, q, n_q_tokens, scores, 1.0f, workspace, workspace_bytes, st, &sc);
    if (rc != KVMEM_OK) return rc;
    cudaError_t e = launch_topk(*p, session_first, n_sessions, sc, p->cfg.max_blocks_per_session, *prm, sel_ids, sel_stride, n_sel, st);
    if (e != cudaSuccess) return cuda_fail("top-k kernel launch", e);
    return KVMEM_OK;
}

int kvmem_materialize(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids,
                      int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v, int32_t view_cap_tokens,
                      void* stream) {
    if (!pool_live(p) || !pages_are(p, false, "kvmem_materialize")) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!sel_ids || !n_sel || !view_k || !view_v || !aligned(view_k, 16) || !aligned(view_v, 16)) {
        set_error("kvmem_materialize: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (sel_stride < 1 || view_cap_tokens < p->cfg.block_tokens || view_cap_tokens % p->cfg.block_tokens != 0) {
        set_error("view_cap_tokens must be a positive multiple of block_tokens and sel_stride positive");
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_gather(*p, session_first, n_sessions, sel_ids, sel_stride, n_sel, (__nv_bfloat16*)view_k,
                                  (__nv_bfloat16*)view_v, view_cap_tokens, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("gather kernel launch", e);
    return KVMEM_OK;
}

int kvmem_materialize_delta(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const int32_t* prev_ids, const int32_t* n_prev,
                            const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v,
                            int32_t view_cap_tokens, int32_t* stats, void* stream) {
    if (!pool_live(p) || !pages_are(p, false, "kvmem_materialize_delta")) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!prev_ids || !n_prev || !sel_ids || !n_sel || !view_k || !view_v || !aligned(view_k, 16) || !aligned(view_v, 16)) {
        set_error("kvmem_materialize_delta: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (sel_stride < 1 || view_cap_tokens < p->cfg.block_tokens || view_cap_tokens % p->cfg.block_tokens != 0) {
        set_error("view_cap_tokens must be a positive multiple of block_tokens and sel_stride positive");
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_gather(*p, session_first, n_sessions, sel_ids, sel_stride, n_sel, (__nv_bfloat16*)view_k,
                                  (__nv_bfloat16*)view_v, view_cap_tokens, (cudaStream_t)stream, prev_ids, n_prev, stats);
    if (e != cudaSuccess) return cuda_fail("incremental gather kernel launch", e);
    return KVMEM_OK;
}

int kvmem_view_attend(kvmem_pool_t* p, int32_t n_sessions, const void* q, int32_t n_q_tokens, const void* view_k,
                      const void* view_v, int32_t view_cap_tokens, const int32_t* n_sel, float scale, float* out,
                      float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (n_sessions < 1) { set_error("n_sessions must be positive"); return KVMEM_E_INVALID; }
    if (!q || !view_k || !view_v || !n_sel || !out || !lse || !workspace || !aligned(q, 16) || !aligned(view_k, 128) ||
        !aligned(view_v, 128) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_view_attend: null or misaligned pointer (views need 128-byte alignment)");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1) { set_error("n_q_tokens must be positive"); return KVMEM_E_INVALID; }
    if (p->cfg.head_dim != 128) {       // any block size the pool accepts (a multiple of 16): the view is walked in 64-token tiles
        set_error("attention kernel is built for head_dim 128");
        return KVMEM_E_UNSUPPORTED;
    }
    if (n_q_tokens * p->geo.r > 64) { set_error("n_q_tokens * (H/G) = %d exceeds 64 rows per call", n_q_tokens * p->geo.r); return KVMEM_E_UNSUPPORTED; }
    if (view_cap_tokens < p->cfg.block_tokens || view_cap_tokens % p->cfg.block_tokens != 0) {
        set_error("view_cap_tokens must be a positive multiple of block_tokens");
        return KVMEM_E_INVALID;
    }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_attend(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, (const __nv_bfloat16*)view_k,
                                  (const __nv_bfloat16*)view_v, view_cap_tokens, n_sel, scale, out, lse, workspace,
                                  (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("attend kernel launch", e);
    return KVMEM_OK;
}

static void step_staging(const kvmem_pool_config_t& c, int ns, int M, size_t* q_b, size_t* out_b, size_t* lse_b) {
    const size_t rows = (size_t)ns * M * c.n_layers * c.n_q_heads;
    *q_b = align_up(rows * c.head_dim * 2, 256);
    *out_b = align_up(rows * c.head_dim * 4, 256);
    *lse_b = align_up(rows * 4, 256);
}

size_t kvmem_step_staging_bytes(const kvmem_pool_config_t* cfg, int32_t n_sessions, int32_t n_q_tokens) {
    const char* why = "";
    if (!cfg || !config_valid(*cfg, &why) || n_sessions < 1 || n_q_tokens < 1) {
        set_error("invalid arguments to kvmem_step_staging_bytes");
        return 0;
    }
    size_t a, b, c;
    step_staging(*cfg, n_sessions, n_q_tokens, &a, &b, &c);
    return a + b + c;
}

// the device-side address of a host buffer that the GPU can write directly (pinned and mapped), else null
static float* mapped_host_pointer(float* host) {
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer) return nullptr;
    return static_cast<float*>(at.devicePointer);
}

int kvmem_recall_step_host(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q_host,
                           int32_t n_q_tokens, const kvmem_select_params_t* prm, int32_t* sel_ids, int32_t sel_stride,
                           int32_t* n_sel, void* view_k, void* view_v, int32_t view_cap_tokens, float scale,
                           float* out_host, float* lse_host, void* staging, size_t staging_bytes, void* select_ws,
                           size_t select_ws_bytes, void* attend_ws, size_t attend_ws_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!q_host || !out_host || !lse_host || !staging || !aligned(staging, 256) || n_q_tokens < 1) {
        set_error("kvmem_recall_step_host: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    size_t q_b, out_b, lse_b;
    step_staging(p->cfg, n_sessions, n_q_tokens, &q_b, &out_b, &lse_b);
    if (staging_bytes < q_b + out_b + lse_b) { set_error("staging holds %zu bytes, %zu needed", staging_bytes, q_b + out_b + lse_b); return KVMEM_E_CAPACITY; }
    char* sb = (char*)staging;
    void* q_dev = sb;
    float* out_dev = (float*)(sb + q_b);
    float* lse_dev = (float*)(sb + q_b + out_b);
    const size_t rows = (size_t)n_sessions * n_q_tokens * p->cfg.n_layers * p->cfg.n_q_heads;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(q_dev, q_host, rows * p->cfg.head_dim * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail("query upload", e);
    int rc = kvmem_select(p, session_first, n_sessions, q_dev, n_q_tokens, prm, sel_ids, sel_stride, n_sel, nullptr,
                          select_ws, select_ws_bytes, stream);
    if (rc != KVMEM_OK) return rc;
    // Result buffers in pinned, device-mapped host memory are written by the merge kernel itself (the stores cross
    // PCIe as they are issued and are complete when the stream is): two copy operations less on the critical path
    // of a synchronous step.  Anything else (pageable memory) takes the staged copies.
    float* out_map = mapped_host_pointer(out_host);
    float* lse_map = mapped_host_pointer(lse_host);
    const bool direct = out_map && lse_map && aligned(out_map, 16);
    rc = kvmem_materialize_attend(p, session_first, n_sessions, q_dev, n_q_tokens, sel_ids, sel_stride, n_sel, view_k, view_v,
                                  view_cap_tokens, scale, direct ? out_map : out_dev, direct ? lse_map : lse_dev, attend_ws,
                                  attend_ws_bytes, stream);
    if (rc != KVMEM_OK) return rc;
    if (!direct) {
        e = cudaMemcpyAsync(out_host, out_dev, rows * p->cfg.head_dim * 4, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(lse_host, lse_dev, rows * 4, cudaMemcpyDeviceToHost, st);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail("result download", e);
    return KVMEM_OK;
}

int kvmem_set_option(const char* name, int32_t value) {
    if (!name) { set_error("option name is null"); return KVMEM_E_INVALID; }
    if (strcmp(name, "gather_mode") == 0 && (value == 0 || value == 1)) { g_gather_mode = value; return KVMEM_OK; }
    if (strcmp(name, "chunk_poly") == 0 && (value == 0 || (value >= 2 && value <= 5))) { g_chunk_poly = value; return KVMEM_OK; }
    if (strcmp(name, "topk_cluster") == 0 && (value == 0 || value == 1)) { g_topk_cluster = value; return KVMEM_OK; }
    if (strcmp(name, "topk_items") == 0 && (value == 0 || value == 1 || value == 2 || value == 4 || value == 8 || value == 16)) {
        g_topk_items = value;
        return KVMEM_OK;
    }
    if (strcmp(name, "gather_ctas") == 0 && value >= 0) { g_gather_ctas = value; return KVMEM_OK; }
    if (strcmp(name, "attend_lookahead") == 0 && value >= 0 && value <= 8) { g_attend_lookahead = value; return KVMEM_OK; }
    if (strcmp(name, "attend_landed") == 0 && (value >= -1 && value <= 1)) { g_attend_landed = value; return KVMEM_OK; }
    if (strcmp(name, "attend_splits") == 0 && value >= 0 && value <= 64) { g_attend_splits = value; return KVMEM_OK; }
    if (strcmp(name, "pdl") == 0 && (value == 0 || value == 1)) { g_pdl = value; return KVMEM_OK; }
    if (strcmp(name, "score_mode") == 0 && (value == 0 || value == 1)) { g_score_mode = value; return KVMEM_OK; }
    set_error("unknown option or value: %s = %d", name, value);
    return KVMEM_E_INVALID;
}

// rope_first_position < 0: plain views; otherwise the position-consistent fused pass (in-block key layout)
static int materialize_attend_impl(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                   const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v,
                                   int32_t view_cap_tokens, int32_t rope_first_position, float scale, float* out, float* lse,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p) || !pages_are(p, false, "kvmem_materialize_attend")) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!q || !sel_ids || !n_sel || !view_k || !view_v || !out || !lse || !workspace || !aligned(q, 16) ||
        !aligned(view_k, 128) || !aligned(view_v, 128) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_materialize_attend: null or misaligned pointer (views need 128-byte alignment)");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1 || sel_stride < 1) { set_error("n_q_tokens and sel_stride must be positive"); return KVMEM_E_INVALID; }
    if (!paged_block_size_ok(p, rope_first_position >= 0 && p->cfg.rope_in_block_keys, "kvmem_materialize_attend")) return KVMEM_E_UNSUPPORTED;
    if (n_q_tokens * p->geo.r > (rope_first_position >= 0 ? 16 : 64)) { set_error("n_q_tokens * (H/G) = %d exceeds %d rows per call", n_q_tokens * p->geo.r, rope_first_position >= 0 ? 16 : 64); return KVMEM_E_UNSUPPORTED; }
    if (view_cap_tokens < p->cfg.block_tokens || view_cap_tokens % p->cfg.block_tokens != 0) {
        set_error("view_cap_tokens must be a positive multiple of block_tokens");
        return KVMEM_E_INVALID;
    }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    if ((int64_t)p->cfg.max_blocks * 2 * p->cfg.n_layers * p->cfg.n_kv_heads * p->cfg.block_tokens > 0x7fffffffll) {
        set_error("page pool too large for 32-bit TMA row coordinates");
        return KVMEM_E_UNSUPPORTED;
    }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_attend(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, (const __nv_bfloat16*)view_k,
                                  (const __nv_bfloat16*)view_v, view_cap_tokens, n_sel, scale, out, lse, workspace,
                                  (cudaStream_t)stream, sel_ids, sel_stride, session_first, nullptr, rope_first_position);
    if (e != cudaSuccess) return cuda_fail("fused materialize+attend kernel launch", e);
    return KVMEM_OK;
}

int kvmem_materialize_attend(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                             const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v,
                             int32_t view_cap_tokens, float scale, float* out, float* lse, void* workspace,
                             size_t workspace_bytes, void* stream) {
    return materialize_attend_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, view_k, view_v,
                                   view_cap_tokens, -1, scale, out, lse, workspace, workspace_bytes, stream);
}

int kvmem_materialize_attend_rope(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                  const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, void* view_k, void* view_v,
                                  int32_t view_cap_tokens, int32_t first_position, float scale, float* out, float* lse,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
    if (sel_stride < 1 || view_cap_tokens < 1) { set_error("sel_stride and view_cap_tokens must be positive"); return KVMEM_E_INVALID; }
    const int64_t last = (int64_t)first_position + std::min<int64_t>((int64_t)sel_stride * p->cfg.block_tokens, view_cap_tokens);
    if (first_position < 0 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last,
                  p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    // One pass either way: on the in-block layout every K tile is rotated by its block position on its way through shared
    // memory; raw keys are rotated by the consumer warps on their way to the tensor cores and handed back for the store.
    // The pass walks whole 64-token tiles and fetches rotary rows up to the 49th position of the last one (the bound is
    // kept at the whole tile).
    if (!p->cfg.rope_in_block_keys) {
        const int64_t tiles_end = (int64_t)first_position + (std::min<int64_t>((int64_t)sel_stride * p->cfg.block_tokens, view_cap_tokens) + 63) / 64 * 64;
        if (tiles_end > p->cfg.rope_max_positions) {
            set_error("the last 64-token tile of the view reaches position %lld, outside the rotary table [0, %d)", (long long)tiles_end,
                      p->cfg.rope_max_positions);
            return KVMEM_E_INVALID;
        }
    }
    return materialize_attend_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, view_k, view_v,
                                   view_cap_tokens, first_position, scale, out, lse, workspace, workspace_bytes, stream);
}

static int paged_attend_impl(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                             const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, int32_t rope_first_position,
                             float scale, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p) || !pages_are(p, false, "kvmem_paged_attend")) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!q || !sel_ids || !n_sel || !out || !lse || !workspace || !aligned(q, 16) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_paged_attend: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1 || sel_stride < 1) { set_error("n_q_tokens and sel_stride must be positive"); return KVMEM_E_INVALID; }
    if (!paged_block_size_ok(p, false, "kvmem_paged_attend")) return KVMEM_E_UNSUPPORTED;     // the query-rotating mode handles every block size too
    if (n_q_tokens * p->geo.r > (rope_first_position >= 0 ? 16 : 64)) { set_error("n_q_tokens * (H/G) = %d exceeds %d rows per call", n_q_tokens * p->geo.r, rope_first_position >= 0 ? 16 : 64); return KVMEM_E_UNSUPPORTED; }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    if ((int64_t)p->cfg.max_blocks * 2 * p->cfg.n_layers * p->cfg.n_kv_heads * p->cfg.block_tokens > 0x7fffffffll) {
        set_error("page pool too large for 32-bit TMA row coordinates");
        return KVMEM_E_UNSUPPORTED;
    }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    // the "view" is only virtual here: its length bound is sel_stride blocks
    const int64_t cap_tokens = (int64_t)sel_stride * p->cfg.block_tokens;
    if (cap_tokens > 0x7fffffffll) { set_error("sel_stride too large"); return KVMEM_E_INVALID; }
    cudaError_t e = launch_attend(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, nullptr, nullptr, (int)cap_tokens, n_sel,
                                  scale, out, lse, workspace, (cudaStream_t)stream, sel_ids, sel_stride, session_first, nullptr,
                                  rope_first_position);
    if (e != cudaSuccess) return cuda_fail("paged attention kernel launch", e);
    return KVMEM_OK;
}

int kvmem_paged_attend(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                       const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, float scale, float* out, float* lse,
                       void* workspace, size_t workspace_bytes, void* stream) {
    return paged_attend_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, -1, scale, out, lse,
                             workspace, workspace_bytes, stream);
}

int kvmem_paged_attend_rope(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                            const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, int32_t first_position,
                            float scale, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
    // the pass walks whole 64-token tiles: the last tile fetches rotary rows up to its 49th position (bound kept at the whole tile)
    const int64_t last = (int64_t)first_position + ((int64_t)sel_stride * p->cfg.block_tokens + 63) / 64 * 64;
    if (first_position < 0 || sel_stride < 1 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last,
                  p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    return paged_attend_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, first_position, scale, out,
                             lse, workspace, workspace_bytes, stream);
}

int kvmem_working_set_delta(kvmem_pool_t* p, int32_t n_sessions, const int32_t* prev_ids, const int32_t* n_prev,
                            const int32_t* next_ids, const int32_t* n_next, int32_t stride, int32_t* retained,
                            int32_t* incoming, int32_t* outgoing, int32_t* counts, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (n_sessions < 1 || stride < 1 || !prev_ids || !n_prev || !next_ids || !n_next || !retained || !incoming || !outgoing ||
        !counts) {
        set_error("kvmem_working_set_delta: null pointer or non-positive size");
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_working_set_delta(*p, n_sessions, prev_ids, n_prev, next_ids, n_next, stride, retained, incoming,
                                             outgoing, counts, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("working-set delta kernel launch", e);
    return KVMEM_OK;
}

// ---- FP8 execution view ----

static int fp8_common_ok(kvmem_pool_t* p, int32_t view_cap_tokens, float k_scale, float v_scale, const char* who) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.head_dim != 128 || p->cfg.block_tokens != 64) {
        set_error("%s: the FP8 view kernels are built for head_dim 128 and 64-token blocks", who);
        return KVMEM_E_UNSUPPORTED;
    }
    if (view_cap_tokens < 64 || view_cap_tokens % 64 != 0) { set_error("%s: view_cap_tokens must be a positive multiple of 64", who); return KVMEM_E_INVALID; }
    if (!(k_scale > 0.0f) || !(v_scale > 0.0f) || !std::isfinite(k_scale) || !std::isfinite(v_scale)) {
        set_error("%s: scales must be positive and finite", who);
        return KVMEM_E_INVALID;
    }
    return KVMEM_OK;
}

int kvmem_materialize_fp8(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids, int32_t sel_stride,
                          const int32_t* n_sel, void* view_k8, void* view_v8t, int32_t view_cap_tokens, float k_scale,
                          float v_scale, void* stream) {
    const int rc = fp8_common_ok(p, view_cap_tokens, k_scale, v_scale, "kvmem_materialize_fp8");
    if (rc != KVMEM_OK) return rc;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!sel_ids || !n_sel || !view_k8 || !view_v8t || !aligned(view_k8, 128) || !aligned(view_v8t, 128) || sel_stride < 1) {
        set_error("kvmem_materialize_fp8: null or misaligned pointer (views need 128-byte alignment), or sel_stride < 1");
        return KVMEM_E_INVALID;
    }
    if (p->cfg.fp8_pages && (k_scale != p->cfg.fp8_k_scale || v_scale != p->cfg.fp8_v_scale)) {
        set_error("kvmem_materialize_fp8: the pool's pages were quantised with scales %g / %g, not %g / %g", p->cfg.fp8_k_scale,
                  p->cfg.fp8_v_scale, k_scale, v_scale);
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_gather_fp8(*p, session_first, n_sessions, sel_ids, sel_stride, n_sel, (uint8_t*)view_k8,
                                      (uint8_t*)view_v8t, view_cap_tokens, k_scale, v_scale, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("FP8 gather kernel launch", e);
    return KVMEM_OK;
}

int kvmem_materialize_fp8_rope(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const int32_t* sel_ids, int32_t sel_stride,
                               const int32_t* n_sel, void* view_k8, void* view_v8t, int32_t view_cap_tokens, int32_t first_position,
                               float k_scale, float v_scale, void* stream) {
    const int rc = fp8_common_ok(p, view_cap_tokens, k_scale, v_scale, "kvmem_materialize_fp8_rope");
    if (rc != KVMEM_OK) return rc;
    if (!pages_are(p, false, "kvmem_materialize_fp8_rope")) return KVMEM_E_STATE;
    if (p->cfg.rope_max_positions <= 0) { set_error("the pool was created without rotary support"); return KVMEM_E_STATE; }
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!sel_ids || !n_sel || !view_k8 || !view_v8t || !aligned(view_k8, 128) || !aligned(view_v8t, 128) || sel_stride < 1) {
        set_error("kvmem_materialize_fp8_rope: null or misaligned pointer (views need 128-byte alignment), or sel_stride < 1");
        return KVMEM_E_INVALID;
    }
    const int64_t last = (int64_t)first_position + std::min<int64_t>((int64_t)sel_stride * 64, view_cap_tokens);
    if (first_position < 0 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last, p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    cudaError_t e = launch_gather_fp8(*p, session_first, n_sessions, sel_ids, sel_stride, n_sel, (uint8_t*)view_k8,
                                      (uint8_t*)view_v8t, view_cap_tokens, k_scale, v_scale, (cudaStream_t)stream, first_position);
    if (e != cudaSuccess) return cuda_fail("rotating FP8 gather kernel launch", e);
    return KVMEM_OK;
}

int kvmem_view_attend_fp8(kvmem_pool_t* p, int32_t n_sessions, const void* q, int32_t n_q_tokens, const void* view_k8,
                          const void* view_v8t, int32_t view_cap_tokens, const int32_t* n_sel, float scale, float k_scale,
                          float v_scale, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = fp8_common_ok(p, view_cap_tokens, k_scale, v_scale, "kvmem_view_attend_fp8");
    if (rc != KVMEM_OK) return rc;
    if (n_sessions < 1 || n_q_tokens < 1) { set_error("n_sessions and n_q_tokens must be positive"); return KVMEM_E_INVALID; }
    if (!q || !view_k8 || !view_v8t || !n_sel || !out || !lse || !workspace || !aligned(q, 16) || !aligned(view_k8, 128) ||
        !aligned(view_v8t, 128) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_view_attend_fp8: null or misaligned pointer (views need 128-byte alignment)");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens * p->geo.r > 16) { set_error("n_q_tokens * (H/G) = %d exceeds 16 rows per call", n_q_tokens * p->geo.r); return KVMEM_E_UNSUPPORTED; }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    if ((int64_t)n_sessions * p->cfg.n_layers * p->cfg.n_kv_heads * view_cap_tokens > 0x7fffffffll) {
        set_error("view too large for 32-bit TMA row coordinates");
        return KVMEM_E_UNSUPPORTED;
    }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_attend_fp8(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, (const uint8_t*)view_k8,
                                      (const uint8_t*)view_v8t, view_cap_tokens, n_sel, scale, k_scale, v_scale, out, lse,
                                      workspace, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("FP8 attention kernel launch", e);
    return KVMEM_OK;
}

static int paged_attend_fp8_impl(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                 const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, int32_t rope_first_position,
                                 float scale, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p) || !pages_are(p, true, "kvmem_paged_attend_fp8")) return KVMEM_E_STATE;
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    if (!q || !sel_ids || !n_sel || !out || !lse || !workspace || !aligned(q, 16) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_paged_attend_fp8: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1 || sel_stride < 1) { set_error("n_q_tokens and sel_stride must be positive"); return KVMEM_E_INVALID; }
    if (n_q_tokens * p->geo.r > 16) { set_error("n_q_tokens * (H/G) = %d exceeds 16 rows per call", n_q_tokens * p->geo.r); return KVMEM_E_UNSUPPORTED; }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    if ((int64_t)p->cfg.max_blocks * 2 * p->cfg.n_layers * p->cfg.n_kv_heads * 64 > 0x7fffffffll) {
        set_error("page pool too large for 32-bit TMA row coordinates");
        return KVMEM_E_UNSUPPORTED;
    }
    if ((int64_t)sel_stride * 64 > 0x7fffffffll) { set_error("sel_stride too large"); return KVMEM_E_INVALID; }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_attend_fp8(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, nullptr, nullptr, sel_stride * 64, n_sel,
                                      scale, p->cfg.fp8_k_scale, p->cfg.fp8_v_scale, out, lse, workspace, (cudaStream_t)stream,
                                      sel_ids, sel_stride, session_first, rope_first_position);
    if (e != cudaSuccess) return cuda_fail("paged FP8 attention kernel launch", e);
    return KVMEM_OK;
}

int kvmem_paged_attend_fp8(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                           const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, float scale, float* out, float* lse,
                           void* workspace, size_t workspace_bytes, void* stream) {
    return paged_attend_fp8_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, -1, scale, out, lse,
                                 workspace, workspace_bytes, stream);
}

int kvmem_paged_attend_fp8_rope(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, int32_t first_position,
                                float scale, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!p->cfg.fp8_pages || !p->cfg.rope_in_block_keys) {
        set_error("kvmem_paged_attend_fp8_rope needs a pool with fp8_pages and rope_in_block_keys");
        return KVMEM_E_STATE;
    }
    const int64_t last = (int64_t)first_position + (int64_t)sel_stride * p->cfg.block_tokens;
    if (first_position < 0 || sel_stride < 1 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last,
                  p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    return paged_attend_fp8_impl(p, session_first, n_sessions, q, n_q_tokens, sel_ids, sel_stride, n_sel, first_position, scale,
                                 out, lse, workspace, workspace_bytes, stream);
}

int kvmem_materialize_attend_fp8(kvmem_pool_t* p, int32_t session_first, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                 const int32_t* sel_ids, int32_t sel_stride, const int32_t* n_sel, void* view_k8, void* view_v8t,
                                 int32_t view_cap_tokens, float scale, float* out, float* lse, void* workspace,
                                 size_t workspace_bytes, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.head_dim != 128 || p->cfg.block_tokens != 64) {
        set_error("kvmem_materialize_attend_fp8: the FP8 view kernels are built for head_dim 128 and 64-token blocks");
        return KVMEM_E_UNSUPPORTED;
    }
    if (!sessions_ok(p, session_first, n_sessions)) return KVMEM_E_INVALID;
    // a bf16 repository is quantised on the way with the pool's scales, 1 where the configuration leaves them unset
    const float k_scale = p->cfg.fp8_k_scale > 0.0f && std::isfinite(p->cfg.fp8_k_scale) ? p->cfg.fp8_k_scale : 1.0f;
    const float v_scale = p->cfg.fp8_v_scale > 0.0f && std::isfinite(p->cfg.fp8_v_scale) ? p->cfg.fp8_v_scale : 1.0f;
    if (!q || !sel_ids || !n_sel || !view_k8 || !view_v8t || !out || !lse || !workspace || !aligned(q, 16) || !aligned(view_k8, 128) ||
        !aligned(view_v8t, 128) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_materialize_attend_fp8: null or misaligned pointer (views need 128-byte alignment)");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1 || sel_stride < 1) { set_error("n_q_tokens and sel_stride must be positive"); return KVMEM_E_INVALID; }
    if (view_cap_tokens < 64 || view_cap_tokens % 64 != 0) { set_error("view_cap_tokens must be a positive multiple of 64"); return KVMEM_E_INVALID; }
    if (n_q_tokens * p->geo.r > 16) { set_error("n_q_tokens * (H/G) = %d exceeds 16 rows per call", n_q_tokens * p->geo.r); return KVMEM_E_UNSUPPORTED; }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    if ((int64_t)p->cfg.max_blocks * 2 * p->cfg.n_layers * p->cfg.n_kv_heads * 64 > 0x7fffffffll ||
        (int64_t)n_sessions * p->cfg.n_layers * p->cfg.n_kv_heads * view_cap_tokens > 0x7fffffffll) {
        set_error("page pool or view too large for 32-bit TMA row coordinates");
        return KVMEM_E_UNSUPPORTED;
    }
    AttendPlan plan = plan_attend(p->cfg, n_sessions, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    cudaError_t e = launch_attend_fp8(*p, n_sessions, (const __nv_bfloat16*)q, n_q_tokens, (const uint8_t*)view_k8,
                                      (const uint8_t*)view_v8t, view_cap_tokens, n_sel, scale, k_scale, v_scale,
                                      out, lse, workspace, (cudaStream_t)stream, sel_ids, sel_stride, session_first);
    if (e != cudaSuccess) return cuda_fail("fused FP8 materialize+attend kernel launch", e);
    return KVMEM_OK;
}

// ---- execution cache: working-set reuse with bounded delta re-RoPE ----

static int cache_ok(kvmem_pool_t* p, const void* cache, size_t cache_bytes, int32_t cap_blocks, const char* who) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (p->cfg.rope_max_positions <= 0) { set_error("%s: the pool was created without rotary support", who); return KVMEM_E_STATE; }
    if (cap_blocks < 1 || cap_blocks > 32768) { set_error("%s: cap_blocks must be in [1, 32768]", who); return KVMEM_E_INVALID; }
    if (!cache || !aligned(cache, 256)) { set_error("%s: cache is null or not 256-byte aligned", who); return KVMEM_E_INVALID; }
    const size_t need = cache_layout(p->lay.page_elems, cap_blocks).total;
    if (cache_bytes < need) { set_error("%s: cache holds %zu bytes, %zu needed", who, cache_bytes, need); return KVMEM_E_CAPACITY; }
    return KVMEM_OK;
}

size_t kvmem_view_cache_bytes(const kvmem_pool_t* p, int32_t cap_blocks) {
    if (!p || cap_blocks < 1 || cap_blocks > 32768) return 0;
    return cache_layout(p->lay.page_elems, cap_blocks).total;
}

int kvmem_view_cache_layout(const kvmem_pool_t* p, int32_t cap_blocks, size_t* offsets) {
    if (!p || !offsets || cap_blocks < 1 || cap_blocks > 32768) { set_error("kvmem_view_cache_layout: bad argument"); return KVMEM_E_INVALID; }
    const CacheLayout c = cache_layout(p->lay.page_elems, cap_blocks);
    offsets[0] = c.pages; offsets[1] = c.slot_block; offsets[2] = c.slot_pos; offsets[3] = c.slot_cnt;
    offsets[4] = c.view_slots; offsets[5] = c.n_view;
    return KVMEM_OK;
}

int kvmem_view_cache_reset(kvmem_pool_t* p, void* cache, size_t cache_bytes, int32_t cap_blocks, void* stream) {
    const int rc = cache_ok(p, cache, cache_bytes, cap_blocks, "kvmem_view_cache_reset");
    if (rc != KVMEM_OK) return rc;
    cudaError_t e = launch_view_cache_reset(*p, cache, cap_blocks, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("execution-cache reset kernel launch", e);
    return KVMEM_OK;
}

int kvmem_view_cache_update(kvmem_pool_t* p, int32_t session, const int32_t* sel_ids, const int32_t* n_sel, void* cache,
                            size_t cache_bytes, int32_t cap_blocks, int32_t max_delta_ropes, int32_t first_position,
                            int32_t* stats, void* stream) {
    const int rc = cache_ok(p, cache, cache_bytes, cap_blocks, "kvmem_view_cache_update");
    if (rc != KVMEM_OK) return rc;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    if (!sel_ids || !n_sel) { set_error("kvmem_view_cache_update: null pointer"); return KVMEM_E_INVALID; }
    if (max_delta_ropes < 0) { set_error("max_delta_ropes must be non-negative"); return KVMEM_E_INVALID; }
    const int64_t last = (int64_t)first_position + (int64_t)cap_blocks * p->cfg.block_tokens;
    if (first_position < 0 || last > p->cfg.rope_max_positions) {
        set_error("compact positions [%d, %lld) outside the rotary table [0, %d)", first_position, (long long)last,
                  p->cfg.rope_max_positions);
        return KVMEM_E_INVALID;
    }
    if (p->cfg.head_dim % 16 != 0) { set_error("rotary kernels need head_dim to be a multiple of 16"); return KVMEM_E_UNSUPPORTED; }
    cudaError_t e = launch_view_cache_update(*p, session, sel_ids, n_sel, cache, cap_blocks, max_delta_ropes, first_position,
                                             stats, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail("execution-cache update kernel launch", e);
    return KVMEM_OK;
}

int kvmem_view_cache_attend(kvmem_pool_t* p, const void* q, int32_t n_q_tokens, void* cache, size_t cache_bytes,
                            int32_t cap_blocks, float scale, float* out, float* lse, void* workspace, size_t workspace_bytes,
                            void* stream) {
    const int rc = cache_ok(p, cache, cache_bytes, cap_blocks, "kvmem_view_cache_attend");
    if (rc != KVMEM_OK) return rc;
    if (!q || !out || !lse || !workspace || !aligned(q, 16) || !aligned(workspace, 256) || !aligned(out, 16)) {
        set_error("kvmem_view_cache_attend: null or misaligned pointer");
        return KVMEM_E_INVALID;
    }
    if (n_q_tokens < 1) { set_error("n_q_tokens must be positive"); return KVMEM_E_INVALID; }
    if (!paged_block_size_ok(p, false, "kvmem_view_cache_attend")) return KVMEM_E_UNSUPPORTED;
    if (n_q_tokens * p->geo.r > 64) { set_error("n_q_tokens * (H/G) = %d exceeds 64 rows per call", n_q_tokens * p->geo.r); return KVMEM_E_UNSUPPORTED; }
    if (!(scale >= 0.0f)) { set_error("scale must be non-negative (0 selects 1/sqrt(d))"); return KVMEM_E_INVALID; }
    AttendPlan plan = plan_attend(p->cfg, 1, n_q_tokens, p->sm_count);
    if (workspace_bytes < plan.total) { set_error("attend workspace holds %zu bytes, %zu needed", workspace_bytes, plan.total); return KVMEM_E_CAPACITY; }
    PagedSource src{};
    view_cache_paged_source(*p, cache, cap_blocks, &src);
    const int64_t cap_tokens = (int64_t)cap_blocks * p->cfg.block_tokens;
    cudaError_t e = launch_attend(*p, 1, (const __nv_bfloat16*)q, n_q_tokens, nullptr, nullptr, (int)cap_tokens, src.n_sel, scale,
                                  out, lse, workspace, (cudaStream_t)stream, src.sel_ids, cap_blocks, 0, &src);
    if (e != cudaSuccess) return cuda_fail("execution-cache attention kernel launch", e);
    return KVMEM_OK;
}

int kvmem_get_index(kvmem_pool_t* p, int32_t session, const void** index, int32_t* n_blocks) {
    if (!pool_ok(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    if (!index || !n_blocks) { set_error("null output pointer"); return KVMEM_E_INVALID; }
    *index = p->index + (size_t)session * p->lay.index_elems_per_session;
    *n_blocks = p->sess_blocks[session];
    return KVMEM_OK;
}

int kvmem_get_block_table(kvmem_pool_t* p, int32_t session, const int32_t** table, int32_t* n_blocks) {
    if (!pool_ok(p)) return KVMEM_E_STATE;
    if (!sessions_ok(p, session, 1)) return KVMEM_E_INVALID;
    if (!table || !n_blocks) { set_error("null output pointer"); return KVMEM_E_INVALID; }
    *table = p->tables + (size_t)session * p->cfg.max_blocks_per_session;
    *n_blocks = p->sess_blocks[session];
    return KVMEM_OK;
}

int kvmem_device_status(kvmem_pool_t* p, int32_t* status, void* stream) {
    if (!pool_live(p)) return KVMEM_E_STATE;
    if (!status) { set_error("status is null"); return KVMEM_E_INVALID; }
    cudaStream_t st = (cudaStream_t)stream;
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, p->status_dev, 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(p->status_dev, 0, 4, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail("reading the device status word", e);
    *status = word;
    return KVMEM_OK;
}

}  // extern "C"
