// FP8 (E4M3) execution view (the paper's evaluation keeps the KV cache in FP8, Sec. 6.1): assembly of
// the view with quantisation on the way, and split-K decode attention over it.
//
// A stored element is the E4M3 code of x * inv_scale (one fp32 product, round to nearest even,
// saturating at +-448), one static scale per tensor.  Layout: keys [heads][cap_tokens][128] bytes; values
// transposed inside every 64-token tile, [heads][cap_tokens / 64][128][64] bytes, so that both
// operands of the two attention contractions are read along their contraction index with plain
// ldmatrix loads: a 32-bit ldmatrix register then holds four consecutive elements of the contraction
// index, which two cvt instructions turn into the two f16x2 registers of an m16n8k16 B fragment.  The
// k-slots of the MMA are a permutation of the contraction index that the A fragments (the query for
// Q K^T, the probabilities for P V) follow, so no data is shuffled.
#include <cuda_fp8.h>
#include <cudaTypedefs.h>
#include <math.h>

#include <algorithm>

#include "kvmem_internal.cuh"
#include "kvmem_ptx.cuh"
#include "kvmem_rope.cuh"

namespace kvmem {

constexpr int kF8Tile = 64;                      // tokens per tile == block_tokens on this path
constexpr int kF8D = 128;

// UNIT: the scale is 1 and the multiplication by its inverse is left out (x * 1 is x: the same codes)
template <bool UNIT = false>
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, float inv) {
    if (!UNIT) { a = __fmul_rn(a, inv); b = __fmul_rn(b, inv); c = __fmul_rn(c, inv); d = __fmul_rn(d, inv); }
    const __nv_fp8x2_storage_t lo = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t hi = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
    return (uint32_t)lo | ((uint32_t)hi << 16);
}

// 8 bf16 (one 128-bit load) -> 8 E4M3 bytes
template <bool UNIT = false>
__device__ __forceinline__ uint2 quant8(const uint4& v, float inv) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
    return make_uint2(quant4<UNIT>(f[0], f[1], f[2], f[3], inv), quant4<UNIT>(f[4], f[5], f[6], f[7], inv));
}

struct GatherF8Args {
    const __nv_bfloat16* pages;
    const int32_t* tables;
    const int32_t* nblocks_dev;
    const int32_t* sel_ids;
    const int32_t* n_sel;
    uint8_t* view_k;
    uint8_t* view_v;
    int32_t* status;
    int session_first, sel_stride, max_bps, max_blocks, LG, cap_tokens;
    float k_inv_scale, v_inv_scale;
    size_t page_elems;
    // position-consistent view: keys are rotated to compact position first_position + j*64 + t before they are quantised
    const float2* rope;          // null: keys quantised as stored
    int first_position, rope_positions, in_block;
};

// One CTA pass = one (selected block, layer x KV head): the K tile is quantised straight through, the V
// tile goes through shared memory to come out transposed.  HBM: 2 bytes read + 1 byte written per element.
constexpr int kF8Pitch = kF8D + 4;               // bytes per token row of the staging buffer (33 words: conflict-free columns)
// (The rotating form is held to 64 registers: four CTAs per SM instead of three.  It is bound by the latency of its loads,
// not by its arithmetic: 322 -> 289 us at a 1M-token history; five CTAs at 48 registers spill and take 311 us.)
template <bool ROPE>
__global__ void __launch_bounds__(256, ROPE ? 4 : 8)
gather_fp8_kernel(GatherF8Args a) {
    pdl_wait();
    __shared__ __align__(16) uint8_t sv[kF8Tile * kF8Pitch];
    const int s = blockIdx.y;
    const int NB = a.nblocks_dev[a.session_first + s];
    int n_blk = a.n_sel[s];
    const int cap_blocks = a.cap_tokens / kF8Tile;
    if (n_blk > a.sel_stride || n_blk > cap_blocks) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE);
        n_blk = min(min(n_blk, a.sel_stride), cap_blocks);
    }
    n_blk = max(n_blk, 0);
    // ROPE: an item is a whole selected block and the (layer, KV head) tiles are walked inside it, so that the rotary rows
    // of the block's 64 positions are fetched once and serve every head
    const int inner = ROPE ? a.LG : 1;
    const long long n_items = ROPE ? (long long)n_blk : (long long)n_blk * a.LG;
    const int tile_elems = kF8Tile * kF8D;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int j = ROPE ? (int)item : (int)(item / a.LG);
        float4 cs[2][4];
        if (ROPE) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int it2 = threadIdx.x + 256 * h, tok = it2 >> 3, c = it2 & 7;
                int pos = a.first_position + j * kF8Tile + (a.in_block ? 0 : tok);
                if (pos < 0 || pos >= a.rope_positions) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); pos = 0; }
                const float4* cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)pos * (kF8D / 2) + c * 8);
#pragma unroll
                for (int w = 0; w < 4; ++w) cs[h][w] = __ldg(cs4 + w);
            }
        }
        for (int in = 0; in < inner; ++in) {
        const int lg = ROPE ? in : (int)(item % a.LG);
        const int id = a.sel_ids[(size_t)s * a.sel_stride + j];
        int page = -1;
        if (id >= 0 && id < NB) page = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
        if (page < 0 || page >= a.max_blocks) { if (threadIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); break; }
        const __nv_bfloat16* ksrc = a.pages + (size_t)page * a.page_elems + (size_t)lg * tile_elems;
        const __nv_bfloat16* vsrc = ksrc + (size_t)a.LG * tile_elems;
        const size_t head = (size_t)s * a.LG + lg;
        uint8_t* kdst = a.view_k + (head * a.cap_tokens + (size_t)j * kF8Tile) * kF8D;
        uint8_t* vdst = a.view_v + (head * cap_blocks + (size_t)j) * (size_t)tile_elems;
        // 1,024 groups of 8 elements per tile: 4 per thread
        uint4 kv[4], vv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = threadIdx.x + 256 * i;
            // ROPE: a thread takes the low-half group (token, c) and its partner (token, c + 8) of the high half, which
            // rotate together: groups 2 i and 2 i + 1 of the four are one such pair
            const int ek = ROPE ? ((threadIdx.x + 256 * (i >> 1)) >> 3) * 16 + ((threadIdx.x + 256 * (i >> 1)) & 7) + 8 * (i & 1) : e;
            kv[i] = __ldg(reinterpret_cast<const uint4*>(ksrc) + ek);
            vv[i] = __ldg(reinterpret_cast<const uint4*>(vsrc) + e);
        }
        if (ROPE) {
            // RoPE at the compact position (arithmetic of kvmem_rope_rotate: fp32 products and sums, one rounding to bf16),
            // then the quantisation of the rotated bf16 key: the code of the position-consistent view's element
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint4 lo_o, hi_o;
                rotate8_cs(kv[2 * h], kv[2 * h + 1], cs[h], 1.0f, lo_o, hi_o);
                kv[2 * h] = lo_o; kv[2 * h + 1] = hi_o;
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = threadIdx.x + 256 * i;                  // token e / 16, dims 8 * (e % 16) ..
            const int ek = ROPE ? ((threadIdx.x + 256 * (i >> 1)) >> 3) * 16 + ((threadIdx.x + 256 * (i >> 1)) & 7) + 8 * (i & 1) : e;
            *reinterpret_cast<uint2*>(kdst + (size_t)ek * 8) = quant8(kv[i], a.k_inv_scale);
            const uint2 q = quant8(vv[i], a.v_inv_scale);
            uint32_t* row = reinterpret_cast<uint32_t*>(sv + (e >> 4) * kF8Pitch + (e & 15) * 8);
            row[0] = q.x; row[1] = q.y;
        }
        __syncthreads();
        // transposed store: 512 pieces of 16 tokens of one dimension, 2 per thread
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int pce = threadIdx.x + 256 * i;
            const int dim = pce >> 2, tg = pce & 3;
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t x = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) x |= (uint32_t)sv[(tg * 16 + k * 4 + b) * kF8Pitch + dim] << (8 * b);
                w[k] = x;
            }
            *reinterpret_cast<uint4*>(vdst + (size_t)dim * kF8Tile + tg * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        __syncthreads();
        }       // tiles of the item
    }
}

// ---------------------------------------------------------------------------------------------------
// FP8 repository (pool created with fp8_pages): the pages hold the tiles of the FP8 view, so the append
// quantises once (K straight, V transposed through shared memory, the same arithmetic as above), builds the
// Mean-K entry from the bf16 keys it was given (Eq. "mean_k_index": fp32 sum in ascending token order, one
// rounding to bf16), and every later pass moves one byte per element.
__global__ void __launch_bounds__(256)
append_fp8_kernel(const __nv_bfloat16* __restrict__ k_in, const __nv_bfloat16* __restrict__ v_in, uint8_t* __restrict__ pages8,
                  __nv_bfloat16* __restrict__ index_sess, const int32_t* __restrict__ table_sess, int32_t* __restrict__ status,
                  int b_first, int L, int G, int max_blocks, int max_bps, size_t page_bytes, float k_inv_scale, float v_inv_scale,
                  const int32_t* __restrict__ pos0_sess, const float2* __restrict__ rope, int rope_positions, int in_block) {
    __shared__ __align__(16) __nv_bfloat16 ktile[kF8Tile * kF8D];      // the bf16 keys: index entry, rotary steps, then quantised
    __shared__ __align__(16) uint8_t sv[kF8Tile * kF8Pitch];
    const int i = blockIdx.x, lg = blockIdx.y, LG = L * G;
    const int page = table_sess[b_first + i];
    if (page < 0 || page >= max_blocks) {
        if (threadIdx.x == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        return;
    }
    const size_t row_stride = (size_t)LG * kF8D;                       // elements between consecutive tokens of the input
    const __nv_bfloat16* ksrc = k_in + (size_t)i * kF8Tile * row_stride + (size_t)lg * kF8D;
    const __nv_bfloat16* vsrc = v_in + (size_t)i * kF8Tile * row_stride + (size_t)lg * kF8D;
    uint8_t* kdst = pages8 + (size_t)page * page_bytes + (size_t)lg * (kF8Tile * kF8D);
    uint8_t* vdst = kdst + (size_t)LG * (kF8Tile * kF8D);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int e = threadIdx.x + 256 * it;                          // token e / 16, dims 8 * (e % 16) ..
        const int t = e >> 4, j = e & 15;
        *reinterpret_cast<uint4*>(ktile + (size_t)e * 8) = *reinterpret_cast<const uint4*>(ksrc + (size_t)t * row_stride + j * 8);
        const uint4 vv = *reinterpret_cast<const uint4*>(vsrc + (size_t)t * row_stride + j * 8);
        const uint2 q = quant8(vv, v_inv_scale);
        uint32_t* row = reinterpret_cast<uint32_t*>(sv + t * kF8Pitch + j * 8);
        row[0] = q.x; row[1] = q.y;
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < 2; ++it) {                                    // transposed store: 16 tokens of one dimension per piece
        const int pce = threadIdx.x + 256 * it;
        const int dim = pce >> 2, tg = pce & 3;
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t x = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) x |= (uint32_t)sv[(tg * 16 + k * 4 + b) * kF8Pitch + dim] << (8 * b);
            w[k] = x;
        }
        *reinterpret_cast<uint4*>(vdst + (size_t)dim * kF8Tile + tg * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    constexpr int half = kF8D / 2;
    if (pos0_sess) {
        // the keys still carry RoPE of positions pos0 + t: rotate back (Sec. 4.3); the arithmetic of a rotated element
        // (fp32 products and sums without fused multiply-add, one rounding to bf16)
        const int pos0 = pos0_sess[b_first + i];
        for (int e = threadIdx.x; e < kF8Tile * half; e += 256) {
            const int t = e / half, x = e % half, pos = pos0 + t;
            if (pos < 0 || pos >= rope_positions) { atomicExch(status, (int)KVMEM_E_DEVICE_RANGE); continue; }
            const float2 cs = rope[(size_t)pos * half + x];
            const float a = __bfloat162float(ktile[t * kF8D + x]), b = __bfloat162float(ktile[t * kF8D + x + half]);
            ktile[t * kF8D + x] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(a, cs.x), __fmul_rn(b, cs.y)));
            ktile[t * kF8D + x + half] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(b, cs.x), __fmul_rn(a, cs.y)));
        }
        __syncthreads();
    }
    // the index entry comes from the raw bf16 keys (position-independent, Sec. 4.3)
    const float inv = 1.0f / (float)kF8Tile;
    __nv_bfloat16* idx_row = index_sess + ((size_t)lg * max_bps + (size_t)(b_first + i)) * kF8D;
    if (threadIdx.x < kF8D) {
        const int c = threadIdx.x;
        float acc = 0.0f;
        for (int t = 0; t < kF8Tile; ++t) acc = __fadd_rn(acc, __bfloat162float(ktile[(size_t)t * kF8D + c]));
        idx_row[c] = __float2bfloat16_rn(__fmul_rn(acc, inv));
    }
    if (in_block) {
        // in-block layout: the page holds the codes of bf16(RoPE(k, t)), t the offset inside the block
        __syncthreads();
        for (int e = threadIdx.x; e < kF8Tile * half; e += 256) {
            const int t = e / half, x = e % half;
            const float2 cs = rope[(size_t)t * half + x];
            const float a = __bfloat162float(ktile[t * kF8D + x]), b = __bfloat162float(ktile[t * kF8D + x + half]);
            ktile[t * kF8D + x] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(a, cs.x), __fmul_rn(b, cs.y)));
            ktile[t * kF8D + x + half] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(b, cs.x), __fmul_rn(a, cs.y)));
        }
        __syncthreads();
    }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int e = threadIdx.x + 256 * it;
        *reinterpret_cast<uint2*>(kdst + (size_t)e * 8) = quant8(*reinterpret_cast<const uint4*>(ktile + (size_t)e * 8), k_inv_scale);
    }
}

cudaError_t launch_append_fp8(const kvmem_pool& p, int session, int b_first, int n_blocks, const __nv_bfloat16* k,
                              const __nv_bfloat16* v, cudaStream_t st, bool derope) {
    const Geometry& g = p.geo;
    const int32_t* table = p.tables + (size_t)session * g.max_bps;
    __nv_bfloat16* index = p.index + (size_t)session * p.lay.index_elems_per_session;
    dim3 grid((unsigned)n_blocks, (unsigned)(g.L * g.G));
    append_fp8_kernel<<<grid, 256, 0, st>>>(k, v, reinterpret_cast<uint8_t*>(p.pages), index, table, p.status_dev, b_first, g.L, g.G,
                                            g.max_blocks, g.max_bps, p.lay.page_elems, 1.0f / p.cfg.fp8_k_scale,
                                            1.0f / p.cfg.fp8_v_scale, derope ? p.pos0_dev + (size_t)session * g.max_bps : nullptr,
                                            p.rope_dev, p.cfg.rope_max_positions, p.cfg.rope_in_block_keys);
    return cudaGetLastError();
}

// materialize_fp8 over an FP8 repository: the tiles are copied as they are (one 8 KiB K tile and one 8 KiB V tile
// per selected block, layer and KV head: 4 x 128-bit loads per thread in flight for each)
__global__ void __launch_bounds__(256)
gather_fp8_pages_kernel(GatherF8Args a) {
    pdl_wait();
    const int s = blockIdx.y;
    const int NB = a.nblocks_dev[a.session_first + s];
    int n_blk = a.n_sel[s];
    const int cap_blocks = a.cap_tokens / kF8Tile;
    if (n_blk > a.sel_stride || n_blk > cap_blocks) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE);
        n_blk = min(min(n_blk, a.sel_stride), cap_blocks);
    }
    n_blk = max(n_blk, 0);
    const long long n_items = (long long)n_blk * a.LG;
    const int tile_bytes = kF8Tile * kF8D;
    const uint8_t* pages8 = reinterpret_cast<const uint8_t*>(a.pages);
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int j = (int)(item / a.LG), lg = (int)(item % a.LG);
        const int id = a.sel_ids[(size_t)s * a.sel_stride + j];
        int page = -1;
        if (id >= 0 && id < NB) page = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
        if (page < 0 || page >= a.max_blocks) { if (threadIdx.x == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); continue; }
        const uint4* ksrc = reinterpret_cast<const uint4*>(pages8 + (size_t)page * a.page_elems + (size_t)lg * tile_bytes);
        const uint4* vsrc = reinterpret_cast<const uint4*>(pages8 + (size_t)page * a.page_elems + (size_t)(a.LG + lg) * tile_bytes);
        const size_t head = (size_t)s * a.LG + lg;
        uint4* kdst = reinterpret_cast<uint4*>(a.view_k + (head * a.cap_tokens + (size_t)j * kF8Tile) * kF8D);
        uint4* vdst = reinterpret_cast<uint4*>(a.view_v + (head * cap_blocks + (size_t)j) * (size_t)tile_bytes);
        uint4 kv[2], vv[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) { kv[i] = __ldg(ksrc + threadIdx.x + 256 * i); vv[i] = __ldg(vsrc + threadIdx.x + 256 * i); }
#pragma unroll
        for (int i = 0; i < 2; ++i) { kdst[threadIdx.x + 256 * i] = kv[i]; vdst[threadIdx.x + 256 * i] = vv[i]; }
    }
}

// ---------------------------------------------------------------------------------------------------
// Split-K decode attention over the FP8 view.  Same structure as the bf16 kernel (producer warp with
// TMA, two groups of four consumer warps, one partial per split, merge kernel), with 16 KiB stages
// (an 8 KiB K tile and an 8 KiB transposed V tile) and f16 tensor-core MMAs on converted fragments.
constexpr int kF8Stages = 8;
constexpr int kF8Consumers = 8;
constexpr int kF8Groups = 2;
static_assert(kF8Stages % kF8Groups == 0, "each group must own whole stages");
constexpr int kF8Threads = (kF8Consumers + 1) * 32;
constexpr int kF8TileBytes = kF8Tile * kF8D;     // 8 KiB: 64 rows of 128 bytes, for K (row = token) and V^T (row = two dims)
constexpr int kF8StageBytes = 2 * kF8TileBytes;
constexpr int kF8RowsPad = 16;
constexpr int kF8MergeStride = 136;
constexpr size_t kF8Smem = (size_t)kF8Stages * kF8StageBytes + 1024;
constexpr int kF8QrotPitch = kF8D * 2 + 32;      // bytes per rotated query row (f16): 288, so that the consumers' 64-bit reads of 4 rows cover all banks
constexpr int kF8QrotBytes = kF8RowsPad * kF8QrotPitch;
constexpr size_t kF8SmemQrot = kF8Smem + (size_t)kF8Stages * kF8QrotBytes;
constexpr int kF8QrotWarps = 3;                  // query-rotator warps; they take tiles in turn (12 warps in all: the register budget of 9)
constexpr int kF8QuantWarps = 4;                 // MODE 4: warps that turn a landed bf16 tile into the FP8 tiles of the view
constexpr int kF8BfStages = 5;                   // MODE 4: ring of bf16 tiles (K lo, K hi, V lo, V hi halves of 8 KiB) in front of
constexpr int kF8QuantStages = 4;                //         a shorter FP8 ring: what is in flight from HBM is the bf16 tiles
constexpr int kF8BfStageBytes = 4 * kF8Tile * 128;
constexpr size_t kF8SmemQuant = (size_t)kF8QuantStages * kF8StageBytes + (size_t)kF8BfStages * kF8BfStageBytes + 1024;
static_assert(kF8QuantStages % kF8Groups == 0, "each group must own whole stages");
static_assert((size_t)kF8Consumers * kF8RowsPad * kF8MergeStride * sizeof(float) <= (size_t)kF8Stages * kF8StageBytes,
              "the ring is reused for the merge of the consumer warps");

// One quantiser warp's share of a landed bf16 tile (MODE 4 of the attention kernel below): srcK / srcV are the tile's K and V
// halves in the bf16 ring, dstK / dstV the FP8 tiles of the view in the FP8 ring.
template <bool UNIT>
__device__ __forceinline__ void quantise_tile_share(const unsigned char* srcK, const unsigned char* srcV, unsigned char* dstK,
                                                    unsigned char* dstV, int qw, int lane, float k_inv, float v_inv) {
    // Both tiles carry the 128-byte swizzle of their TMA maps: the 16-byte chunk c of row r sits at chunk c ^ (r & 7).
    // K: a lane takes chunk c = lane & 7 (8 dims) of half h = (lane >> 3) & 1 of one token per step; half a warp reads
    // and writes one token's row, conflict-free.
    {
        const int c = lane & 7, h = (lane >> 3) & 1;
#pragma unroll 4
        for (int i = 0; i < kF8Tile / (2 * kF8QuantWarps); ++i) {
            const int t = i * 2 * kF8QuantWarps + qw * 2 + (lane >> 4);
            const uint4 u = *reinterpret_cast<const uint4*>(srcK + h * kF8TileBytes + t * 128 + ((c ^ (t & 7)) << 4));
            const int cc = 4 * h + (c >> 1);                                 // dims 64 h + 8 c .. are bytes 64 h + 8 c .. of the row
            *reinterpret_cast<uint2*>(dstK + t * 128 + ((cc ^ (t & 7)) << 4) + 8 * (c & 1)) = quant8<UNIT>(u, k_inv);
        }
    }
    // V: a lane takes 8 dims (chunk c of half h) of 8 consecutive tokens (group tg) and leaves, for each of the 8 dims, the
    // 8 bytes of its tokens in the transposed tile: row = dim / 2, bytes (dim & 1) * 64 + token.  The items are dealt so
    // that both sides of the transposition are conflict-free: a quarter-warp reads eight different chunks (one 128-bit
    // load each), and the sixteen 64-bit stores of half a warp fall on sixteen different bank pairs (the chunk a store
    // lands in depends on tg and on the parity of c only).
    {
        static_assert(kF8QuantWarps == 4, "the item assignment below is for four quantiser warps: 16 chunks x 8 token groups = 128 lanes");
        const int c = lane & 7, u = (lane >> 3) & 1, h = lane >> 4, tg = ((c >> 1) + 4 * u + qw) & 7;
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int t = tg * 8 + k;
            v[k] = *reinterpret_cast<const uint4*>(srcV + h * kF8TileBytes + t * 128 + ((c ^ (t & 7)) << 4));
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int dim = 64 * h + 8 * c + e, vr = dim >> 1, col = (dim & 1) * 64 + tg * 8;
            uint32_t w[2];
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                float fv[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint4& x = v[4 * kk + b];
                    const uint32_t word = (e >> 1) == 0 ? x.x : (e >> 1) == 1 ? x.y : (e >> 1) == 2 ? x.z : x.w;
                    fv[b] = (e & 1) ? __uint_as_float(word & 0xffff0000u) : __uint_as_float(word << 16);
                }
                w[kk] = quant4<UNIT>(fv[0], fv[1], fv[2], fv[3], v_inv);
            }
            *reinterpret_cast<uint2*>(dstV + vr * 128 + ((((col >> 4) ^ (vr & 7)) << 4) | (col & 15))) = make_uint2(w[0], w[1]);
        }
    }
}

struct AttendF8Args {
    const __nv_bfloat16* q;
    const int32_t* n_sel;
    float* part_o;      // [ns*LG][n_splits][16][128]
    float2* part_ml;    // [ns*LG][n_splits][16]
    int32_t* status;
    int M, L, H, G, r, rows, n_splits, cap_tokens;
    float scale_log2e;  // softmax scale * k_scale * log2(e)
    float v_scale;
    // copy-free view over an FP8 repository (attend_fp8_split_kernel<true>): tiles come from the pages through the block table
    const int32_t* sel_ids;      // [n_sessions][sel_stride]
    const int32_t* tables;       // [max_sessions][max_bps]
    const int32_t* nblocks_dev;  // [max_sessions]
    int session_first, sel_stride, max_bps, max_blocks;
    int lookahead;               // MODE 2: tiles the producer may have in flight that have not landed (0: every stage)
    float k_inv_scale, v_inv_scale;      // MODE 4: what the bf16 keys and values are multiplied by before their conversion to E4M3
    // MODE 3: the pages hold the codes of RoPE(k, offset in block); the query is rotated back per tile
    const float2* rope;          // [rope_positions][64] (cos, sin)
    int first_position, rope_positions;
};

// MODE 0: tiles come from the FP8 view (map_k, map_v).
// MODE 1: copy-free view over an FP8 repository: tiles come from the page pool (map_pages: [pages * 2 * L*G * 64 rows][128
//         bytes]) through the block table; nothing is written.
// MODE 2: MODE 1 plus a view-writer warp that stores every landed tile to the FP8 view (map_k, map_v) while the consumers
//         attend over it: materialize_fp8 + view_attend_fp8 in one pass, 1 byte read + 1 byte written per element.
// MODE 3: MODE 1 over pages whose keys are the codes of RoPE(k, t), t the offset inside the block: two extra warps, taking
//         tiles alternately, rotate the 16 query rows back by the tile's compact position p0 (q . R(p0 + t) k = (R(-p0) q) .
//         RoPE(k, t)), round them to bf16 as the definition says, widen them to f16 and leave them in a small ring of
//         shared memory from which the consumers fetch their A fragments; no key is touched.
// MODE 4: MODE 2 over a bf16 repository (kvmem_materialize_fp8 + kvmem_view_attend_fp8 in one pass, 2 bytes read + 1 byte
//         written per element): the producer brings bf16 tiles (map_pages: [pages * 2 * L*G * 64 rows][128 bf16], 64-dim
//         halves) into a ring of their own; two quantiser warps turn each landed tile into the view's FP8 tiles (K straight,
//         V transposed; arithmetic of the quantising gather) in the FP8 ring, from where the consumers attend over it and
//         the view writer stores it, exactly as in MODE 2.
template <int MODE>
__global__ void __launch_bounds__(kF8Threads + (MODE == 2 ? 32 : MODE == 3 ? 32 * kF8QrotWarps : MODE == 4 ? 32 + 32 * kF8QuantWarps : 0), 1)
attend_fp8_split_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                        const __grid_constant__ CUtensorMap map_pages, AttendF8Args a) {
    constexpr bool PAGED = MODE != 0, QUANT = MODE == 4, FUSED = MODE == 2 || QUANT, QROT = MODE == 3;
    pdl_wait();
    extern __shared__ unsigned char smem_dyn[];
    constexpr int NST = QUANT ? kF8QuantStages : kF8Stages;      // stages of the FP8 ring
    __shared__ uint64_t full_bar[kF8Stages], empty_bar[kF8Stages], q_full[kF8Stages];
    __shared__ uint64_t bf_full[kF8BfStages], bf_empty[kF8BfStages];       // MODE 4: the ring of bf16 tiles
    __shared__ float merge_m[kF8Consumers][kF8RowsPad], merge_l[kF8Consumers][kF8RowsPad];

    unsigned char* stages = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, lg = blockIdx.y, s = blockIdx.z;
    const int LG = a.L * a.G;
    const int z = s * LG + lg;
    const int l = lg / a.G, g = lg % a.G;

    const int n_blk = max(0, min(a.n_sel[s], (MODE == 1 || MODE == 3) ? a.sel_stride : FUSED ? min(a.sel_stride, a.cap_tokens / kF8Tile) : a.cap_tokens / kF8Tile));
    const int t0 = (int)((long long)n_blk * split / a.n_splits);
    const int t1 = (int)((long long)n_blk * (split + 1) / a.n_splits);
    const int n_tiles = t1 - t0;
    const int cap_tiles = a.cap_tokens / kF8Tile;

    if (tid == 0) {
        // MODE 4: a stage of the FP8 ring is full when both quantiser warps have written their share of it
        for (int i = 0; i < NST; ++i) { ptx::mbar_init(&full_bar[i], QUANT ? kF8QuantWarps : 1); ptx::mbar_init(&empty_bar[i], kF8Consumers / kF8Groups + (FUSED ? 1 : 0)); ptx::mbar_init(&q_full[i], 1); }
        for (int i = 0; i < kF8BfStages; ++i) { ptx::mbar_init(&bf_full[i], 1); ptx::mbar_init(&bf_empty[i], kF8QuantWarps); }
        ptx::fence_mbar_init();
    }
    __syncthreads();

    float o[16][4];           // O accumulators: 16 n-tiles of 8 dims
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f; }

    if (PAGED && warp == kF8Consumers) {
        // ---------------- producer over pages: the whole warp looks pages up, 32 tiles at a time; lane 0 issues the loads
        if (n_tiles > 0) {
            if (lane == 0) ptx::prefetch_tensormap(&map_pages);
            const int NB = a.nblocks_dev[a.session_first + s];
            const int ahead = MODE == 2 && a.lookahead > 0 ? min(a.lookahead, NST) : NST;
            auto lookup = [&](int it) -> int {
                if (it >= n_tiles) return 0;
                const int id = a.sel_ids[(size_t)s * a.sel_stride + t0 + it];
                int pg = -1;
                if (id >= 0 && id < NB) pg = a.tables[(size_t)(a.session_first + s) * a.max_bps + id];
                if (pg < 0 || pg >= a.max_blocks) { atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); pg = 0; }
                return pg;           // a flagged id reads page 0 instead of faulting; the status word reports it
            };
            int base_it = 0, my_page = lookup(lane);
            bool ok = true;
            for (int it = 0; it < n_tiles; ++it) {
                if (it >= base_it + 32) { base_it = it; my_page = lookup(base_it + lane); }
                const int page = __shfl_sync(0xffffffffu, my_page, it - base_it);
                if (QUANT) {
                    if (lane == 0) {
                        // bf16 tile into its own ring; the ring's depth bounds the tiles in flight
                        const int sb = it % kF8BfStages;
                        if (it >= kF8BfStages) ok = ptx::mbar_wait(&bf_empty[sb], (uint32_t)(((it / kF8BfStages) & 1) ^ 1));
                        if (ok) {
                            unsigned char* dst = stages + (size_t)NST * kF8StageBytes + (size_t)sb * kF8BfStageBytes;
                            // page layout [K|V][L*G][64 tokens][128 bf16]: rows of 256 B, fetched as two 64-dim halves
                            const int yk = ((page * 2 + 0) * LG + lg) * kF8Tile, yv = ((page * 2 + 1) * LG + lg) * kF8Tile;
                            ptx::mbar_expect_tx(&bf_full[sb], kF8BfStageBytes);
                            ptx::tma_load_2d(dst, &map_pages, 0, yk, &bf_full[sb]);
                            ptx::tma_load_2d(dst + kF8TileBytes, &map_pages, 64, yk, &bf_full[sb]);
                            ptx::tma_load_2d(dst + 2 * kF8TileBytes, &map_pages, 0, yv, &bf_full[sb]);
                            ptx::tma_load_2d(dst + 3 * kF8TileBytes, &map_pages, 64, yv, &bf_full[sb]);
                        }
                    }
                } else if (lane == 0) {
                    const int st = it % NST;
                    if (ahead < NST && it >= ahead) {       // at most `ahead` tiles that have not landed yet
                        const int jt = it - ahead;
                        ok = ptx::mbar_wait(&full_bar[jt % NST], (uint32_t)((jt / NST) & 1));
                    }
                    if (ok && it >= NST) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / NST) & 1) ^ 1));
                    if (ok) {
                        unsigned char* dst = stages + (size_t)st * kF8StageBytes;
                        // page layout [K|V][L*G][64 rows][128 bytes]
                        ptx::mbar_expect_tx(&full_bar[st], kF8StageBytes);
                        ptx::tma_load_2d(dst, &map_pages, 0, ((page * 2 + 0) * LG + lg) * kF8Tile, &full_bar[st]);
                        ptx::tma_load_2d(dst + kF8TileBytes, &map_pages, 0, ((page * 2 + 1) * LG + lg) * kF8Tile, &full_bar[st]);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
            }
        }
    } else if (QROT && warp > kF8Consumers) {
        // ---------------- query rotators: Q'(tile) = RoPE^-1(q, p0(tile)), rounded to bf16, stored as f16 ----------------
        // lane -> 16-byte chunk c = lane & 7 of the low half (dims 8c..8c+7, paired with 64+8c..) of rows (lane >> 3) + 4 i
        if (n_tiles > 0) {
            const int c = lane & 7;
            uint4 raw_lo[4], raw_hi[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = (lane >> 3) + 4 * i;
                raw_lo[i] = raw_hi[i] = make_uint4(0u, 0u, 0u, 0u);
                if (row < a.rows) {
                    const __nv_bfloat16* qr = a.q + ((((size_t)s * a.M + row / a.r) * a.L + l) * a.H + (size_t)g * a.r + row % a.r) * kF8D;
                    raw_lo[i] = *reinterpret_cast<const uint4*>(qr + c * 8);
                    raw_hi[i] = *reinterpret_cast<const uint4*>(qr + kF8D / 2 + c * 8);
                }
            }
            unsigned char* qring = stages + (size_t)NST * kF8StageBytes;
            auto fetch_row = [&](int it, float4 (&t4)[4]) {
                int p0 = a.first_position + (t0 + min(it, n_tiles - 1)) * kF8Tile;
                if (p0 < 0 || p0 >= a.rope_positions) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_DEVICE_RANGE); p0 = 0; }
                const float4* cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)p0 * (kF8D / 2) + c * 8);
#pragma unroll
                for (int w = 0; w < 4; ++w) t4[w] = __ldg(cs4 + w);
            };
            auto to_f16 = [](const uint4& v) -> uint4 {       // 8 bf16 -> 8 f16 (exact for the values a query takes)
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) o[i] = ptx::pack_f16x2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
                return make_uint4(o[0], o[1], o[2], o[3]);
            };
            const int it_first = warp - kF8Consumers - 1;
            float4 t4[4], t4_next[4];
            fetch_row(it_first, t4_next);
            for (int it = it_first; it < n_tiles; it += kF8QrotWarps) {
                const int st = it % NST;
#pragma unroll
                for (int w = 0; w < 4; ++w) t4[w] = t4_next[w];
                fetch_row(it + kF8QrotWarps, t4_next);
                bool ok = true;
                if (it >= NST) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / NST) & 1) ^ 1));
                if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
                unsigned char* qb = qring + (size_t)st * kF8QrotBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = (lane >> 3) + 4 * i;
                    uint4 lo_o, hi_o;
                    rotate8_cs(raw_lo[i], raw_hi[i], t4, -1.0f, lo_o, hi_o);
                    *reinterpret_cast<uint4*>(qb + row * kF8QrotPitch + c * 16) = to_f16(lo_o);
                    *reinterpret_cast<uint4*>(qb + row * kF8QrotPitch + (kF8D / 2) * 2 + c * 16) = to_f16(hi_o);
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&q_full[st]);
            }
        }
    } else if (QUANT && warp > kF8Consumers + 1) {
        // ---------------- quantisers: landed bf16 tile -> the view's FP8 tiles (K [token][128 B], V^T [dim / 2][128 B]) ----------------
        const int qw = warp - kF8Consumers - 2;
        for (int it = 0; it < n_tiles; ++it) {
            const int sb = it % kF8BfStages, st = it % NST;
            bool ok = ptx::mbar_wait(&bf_full[sb], (uint32_t)((it / kF8BfStages) & 1));
            if (ok && it >= NST) ok = ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / NST) & 1) ^ 1));
            if (!__all_sync(0xffffffffu, ok)) { if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT); break; }
            const unsigned char* srcK = stages + (size_t)NST * kF8StageBytes + (size_t)sb * kF8BfStageBytes;
            const unsigned char* srcV = srcK + 2 * kF8TileBytes;
            unsigned char* dstK = stages + (size_t)st * kF8StageBytes;
            unsigned char* dstV = dstK + kF8TileBytes;
            if (a.k_inv_scale == 1.0f && a.v_inv_scale == 1.0f) quantise_tile_share<true>(srcK, srcV, dstK, dstV, qw, lane, 1.0f, 1.0f);
            else quantise_tile_share<false>(srcK, srcV, dstK, dstV, qw, lane, a.k_inv_scale, a.v_inv_scale);
            ptx::fence_proxy_async_smem();      // the view writer's bulk stores read these bytes through the async proxy
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(&full_bar[st]);
                ptx::mbar_arrive(&bf_empty[sb]);
            }
        }
    } else if (FUSED && warp == kF8Consumers + 1) {
        // ---------------- view writer: every tile that lands in shared memory is stored to the FP8 view ----------------
        if (lane == 0 && n_tiles > 0) {
            ptx::prefetch_tensormap(&map_k);
            ptx::prefetch_tensormap(&map_v);
            bool ok = true;
            for (int it = 0; it < n_tiles; ++it) {
                const int st = it % NST;
                ok = ptx::mbar_wait(&full_bar[st], (uint32_t)((it / NST) & 1));
                if (!ok) break;
                unsigned char* src = stages + (size_t)st * kF8StageBytes;
                const int y = (z * cap_tiles + t0 + it) * kF8Tile;
                ptx::tma_store_2d(&map_k, src, 0, y);
                ptx::tma_store_2d(&map_v, src + kF8TileBytes, 0, y);
                ptx::bulk_commit();
                if (it > 0) {                              // all but the newest store have left shared memory
                    ptx::bulk_wait_read<1>();
                    ptx::mbar_arrive(&empty_bar[(it - 1) % NST]);
                }
            }
            ptx::bulk_wait_read<0>();
            if (ok) ptx::mbar_arrive(&empty_bar[(n_tiles - 1) % NST]);
            else atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
            ptx::bulk_wait<0>();                           // the view is complete before the kernel ends
        }
    } else if (warp == kF8Consumers) {
        // ---------------- producer ----------------
        if (lane == 0 && n_tiles > 0) {
            ptx::prefetch_tensormap(&map_k);
            ptx::prefetch_tensormap(&map_v);
            for (int it = 0; it < n_tiles; ++it) {
                const int st = it % NST;
                if (it >= NST && !ptx::mbar_wait(&empty_bar[st], (uint32_t)(((it / NST) & 1) ^ 1))) {
                    atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                    break;
                }
                unsigned char* dst = stages + (size_t)st * kF8StageBytes;
                ptx::mbar_expect_tx(&full_bar[st], kF8StageBytes);
                ptx::tma_load_2d(dst, &map_k, 0, (z * cap_tiles + t0 + it) * kF8Tile, &full_bar[st]);                 // 64 tokens x 128 B
                ptx::tma_load_2d(dst + kF8TileBytes, &map_v, 0, (z * cap_tiles + t0 + it) * kF8Tile, &full_bar[st]);  // 64 dim pairs x 128 B
            }
        }
    } else {
        // ---------------- consumers ----------------
        // Q fragments in f16.  k-slot permutation inside a k16 step: slots {2c, 2c+1} of lane quad position c hold
        // dims 16 ks + 4c + {0, 1}, slots {2c+8, 2c+9} hold dims 16 ks + 4c + {2, 3}: what one ldmatrix register of
        // FP8 keys (four consecutive dims of a token) converts to.
        uint32_t qf[8][4];
        if (!QROT) {
            const int row_a = lane >> 2, row_b = row_a + 8;
            const __nv_bfloat16* qa = nullptr;
            const __nv_bfloat16* qb = nullptr;
            if (row_a < a.rows) qa = a.q + ((((size_t)s * a.M + row_a / a.r) * a.L + l) * a.H + (size_t)g * a.r + row_a % a.r) * kF8D;
            if (row_b < a.rows) qb = a.q + ((((size_t)s * a.M + row_b / a.r) * a.L + l) * a.H + (size_t)g * a.r + row_b % a.r) * kF8D;
            const int kq = 4 * (lane & 3);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                float fa[4] = {0.f, 0.f, 0.f, 0.f}, fb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (qa) fa[i] = __bfloat162float(qa[ks * 16 + kq + i]);
                    if (qb) fb[i] = __bfloat162float(qb[ks * 16 + kq + i]);
                }
                qf[ks][0] = ptx::pack_f16x2(fa[0], fa[1]);
                qf[ks][1] = ptx::pack_f16x2(fb[0], fb[1]);
                qf[ks][2] = ptx::pack_f16x2(fa[2], fa[3]);
                qf[ks][3] = ptx::pack_f16x2(fb[2], fb[3]);
            }
        }
        const uint32_t stage0 = ptx::smem_u32(stages);
        const int mj = lane >> 3, mr = lane & 7;        // ldmatrix: matrix index and row within it
        const int grp = warp >> 2, wq = warp & 3;       // group grp takes tiles grp, grp + 2, ...; warp wq tokens [16 wq, 16 wq + 16)

        for (int it = grp; it < n_tiles; it += kF8Groups) {
            const int st = it % NST;
            bool arrived = ptx::mbar_wait(&full_bar[st], (uint32_t)((it / NST) & 1));
            if (QROT) arrived = arrived && ptx::mbar_wait(&q_full[st], (uint32_t)((it / NST) & 1));
            if (!__all_sync(0xffffffffu, arrived)) {
                if (lane == 0) atomicExch(a.status, (int)KVMEM_E_TIMEOUT);
                break;
            }
            const uint32_t kbase = stage0 + (uint32_t)st * kF8StageBytes;
            const uint32_t vbase = kbase + kF8TileBytes;
            if (QROT) {
                // this tile's rotated query: four consecutive dims (two f16x2 words) per k-step for rows lane / 4 and + 8
                const unsigned char* qb = stages + (size_t)NST * kF8StageBytes + (size_t)st * kF8QrotBytes;
                const unsigned char* pa = qb + (lane >> 2) * kF8QrotPitch + 8 * (lane & 3);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint2 va = *reinterpret_cast<const uint2*>(pa + ks * 32);
                    const uint2 vb = *reinterpret_cast<const uint2*>(pa + 8 * kF8QrotPitch + ks * 32);
                    qf[ks][0] = va.x; qf[ks][2] = va.y; qf[ks][1] = vb.x; qf[ks][3] = vb.y;
                }
            }

            // S = Q K^T for this warp's 16 tokens.  Column n of n-tile nt is token 4 (n / 2) + 2 nt + (n % 2) of the 16,
            // so that a lane ends up with the probabilities of four consecutive tokens: the same four an ldmatrix register
            // of transposed FP8 values carries.
            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f; }
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                const int tok = wq * 16 + 4 * (mr >> 1) + 2 * nt + (mr & 1);
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {            // 64 dims = 4 chunks of 16 B = 4 k-steps
                    const int c = kh * 4 + mj;
                    const uint32_t addr = kbase + (uint32_t)tok * 128u + (uint32_t)((c ^ (tok & 7)) << 4);
                    uint32_t kr[4];
                    ptx::ldmatrix_x4(addr, kr[0], kr[1], kr[2], kr[3]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t b0, b1;
                        ptx::e4m3x4_to_f16x2x2(kr[j], b0, b1);
                        ptx::mma_f16_16816(sc[nt], qf[kh * 4 + j], b0, b1);
                    }
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
            if (__any_sync(0xffffffffu, grew)) {
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
                pa[0] = ptx::pack_f16x2(p00, p01); pa[1] = ptx::pack_f16x2(p02, p03);
                pa[2] = ptx::pack_f16x2(p10, p11); pa[3] = ptx::pack_f16x2(p12, p13);
            }
            // O += P V: the transposed V tile has row = dim / 2; the 16 bytes of chunk (dim & 1) * 4 + wq are this warp's
            // 16 tokens of that dim, and a lane's register holds tokens 4 (lane & 3) .. + 3 of dim 8 nd + lane / 4
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int dim = (np * 4 + mj) * 8 + mr;
                const int vr = dim >> 1, c = (dim & 1) * 4 + wq;
                const uint32_t addr = vbase + (uint32_t)vr * 128u + (uint32_t)((c ^ (vr & 7)) << 4);
                uint32_t vreg[4];
                ptx::ldmatrix_x4(addr, vreg[0], vreg[1], vreg[2], vreg[3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t b0, b1;
                    ptx::e4m3x4_to_f16x2x2(vreg[j], b0, b1);
                    ptx::mma_f16_16816(o[np * 4 + j], pa, b0, b1);
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&empty_bar[st]);
        }
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1); l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1); l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    }

    __syncthreads();
    float* merge_o = reinterpret_cast<float*>(stages);          // [consumer][16][kF8MergeStride]
    if (warp < kF8Consumers) {
        const int row_a = lane >> 2, row_b = row_a + 8, col = 2 * (lane & 3);
        float* base = merge_o + (size_t)warp * kF8RowsPad * kF8MergeStride;
#pragma unroll
        for (int nd = 0; nd < 16; ++nd) {
            *reinterpret_cast<float2*>(base + row_a * kF8MergeStride + nd * 8 + col) = make_float2(o[nd][0], o[nd][1]);
            *reinterpret_cast<float2*>(base + row_b * kF8MergeStride + nd * 8 + col) = make_float2(o[nd][2], o[nd][3]);
        }
        if ((lane & 3) == 0) {
            merge_m[warp][row_a] = m_run[0]; merge_l[warp][row_a] = l_run[0];
            merge_m[warp][row_b] = m_run[1]; merge_l[warp][row_b] = l_run[1];
        }
    }
    __syncthreads();
    if (tid < 256) {
        const int col = tid & 127, r0 = (tid >> 7) * 8;
        const size_t pbase = ((size_t)z * a.n_splits + split) * kF8RowsPad;
        for (int row = r0; row < r0 + 8; ++row) {
            float mx = -INFINITY;
#pragma unroll
            for (int w = 0; w < kF8Consumers; ++w) mx = fmaxf(mx, merge_m[w][row]);
            float acc = 0.0f, lsum = 0.0f;
#pragma unroll
            for (int w = 0; w < kF8Consumers; ++w) {
                const float mw = merge_m[w][row];
                if (mw > -INFINITY) {
                    const float f = exp2f(mw - mx);
                    acc += f * merge_o[((size_t)w * kF8RowsPad + row) * kF8MergeStride + col];
                    lsum += f * merge_l[w][row];
                }
            }
            a.part_o[(pbase + row) * kF8D + col] = acc * a.v_scale;
            if (col == 0) a.part_ml[pbase + row] = make_float2(mx, lsum);
        }
    }
}


static PFN_cuTensorMapEncodeTiled_v12000 f8_encode() {
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

// [rows][128] bytes; box = 128 bytes x 64 rows, 128-byte swizzle
static bool make_f8_map(CUtensorMap* map, const uint8_t* base, long long rows) {
    PFN_cuTensorMapEncodeTiled_v12000 enc = f8_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {128, (cuuint32_t)kF8Tile};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 page pool as [rows][128 bf16]; box = one 64-dim half (128 bytes) x 64 rows, 128-byte swizzle
static bool make_bf16_pages_map(CUtensorMap* map, const __nv_bfloat16* base, long long rows) {
    PFN_cuTensorMapEncodeTiled_v12000 enc = f8_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kF8D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kF8D * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kF8Tile};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_gather_fp8(const kvmem_pool& p, int session_first, int n_sessions, const int32_t* sel_ids, int sel_stride,
                              const int32_t* n_sel, uint8_t* view_k, uint8_t* view_v, int view_cap_tokens, float k_scale,
                              float v_scale, cudaStream_t st, int rope_first_position) {
    const Geometry& g = p.geo;
    GatherF8Args a{};
    a.pages = p.pages; a.tables = p.tables; a.nblocks_dev = p.nblocks_dev; a.sel_ids = sel_ids; a.n_sel = n_sel;
    a.view_k = view_k; a.view_v = view_v; a.status = p.status_dev;
    a.session_first = session_first; a.sel_stride = sel_stride; a.max_bps = g.max_bps; a.max_blocks = g.max_blocks;
    a.LG = g.L * g.G; a.cap_tokens = view_cap_tokens; a.k_inv_scale = 1.0f / k_scale; a.v_inv_scale = 1.0f / v_scale;
    a.page_elems = p.lay.page_elems;
    // about 64 short-lived CTAs per SM over the kernel's life (8 resident): 250 -> 240 us (quantising) and 176 -> 164 us (tile copy) at 1M
    const int ctas = g_gather_ctas > 0 ? g_gather_ctas : std::max(1, p.sm_count * 64 / n_sessions + 1);
    a.rope = rope_first_position >= 0 ? p.rope_dev : nullptr;
    a.first_position = rope_first_position; a.rope_positions = p.cfg.rope_max_positions; a.in_block = p.cfg.rope_in_block_keys;
    if (p.cfg.fp8_pages)
        launch_pdl(gather_fp8_pages_kernel, dim3((unsigned)ctas, (unsigned)n_sessions), dim3(256), 0, st, a);
    else if (rope_first_position >= 0)
        launch_pdl(gather_fp8_kernel<true>, dim3((unsigned)ctas, (unsigned)n_sessions), dim3(256), 0, st, a);
    else
        launch_pdl(gather_fp8_kernel<false>, dim3((unsigned)ctas, (unsigned)n_sessions), dim3(256), 0, st, a);
    return cudaGetLastError();
}

static int f8_choose_splits(int heads, int max_tiles, int sms) {
    const int overhead = 6;
    long long best_cost = -1;
    int best = 1;
    for (int s = 1; s <= 64 && s <= std::max(1, max_tiles); ++s) {
        const long long waves = ((long long)heads * s + sms - 1) / sms;
        const long long cost = waves * ((max_tiles + s - 1) / s + overhead);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

cudaError_t launch_attend_fp8(const kvmem_pool& p, int n_sessions, const __nv_bfloat16* q, int M, const uint8_t* view_k,
                              const uint8_t* view_v, int view_cap_tokens, const int32_t* n_sel, float scale, float k_scale,
                              float v_scale, float* out, float* lse, void* workspace, cudaStream_t st, const int32_t* sel_ids,
                              int sel_stride, int session_first, int rope_first_position) {
    const Geometry& g = p.geo;
    const int LG = g.L * g.G, heads = n_sessions * LG;
    const bool paged = sel_ids != nullptr;                  // straight over the pages of an FP8 repository ...
    const bool fused = paged && view_k != nullptr;          // ... and, with view buffers, storing the view on the way
    const bool quant = fused && !p.cfg.fp8_pages;           // bf16 repository: tiles are quantised on their way through
    CUtensorMap map_k, map_v, map_pages;
    if (quant) {
        if (!make_bf16_pages_map(&map_pages, p.pages, (long long)g.max_blocks * 2 * LG * kF8Tile)) return cudaErrorInvalidValue;
    } else if (paged && !make_f8_map(&map_pages, reinterpret_cast<const uint8_t*>(p.pages), (long long)g.max_blocks * 2 * LG * kF8Tile))
        return cudaErrorInvalidValue;
    if (paged && !fused) {
        map_k = map_pages; map_v = map_pages;               // unused by this mode
    } else if (!make_f8_map(&map_k, view_k, (long long)heads * view_cap_tokens) || !make_f8_map(&map_v, view_v, (long long)heads * view_cap_tokens)) {
        return cudaErrorInvalidValue;
    }
    if (!paged) map_pages = map_k;
    static PerDeviceOnce attr_done;
    if (attr_done.pending(p.cfg.device)) {
        cudaError_t e = cudaFuncSetAttribute(attend_fp8_split_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF8Smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_fp8_split_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF8Smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_fp8_split_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF8Smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_fp8_split_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF8SmemQrot);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attend_fp8_split_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF8SmemQuant);
        if (e != cudaSuccess) return e;
        attr_done.mark(p.cfg.device);
    }
    AttendPlan plan = plan_attend(p.cfg, n_sessions, M, p.sm_count);
    AttendF8Args a{};
    a.q = q; a.n_sel = n_sel;
    a.part_o = reinterpret_cast<float*>(workspace);
    a.part_ml = reinterpret_cast<float2*>(reinterpret_cast<char*>(workspace) + plan.part_o_bytes);
    a.status = p.status_dev;
    a.M = M; a.L = g.L; a.H = g.H; a.G = g.G; a.r = g.r; a.rows = M * g.r;
    a.n_splits = f8_choose_splits(heads, view_cap_tokens / kF8Tile, p.sm_count);
    a.cap_tokens = view_cap_tokens;
    const float sc = scale > 0.0f ? scale : 1.0f / sqrtf((float)g.d);
    a.scale_log2e = sc * k_scale * 1.4426950408889634f;
    a.v_scale = v_scale;
    a.k_inv_scale = 1.0f / k_scale; a.v_inv_scale = 1.0f / v_scale;
    a.sel_ids = sel_ids; a.tables = p.tables; a.nblocks_dev = p.nblocks_dev;
    a.session_first = session_first; a.sel_stride = sel_stride; a.max_bps = g.max_bps; a.max_blocks = g.max_blocks;
    dim3 grid((unsigned)a.n_splits, (unsigned)LG, (unsigned)n_sessions);
    // the view-writing pass is fastest with about 9.5 MiB of tiles that have not landed yet over all SMs (as its bf16 counterpart)
    a.lookahead = g_attend_lookahead;
    if (fused && a.lookahead == 0) {
        const long long ctas = (long long)a.n_splits * heads;
        const int tiles_per_cta = (view_cap_tokens / kF8Tile + a.n_splits - 1) / a.n_splits;
        if (ctas <= p.sm_count && tiles_per_cta >= 64)
            a.lookahead = std::max(2, std::min(kF8Stages, (int)(9.5 * 1024.0 * 1024.0 / ((double)ctas * kF8StageBytes) + 0.5)));
    }
    a.rope = p.rope_dev; a.first_position = rope_first_position; a.rope_positions = p.cfg.rope_max_positions;
    if (paged && !fused && rope_first_position >= 0)
        launch_pdl(attend_fp8_split_kernel<3>, dim3(grid), dim3(kF8Threads + 32 * kF8QrotWarps), kF8SmemQrot, st, map_k, map_v, map_pages, a);
    else if (quant)
        launch_pdl(attend_fp8_split_kernel<4>, dim3(grid), dim3(kF8Threads + 32 + 32 * kF8QuantWarps), kF8SmemQuant, st, map_k, map_v, map_pages, a);
    else if (fused)
        launch_pdl(attend_fp8_split_kernel<2>, dim3(grid), dim3(kF8Threads + 32), kF8Smem, st, map_k, map_v, map_pages, a);
    else if (paged)
        launch_pdl(attend_fp8_split_kernel<1>, dim3(grid), dim3(kF8Threads), kF8Smem, st, map_k, map_v, map_pages, a);
    else
        launch_pdl(attend_fp8_split_kernel<0>, dim3(grid), dim3(kF8Threads), kF8Smem, st, map_k, map_v, map_pages, a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_attend_merge(a.part_o, a.part_ml, out, lse, a.rows, heads, M, g.L, g.H, g.G, g.r, a.n_splits, plan.rows_pad, st);
}

}  // namespace kvmem
