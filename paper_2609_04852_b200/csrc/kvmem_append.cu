// Repository append + Mean-K index construction (Eq. "mean_k_index", Sec. 4.3; "Incremental
// Indexing", Sec. 5.3: the index entry is computed while the block's keys pass through the SM).
//
// One CTA per (new block, layer, KV head).  The caller's token-major rows (256 B each at d = 128,
// strided by L*G*d) are read once with 128-bit loads, written to the page's contiguous [B][d]
// tile, and the K tile is kept in shared memory so that thread c can walk tokens 0..B-1 of
// dimension c in order: an fp32 running sum in ascending token order, one multiply by 1/B and one
// round-to-nearest-even to bf16.  That order is the definition of the stored index value.
#include "kvmem_internal.cuh"

namespace kvmem {

__global__ void __launch_bounds__(256)
append_kernel(const __nv_bfloat16* __restrict__ k_in, const __nv_bfloat16* __restrict__ v_in,
              __nv_bfloat16* __restrict__ pages, __nv_bfloat16* __restrict__ index_sess,
              const int32_t* __restrict__ table_sess, int32_t* __restrict__ status,
              int b_first, int L, int G, int B, int d, int max_blocks, int max_bps, size_t page_elems,
              const int32_t* __restrict__ pos0_sess, const float2* __restrict__ rope, int rope_positions, int in_block) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* tile = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [B][d]

    const int i = blockIdx.x;          // new block index within this call
    const int lg = blockIdx.y;         // l * G + g
    const int page = table_sess[b_first + i];
    if (page < 0 || page >= max_blocks) {
        if (threadIdx.x == 0) atomicExch(status, (int)KVMEM_E_DEVICE_RANGE);
        return;
    }
    const int chunks_per_row = d / 8;                     // 16-byte chunks
    const int n_chunks = B * chunks_per_row;
    const size_t row_stride = (size_t)L * G * d;          // elements between consecutive tokens
    const __nv_bfloat16* ksrc = k_in + (size_t)i * B * row_stride + (size_t)lg * d;
    const __nv_bfloat16* vsrc = v_in + (size_t)i * B * row_stride + (size_t)lg * d;
    const size_t tile_elems = (size_t)B * d;
    __nv_bfloat16* kdst = pages + (size_t)page * page_elems + (size_t)lg * tile_elems;
    __nv_bfloat16* vdst = kdst + (size_t)L * G * tile_elems;

    for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) {
        const int t = c / chunks_per_row, j = c % chunks_per_row;
        const uint4 kk = *reinterpret_cast<const uint4*>(ksrc + (size_t)t * row_stride + j * 8);
        const uint4 vv = *reinterpret_cast<const uint4*>(vsrc + (size_t)t * row_stride + j * 8);
        *reinterpret_cast<uint4*>(tile + (size_t)t * d + j * 8) = kk;
        *reinterpret_cast<uint4*>(vdst + (size_t)t * d + j * 8) = vv;
    }
    __syncthreads();
    if (pos0_sess) {
        // the keys still carry RoPE of positions pos0 + t: rotate back by the same angles (Sec. 4.3), so
        // that the pages hold raw keys and the index is position-independent.  fp32 products and sums
        // without fused multiply-add, one rounding to bf16: the defined arithmetic of a rotated element.
        const int pos0 = pos0_sess[b_first + i];
        const int half = d / 2;
        for (int e = threadIdx.x; e < B * half; e += blockDim.x) {
            const int t = e / half, x = e % half;
            const int pos = pos0 + t;
            if (pos < 0 || pos >= rope_positions) { atomicExch(status, (int)KVMEM_E_DEVICE_RANGE); continue; }
            const float2 cs = rope[(size_t)pos * half + x];
            const float a = __bfloat162float(tile[(size_t)t * d + x]), b = __bfloat162float(tile[(size_t)t * d + x + half]);
            const float lo = __fadd_rn(__fmul_rn(a, cs.x), __fmul_rn(b, cs.y));     // inverse rotation: sin -> -sin
            const float hi = __fsub_rn(__fmul_rn(b, cs.x), __fmul_rn(a, cs.y));
            tile[(size_t)t * d + x] = __float2bfloat16_rn(lo);
            tile[(size_t)t * d + x + half] = __float2bfloat16_rn(hi);
        }
        __syncthreads();
    }
    // the index entry comes from the raw keys (position-independent, Sec. 4.3), whatever the pages hold
    const float inv = 1.0f / (float)B;
    __nv_bfloat16* idx_row = index_sess + ((size_t)lg * max_bps + (size_t)(b_first + i)) * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float acc = 0.0f;
        for (int t = 0; t < B; ++t) acc = __fadd_rn(acc, __bfloat162float(tile[(size_t)t * d + c]));
        idx_row[c] = __float2bfloat16_rn(__fmul_rn(acc, inv));
    }
    if (in_block) {
        // in-block layout: the page holds RoPE(k, t), t the offset inside the block, so that a later placement at
        // compact position p0 is the rotation of p0 alone for the whole block.  Same defined arithmetic.
        __syncthreads();
        const int half = d / 2;
        for (int e = threadIdx.x; e < B * half; e += blockDim.x) {
            const int t = e / half, x = e % half;
            const float2 cs = rope[(size_t)t * half + x];
            const float a = __bfloat162float(tile[(size_t)t * d + x]), b = __bfloat162float(tile[(size_t)t * d + x + half]);
            const float lo = __fsub_rn(__fmul_rn(a, cs.x), __fmul_rn(b, cs.y));
            const float hi = __fadd_rn(__fmul_rn(b, cs.x), __fmul_rn(a, cs.y));
            tile[(size_t)t * d + x] = __float2bfloat16_rn(lo);
            tile[(size_t)t * d + x + half] = __float2bfloat16_rn(hi);
        }
        __syncthreads();
    }
    for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) {
        const int t = c / chunks_per_row, j = c % chunks_per_row;
        *reinterpret_cast<uint4*>(kdst + (size_t)t * d + j * 8) = *reinterpret_cast<const uint4*>(tile + (size_t)t * d + j * 8);
    }
}

cudaError_t launch_append(const kvmem_pool& p, int session, int b_first, int n_blocks, const __nv_bfloat16* k,
                          const __nv_bfloat16* v, cudaStream_t st, bool derope) {
    const Geometry& g = p.geo;
    const size_t smem = (size_t)g.B * g.d * sizeof(__nv_bfloat16);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(append_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int32_t* table = p.tables + (size_t)session * g.max_bps;
    __nv_bfloat16* index = p.index + (size_t)session * p.lay.index_elems_per_session;
    // gridDim.x is limited to 2^31-1 blocks and gridDim.y to 65535: L*G stays far below that
    dim3 grid((unsigned)n_blocks, (unsigned)(g.L * g.G));
    append_kernel<<<grid, 256, smem, st>>>(k, v, p.pages, index, table, p.status_dev, b_first, g.L, g.G, g.B, g.d,
                                           g.max_blocks, g.max_bps, p.lay.page_elems,
                                           derope ? p.pos0_dev + (size_t)session * g.max_bps : nullptr,
                                           p.rope_dev, p.cfg.rope_max_positions, p.cfg.rope_in_block_keys);
    return cudaGetLastError();
}

}  // namespace kvmem
