// Cosine matrix of shared signatures (Algorithm 1's "Sims <- V V^T", formed once and used by every event that
// shares the signatures: all layers and heads of a sequence with Eq. 1's flat signature, all heads of a layer
// with the per-layer one). gram[g][i][j] = <sig_i, sig_j> for the unit rows of group g, fp32, d = 128.
//
// The signatures are fp32 averages, and a pick is decided at the 1e-6 level, so a bf16 or tf32 product is not
// accurate enough. Each fp32 row is split into three bf16 parts, x = x1 + x2 + x3 (exact to 2^-24 |x|), and
//   <x, y> = <x1,y1> + <x1,y2> + <x2,y1> + <x1,y3> + <x3,y1> + <x2,y2> + (terms below 2^-24 |x||y|)
// runs as six tcgen05.mma sequences (bf16 x bf16 products are exact, accumulation is fp32 in tensor memory)
// into one accumulator. One CTA per (group, 128 x 128 tile of the matrix).
#pragma once
#include "akv_event_tri.cuh"

namespace akv {

constexpr int kGramThreads = 128;
constexpr unsigned kGramPart = 128u * 256u;                       // one bf16 part of 128 rows: 32 KB
constexpr unsigned kGramSmem = 6u * kGramPart + 64u + 1024u;      // A and B parts, barrier + holder, alignment

// round-to-nearest-even bf16 of x as the high half of a float (the value itself, still fp32)
__device__ __forceinline__ float bf16_part(float x) {
    const uint32_t u = __float_as_uint(x);
    const uint32_t r = u + 0x7FFFu + ((u >> 16) & 1u);
    return __uint_as_float(r & 0xFFFF0000u);
}

// rows [row0, row0 + 128) of `sig` (fp32 [N, 128]; rows >= n read as zero) as three swizzled bf16 operand tiles
__device__ __forceinline__ void gram_split_rows(const float* sig, int row0, int n, unsigned char* parts, int tid) {
    // one (row, 16-byte chunk of 8 elements) per step
    for (int x = tid; x < 128 * 16; x += kGramThreads) {
        const int rr = x >> 4, c = x & 15;
        float v[8];
        if (row0 + rr < n) {
            const float4 a = *reinterpret_cast<const float4*>(sig + (long long)(row0 + rr) * 128 + c * 8);
            const float4 b = *reinterpret_cast<const float4*>(sig + (long long)(row0 + rr) * 128 + c * 8 + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = 0.f;
        }
        uint32_t w[3][4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            uint32_t hi[3][2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const float x1 = bf16_part(v[e + q]);
                const float r1 = v[e + q] - x1;   // exact
                const float x2 = bf16_part(r1);
                const float x3 = bf16_part(r1 - x2);
                hi[0][q] = __float_as_uint(x1) >> 16;
                hi[1][q] = __float_as_uint(x2) >> 16;
                hi[2][q] = __float_as_uint(x3) >> 16;
            }
#pragma unroll
            for (int p = 0; p < 3; ++p) w[p][e >> 1] = hi[p][0] | (hi[p][1] << 16);
        }
#pragma unroll
        for (int p = 0; p < 3; ++p)
            *reinterpret_cast<uint4*>(parts + p * kGramPart + tile_chunk(rr, c, 128u * 128u)) = make_uint4(w[p][0], w[p][1], w[p][2], w[p][3]);
    }
}

// sig: [groups, N, 128] fp32; n_cand: valid rows per sequence (or null); seq_div: groups per sequence
// (1 for flat signatures, L for per-layer ones); gram: [groups, N, N] fp32, rows/columns >= n left untouched.
__global__ void __launch_bounds__(kGramThreads, 1) gram_shared_kernel(const float* sig, const int* n_cand, int seq_div, int N, float* gram,
                                                                     int* error_flag) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tiles = (N + 127) >> 7;
    const int g = blockIdx.x / (tiles * tiles), tt = blockIdx.x % (tiles * tiles);
    const int mb = tt / tiles, nb = tt % tiles;
    int n = n_cand ? n_cand[g / seq_div] : N;
    n = n < 0 ? 0 : (n > N ? N : n);
    if (mb * 128 >= n || nb * 128 >= n) return;
    unsigned char* partsA = smem;
    unsigned char* partsB = smem + 3 * kGramPart;
    const uint32_t barM = smem_u32(smem + 6 * kGramPart);
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + 6 * kGramPart + 16);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* sg = sig + (long long)g * N * 128;
    if (tid == 0) {
        mbar_init(barM, 1);
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_holder), 128u);
    gram_split_rows(sg, mb * 128, n, partsA, tid);
    gram_split_rows(sg, nb * 128, n, partsB, tid);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_holder;
    if (tid == 0) {
        const uint32_t idesc = umma_idesc_bf16(128, 128);
        const uint32_t a_u32 = smem_u32(partsA), b_u32 = smem_u32(partsB);
        // (part of x, part of y): the six products that matter
        const int pa[6] = {0, 0, 1, 0, 2, 1}, pb[6] = {0, 1, 0, 2, 0, 1};
        bool first = true;
        // smallest terms first
        for (int q = 5; q >= 0; --q) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t koff = (uint32_t)(kk >> 2) * (128u * 128u) + (uint32_t)(kk & 3) * 32u;
                umma_bf16(tbase, umma_desc_sw128(a_u32 + (uint32_t)pa[q] * kGramPart + koff),
                          umma_desc_sw128(b_u32 + (uint32_t)pb[q] * kGramPart + koff), idesc, first ? 0u : 1u);
                first = false;
            }
        }
        umma_commit(barM);
    }
    const bool ok = mbar_wait_bounded(barM, 0, kWaitPolls);
    tc_fence_after();
    if (!ok && tid == 0 && error_flag) atomicExch(error_flag, 3);
    // row mb*128 + 32 warp + lane of the tile: 128 columns, 32 at a time
    const int row = mb * 128 + 32 * warp + lane;
    for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tbase + ((uint32_t)(32 * warp) << 16) + (uint32_t)(32 * cb), v);
        tmem_ld_wait();
        if (ok && row < n) {
            float* out = gram + ((long long)g * N + row) * N + nb * 128 + 32 * cb;
#pragma unroll
            for (int k = 0; k < 32; ++k)
                if (nb * 128 + 32 * cb + k < n) out[k] = __uint_as_float(v[k]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, 128u);
}

}  // namespace akv
