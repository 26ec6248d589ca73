// CTA-wide building blocks of one compression event: score, reciprocal norms, greedy
// selection, index ordering. Every block is called by all kThreads threads of the CTA.
#pragma once
#include "akv_common.cuh"

namespace akv {

// ---- row sources -----------------------------------------------------------------------------
// Rows at a fixed stride (a tile in shared memory, or a dense global tensor).
template <typename T>
struct StridedRows {
    const T* base;
    long long stride;  // elements
    __device__ __forceinline__ const T* operator()(int j) const { return base + (long long)j * stride; }
};
// Rows of one event addressed through the K/V layout (dense or paged) in global memory.
template <typename T>
struct LayoutRows {
    const T* base;
    const DevLayout* lay;
    int b, l, h;
    __device__ __forceinline__ const T* operator()(int j) const { return base + row_offset(*lay, b, l, h, j); }
};

// ---- score ------------------------------------------------------------------------------------
// cos and sin of 2*pi*(top / 2^32): octant reduction on the fixed-point phase, then short polynomials
// in y = (angle offset)/(pi/4) in [-1, 1) (least-squares fits at Chebyshev nodes, |error| < 1e-7).
__device__ __forceinline__ void sincos_phase(uint32_t top, float& sn, float& cs) {
    const uint32_t u = top + 0x20000000u;
    const uint32_t quad = u >> 30;
    const int t = (int)(u & 0x3FFFFFFFu) - 0x20000000;
    const float y = (float)t * 1.862645149230957e-09f;  // 2^-29
    const float z = y * y;
    const float sp = y * fmaf(z, fmaf(z, fmaf(z, -3.587714997811334e-05f, 0.0024898717780787645f), -0.08074536717605851f),
                              0.7853981525308736f);
    const float cp = fmaf(z, fmaf(z, fmaf(z, -0.0003191315544232772f, 0.01585035496683941f), -0.308424473701413f), 1.0f);
    const bool swap = quad & 1u;
    const float c0 = swap ? sp : cp;
    const float s0 = swap ? cp : sp;
    cs = ((quad + 1u) & 2u) ? -c0 : c0;  // quadrants 1, 2
    sn = (quad & 2u) ? -s0 : s0;         // quadrants 2, 3
}

// Score of one row, computed by the G lanes of a group; lane `lig` covers frequencies
// [4*lig, 4*lig+4). All lanes of the warp must call (shuffles inside). dist = p_ref - p_i.
template <typename T>
__device__ __forceinline__ float score_row(const T* krow, bool valid, long long dist, bool rotate, int d,
                                           const unsigned long long* phi, const float2* g, int lig, int G) {
    const int half = d >> 1;
    const int f0 = lig * 4;
    float acc = 0.f;
    if (valid && f0 < half) {
        float kr[4], ki[4];
        load4(krow + f0, kr);
        load4(krow + half + f0, ki);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 gf = g[f0 + u];
            const float tr = fmaf(gf.x, kr[u], gf.y * ki[u]);
            const float ti = fmaf(gf.y, kr[u], -gf.x * ki[u]);
            if (rotate) {
                const unsigned long long turns = (unsigned long long)dist * phi[f0 + u];
                float sn, cs;
                sincos_phase((uint32_t)(turns >> 32), sn, cs);
                acc += fmaf(tr, cs, -ti * sn);
            } else {
                acc += tr;
            }
        }
    }
    return group_sum(acc, G);
}

// sum of squares of one row by a lane group; lane `lig` covers elements [8*lig, 8*lig+8)
template <typename T>
__device__ __forceinline__ float sumsq_row(const T* vrow, bool valid, int d, int lig, int G) {
    float acc = 0.f;
    if (valid && lig * 8 < d) {
        float x[8];
        load8(vrow + lig * 8, x);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc = fmaf(x[u], x[u], acc);
    }
    return group_sum(acc, G);
}

// ---- greedy selection (Algorithm 1) ---------------------------------------------------------------
// s, m, taken, order, gain and red live in shared memory. s holds sanitised scores (non-finite ->
// -inf), m starts at 0, taken at 0. r holds 1/(||V_j||+eps) per candidate, or nullptr when the
// signature rows are already unit-normalised. `rows` yields the signature row of candidate j.
// Performs `picks` picks; with similarity == false no row is ever read and the loop is a plain
// repeated argmax (top-k in pick order). red: 2*kWarps keys.
template <typename T, typename Rows>
__device__ void greedy_cta(int n, int picks, float lam, bool similarity, int d, const float* s, const float* r,
                           float* m, unsigned char* taken, int* order, float* gain, const Rows& rows,
                           unsigned long long* red) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = pow2_ceil(d >> 3) > 32 ? 32 : pow2_ceil(d >> 3);  // lanes per row
    const int RPW = 32 / G;                                         // rows per warp and pass
    const int grp = lane / G, lig = lane % G;
    for (int t = 0; t < picks; ++t) {
        // Eq. 2 for every candidate still outside the set, Eq. 3's arg-max (ties to the lower slot)
        unsigned long long best = 0ull;
        for (int j = tid; j < n; j += kThreads) {
            if (!taken[j]) {
                const float a = fmaf(-lam, m[j], s[j]);
                const unsigned long long key = pack_key(a, j);
                best = key > best ? key : best;
            }
        }
        best = warp_max_u64(best);
        unsigned long long* slot = red + (t & 1) * kWarps;
        if (lane == 0) slot[warp] = best;
        __syncthreads();
        best = slot[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) best = slot[w] > best ? slot[w] : best;
        const int i = key_index(best);
        if (tid == 0) {
            order[t] = i;
            gain[t] = key_value(best);
            taken[i] = 1;
        }
        // fold the new member's cosines <V_i, V_j> r_i r_j into every candidate's running maximum
        if (similarity && t + 1 < picks) {
            float vi[8];
            const bool act = lig * 8 < d;
            if (act) load8(rows(i) + lig * 8, vi);
            const float ri = r ? r[i] : 1.f;
            for (int j0 = warp * RPW; j0 < n; j0 += kWarps * RPW) {
                const int j = j0 + grp;
                const bool live = j < n && j != i && !taken[j];
                float acc = 0.f;
                if (live && act) {
                    float vj[8];
                    load8(rows(j) + lig * 8, vj);
#pragma unroll
                    for (int u = 0; u < 8; ++u) acc = fmaf(vi[u], vj[u], acc);
                }
                acc = group_sum(acc, G);
                if (live && lig == 0) {
                    const float c = acc * (ri * (r ? r[j] : 1.f));
                    m[j] = fmaxf(m[j], c);
                }
            }
        }
        __syncthreads();
    }
}

// sort(S): ascending slot indices of the taken flags, written by warp 0. Returns nothing; idx has
// `budget` entries, the tail beyond the kept count is set to -1.
__device__ __forceinline__ void ordered_indices(int n, int budget, const unsigned char* taken, int* idx) {
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int off = 0;
        for (int base = 0; base < n; base += 32) {
            const int j = base + lane;
            const bool f = j < n && taken[j];
            const unsigned mask = __ballot_sync(0xFFFFFFFFu, f);
            if (f) idx[off + __popc(mask & ((1u << lane) - 1u))] = j;
            off += __popc(mask);
        }
        for (int t = off + lane; t < budget; t += 32) idx[t] = -1;
    }
}

}  // namespace akv
