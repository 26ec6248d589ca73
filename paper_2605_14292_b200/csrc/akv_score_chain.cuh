// Scores of the fused on-chip kernels (bf16, d = 128): eight lanes per key row, eight frequencies per
// lane, the rotation of the query statistic carried from row to row.
#pragma once
#include "akv_kernels.cuh"

namespace akv {

// (cos, sin) of the angle 2 pi ph / 2^32: nearest of the 32 sector angles from the shared-memory table,
// remainder by the short polynomials of score_lane8
__device__ __forceinline__ float2 phase_cos_sin(uint32_t ph, const float2* sect) {
    const float2 e = sect[(ph + 0x04000000u) >> 27];
    const float w = (float)(int32_t)(ph << 5) * 4.5716245e-11f, z = w * w;
    const float sw = w * fmaf(z, fmaf(z, 8.3333333e-3f, -0.16666667f), 1.f);
    const float cw = fmaf(z, fmaf(z, 4.1666667e-2f, -0.5f), 1.f);
    return make_float2(e.x * cw - e.y * sw, e.y * cw + e.x * sw);
}
// bits 32..63 of dist * phi (mod 2^64) for a signed 64-bit distance: the angle dist * theta_f in 2^-32 turns
__device__ __forceinline__ uint32_t phase_of(long long dist, unsigned long long phi) {
    const uint32_t dl = (uint32_t)dist, dh = (uint32_t)((unsigned long long)dist >> 32);
    const uint32_t pl = (uint32_t)phi, ph = (uint32_t)(phi >> 32);
    return __umulhi(dl, pl) + dl * ph + dh * pl;
}

// Scoring state of a lane: the folded statistic already turned to the row at hand,
// G_f = g_f e^{i dist theta_f} for the lane's eight frequencies, so that a row's score is
// sum_f Re(G_f conj(k_f)); and the turn S_f = e^{-i D theta_f} that takes G from one row of a lane
// group to its next one when the two rows' positions differ by D (rows 16 slots apart: D = 16 for a
// cache filled token by token). G is taken afresh (sector table + polynomials) whenever the spacing is
// not D, and every kChainRounds-th (kChainRoundsShort-th) round in any case: a chained complex product adds
// about 3e-9 of the score's scale to the error (fp32 summation of the 64 terms gives 4e-8 by itself; a chain
// of twelve products measured 8e-8 in all).
struct ChainScore {
    float2 Gx[4], Gy[4], Sx[4], Sy[4], nSy[4];
    // S from D (any sign); phitab: phi_f for the lane's frequencies (shared memory)
    __device__ __forceinline__ void set_step(long long D, const unsigned long long* phitab, const float2* sect) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float2 e = phase_cos_sin(phase_of(-D, phitab[u]), sect);
            if (u & 1) { Sx[u >> 1].y = e.x; Sy[u >> 1].y = e.y; nSy[u >> 1].y = -e.y; }
            else { Sx[u >> 1].x = e.x; Sy[u >> 1].x = e.y; nSy[u >> 1].x = -e.y; }
        }
    }
    // G afresh for a row at distance dist (any sign); gtab: folded statistic g_f for the lane's frequencies
    __device__ __forceinline__ void anchor(long long dist, const float2* gtab, const unsigned long long* phitab,
                                           const float2* sect) {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const float4 g2 = *reinterpret_cast<const float4*>(gtab + 2 * p);       // g of frequencies 2p, 2p + 1
            const ulonglong2 ph = *reinterpret_cast<const ulonglong2*>(phitab + 2 * p);
            const float2 ea = phase_cos_sin(phase_of(dist, ph.x), sect), eb = phase_cos_sin(phase_of(dist, ph.y), sect);
            Gx[p] = make_float2(g2.x * ea.x - g2.y * ea.y, g2.z * eb.x - g2.w * eb.y);
            Gy[p] = make_float2(g2.x * ea.y + g2.y * ea.x, g2.z * eb.y + g2.w * eb.x);
        }
    }
    __device__ __forceinline__ void advance() {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const float2 nx = __ffma2_rn(Gy[p], nSy[p], __fmul2_rn(Gx[p], Sx[p]));
            const float2 ny = __ffma2_rn(Gy[p], Sx[p], __fmul2_rn(Gx[p], Sy[p]));
            Gx[p] = nx; Gy[p] = ny;
        }
    }
    // the same turn, taken from another state's S (two rows of a lane group chained side by side share one S)
    __device__ __forceinline__ void advance_by(const ChainScore& o) {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const float2 nx = __ffma2_rn(Gy[p], o.nSy[p], __fmul2_rn(Gx[p], o.Sx[p]));
            const float2 ny = __ffma2_rn(Gy[p], o.Sx[p], __fmul2_rn(Gx[p], o.Sy[p]));
            Gx[p] = nx; Gy[p] = ny;
        }
    }
    // the lane's partial sum of Re(G conj(k)) over its 8 frequencies
    __device__ __forceinline__ float dot(const uint4& wr, const uint4& wi) const {
        const uint32_t wre[4] = {wr.x, wr.y, wr.z, wr.w}, wim[4] = {wi.x, wi.y, wi.z, wi.w};
        float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            acc2 = __ffma2_rn(Gx[p], make_float2(bf16lo(wre[p]), bf16hi(wre[p])), acc2);
            acc2 = __ffma2_rn(Gy[p], make_float2(bf16lo(wim[p]), bf16hi(wim[p])), acc2);
        }
        return acc2.x + acc2.y;
    }
    // the same sum with four independent accumulators (a chain of two dependent products instead of eight)
    __device__ __forceinline__ float dot4(const uint4& wr, const uint4& wi) const {
        const uint32_t wre[4] = {wr.x, wr.y, wr.z, wr.w}, wim[4] = {wi.x, wi.y, wi.z, wi.w};
        float2 acc[4];
#pragma unroll
        for (int p = 0; p < 4; ++p)
            acc[p] = __ffma2_rn(Gy[p], make_float2(bf16lo(wim[p]), bf16hi(wim[p])),
                                __fmul2_rn(Gx[p], make_float2(bf16lo(wre[p]), bf16hi(wre[p]))));
        const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
        const float2 a = __fadd2_rn(a01, a23);
        return a.x + a.y;
    }
};
constexpr int kChainRounds = 8;        // rounds between two fresh computations of G (long events, streamed)
constexpr int kChainRoundsShort = 16;  // the same for events of at most 256 rows: one or two fresh computations per lane
                                       // group; fifteen chained products add 1e-7 of the score's scale at most

// The 32 sector angles' cosines and sines, written by one warp: sect[h] = (cos, sin)(2 pi h / 32)
__device__ __forceinline__ void fill_sector_table(float2* sect, int lane) {
    float sn, cs;
    sincospif((float)lane * 0.0625f, &sn, &cs);
    sect[lane] = make_float2(cs, sn);
}
// Folded statistic g_f = c_f z(q)_f / sqrt(d) and the frequencies' phase steps for d = 128, written by
// threads 0..63 into gtab[64] and phitab[64]
__device__ __forceinline__ void fill_statistic_tables(const float* q, const ScoreTab& tab, int tid, float2* gtab,
                                                      unsigned long long* phitab) {
    if (tid < 64) {
        const float inv = rsqrtf(128.f);
        const float qr = q[tid] * inv, qi = q[tid + 64] * inv;
        const float2 c = tab.cw[tid];
        gtab[tid] = make_float2(c.x * qr - c.y * qi, c.x * qi + c.y * qr);
        phitab[tid] = tab.phi[tid];
    }
}

}  // namespace akv
