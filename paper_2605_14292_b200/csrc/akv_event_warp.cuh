// Fast path for bf16, d = 128, per-head signatures: one CTA of four warps per event.
//   - V rows are brought into shared memory by per-row bulk copies (cp.async.bulk + mbarrier),
//     K rows are scored straight from global memory (each is needed once),
//   - the greedy loop of Algorithm 1 runs in ONE warp: every lane owns N/32 candidates and keeps
//     s, the running maximum and lambda*r in registers; the argmax is two warp reductions,
//   - rows of the cosine matrix come from tensor-core batches: the similarity of all candidates
//     to the 8 most promising ones is computed at once (mma.sync m16n8k16, bf16 x bf16 products
//     are exact in fp32) and reused for as long as the picks stay inside the batch,
//   - kept rows are written back in place at the end.
#pragma once
#include "akv_kernels.cuh"

namespace akv {

constexpr int kWThreads = 128;
constexpr int kWWarps = 4;
constexpr int kWD = 128;          // head dimension of this path
constexpr int kVRowBytes = 272;   // 256 bytes of bf16 + 16 bytes pad: 8 consecutive rows fall in 8 distinct 16-byte bank groups
constexpr int kBatch = 8;         // candidates per tensor-core batch

struct WarpSmem {
    unsigned vt, gcol, s, r, order, gain, idx, red, mbar, total;
    int gstride;
};
__host__ __device__ inline WarpSmem plan_warp_smem(int NT, int budget) {
    WarpSmem p;
    const int rows = 16 * NT;
    p.gstride = rows + 4;  // 2*gstride = 8 (mod 32): the four column pairs of a quad land in distinct banks
    unsigned o = 0;
    p.vt = o;    o += align16((unsigned)rows * kVRowBytes);
    p.gcol = o;  o += align16((unsigned)kBatch * p.gstride * 4);
    p.s = o;     o += align16((unsigned)rows * 4);
    p.r = o;     o += align16((unsigned)rows * 4);
    p.order = o; o += align16((unsigned)budget * 4);
    p.gain = o;  o += align16((unsigned)budget * 4);
    p.idx = o;   o += align16((unsigned)budget * 4);
    p.red = o;   o += 64;
    p.mbar = o;  o += 16;
    p.total = o;
    return p;
}

// ---- PTX wrappers --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after a fixed number of polls instead of spinning for ever.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (int it = 0; it < (1 << 22); ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- the kernel ------------------------------------------------------------------------------------
// NT: row tiles of 16 (N <= 16*NT). FUSED: score + select + compact; otherwise selection only
// (scores are read from a.scores and nothing is rewritten).
template <int NT, bool FUSED>
__global__ void __launch_bounds__(kWThreads) event_warp_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab) {
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int CPL = NT / 2;  // candidates per lane
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int N = lay.N;
    const int picks = min(a.budget, n);
    const WarpSmem sp = plan_warp_smem(NT, a.budget);
    unsigned char* vt = smem + sp.vt;
    float* gcol = reinterpret_cast<float*>(smem + sp.gcol);
    float* s = reinterpret_cast<float*>(smem + sp.s);
    float* r = reinterpret_cast<float*>(smem + sp.r);
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    int* redi = reinterpret_cast<int*>(smem + sp.red);
    const uint32_t bar = smem_u32(smem + sp.mbar);
    const uint32_t vt_u32 = smem_u32(vt);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(a.K);
    __nv_bfloat16* Vg = reinterpret_cast<__nv_bfloat16*>(a.V);
    const bool similarity = a.greedy != 0;
    const bool needV = similarity || FUSED;

    if (tid == 0) mbar_init(bar, 1);
    __syncthreads();
    if (needV) {
        if (tid == 0) mbar_expect_tx(bar, (uint32_t)n * 256u);
        for (int row = tid; row < n; row += kWThreads)
            bulk_g2s(vt_u32 + row * kVRowBytes, Vg + row_offset(lay, id.b, id.l, id.h, row), 256u, bar);
    }

    // ---- scores ---------------------------------------------------------------------------------
    int bad = 0;
    if (FUSED) {
        const int* gpos = event_pos(a.pos, id);
        const bool rotate = gpos != nullptr;
        long long pref = 0;
        if (rotate) {
            if (a.p_ref) pref = a.p_ref[id.b];
            else {
                int pmax = INT_MIN;
                for (int j = tid; j < n; j += kWThreads) pmax = max(pmax, gpos[j]);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) pmax = max(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, off));
                if (lane == 0) redi[warp] = pmax;
                __syncthreads();
                pref = (long long)max(max(redi[0], redi[1]), max(redi[2], redi[3])) + 1;
            }
        }
        // lane covers frequencies f0..f0+3 of the row handled by its half warp
        const int grp = lane >> 4, f0 = (lane & 15) * 4;
        const float* q = a.qstat + ((long long)id.l * lay.H + id.h) * kWD;
        const float inv = rsqrtf((float)kWD);
        float2 g[4];
        uint32_t phi_lo[4], phi_hi[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float qr = q[f0 + u] * inv, qi = q[f0 + u + 64] * inv;
            const float2 c = tab.cw[f0 + u];
            g[u] = make_float2(c.x * qr - c.y * qi, c.x * qi + c.y * qr);
            phi_lo[u] = (uint32_t)tab.phi[f0 + u];
            phi_hi[u] = (uint32_t)(tab.phi[f0 + u] >> 32);
        }
        // two rows per warp and step, the next step's loads in flight while this one is computed
        const int jstep = 2 * kWWarps;
        int j = 2 * warp + grp;
        uint2 kr = make_uint2(0, 0), ki = make_uint2(0, 0);
        int pj = 0;
        if (j < n) {
            const __nv_bfloat16* row = Kg + row_offset(lay, id.b, id.l, id.h, j);
            kr = __ldg(reinterpret_cast<const uint2*>(row + f0));
            ki = __ldg(reinterpret_cast<const uint2*>(row + 64 + f0));
            if (rotate) pj = gpos[j];
        }
        for (int j0 = 2 * warp; j0 < n; j0 += jstep) {
            const int jn = j + jstep;
            uint2 nkr = make_uint2(0, 0), nki = make_uint2(0, 0);
            int npj = 0;
            if (jn < n) {
                const __nv_bfloat16* row = Kg + row_offset(lay, id.b, id.l, id.h, jn);
                nkr = __ldg(reinterpret_cast<const uint2*>(row + f0));
                nki = __ldg(reinterpret_cast<const uint2*>(row + 64 + f0));
                if (rotate) npj = gpos[jn];
            }
            const float kre[4] = {bf16lo(kr.x), bf16hi(kr.x), bf16lo(kr.y), bf16hi(kr.y)};
            const float kim[4] = {bf16lo(ki.x), bf16hi(ki.x), bf16lo(ki.y), bf16hi(ki.y)};
            const long long dist = pref - (long long)pj;
            const uint32_t dlo = (uint32_t)dist, dhi = (uint32_t)((unsigned long long)dist >> 32);
            float acc = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float tr = fmaf(g[u].x, kre[u], g[u].y * kim[u]);
                const float ti = fmaf(g[u].y, kre[u], -g[u].x * kim[u]);
                if (rotate) {
                    // bits 32..63 of dist * phi (mod 2^64)
                    const uint32_t top = __umulhi(dlo, phi_lo[u]) + dlo * phi_hi[u] + dhi * phi_lo[u];
                    float sn, cs;
                    sincos_phase(top, sn, cs);
                    acc += fmaf(tr, cs, -ti * sn);
                } else {
                    acc += tr;
                }
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
            if (j < n && (lane & 15) == 0) {
                if (a.scores) a.scores[(long long)id.e * N + j] = acc;
                const bool fin = isfinite(acc);
                bad |= !fin;
                s[j] = fin ? acc : -INFINITY;
            }
            j = jn; kr = nkr; ki = nki; pj = npj;
        }
    } else {
        for (int j = tid; j < n; j += kWThreads) {
            const float sc = a.scores[(long long)id.e * N + j];
            const bool fin = isfinite(sc);
            bad |= !fin;
            s[j] = fin ? sc : -INFINITY;
        }
    }

    // ---- V tile arrival (bounded) ----------------------------------------------------------------
    int timeout = 0;
    if (needV) timeout = !mbar_wait_bounded(bar, 0);
    timeout = __syncthreads_or(timeout);
    bad = __syncthreads_or(bad);
    if (timeout) {
        if (tid == 0 && a.status) a.status[id.e] = 3;
        if (needV) mbar_wait_bounded(bar, 0);  // give copies still in flight another bounded chance to land
        return;
    }

    // ---- reciprocal norms from the diagonal of V V^T, one 16-row tile per warp and pass ------------
    const int g8 = lane >> 2, q4 = lane & 3;
    const int ntile = (n + 15) >> 4;
    if (similarity) {
        for (int t = warp; t < ntile; t += kWWarps) {
            float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t abase = vt_u32 + (16 * t + (lane & 7) + ((lane >> 3) & 1) * 8) * kVRowBytes + (lane >> 4) * 16;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                uint32_t a0, a1, a2, a3;
                ldsm_x4(abase + kk * 32, a0, a1, a2, a3);
                mma_bf16(d0, a0, a1, a2, a3, a0, a2);  // columns = rows 0..7 of the tile
                mma_bf16(d1, a0, a1, a2, a3, a1, a3);  // columns = rows 8..15
            }
            if ((g8 >> 1) == q4) {
                const float n0 = (g8 & 1) ? d0[1] : d0[0];
                const float n1 = (g8 & 1) ? d1[3] : d1[2];
                r[16 * t + g8] = 1.f / (sqrtf(n0) + a.eps);
                r[16 * t + g8 + 8] = 1.f / (sqrtf(n1) + a.eps);
            }
        }
    }
    __syncthreads();

    // ---- Algorithm 1 in warp 0 ---------------------------------------------------------------------
    if (warp == 0) {
        float sv[CPL], M[CPL], lr[CPL];
        uint32_t alive = 0;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const int j = lane + 32 * k;
            sv[k] = 0.f; M[k] = 0.f; lr[k] = 0.f;
            if (j < n) {
                sv[k] = s[j];
                lr[k] = similarity ? a.lam * r[j] : 0.f;
                alive |= 1u << k;
            }
        }
        const uint32_t alive0 = alive;
        int mycand = -1;  // lanes 0..7: the batch's candidates
        for (int t = 0; t < picks; ++t) {
            // a = s - lambda m (a[S] = -inf by the alive mask); i = argmax a, ties to the lower index
            uint32_t bk = 0;
            int bj = 0;
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                const uint32_t key = orderable(fmaf(-lr[k], M[k], sv[k]));
                if (((alive >> k) & 1u) && key > bk) { bk = key; bj = lane + 32 * k; }
            }
            const uint32_t gmax = __reduce_max_sync(0xFFFFFFFFu, bk);
            const int i = (int)__reduce_min_sync(0xFFFFFFFFu, (bk == gmax && bk != 0u) ? (uint32_t)bj : 0xFFFFFFFFu);
            const int owner = i & 31;
            if (lane == owner) alive &= ~(1u << (i >> 5));
            if (lane == 0) { order[t] = i; gain[t] = from_orderable(gmax); }
            if (!similarity || t + 1 == picks) continue;

            // m <- max(m, Sims[i, :]); the row comes from the current batch, or a new batch is made
            uint32_t hit = __ballot_sync(0xFFFFFFFFu, lane < kBatch && mycand == i);
            if (!hit) {
                // batch = i plus the best remaining candidate of up to 7 other lanes
                uint32_t k2 = (lane == owner) ? 0u : bk;
                int mine = (lane == 0) ? i : -1;
#pragma unroll
                for (int slot = 1; slot < kBatch; ++slot) {
                    const uint32_t gm = __reduce_max_sync(0xFFFFFFFFu, k2);
                    int jj = (int)__reduce_min_sync(0xFFFFFFFFu, (k2 == gm && k2 != 0u) ? (uint32_t)bj : 0xFFFFFFFFu);
                    if (gm == 0u) jj = i;
                    else if ((jj & 31) == lane) k2 = 0u;
                    if (lane == slot) mine = jj;
                }
                mycand = mine;
                const int crow = __shfl_sync(0xFFFFFFFFu, mycand, lane & 7);
                uint32_t bf[8][2];
                const uint32_t bbase = vt_u32 + crow * kVRowBytes + (lane >> 3) * 16;
#pragma unroll
                for (int p = 0; p < 4; ++p) ldsm_x4(bbase + p * 64, bf[2 * p][0], bf[2 * p][1], bf[2 * p + 1][0], bf[2 * p + 1][1]);
                float acc[NT][4];
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) { acc[tt][0] = acc[tt][1] = acc[tt][2] = acc[tt][3] = 0.f; }
                const uint32_t arow = vt_u32 + ((lane & 7) + ((lane >> 3) & 1) * 8) * kVRowBytes + (lane >> 4) * 16;
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) {
                    if (tt < ntile) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            uint32_t a0, a1, a2, a3;
                            ldsm_x4(arow + tt * 16 * kVRowBytes + kk * 32, a0, a1, a2, a3);
                            mma_bf16(acc[tt], a0, a1, a2, a3, bf[kk][0], bf[kk][1]);
                        }
                    }
                }
                __syncwarp();
#pragma unroll
                for (int tt = 0; tt < NT; ++tt) {
                    float* col = gcol + (2 * q4) * sp.gstride + 16 * tt + g8;
                    col[0] = acc[tt][0];
                    col[sp.gstride] = acc[tt][1];
                    col[8] = acc[tt][2];
                    col[sp.gstride + 8] = acc[tt][3];
                }
                __syncwarp();
                hit = 1u;  // slot 0 holds i
            }
            const int c = __ffs(hit) - 1;
            const float ri = r[i];
            const float* col = gcol + c * sp.gstride + lane;
#pragma unroll
            for (int k = 0; k < CPL; ++k) M[k] = fmaxf(M[k], ri * col[32 * k]);
        }
        // sort(S): ascending indices of the taken candidates
        const uint32_t taken = alive0 & ~alive;
        int base = 0;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const bool f = (taken >> k) & 1u;
            const uint32_t mask = __ballot_sync(0xFFFFFFFFu, f);
            if (f) idx[base + __popc(mask & ((1u << lane) - 1u))] = lane + 32 * k;
            base += __popc(mask);
        }
        for (int t = base + lane; t < a.budget; t += 32) idx[t] = -1;
    }
    __syncthreads();

    // ---- outputs -----------------------------------------------------------------------------------
    const long long ob = (long long)id.e * a.budget;
    for (int t = tid; t < a.budget; t += kWThreads) {
        a.idx_sorted[ob + t] = idx[t];
        if (a.pick_order) a.pick_order[ob + t] = t < picks ? order[t] : -1;
        if (a.pick_gain) a.pick_gain[ob + t] = t < picks ? gain[t] : 0.f;
    }
    if (tid == 0) {
        if (a.n_kept) a.n_kept[id.e] = picks;
        if (a.status) a.status[id.e] = n < a.budget ? 2 : (bad ? 1 : 0);
    }
    if (!FUSED) return;

    // ---- compaction in place: V from the tile; K and positions staged on chip before any store -----
    for (int x = tid; x < picks * 16; x += kWThreads) {
        const int rr = x >> 4, c = x & 15;
        copy16(reinterpret_cast<char*>(Vg + row_offset(lay, id.b, id.l, id.h, rr)) + c * 16,
               vt + idx[rr] * kVRowBytes + c * 16);
    }
    int* wpos = a.pos.p ? a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh : nullptr;
    __syncthreads();  // the V tile is free from here on
    __nv_bfloat16* Kw = reinterpret_cast<__nv_bfloat16*>(a.K);
    for (int x = tid; x < picks * 16; x += kWThreads) {
        const int rr = x >> 4, c = x & 15;
        copy16(vt + rr * kVRowBytes + c * 16,
               reinterpret_cast<const char*>(Kw + row_offset(lay, id.b, id.l, id.h, idx[rr])) + c * 16);
    }
    if (wpos)
        for (int t = tid; t < picks; t += kWThreads) order[t] = wpos[idx[t]];
    __syncthreads();
    for (int x = tid; x < picks * 16; x += kWThreads) {
        const int rr = x >> 4, c = x & 15;
        copy16(reinterpret_cast<char*>(Kw + row_offset(lay, id.b, id.l, id.h, rr)) + c * 16, vt + rr * kVRowBytes + c * 16);
    }
    if (wpos)
        for (int t = tid; t < picks; t += kWThreads) wpos[t] = order[t];
}

}  // namespace akv
