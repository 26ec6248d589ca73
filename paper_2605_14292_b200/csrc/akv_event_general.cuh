// Fused event for every shape the tensor-memory kernels do not take (fp32, head dimensions other than 128,
// grouped query statistics, shared signatures without a cosine matrix), when the event's K and V tiles fit in
// shared memory.
//
// Selection, when lambda > 0: the exact pool (s_i >= s_(b) - lambda (1 + slack), see akv_select_pool.cuh) is
// formed, and when the lower triangle of its cosine matrix fits in the shared memory left beside the tiles, the
// triangle is filled by plain fp32 dot products (every thread its own pairs of rows, each walking the head
// dimension from its own starting column so that a warp's loads fall into different banks) and Algorithm 1 runs
// as the one-warp loop of the tensor-memory kernels. Otherwise, and for lambda = 0, the CTA-wide loop with rows
// of the cosine matrix on demand (greedy_cta).
#pragma once
#include "akv_event_tri.cuh"

namespace akv {

// n rows of one event from global memory into a dense shared tile by 16-byte asynchronous copies, all in flight
// at once; the caller waits (cp_async_wait_all) and synchronises before reading the tile
template <typename T>
__device__ __forceinline__ void load_tile_async(T* tile, const T* base, const DevLayout& lay, const EventId& id, int n) {
    const int cpr = lay.d * (int)sizeof(T) / 16;  // 16-byte chunks per row
    const uint32_t t0 = smem_u32(tile);
    for (int x = threadIdx.x; x < n * cpr; x += kThreads) {
        const int row = x / cpr, c = x - row * cpr;
        cp_async16(t0 + (uint32_t)x * 16u, reinterpret_cast<const char*>(base + row_offset(lay, id.b, id.l, id.h, row)) + c * 16);
    }
}

// ---------------------------------------------------------------------------------------------
// Fused event, tiles resident in shared memory: K and V are read from HBM once and the kept rows
// are written once. One CTA per (sequence, layer, KV head).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) event_resident_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab, int extra_bytes) {
    extern __shared__ __align__(16) unsigned char smem[];
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int d = lay.d, N = lay.N;
    const SmemPlan sp = plan_smem(N, d, sizeof(T), a.budget, true, true);
    T* Kt = reinterpret_cast<T*>(smem + sp.tileK);
    T* Vt = reinterpret_cast<T*>(smem + sp.tileV);
    unsigned long long* phi = reinterpret_cast<unsigned long long*>(smem + sp.phi);
    float2* g = reinterpret_cast<float2*>(smem + sp.g);
    int* spos = reinterpret_cast<int*>(smem + sp.pos);
    float* s = reinterpret_cast<float*>(smem + sp.s);
    float* r = reinterpret_cast<float*>(smem + sp.r);
    float* m = reinterpret_cast<float*>(smem + sp.m);
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    unsigned char* taken = smem + sp.taken;
    unsigned long long* red = reinterpret_cast<unsigned long long*>(smem + sp.red);
    int* redi = reinterpret_cast<int*>(smem + sp.red + 2 * kWarps * 8);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int* gpos = event_pos(a.pos, id);
    T* Kg = reinterpret_cast<T*>(a.K);
    T* Vg = reinterpret_cast<T*>(a.V);

    // stage the event on chip
    load_tile_async(Kt, Kg, lay, id, n);
    load_tile_async(Vt, Vg, lay, id, n);
    int pmax = INT_MIN;
    for (int j = tid; j < n; j += kThreads) {
        const int p = gpos ? gpos[j] : 0;
        spos[j] = p;
        pmax = max(pmax, p);
        taken[j] = 0;
        m[j] = 0.f;
    }
    for (int f = tid; f < d / 2; f += kThreads) phi[f] = tab.phi[f];
    const int members = fold_group(a, id, tab, d, g);
    long long pref = 0;
    if (gpos) pref = a.p_ref ? (long long)a.p_ref[id.b] : (long long)block_max_int(pmax, redi) + 1;
    cp_async_wait_all();
    __syncthreads();

    // scores and reciprocal norms
    const int G = pow2_ceil(d >> 3) > 32 ? 32 : pow2_ceil(d >> 3);
    const int RPW = 32 / G, grp = lane / G, lig = lane % G;
    int bad = 0;
    for (int j0 = warp * RPW; j0 < n; j0 += kWarps * RPW) {
        const int j = j0 + grp;
        const bool valid = j < n;
        const long long dist = valid ? pref - (long long)spos[j] : 0;
        const float sc = score_group(Kt + (size_t)j * d, valid, dist, gpos != nullptr, d, phi, g, lig, G, members);
        const float ss = a.flat_sig ? 1.f : sumsq_row(Vt + (size_t)j * d, valid, d, lig, G);
        if (valid && lig == 0) {
            if (a.scores) a.scores[(long long)id.e * N + j] = sc;
            const bool fin = isfinite(sc);
            bad |= !fin;
            s[j] = fin ? sc : -INFINITY;
            r[j] = 1.f / (sqrtf(ss) + a.eps);
        }
    }
    bad = __syncthreads_or(bad);

    // selection
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);
    // ---- pool + triangle + one-warp loop, when it fits --------------------------------------------------------
    bool done = false;
    const unsigned lists = align16((unsigned)N * 2u) + align16((unsigned)N * 4u);
    if (a.greedy != 0 && picks > 1 && extra_bytes > (int)lists) {
        unsigned short* bypool = reinterpret_cast<unsigned short*>(smem + sp.total);
        float* rp = reinterpret_cast<float*>(smem + sp.total + align16((unsigned)N * 2u));
        float* tri = reinterpret_cast<float*>(smem + sp.total + lists);
        const int tri_floats = (extra_bytes - (int)lists) / 4;
        float* sb_holder = reinterpret_cast<float*>(red);
        int* pool_holder = redi;
        // s_(b): the value v with fewer than `picks` scores above it and at least `picks` not below it
        for (int j = tid; j < n; j += kThreads) {
            const uint32_t kj = orderable(s[j]);
            int gt = 0, ge = 0;
            for (int i = 0; i < n; ++i) {
                const uint32_t ki = orderable(s[i]);
                gt += ki > kj;
                ge += ki >= kj;
            }
            if (gt < picks && picks <= ge) *sb_holder = s[j];
        }
        __syncthreads();
        const float sb = *sb_holder;
        const float thr = a.no_prune ? -INFINITY : fmaf(-1.001f, a.lam, sb) - 1e-6f * fabsf(sb);
        if (warp == 0) {
            int base = 0;
            for (int j0 = 0; j0 < n; j0 += 32) {
                const int j = j0 + lane;
                const bool in = j < n && !(s[j] < thr);
                const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
                if (in) bypool[base + __popc(mask & ((1u << lane) - 1u))] = (unsigned short)j;
                base += __popc(mask);
            }
            if (lane == 0) *pool_holder = base;
        }
        __syncthreads();
        const int P = *pool_holder;
        const long long need = (long long)P * (P + 1) / 2;
        if (P <= 256 && need <= (long long)tri_floats) {
            done = true;
            const float* sig = a.flat_sig ? event_sig(a, id) : nullptr;
            for (int rho = tid; rho < P; rho += kThreads) rp[rho] = sig ? 1.f : r[bypool[rho]];
            // raw dot products of every pair of pool rows (i >= j): thread x takes pairs x, x + 256, ...; the
            // pair's row and column come from the inverse of the triangular numbering
            const int G4 = d >> 2;  // groups of four elements per row
            for (long long x = tid; x < need; x += kThreads) {
                int i = (int)((sqrtf(8.f * (float)x + 1.f) - 1.f) * 0.5f);
                while ((long long)i * (i + 1) / 2 > x) --i;
                while ((long long)(i + 1) * (i + 2) / 2 <= x) ++i;
                const int j = (int)(x - (long long)i * (i + 1) / 2);
                float acc = 0.f;
                int gq = tid % G4;
                if (sig) {
                    const float* vi = sig + (long long)bypool[i] * d;
                    const float* vj = sig + (long long)bypool[j] * d;
                    for (int c = 0; c < G4; ++c) {
                        float xi[4], xj[4];
                        load4(vi + 4 * gq, xi);
                        load4(vj + 4 * gq, xj);
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc = fmaf(xi[e], xj[e], acc);
                        gq = gq + 1 == G4 ? 0 : gq + 1;
                    }
                } else {
                    const T* vi = Vt + (size_t)bypool[i] * d;
                    const T* vj = Vt + (size_t)bypool[j] * d;
                    for (int c = 0; c < G4; ++c) {
                        float xi[4], xj[4];
                        load4(vi + 4 * gq, xi);
                        load4(vj + 4 * gq, xj);
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc = fmaf(xi[e], xj[e], acc);
                        gq = gq + 1 == G4 ? 0 : gq + 1;
                    }
                }
                tri[x] = acc;
            }
            __syncthreads();
            uint32_t* park_key = reinterpret_cast<uint32_t*>(gain);
            if (warp == 0) picks_cosine<8, false>(lane, P, picks, s, bypool, rp, a.lam, tri, park_key, order);
            __syncthreads();
            for (int t = tid; t < picks; t += kThreads) {
                const int j = bypool[order[t]];
                gain[t] = from_orderable(park_key[t]);
                order[t] = j;
                taken[j] = 1;
            }
            __syncthreads();
        }
    }
    if (!done) {
        if (a.flat_sig) {
            StridedRows<float> rows{event_sig(a, id), d};
            greedy_cta<float>(n, picks, a.lam, a.greedy != 0, d, s, nullptr, m, taken, order, gain, rows, red);
        } else {
            StridedRows<T> rows{Vt, d};
            greedy_cta<T>(n, picks, a.lam, a.greedy != 0, d, s, r, m, taken, order, gain, rows, red);
        }
    }
    ordered_indices(n, a.budget, taken, idx);
    __syncthreads();

    // outputs
    const long long ob = (long long)id.e * a.budget;
    for (int t = tid; t < a.budget; t += kThreads) {
        a.idx_sorted[ob + t] = idx[t];
        if (a.pick_order) a.pick_order[ob + t] = t < picks ? order[t] : -1;
        if (a.pick_gain) a.pick_gain[ob + t] = t < picks ? gain[t] : 0.f;
    }
    if (tid == 0) {
        if (a.n_kept) a.n_kept[id.e] = picks;
        if (a.status) a.status[id.e] = n < bud ? 2 : (bad ? 1 : 0);
    }
    // compaction: kept rows go to slots 0..picks-1 of the same buffer (all sources are on chip)
    const int cpr = d * (int)sizeof(T) / 16;
    for (int x = tid; x < picks * cpr; x += kThreads) {
        const int rr = x / cpr, c = x - rr * cpr;
        const int src = idx[rr];
        const long long off = row_offset(lay, id.b, id.l, id.h, rr);
        copy16(reinterpret_cast<char*>(Kg + off) + c * 16, reinterpret_cast<const char*>(Kt + (size_t)src * d) + c * 16);
        copy16(reinterpret_cast<char*>(Vg + off) + c * 16, reinterpret_cast<const char*>(Vt + (size_t)src * d) + c * 16);
    }
    if (gpos) {
        int* wpos = a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh;
        for (int t = tid; t < picks; t += kThreads) wpos[t] = spos[idx[t]];
    }
}

}  // namespace akv
