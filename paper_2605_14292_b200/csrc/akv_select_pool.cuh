// General selection kernel (any dtype, d, N): Algorithm 1 restricted to the candidates that can be
// picked at all. With m <= 1, a candidate with s_i < s_(b) - lambda (1 + slack) is never an arg-max
// while fewer than b are chosen, so the loop runs over that pool only (slot order, exact same picks)
// and only the pool's signature rows are read; they are kept in shared memory when they fit.
#pragma once
#include "akv_kernels.cuh"

namespace akv {

// Signature rows of pool members: pool row rho is slot pool[rho] of the event's V (or flat signature).
template <typename T>
struct PoolLayoutRows {
    const T* base;
    const DevLayout* lay;
    int b, l, h;
    const int* pool;
    __device__ __forceinline__ const T* operator()(int rho) const { return base + row_offset(*lay, b, l, h, pool[rho]); }
};
template <typename T>
struct PoolStridedRows {
    const T* base;
    long long stride;
    const int* pool;
    __device__ __forceinline__ const T* operator()(int rho) const { return base + (long long)pool[rho] * stride; }
};

struct PoolSmem {
    unsigned s, pool, ps, r, m, ptaken, taken, order, gain, idx, red, tile, total;
};
// tile_rows: pool rows that fit in the tile (0: rows are always read from global memory)
__host__ __device__ inline PoolSmem plan_pool_smem(int N, int budget, int row_bytes, int tile_rows) {
    PoolSmem p;
    const unsigned np = (unsigned)((N + 3) & ~3);
    unsigned o = 0;
    p.s = o;      o += align16(np * 4);
    p.pool = o;   o += align16(np * 4);
    p.ps = o;     o += align16(np * 4);
    p.r = o;      o += align16(np * 4);
    p.m = o;      o += align16(np * 4);
    p.ptaken = o; o += align16(np);
    p.taken = o;  o += align16(np);
    p.order = o;  o += align16((unsigned)budget * 4);
    p.gain = o;   o += align16((unsigned)budget * 4);
    p.idx = o;    o += align16((unsigned)budget * 4);
    p.red = o;    o += align16(2u * kWarps * 8u + 4u * kWarps * 4u);
    p.tile = o;   o += (unsigned)tile_rows * (unsigned)row_bytes;
    p.total = o;
    return p;
}

// block-wide sum of a per-thread count (all threads call); scratch: kWarps ints
__device__ __forceinline__ int block_sum_int(int v, int* scratch) {
    v = __reduce_add_sync(0xFFFFFFFFu, v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += scratch[w];
    return t;
}

// T: storage type of the rows the cosine is taken on (V's element type, or float for flat signatures)
template <typename T, bool FLAT>
__global__ void __launch_bounds__(kThreads) select_pool_kernel(const EventArgs a, int tile_rows) {
    extern __shared__ __align__(16) unsigned char smem[];
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int d = lay.d, N = lay.N;
    const int row_bytes = d * (int)sizeof(T);
    const PoolSmem sp = plan_pool_smem(N, a.budget, row_bytes, tile_rows);
    float* s = reinterpret_cast<float*>(smem + sp.s);
    int* pool = reinterpret_cast<int*>(smem + sp.pool);
    float* ps = reinterpret_cast<float*>(smem + sp.ps);
    float* r = reinterpret_cast<float*>(smem + sp.r);
    float* m = reinterpret_cast<float*>(smem + sp.m);
    unsigned char* ptaken = smem + sp.ptaken;
    unsigned char* taken = smem + sp.taken;
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    unsigned long long* red = reinterpret_cast<unsigned long long*>(smem + sp.red);
    int* redi = reinterpret_cast<int*>(smem + sp.red + 2 * kWarps * 8);
    T* tile = reinterpret_cast<T*>(smem + sp.tile);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool similarity = a.greedy != 0;
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);

    int bad = 0;
    for (int j = tid; j < n; j += kThreads) {
        const float sc = a.scores[(long long)id.e * N + j];
        const bool fin = isfinite(sc);
        bad |= !fin;
        s[j] = fin ? sc : -INFINITY;
        taken[j] = 0;
    }
    bad = __syncthreads_or(bad);

    // ---- s_(b): the picks-th largest score, by bisection over order-preserving integer keys -----------
    uint32_t kb = 0u;
    if (picks > 0) {
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t v = kb | (1u << bit);
            int cnt = 0;
            for (int j = tid; j < n; j += kThreads) cnt += orderable(s[j]) >= v;
            if (block_sum_int(cnt, redi) >= picks) kb = v;
        }
    }
    const float sb = from_orderable(kb);
    const float thr = a.no_prune ? -INFINITY : fmaf(-1.001f, a.lam, sb) - 1e-6f * fabsf(sb);  // -inf keeps everyone

    // ---- pool, in slot order (block-wide scan over chunks of kThreads slots) --------------------------
    int P = 0;
    for (int j0 = 0; j0 < n; j0 += kThreads) {
        const int j = j0 + tid;
        const bool in = j < n && (similarity ? !(s[j] < thr) : orderable(s[j]) >= kb);
        const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
        __syncthreads();
        if (lane == 0) redi[warp] = __popc(mask);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            before += w < warp ? redi[w] : 0;
            total += redi[w];
        }
        if (in) {
            const int rho = P + before + __popc(mask & ((1u << lane) - 1u));
            pool[rho] = j;
            ps[rho] = s[j];
        }
        P += total;
    }
    __syncthreads();
    for (int rho = tid; rho < P; rho += kThreads) {
        m[rho] = 0.f;
        ptaken[rho] = 0;
    }

    // ---- the pool's rows: into the tile when they fit, reciprocal norms (Eq. 1) ---------------------------
    const T* gbase = FLAT ? reinterpret_cast<const T*>(event_sig(a, id)) : reinterpret_cast<const T*>(a.V);
    PoolLayoutRows<T> lrows{gbase, &lay, id.b, id.l, id.h, pool};
    PoolStridedRows<T> frows{gbase, d, pool};
    StridedRows<T> trows{tile, d};
    const bool resident = similarity && P <= tile_rows;
    if (resident) {
        const int cpr = row_bytes / 16;
        for (int x = tid; x < P * cpr; x += kThreads) {
            const int rho = x / cpr, c = x - rho * cpr;
            const T* src = FLAT ? frows(rho) : lrows(rho);
            copy16(reinterpret_cast<char*>(tile) + (size_t)x * 16, reinterpret_cast<const char*>(src) + c * 16);
        }
        __syncthreads();
    }
    if (similarity && !FLAT) {
        const int G = pow2_ceil(d >> 3) > 32 ? 32 : pow2_ceil(d >> 3);
        const int RPW = 32 / G, grp = lane / G, lig = lane % G;
        for (int j0 = warp * RPW; j0 < P; j0 += kWarps * RPW) {
            const int rho = j0 + grp;
            const bool valid = rho < P;
            const T* row = resident ? trows(valid ? rho : 0) : lrows(valid ? rho : 0);
            const float ss = sumsq_row(row, valid, d, lig, G);
            if (valid && lig == 0) r[rho] = 1.f / (sqrtf(ss) + a.eps);
        }
    }
    __syncthreads();

    // ---- Algorithm 1 over the pool ----------------------------------------------------------------------
    const float* rr = FLAT ? nullptr : r;  // flat signatures are unit rows already
    if (resident) greedy_cta<T>(P, picks, a.lam, similarity, d, ps, rr, m, ptaken, order, gain, trows, red);
    else if (FLAT) greedy_cta<T>(P, picks, a.lam, similarity, d, ps, rr, m, ptaken, order, gain, frows, red);
    else greedy_cta<T>(P, picks, a.lam, similarity, d, ps, rr, m, ptaken, order, gain, lrows, red);
    for (int t = tid; t < picks; t += kThreads) {
        const int j = pool[order[t]];
        order[t] = j;
        taken[j] = 1;
    }
    __syncthreads();
    ordered_indices(n, a.budget, taken, idx);
    __syncthreads();
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
}

}  // namespace akv
