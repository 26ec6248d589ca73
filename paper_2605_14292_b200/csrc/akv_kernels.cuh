// Kernels: fused resident event, stand-alone score / compact, flat signature (Eq. 1).
#pragma once
#include "akv_steps.cuh"

namespace akv {

struct EventArgs {
    DevLayout lay;
    void* K;
    void* V;
    PosDesc pos;
    const int* n_cand;      // [B] or null
    const float* qstat;     // [L,H,d]
    const int* p_ref;       // [B] or null
    const float* flat_sig;  // shared signatures, or null: [B,N,d] (Eq. 1) or [B,L,N,d] (per layer)
    long long sig_sb, sig_sl;  // element strides of flat_sig over sequences and layers (0 for the flat mode's layers)
    const float* gram;         // cosine matrix of the shared signatures, or null: [B,N,N] (Eq. 1) or [B,L,N,N] (per layer)
    long long gram_sb, gram_sl;  // its element strides over sequences and layers
    const int* head_budgets;   // [L,H] or null: per-(layer, head) budgets, each <= budget
    int budget;             // largest budget of the call = row length of the index outputs
    float lam, eps;
    int greedy;             // 1: run the loop with similarity updates; 0: top-k
    int no_prune;           // 1: keep every candidate in the pool the loop runs over
    int tmem_cols;          // tensor-memory columns the tensor-memory kernel claims per CTA (0: none)
    int no_chain;           // testing aid: score every row from scratch even when positions are regular
    int gqa_group;          // query statistics per KV head (>= 1)
    int gqa_max;            // 1: a key's score is the largest over the group, 0: their mean
    int starve;             // testing aid: request no K row, so that the bounded waits run out
    int wait_polls;         // polls after which a bounded wait gives up
    int* idx_sorted;
    int* pick_order;
    float* pick_gain;
    float* scores;          // in (select) / out (score, fused)
    int* n_kept;
    int* status;
};

__device__ __forceinline__ int event_n(const EventArgs& a, int b) {
    int n = a.n_cand ? a.n_cand[b] : a.lay.N;
    return n < 0 ? 0 : (n > a.lay.N ? a.lay.N : n);
}

// rows this event keeps at most: its (layer, head) budget when budgets are given per head
__device__ __forceinline__ int event_budget(const EventArgs& a, const EventId& id) {
    if (!a.head_budgets) return a.budget;
    const int b = a.head_budgets[id.l * a.lay.H + id.h];
    return b < 1 ? 1 : (b > a.budget ? a.budget : b);
}
// shared signature rows of this event's (sequence, layer)
__device__ __forceinline__ const float* event_sig(const EventArgs& a, const EventId& id) {
    return a.flat_sig + id.b * a.sig_sb + id.l * a.sig_sl;
}

// Folded statistics of the event's query group into g[member * (d / 2) + f]; returns how many a row's score is
// the maximum of (1 when the group is averaged: the score is linear in the statistic, so the mean of the
// members' scores is the score of their mean statistic).
constexpr int kMaxGroup = 8;
__device__ __forceinline__ int fold_group(const EventArgs& a, const EventId& id, const ScoreTab& tab, int d, float2* g) {
    const int G = a.gqa_group < 1 ? 1 : a.gqa_group, half = d >> 1;
    const float* q = a.qstat + ((long long)id.l * a.lay.H + id.h) * G * d;
    const float inv = rsqrtf((float)d);
    if (a.gqa_max) {
        for (int x = threadIdx.x; x < G * half; x += blockDim.x) {
            const int m = x / half, f = x - m * half;
            const float qr = q[m * d + f] * inv, qi = q[m * d + f + half] * inv;
            const float2 c = tab.cw[f];
            g[x] = make_float2(c.x * qr - c.y * qi, c.x * qi + c.y * qr);
        }
        return G;
    }
    for (int f = threadIdx.x; f < half; f += blockDim.x) {
        float qr = 0.f, qi = 0.f;
        for (int m = 0; m < G; ++m) {
            qr += q[m * d + f];
            qi += q[m * d + f + half];
        }
        qr *= inv / (float)G;
        qi *= inv / (float)G;
        const float2 c = tab.cw[f];
        g[f] = make_float2(c.x * qr - c.y * qi, c.x * qi + c.y * qr);
    }
    return 1;
}
// score of one row against every member's statistic, reduced by the maximum (one member: the plain score)
template <typename T>
__device__ __forceinline__ float score_group(const T* krow, bool valid, long long dist, bool rotate, int d,
                                             const unsigned long long* phi, const float2* g, int lig, int G, int members) {
    float best = score_row(krow, valid, dist, rotate, d, phi, g, lig, G);
    for (int m = 1; m < members; ++m) best = fmaxf(best, score_row(krow, valid, dist, rotate, d, phi, g + m * (d >> 1), lig, G));
    return best;
}

__device__ __forceinline__ const int* event_pos(const PosDesc& p, const EventId& id) {
    return p.p ? p.p + id.b * p.sb + id.l * p.sl + id.h * p.sh : nullptr;
}

// block-wide max of int values (all threads call); scratch: kWarps ints
__device__ __forceinline__ int block_max_int(int v, int* scratch) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    int r = scratch[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) r = max(r, scratch[w]);
    return r;
}

// Shared-memory carve-up used by the per-event kernels. Offsets in bytes, 16-byte aligned blocks.
struct SmemPlan {
    unsigned tileK, tileV, phi, g, pos, s, r, m, order, gain, idx, taken, red, total;
};
__host__ __device__ inline unsigned align16(unsigned x) { return (x + 15u) & ~15u; }
__host__ __device__ inline SmemPlan plan_smem(int N, int d, int esize, int budget, bool withK, bool withV) {
    SmemPlan p;
    unsigned o = 0;
    p.tileK = o; o += withK ? align16((unsigned)N * d * esize) : 0;
    p.tileV = o; o += withV ? align16((unsigned)N * d * esize) : 0;
    p.phi = o;   o += align16((unsigned)(d / 2) * 8);
    p.g = o;     o += align16((unsigned)(d / 2) * 8) * kMaxGroup;  // folded statistic of every member of a query group
    p.pos = o;   o += align16((unsigned)N * 4);
    p.s = o;     o += align16((unsigned)N * 4);
    p.r = o;     o += align16((unsigned)N * 4);
    p.m = o;     o += align16((unsigned)N * 4);
    p.order = o; o += align16((unsigned)budget * 4);
    p.gain = o;  o += align16((unsigned)budget * 4);
    p.idx = o;   o += align16((unsigned)budget * 4);
    p.taken = o; o += align16((unsigned)N);
    p.red = o;   o += align16(2u * kWarps * 8u + kWarps * 4u);
    p.total = o;
    return p;
}

// ---------------------------------------------------------------------------------------------
// Stand-alone score: one CTA per (event, block of kScoreRows rows), both folded into grid.x; K
// streamed from global memory once.
// ---------------------------------------------------------------------------------------------
constexpr int kScoreRows = 64;  // rows per CTA

template <typename T>
__global__ void __launch_bounds__(kThreads) score_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab) {
    __shared__ unsigned long long phi[kMaxHalf];
    __shared__ float2 g[kMaxGroup * kMaxHalf];
    __shared__ int redi[kWarps];
    const DevLayout& lay = a.lay;
    const int row_blocks = (lay.N + kScoreRows - 1) / kScoreRows;
    const EventId id = decode_event(lay, blockIdx.x / row_blocks);
    const int n = event_n(a, id.b);
    const int d = lay.d;
    const int row0 = (blockIdx.x % row_blocks) * kScoreRows;
    if (row0 >= n) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int* gpos = event_pos(a.pos, id);
    for (int f = tid; f < d / 2; f += kThreads) phi[f] = tab.phi[f];
    const int members = fold_group(a, id, tab, d, g);
    long long pref = 0;
    if (gpos) {
        if (a.p_ref) pref = a.p_ref[id.b];
        else {
            int pmax = INT_MIN;
            for (int j = tid; j < n; j += kThreads) pmax = max(pmax, gpos[j]);
            pref = (long long)block_max_int(pmax, redi) + 1;
        }
    }
    __syncthreads();
    const int G = pow2_ceil(d >> 3) > 32 ? 32 : pow2_ceil(d >> 3);
    const int RPW = 32 / G, grp = lane / G, lig = lane % G;
    const T* Kg = reinterpret_cast<const T*>(a.K);
    int bad = 0;
    const int rend = min(n, row0 + kScoreRows);
    for (int j0 = row0 + warp * RPW; j0 < rend; j0 += kWarps * RPW) {
        const int j = j0 + grp;
        const bool valid = j < rend;
        const long long dist = (valid && gpos) ? pref - (long long)gpos[j] : 0;
        const T* krow = Kg + (valid ? row_offset(lay, id.b, id.l, id.h, j) : 0);
        const float sc = score_group(krow, valid, dist, gpos != nullptr, d, phi, g, lig, G, members);
        if (valid && lig == 0) {
            a.scores[(long long)id.e * lay.N + j] = sc;
            bad |= !isfinite(sc);
        }
    }
    if (a.status) {
        bad = __syncthreads_or(bad);
        if (tid == 0 && bad) atomicMax(a.status + id.e, 1);
    }
}

// zero a status array before the score kernel's atomicMax
__global__ void fill_int_kernel(int* p, long long n, int v) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

// ---------------------------------------------------------------------------------------------
// Stand-alone compaction, in place. Rows move in ascending chunks staged through shared memory:
// a chunk's destinations [c0, c1) can only overlap sources of the same chunk (idx[r] >= r and idx
// ascending), which are on chip before the first store.
// ---------------------------------------------------------------------------------------------
struct CompactArgs {
    DevLayout lay;
    void* K;
    void* V;
    PosDesc pos;
    const int* idx_sorted;
    int budget;
    int chunk_rows;
};

template <typename T>
__global__ void __launch_bounds__(kThreads) compact_kernel(const CompactArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int d = lay.d;
    const int tid = threadIdx.x;
    const int rowB = d * (int)sizeof(T);
    const int cpr = rowB / 16;
    unsigned char* stK = smem;
    unsigned char* stV = smem + (size_t)a.chunk_rows * rowB;
    int* sidx = reinterpret_cast<int*>(smem + 2 * (size_t)a.chunk_rows * rowB);
    int* spos = sidx + a.chunk_rows;
    const int* gidx = a.idx_sorted + (long long)id.e * a.budget;
    T* Kg = reinterpret_cast<T*>(a.K);
    T* Vg = reinterpret_cast<T*>(a.V);
    int* gpos = a.pos.p ? a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh : nullptr;
    for (int c0 = 0; c0 < a.budget; c0 += a.chunk_rows) {
        const int cn = min(a.chunk_rows, a.budget - c0);
        __syncthreads();
        for (int t = tid; t < cn; t += kThreads) {
            const int src = gidx[c0 + t];
            sidx[t] = (src >= 0 && src < lay.N) ? src : -1;
            if (gpos && sidx[t] >= 0) spos[t] = gpos[src];
        }
        __syncthreads();
        for (int x = tid; x < cn * cpr; x += kThreads) {
            const int rr = x / cpr, c = x - rr * cpr;
            const int src = sidx[rr];
            if (src < 0) continue;
            const long long off = row_offset(lay, id.b, id.l, id.h, src);
            if (Kg) copy16(stK + (size_t)x * 16, reinterpret_cast<const char*>(Kg + off) + c * 16);
            if (Vg) copy16(stV + (size_t)x * 16, reinterpret_cast<const char*>(Vg + off) + c * 16);
        }
        __syncthreads();
        for (int x = tid; x < cn * cpr; x += kThreads) {
            const int rr = x / cpr, c = x - rr * cpr;
            if (sidx[rr] < 0) continue;
            const long long off = row_offset(lay, id.b, id.l, id.h, c0 + rr);
            if (Kg) copy16(reinterpret_cast<char*>(Kg + off) + c * 16, stK + (size_t)x * 16);
            if (Vg) copy16(reinterpret_cast<char*>(Vg + off) + c * 16, stV + (size_t)x * 16);
        }
        if (gpos)
            for (int t = tid; t < cn; t += kThreads)
                if (sidx[t] >= 0) gpos[c0 + t] = spos[t];
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 1: shared signatures. u = mean over (l, h) of the V rows of one (sequence, slot), v = u / (||u|| + eps),
// written as fp32 [B, N, d]; per_layer: one signature per (sequence, layer, slot), the mean runs over the heads
// of that layer only, written as fp32 [B, L, N, d]. One CTA per (group, 32 / G slots), G = lanes per row: its
// eight warps split the (layer, head) pairs among themselves (every thread has a dozen independent 16-byte
// loads in flight), partial sums meet in shared memory in a fixed order.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) flat_signature_kernel(const DevLayout lay, const void* V, const int* n_cand,
                                                                 float eps, float* out, int per_layer) {
    __shared__ float part[kWarps][32][8];
    const int d = lay.d;
    const int G = pow2_ceil(d >> 3) > 32 ? 32 : pow2_ceil(d >> 3);
    const int RPW = 32 / G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane / G, lig = lane % G;
    const int slot_blocks = (lay.N + RPW - 1) / RPW;
    const int grpi = blockIdx.x / slot_blocks;                         // sequence, or (sequence, layer)
    const int j = (blockIdx.x % slot_blocks) * RPW + grp;
    const int b = per_layer ? grpi / lay.L : grpi;
    const int l0 = per_layer ? grpi % lay.L : 0, l1 = per_layer ? l0 + 1 : lay.L;
    int n = n_cand ? n_cand[b] : lay.N;
    n = n < 0 ? 0 : (n > lay.N ? lay.N : n);
    const bool valid = j < n;
    const bool act = valid && lig * 8 < d;
    const T* Vg = reinterpret_cast<const T*>(V);
    const int pairs = (l1 - l0) * lay.H;
    float u[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (act) {
        for (int p = warp; p < pairs; p += kWarps) {
            float x[8];
            load8(Vg + row_offset(lay, b, l0 + p / lay.H, p % lay.H, j) + lig * 8, x);
#pragma unroll
            for (int q = 0; q < 8; ++q) u[q] += x[q];
        }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) part[warp][lane][q] = u[q];
    __syncthreads();
    if (warp != 0) return;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) acc += part[w][lane][q];
        u[q] = acc * (1.f / (float)pairs);
    }
    float ss = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) ss = fmaf(u[q], u[q], ss);
    ss = group_sum(ss, G);
    if (act) {
        const float r = 1.f / (sqrtf(ss) + eps);
        float* o = out + ((long long)grpi * lay.N + j) * d + lig * 8;
        *reinterpret_cast<float4*>(o) = make_float4(u[0] * r, u[1] * r, u[2] * r, u[3] * r);
        *reinterpret_cast<float4*>(o + 4) = make_float4(u[4] * r, u[5] * r, u[6] * r, u[7] * r);
    }
}

}  // namespace akv
