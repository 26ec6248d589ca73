// Fast event kernel for bf16, d = 128, per-head signatures, N <= 256, used when the pool that
// survives pruning is expected to stay within 127 rows (N <= 128 or budget <= 64). One CTA of four
// warps per event, six CTAs resident per SM (37 KB of shared memory and 72 registers each).
//
//   1. K rows arrive in shared memory by bulk copies (cp.async.bulk + mbarrier) and are scored there
//      (fused RoPE rotate-and-dot against the folded query statistic). The tile holds 128 rows: rows
//      from 128 on arrive later, in the slots of the first rows once those have been scored.
//   2. Only candidates with  s_i >= s_(b) - lambda * (1 + slack)  can ever be an argmax of Eq. 2
//      (the running maximum m never exceeds 1, so every still unchosen member of the top-b scores
//      beats the others). s_(b) comes from a bisection over the score keys; that pool of P rows,
//      in slot order, is the only part of V that is read for the selection.
//   3. P <= 127: the pool's V rows form a K-major, 128-byte-swizzled operand tile, one
//      tcgen05.mma sequence writes the pool's cosine matrix (raw dot products, fp32) into tensor
//      memory, and the four warps move its lower triangle to shared memory (tcgen05.ld), taking
//      the squared norms of Eq. 1 from the diagonal on the way.
//      P > 127 (hardly any pruning): no tensor-core product; rows of the cosine matrix are plain
//      dot products of V rows read in place, one picked row at a time.
//   4. Algorithm 1 runs in ONE warp: every lane owns up to P/32 candidates and keeps s, the
//      running maximum and lambda/norm in registers; the argmax is two warp reductions, the picked
//      row of the cosine matrix is read from the triangle without bank conflicts.
//   5. Kept rows are written back in place: K and V rows are re-read (L2) into the tile, which is
//      free by then, and stored after a barrier; positions come from their shared-memory copy.
#pragma once
#include "akv_event_tc.cuh"

namespace akv {

constexpr int kTriTileRows = 128;           // K rows resident at a time = rows of the V operand tile
constexpr unsigned kTriTileBytes = 32768u;  // 128 rows of 256 bytes; holds the triangle of up to 127 rows
constexpr int kTriMaxPool = 127;            // largest pool whose cosine matrix goes through the tile

struct TriSmem {
    unsigned tile, s, key, spos, bypool, taken, order, gain, idx, row, sect, misc, total;
};
// Layout after the 1024-byte aligned base. `key` (score keys) and `r` (reciprocal norms) share storage.
__host__ __device__ inline TriSmem plan_tri_smem(int N, int budget) {
    TriSmem p;
    const unsigned np = (unsigned)((N + 3) & ~3);
    unsigned o = 0;
    p.tile = o;   o += kTriTileBytes;
    p.s = o;      o += align16(np * 4);
    p.key = o;    o += align16(np * 4);
    p.spos = o;   o += align16(np * 4);
    p.bypool = o; o += align16(np * 2);
    p.taken = o;  o += align16(np);
    p.order = o;  o += align16((unsigned)budget * 4);
    p.gain = o;   o += align16((unsigned)budget * 4);
    p.idx = o;    o += align16((unsigned)budget * 4);
    if (o - p.bypool < 1024u) o = p.bypool + 1024u;  // bypool..idx also hold the folded statistic and the phase steps (1 KB) while scoring
    p.row = p.tile;               // one row of the cosine matrix: plain-dot route only, which leaves the tile unused
    p.sect = o;   o += 256;       // cosine and sine of the 32 sector angles
    p.misc = o;   o += 64;        // mbarriers (K, product, late K rows), tmem base, pool size, block-max scratch
    p.total = o + 1024;           // room to align the base to 1024 bytes
    return p;
}

// 32 consecutive columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// entry (a, b), a >= b, of a lower triangle stored row by row; rows a = lane + 32 k of one warp
// fall into 32 different banks for a fixed b, and so do consecutive b for a fixed a
__device__ __forceinline__ int tri_row(int a) { return (a * (a + 1)) >> 1; }

// Per-lane state of the single-warp greedy loop: candidates rho = lane + 32 k, k < CPL.
template <int CPL>
struct GreedyLane {
    float sv[CPL], lr[CPL], M[CPL];
    uint32_t am[CPL];  // all ones while the candidate competes; 0 once chosen, or when the row is empty
    __device__ __forceinline__ void init(int lane, int P, const float* s, const unsigned short* bypool, const float* r, float lam,
                                         bool use_r) {
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const int rho = lane + 32 * k;
            sv[k] = 0.f; lr[k] = 0.f; M[k] = 0.f; am[k] = 0u;
            if (rho < P) {
                sv[k] = s[bypool[rho]];
                lr[k] = use_r ? lam * r[rho] : 0.f;
                am[k] = 0xFFFFFFFFu;
            }
        }
    }
    // a = s - lambda m over the candidates still competing; returns the key of the best one and its
    // pool row (ties to the lower row, which is the lower slot) and retires it
    __device__ __forceinline__ int pick(int lane, uint32_t& best_key) {
        uint32_t key[CPL];
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const uint32_t u = __float_as_uint(fmaf(-lr[k], M[k], sv[k]));
            key[k] = (u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u)) & am[k];  // orderable(a), 0 when retired
        }
        uint32_t bk = key[0];
#pragma unroll
        for (int k = 1; k < CPL; ++k) bk = max(bk, key[k]);
        const uint32_t whi = __reduce_max_sync(0xFFFFFFFFu, bk);
        // lowest row among the candidates that reach the maximum (0xFFFF - row, so that max picks the lowest)
        uint32_t cand = 0u;
#pragma unroll
        for (int k = 0; k < CPL; ++k) cand = max(cand, key[k] == whi ? 0xFFFFu - (uint32_t)(lane + 32 * k) : 0u);
        const uint32_t wlo = __reduce_max_sync(0xFFFFFFFFu, cand);
        const int irho = (int)(0xFFFFu - wlo);
#pragma unroll
        for (int k = 0; k < CPL; ++k) am[k] = (lane + 32 * k == irho) ? 0u : am[k];
        best_key = whi;
        return irho;
    }
};

// One float of shared memory, as a volatile load: a group of these is issued back to back and in
// program order, where plain loads get strung out one per use (a picked row's four entries cost four
// exposed latencies that way).
__device__ __forceinline__ float lds_in_order(uint32_t addr) {
    float v;
    asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// The loop of Algorithm 1 run by one warp without any block-wide barrier. with_sims: the running
// maximum is updated from the triangle `tri` of raw dot products (needs P <= 128 and r); otherwise
// the picks are the plain arg-max sequence (top-k in pick order). The winning key and pool row of
// pick t are parked in park_key[t] / park_row[t]; inside the loop they stay in registers (lane t mod
// 32 keeps them) and reach shared memory once per 32 picks: a store per pick would order itself
// against the loads of the next row and lengthen every step.
template <int CPL>
__device__ __forceinline__ void picks_in_one_warp(int lane, int P, int picks, bool with_sims, const float* s,
                                                  const unsigned short* bypool, const float* r, float lam, const float* tri,
                                                  uint32_t* park_key, int* park_row) {
    GreedyLane<CPL> g;
    g.init(lane, P, s, bypool, r, lam, with_sims);
    const uint32_t tb = smem_u32(tri), rb = smem_u32(r);
    // Rows beyond the pool are clamped to its last row: their loads stay inside the triangle and the
    // loop needs no branch (a divergent branch per candidate costs far more than the wasted load);
    // what they compute is never looked at, those candidates are retired from the start.
    int rc4[CPL], trowB[CPL];  // 4 * row, and the byte offset of that row of the triangle
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
        const int rc = min(lane + 32 * k, max(P - 1, 0));
        rc4[k] = 4 * rc;
        trowB[k] = 4 * tri_row(rc);
    }
    for (int t0 = 0; t0 < picks; t0 += 32) {
        uint32_t my_key = 0u;
        int my_row = 0;
        const int t1 = min(t0 + 32, picks);
        for (int t = t0; t < t1; ++t) {
            uint32_t bk;
            const int irho = g.pick(lane, bk);
            const bool mine = lane == t - t0;
            my_key = mine ? bk : my_key;
            my_row = mine ? irho : my_row;
            if (!with_sims || t + 1 == picks) continue;
            // m <- max(m, Sims[i, :]) from the triangle: entry (max, min)
            const int tiB = 4 * tri_row(irho), irho4 = 4 * irho;
            uint32_t addr[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) addr[k] = tb + (uint32_t)(rc4[k] > irho4 ? trowB[k] + irho4 : tiB + rc4[k]);
            const float ri = lds_in_order(rb + irho4);
            float x[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) x[k] = lds_in_order(addr[k]);
#pragma unroll
            for (int k = 0; k < CPL; ++k) g.M[k] = fmaxf(g.M[k], ri * x[k]);
        }
        if (t0 + lane < picks) {
            park_key[t0 + lane] = my_key;
            park_row[t0 + lane] = my_row;
        }
    }
}

// Warp-wide maximum of a float (sm_100a has the reduction for f32).
__device__ __forceinline__ float warp_max_f32(float v) {
    float m;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
    return m;
}

// A non-finite score competes as this value: below every real score, above a retired candidate's -inf.
constexpr float kLowestScore = -3.0e38f;

// The loop of Algorithm 1 with the cosine penalty, Eq. 2 evaluated and compared as floats (no integer keys):
// a candidate is retired through the triangle itself. The diagonal entries are set to +inf before the first
// pick, so the update m <- max(m, Sims[i, :]) gives the picked row m = +inf and a = -inf from then on: no
// mask, no per-candidate retirement. Each lane reduces its candidates to one maximum before the warp-wide
// reduction and finds which candidate that was while the reduction is in flight. Winning values are parked as order-preserving keys, like the other loops'.
// BOUNDED as for picks_bounded; when the bound is reached the state of the loop can be handed back (see there).
// `tri` is modified (its diagonal).
template <int CPL, bool BOUNDED>
__device__ __forceinline__ bool picks_cosine(int lane, int P, int picks, const float* s, const unsigned short* bypool,
                                             const float* r, float lam, float* tri, uint32_t* park_key, int* park_row,
                                             uint32_t bound_key = 0u, float* m_out = nullptr, int* t_out = nullptr) {
    const uint32_t tb = smem_u32(tri), rb = smem_u32(r);
    const float ninf = __int_as_float(0xff800000), pinf = __int_as_float(0x7f800000);
    float sv[CPL], lr[CPL], M[CPL];
    int rc4[CPL];
    uint32_t trowB[CPL];  // 4 * row, and the shared-memory address of that row of the triangle
    const int last = max(P - 1, 0);
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
        const int rho = lane + 32 * k;
        const bool in = rho < P;
        // rows beyond the pool: -inf from the start, and a positive factor so that -inf - lr * m stays -inf
        sv[k] = in ? fmaxf(s[bypool[min(rho, last)]], kLowestScore) : ninf;
        lr[k] = in ? fmaxf(lam * r[rho], 1e-30f) : 1.f;
        M[k] = 0.f;
        const int rc = min(rho, last);  // clamped: the loads stay inside the triangle, the loop needs no branch
        rc4[k] = 4 * rc;
        trowB[k] = tb + 4u * (uint32_t)tri_row(rc);
        if (in) tri[tri_row(rho) + rho] = pinf;
    }
    __syncwarp();
    const float bound = from_orderable(bound_key);
    for (int t0 = 0; t0 < picks; t0 += 32) {
        float my_val = 0.f;
        int my_row = 0;
        const int t1 = min(t0 + 32, picks);
        for (int t = t0; t < t1; ++t) {
            float bv[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) bv[k] = fmaf(-lr[k], M[k], sv[k]);
            float lm = bv[0];
#pragma unroll
            for (int k = 1; k < CPL; ++k) lm = fmaxf(lm, bv[k]);
            const float whi = warp_max_f32(lm);
            // which of the lane's candidates that was, the lower row on equal values (a compare tree, independent of
            // the reduction in flight)
            int bi[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) bi[k] = lane + 32 * k;
#pragma unroll
            for (int w = 1; w < CPL; w *= 2) {
#pragma unroll
                for (int k = 0; k + w < CPL; k += 2 * w) {
                    const bool gt = bv[k + w] > bv[k];
                    bv[k] = gt ? bv[k + w] : bv[k];
                    bi[k] = gt ? bi[k + w] : bi[k];
                }
            }
            const int row = bi[0];
            const uint32_t wlo = __reduce_max_sync(0xFFFFFFFFu, lm == whi ? 0xFFFFu - (uint32_t)row : 0u);
            const int irho = min((int)(0xFFFFu - wlo), last);
            if (BOUNDED && whi <= bound) {
                // The picks made so far stand. They are parked, and with m_out / t_out given the running maxima
                // (by pool row; +inf for the rows already picked) and the number of picks are left for the caller
                // to continue from.
                if (t0 + lane < t) {
                    park_key[t0 + lane] = orderable(my_val <= -2.9e38f ? ninf : my_val);
                    park_row[t0 + lane] = my_row;
                }
                if (m_out) {
#pragma unroll
                    for (int k = 0; k < CPL; ++k)
                        if (lane + 32 * k < P) m_out[lane + 32 * k] = M[k];
                }
                if (t_out && lane == 0) *t_out = t;
                return false;
            }
            const bool mine = lane == t - t0;
            my_val = mine ? whi : my_val;
            my_row = mine ? irho : my_row;
            if (t + 1 == picks) continue;
            // m <- max(m, Sims[i, :]) from the triangle: entry (max, min); the picked row meets its diagonal
            const int irho4 = 4 * irho;
            const uint32_t tiB = tb + 4u * (uint32_t)tri_row(irho);
            uint32_t addr[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) addr[k] = rc4[k] > irho4 ? trowB[k] + (uint32_t)irho4 : tiB + (uint32_t)rc4[k];
            const float ri = fmaxf(lds_in_order(rb + (uint32_t)irho4), 1e-30f);
            float x[CPL];
#pragma unroll
            for (int k = 0; k < CPL; ++k) x[k] = lds_in_order(addr[k]);
#pragma unroll
            for (int k = 0; k < CPL; ++k) M[k] = fmaxf(M[k], ri * x[k]);
        }
        if (t0 + lane < picks) {
            park_key[t0 + lane] = orderable(my_val <= -2.9e38f ? ninf : my_val);
            park_row[t0 + lane] = my_row;
        }
    }
    return true;
}

// FUSED: score + select + compact; otherwise selection only (scores are read from a.scores and
// nothing is rewritten).
template <bool FUSED>
__global__ void __launch_bounds__(kTcThreads) event_tri_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int N = lay.N;
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);
    const TriSmem sp = plan_tri_smem(N, a.budget);
    unsigned char* tile = smem + sp.tile;
    float* tri = reinterpret_cast<float*>(tile);  // lower triangle of the cosine matrix, after the product
    float* s = reinterpret_cast<float*>(smem + sp.s);
    uint32_t* key = reinterpret_cast<uint32_t*>(smem + sp.key);
    float* r = reinterpret_cast<float*>(smem + sp.key);  // reuses the score keys' storage
    int* spos = reinterpret_cast<int*>(smem + sp.spos);
    unsigned short* bypool = reinterpret_cast<unsigned short*>(smem + sp.bypool);
    unsigned char* taken = smem + sp.taken;
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    float* rowbuf = reinterpret_cast<float*>(smem + sp.row);
    float2* sect = reinterpret_cast<float2*>(smem + sp.sect);
    const uint32_t barK = smem_u32(smem + sp.misc);
    const uint32_t barM = barK + 8;
    const uint32_t barL = barK + 48;  // K rows from 128 on
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sp.misc + 16);
    int* pool_holder = reinterpret_cast<int*>(smem + sp.misc + 20);
    int* pick_holder = reinterpret_cast<int*>(smem + sp.misc + 24);
    int* redi = reinterpret_cast<int*>(smem + sp.misc + 32);
    const uint32_t tile_u32 = smem_u32(tile);
    const uint32_t half_bytes = (uint32_t)kTriTileRows * 128u;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool similarity = a.greedy != 0;
    const int np4 = (N + 3) & ~3;
    // row addressing: dense events are one base offset plus a row stride
    const bool dense = lay.page_size == 0;
    const long long ev_off = dense ? id.b * lay.sb + id.l * lay.sl + id.h * lay.sh : 0;
    auto rowoff = [&](int j) -> long long {
        return dense ? ev_off + (long long)j * lay.sn : row_offset(lay, id.b, id.l, id.h, j);
    };
    __nv_bfloat16* Kg = reinterpret_cast<__nv_bfloat16*>(a.K);
    __nv_bfloat16* Vg = reinterpret_cast<__nv_bfloat16*>(a.V);

    phase_stamp(id.e, 0);  // phases: 0 start, 1 tensor memory claimed, 2 K scored, 3 pool, 4 V operand, 5 product, 6 triangle, 7 picks, 8 outputs, 9 end
    // Tensor memory is claimed first and the right to allocate given up at once: the SM starts its
    // next CTA of this kernel only after that, so a late allocation would serialise the CTAs.
    const bool use_tc = similarity;
    // K rows [r0, r1) -> tile slots from slot0 on: as few bulk copies as the layout allows (whole event
    // when its rows are contiguous, whole pages when pages are, else row by row), all issued by one
    // thread (a bulk copy is a per-warp instruction)
    auto request_k_rows = [&](int r0, int r1, int slot0, uint32_t bar) {
        mbar_expect_tx(bar, (uint32_t)(r1 - r0) * 256u);
        for (int row = r0; row < r1 && !a.starve;) {  // starve (testing aid): nothing is requested, the waits run out
            int run = 1;
            if (dense && lay.sn == kTcD) run = min(r1 - row, 128);
            else if (!dense && lay.s_page_n == kTcD) run = min(r1 - row, lay.page_size - row % lay.page_size);
            bulk_g2s(tile_u32 + (uint32_t)(slot0 + row - r0) * 256u, Kg + rowoff(row), (uint32_t)run * 256u, bar);
            row += run;
        }
    };
    const int n_late = FUSED && n > kTriTileRows ? n - kTriTileRows : 0;  // rows that wait for a free slot
    if (tid == 0) {
        mbar_init(barK, 1);
        mbar_init(barM, 1);
        mbar_init(barL, 1);
        mbar_init_fence();
    }
    if (FUSED && tid >= 32 && tid < 64) {
        float sn, cs;
        sincospif((float)(tid - 32) * 0.0625f, &sn, &cs);  // angle 2 pi h / 32
        sect[tid - 32] = make_float2(cs, sn);
    }
    if (warp == 0) {
        if (use_tc) tmem_alloc(smem_u32(tmem_holder), kTcCols);
        else tmem_relinquish();  // top-k events take no tensor memory, and must not hold up the next CTA's start
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = use_tc ? *tmem_holder : 0u;

    phase_stamp(id.e, 1);
    // ---- scores ---------------------------------------------------------------------------------
    int bad = 0;
    int timeout = 0;
    if (FUSED) {
        if (tid == 0) request_k_rows(0, n - n_late, 0, barK);
        const int* gpos = event_pos(a.pos, id);
        const bool rotate = gpos != nullptr;
        int pmax = INT_MIN;
        for (int j = tid; j < n; j += kTcThreads) {
            const int p = rotate ? gpos[j] : 0;
            spos[j] = p;
            pmax = max(pmax, p);
        }
        // folded statistic g_f = c_f z(q)_f / sqrt(d) and the frequencies' phase steps, once per event, in
        // shared memory (storage that the selection uses later)
        float2* gtab = reinterpret_cast<float2*>(smem + sp.bypool);
        unsigned long long* phitab = reinterpret_cast<unsigned long long*>(gtab + 64);
        if (tid < 64) {
            const float* q = a.qstat + ((long long)id.l * lay.H + id.h) * kTcD;
            const float inv = rsqrtf((float)kTcD);
            const float qr = q[tid] * inv, qi = q[tid + 64] * inv;
            const float2 c = tab.cw[tid];
            gtab[tid] = make_float2(c.x * qr - c.y * qi, c.x * qi + c.y * qr);
            phitab[tid] = tab.phi[tid];
        }
        if (rotate) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pmax = max(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, off));
            if (lane == 0) redi[warp] = pmax;
        }
        __syncthreads();
        long long pref = 0;
        if (rotate) pref = a.p_ref ? (long long)a.p_ref[id.b] : (long long)max(max(redi[0], redi[1]), max(redi[2], redi[3])) + 1;
        // lane covers frequencies f0..f0+7 of the row handled by its group of eight lanes
        const int grp = lane >> 3, f0 = (lane & 7) * 8;
        // spacing of rows 16 slots apart at the newest end of the event: what a token-by-token cache has everywhere
        const long long D16 = n > 16 ? (long long)spos[n - 1] - (long long)spos[n - 17] : 0;
        ChainScore cs;
        cs.set_step(D16, phitab + f0, sect);
        const int rounds = (n + 15) >> 4, late_round = (n_late + 15) >> 4;
        // 16 rows per round (4 per warp), in three stretches. Rows from 128 on reuse the slots of rows
        // 0..n_late-1: they are requested after the first stretch, once every warp is past those rows,
        // and awaited before the third. The rounds also run after a timeout (over whatever the tile
        // holds), so that the barrier between them is reached by every thread.
        auto score_rounds = [&](int round0, int round1) {
            for (int round = round0; round < round1; ++round) {
                const int j = 16 * round + 4 * warp + grp;
                const bool live = j < n;
                // G follows from the previous round's by the constant turn when all four rows of the warp sit
                // D16 after the rows 16 slots before them
                bool fresh = (round & (kChainRoundsShort - 1)) == 0 || a.no_chain;
                if (!fresh) fresh = !__all_sync(0xFFFFFFFFu, !live || (long long)spos[j] - (long long)spos[j - 16] == D16);
                if (fresh) {
                    if (live) cs.anchor(pref - (long long)spos[j], gtab + f0, phitab + f0, sect);
                } else {
                    cs.advance();
                }
                float acc = 0.f;
                if (live) {
                    const unsigned char* krow = tile + (j & (kTriTileRows - 1)) * 256 + (lane & 7) * 16;
                    acc = cs.dot(*reinterpret_cast<const uint4*>(krow), *reinterpret_cast<const uint4*>(krow + 128));
                }
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
                if (live && (lane & 7) == 0) {
                    if (a.scores) a.scores[(long long)id.e * N + j] = acc;
                    const bool fin = isfinite(acc);
                    bad |= !fin;
                    const float sj = fin ? acc : -INFINITY;
                    s[j] = sj;
                    key[j] = orderable(sj);
                }
            }
        };
        timeout = !mbar_wait_polls(barK, 0, a.wait_polls);
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            // first and third stretch share one copy of the loop (the kernel's code should stay small)
            if (pass && n_late > 0) timeout |= !mbar_wait_polls(barL, 0, a.wait_polls);
            score_rounds(pass ? kTriTileRows / 16 : 0, pass ? rounds : late_round);
            if (!pass) {
                if (n_late > 0) {
                    __syncthreads();
                    if (tid == 0) request_k_rows(kTriTileRows, n, 0, barL);
                }
                score_rounds(late_round, min(rounds, kTriTileRows / 16));
            }
        }
    } else {
        for (int j = tid; j < n; j += kTcThreads) {
            const float sc = a.scores[(long long)id.e * N + j];
            const bool fin = isfinite(sc);
            bad |= !fin;
            const float sj = fin ? sc : -INFINITY;
            s[j] = sj;
            key[j] = orderable(sj);
        }
    }
    for (int j = n + tid; j < np4; j += kTcThreads) key[j] = 0u;  // below every real key
    timeout = __syncthreads_or(timeout);
    if (timeout) {
        if (tid == 0 && a.status) a.status[id.e] = 3;
        mbar_wait_polls(barK, 0, a.wait_polls);  // give copies still in flight another bounded chance to land
        if (n_late > 0) mbar_wait_polls(barL, 0, a.wait_polls);
        if (use_tc && warp == 0) tmem_dealloc(tbase, kTcCols);
        return;
    }
    bad = __syncthreads_or(bad);
    // (only now: while scoring, this storage holds the statistic's table, which slower warps may still read)
    for (int j = tid; j < np4; j += kTcThreads) taken[j] = 0;

    phase_stamp(id.e, 2);
    // ---- s_(b) by bisection over the score keys, then the pool in slot order (warp 0) -------------
    if (warp == 0) {
        uint32_t kk[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = lane + 32 * k;
            kk[k] = j < np4 ? key[j] : 0u;
        }
        uint32_t kb = 0u;  // the picks-th largest key: the largest v with at least `picks` keys >= v
        if (picks > 0) {
            // two bits per round: the three counts are independent, so their reductions overlap.
            // Pruning only needs a lower bound of s_(b) (the pool may be a little larger than necessary),
            // so the low 14 key bits (0.2 % of the value) are not resolved; top-k needs the exact key.
            const int lo_end = similarity ? 14 : 0;
            for (int lo = 30; lo >= lo_end; lo -= 2) {
                const uint32_t v1 = kb | (1u << lo), v2 = kb | (2u << lo), v3 = kb | (3u << lo);
                int c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    c1 += kk[k] >= v1;
                    c2 += kk[k] >= v2;
                    c3 += kk[k] >= v3;
                }
                c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
                c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
                c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
                kb = c3 >= picks ? v3 : (c2 >= picks ? v2 : (c1 >= picks ? v1 : kb));
            }
        }
        const float sb = from_orderable(kb);
        // -inf keeps everyone
        const float thr = a.no_prune ? -INFINITY : fmaf(-1.001f, a.lam, sb) - 1e-6f * fabsf(sb);
        int base = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool in = kk[k] != 0u && (similarity ? !(from_orderable(kk[k]) < thr) : kk[k] >= kb);
            const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
            if (in) bypool[base + __popc(mask & ((1u << lane) - 1u))] = (unsigned short)(lane + 32 * k);
            base += __popc(mask);
        }
        if (lane == 0) *pool_holder = base;
    }
    __syncthreads();  // every key has been read: its storage becomes r below
    const int P = *pool_holder;
    const bool fast = similarity && P <= kTriMaxPool && picks > 1;
    const bool slow = similarity && P > kTriMaxPool;

    phase_stamp(id.e, 3);
    // ---- V rows of the pool as the swizzled operand tile ---------------------------------------------
    if (similarity && !slow) {
        // thread -> 16-byte column c of rows r0, r0 + 8, ...: the swizzle term (c ^ row) & 7 is the same for
        // all of them, so a row costs one pool lookup, one address and one copy
        const int c = tid & 15, r0 = tid >> 4;
        const uint32_t dst0 = tile_u32 + tile_chunk(r0, c, half_bytes);
        if (dense) {
            const __nv_bfloat16* vcol = Vg + ev_off + c * 8;
            for (int rho = r0; rho < P; rho += 8)
                cp_async16(dst0 + (uint32_t)(rho - r0) * 128u, vcol + (long long)bypool[rho] * lay.sn);
        } else {
            for (int rho = r0; rho < P; rho += 8)
                cp_async16(dst0 + (uint32_t)(rho - r0) * 128u, Vg + rowoff(bypool[rho]) + c * 8);
        }
        cp_async_wait_all();
        fence_proxy_async();
        __syncthreads();
    }
    phase_stamp(id.e, 4);
    if (fast) {
        if (tid == 0) {
            tc_fence_after();
            const uint32_t idesc = umma_idesc_bf16(128, (P + 15) & ~15);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                umma_bf16(tbase, umma_desc_sw128(tile_u32 + koff), umma_desc_sw128(tile_u32 + koff), idesc, kk > 0 ? 1u : 0u);
            }
            umma_commit(barM);
        }
        timeout = !mbar_wait_polls(barM, 0, a.wait_polls);
        tc_fence_after();
    }
    timeout = __syncthreads_or(timeout);  // also: the product has read the whole tile before the triangle lands on it
    if (timeout) {
        if (tid == 0 && a.status) a.status[id.e] = 3;
        if (use_tc && warp == 0) tmem_dealloc(tbase, kTcCols);
        return;
    }
    phase_stamp(id.e, 5);
    if (fast) {
        // lower triangle -> shared memory; row rho = 32 warp + lane needs columns 0..rho
        const int rho = 32 * warp + lane;
        if (32 * warp < P) {
            const int trow = tri_row(rho);
            const uint32_t lanes = tbase + ((uint32_t)(warp * 32) << 16);
            // column blocks left of the diagonal one: every column is below the row
            for (int cb = 0; cb < warp; ++cb) {
                uint32_t v[32];
                tmem_ld32(lanes + (uint32_t)(32 * cb), v);
                tmem_ld_wait();
                if (rho < P) {
#pragma unroll
                    for (int k = 0; k < 32; ++k) tri[trow + 32 * cb + k] = __uint_as_float(v[k]);
                }
            }
            // the diagonal block: columns up to the row itself, whose last entry is the squared norm
            {
                uint32_t v[32];
                tmem_ld32(lanes + (uint32_t)(32 * warp), v);
                tmem_ld_wait();
                if (rho < P) {
#pragma unroll
                    for (int k = 0; k < 32; ++k)
                        if (k <= lane) tri[trow + 32 * warp + k] = __uint_as_float(v[k]);
                    r[rho] = 1.f / (sqrtf(tri[trow + rho]) + a.eps);  // read back: this thread stored it
                }
            }
        }
    } else if (slow) {
        // reciprocal norms (Eq. 1); this pool does not fit the tile, its V rows are read in place
        for (int rho = tid; rho < P; rho += kTcThreads) {
            const __nv_bfloat16* vrow = Vg + rowoff(bypool[rho]);
            float ss = 0.f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                float x[8];
                load8(vrow + c * 8, x);
#pragma unroll
                for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
            }
            r[rho] = 1.f / (sqrtf(ss) + a.eps);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (use_tc && warp == 0) tmem_dealloc(tbase, kTcCols);

    phase_stamp(id.e, 6);
    // ---- Algorithm 1 in warp 0 -------------------------------------------------------------------------
    // The winning key of every pick is parked in gain[] and its pool row in order[]; both are decoded
    // after the loop.
    uint32_t* park_key = reinterpret_cast<uint32_t*>(gain);
    if (!slow) {
        if (warp == 0) {
            if (fast) picks_cosine<4, false>(lane, P, picks, s, bypool, r, a.lam, tri, park_key, order);
            else if (P <= 128) picks_in_one_warp<4>(lane, P, picks, false, s, bypool, r, a.lam, tri, park_key, order);
            else picks_in_one_warp<8>(lane, P, picks, false, s, bypool, r, a.lam, tri, park_key, order);
        }
    } else {
        GreedyLane<8> g;
        if (warp == 0) g.init(lane, P, s, bypool, r, a.lam, true);
        for (int t = 0; t < picks; ++t) {
            if (warp == 0) {
                uint32_t bk;
                const int irho = g.pick(lane, bk);
                if (lane == 0) { park_key[t] = bk; order[t] = irho; *pick_holder = irho; }
            }
            if (t + 1 == picks) break;
            __syncthreads();
            const int irho = *pick_holder;
            // row irho of the cosine matrix by plain dot products
            const __nv_bfloat16* vpick = Vg + rowoff(bypool[irho]);
            for (int rho = tid; rho < P; rho += kTcThreads) {
                const __nv_bfloat16* vrow = Vg + rowoff(bypool[rho]);
                float acc = 0.f;
#pragma unroll 4
                for (int c = 0; c < 16; ++c) {
                    float vi[8], vj[8];
                    load8(vpick + c * 8, vi);
                    load8(vrow + c * 8, vj);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc = fmaf(vi[e], vj[e], acc);
                }
                rowbuf[rho] = acc;
            }
            __syncthreads();
            if (warp == 0) {
                const float ri = r[irho];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int rho = lane + 32 * k;
                    if (rho < P) g.M[k] = fmaxf(g.M[k], ri * rowbuf[rho]);
                }
            }
        }
    }
    __syncthreads();
    for (int t = tid; t < picks; t += kTcThreads) {
        const int j = bypool[order[t]];
        gain[t] = from_orderable(park_key[t]);
        order[t] = j;
        taken[j] = 1;
    }
    __syncthreads();

    phase_stamp(id.e, 7);
    // ---- sort(S) and outputs -------------------------------------------------------------------------
    ordered_indices(n, a.budget, taken, idx);
    __syncthreads();
    const long long ob = (long long)id.e * a.budget;
    for (int t = tid; t < a.budget; t += kTcThreads) {
        a.idx_sorted[ob + t] = idx[t];
        if (a.pick_order) a.pick_order[ob + t] = t < picks ? order[t] : -1;
        if (a.pick_gain) a.pick_gain[ob + t] = t < picks ? gain[t] : 0.f;
    }
    if (tid == 0) {
        if (a.n_kept) a.n_kept[id.e] = picks;
        if (a.status) a.status[id.e] = n < bud ? 2 : (bad ? 1 : 0);
    }
    if (!FUSED) return;

    phase_stamp(id.e, 8);
    // ---- compaction in place ----------------------------------------------------------------------
    // Every kept K and V row and position is on chip before the first store: a destination slot can be
    // another kept row's source. Up to 64 rows: K in registers, V through the (by now free) tile by
    // cp.async, one barrier. Both in registers would make this the kernel's register peak and cost a
    // resident CTA per SM.
    int* wpos = a.pos.p ? a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh : nullptr;
    if (picks <= 64) {
        // thread -> 16-byte column c of kept rows r0, r0 + 8, ...
        const int c = tid & 15, r0 = tid >> 4;
        const uint32_t slot0 = (uint32_t)(r0 * 256 + c * 16);
        const long long col = (dense ? ev_off : 0) + c * 8;
        for (int t = r0; t < picks; t += 8) {
            const long long off = col + (dense ? (long long)idx[t] * lay.sn : rowoff(idx[t]));
            cp_async16(tile_u32 + slot0 + (uint32_t)(t - r0) * 256u, Kg + off);
            cp_async16(tile_u32 + 16384u + slot0 + (uint32_t)(t - r0) * 256u, Vg + off);
        }
        cp_async_wait_all();
        __syncthreads();  // every load above has been performed
        for (int t = r0; t < picks; t += 8) {
            const long long off = col + (dense ? (long long)t * lay.sn : rowoff(t));
            const unsigned char* src = tile + slot0 + (t - r0) * 256;
            *reinterpret_cast<uint4*>(Kg + off) = *reinterpret_cast<const uint4*>(src);
            *reinterpret_cast<uint4*>(Vg + off) = *reinterpret_cast<const uint4*>(src + 16384);
        }
    } else {
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            __nv_bfloat16* X = pass ? Vg : Kg;
            __syncthreads();  // the tile is free (greedy loop, or the previous pass, is done with it)
            for (int x = tid; x < picks * 16; x += kTcThreads)
                copy16(tile + x * 16, reinterpret_cast<const char*>(X + rowoff(idx[x >> 4])) + (x & 15) * 16);
            __syncthreads();
            for (int x = tid; x < picks * 16; x += kTcThreads)
                copy16(reinterpret_cast<char*>(X + rowoff(x >> 4)) + (x & 15) * 16, tile + x * 16);
        }
    }
    if (wpos)
        for (int t = tid; t < picks; t += kTcThreads) wpos[t] = spos[idx[t]];
    phase_stamp(id.e, 9);
}

}  // namespace akv
