// Event kernel for bf16, d = 128, per-head signatures, N <= 256 and budgets up to 128 (the shapes of the
// Qwen-7B-shaped batch and of the decode cadence: 256 candidates -> 128). Same structure as event_tri_kernel
// (K rows scored from a 128-row tile, pool by bisection, cosine matrix on tcgen05, its lower triangle in shared
// memory, Algorithm 1 as a one-warp loop), for an ACTIVE SET instead of the whole pool:
//
//   The picks hardly ever reach beyond the best-scored few dozen rows past the budget. The cosine matrix is
//   therefore formed only for the pool's best-scored rows, at most 180 of them (64 KB of triangle: three CTAs
//   per SM), and only their V rows are read. Every candidate left out scores at most `bound`, the 181st largest
//   key, and its Eq. 2 value never exceeds its score: the loop over the active set is exact as long as its
//   winning value stays above that bound. In the rare event where it does not, the picks made so far stand and
//   the remaining ones (a few, as a rule) are taken over the whole pool with rows of the cosine matrix as plain
//   dot products, starting from the running maxima the loop had reached.
//
//   Rows 128.. of the active set: a second product (the operand's last 128 rows against rows 128..) gives their
//   cosines against one another; their cosines against rows < 128 are those rows' columns 128.. by symmetry.
#pragma once
#include "akv_event_tri.cuh"

namespace akv {

// Two sizes of the kernel. The small one (budgets up to 64): a tile of 128 rows of 256 bytes, which holds the V
// operand and then the triangle of a pool of up to 127 rows; six CTAs per SM. The large one (budgets up to 128,
// N up to 256): 64 KB, for a whole event's K rows, then the triangle of an active set of up to 180 rows (see the kernel); three CTAs per SM.
// Scratch of the continuation after the active set's bound was reached, as byte offsets into the tile (the triangle
// is dead by then): the loop's running maxima, and behind the plain-dot route's row buffer the arrays of the hand-over.
constexpr unsigned kContScratch = 2048u;   // 2 KB + 2 x 1 KB + 2 x 512 B + 512 B + 256 B + 4 B
constexpr unsigned kContMact = 8192u;      // 1 KB

template <bool BIG>
struct TriCfg {
    static constexpr unsigned kTileBytes = BIG ? 65536u : 32768u;
    static constexpr int kKRows = BIG ? 256 : 128;       // K rows resident at a time (the large tile holds a whole event)
    static constexpr int kMaxPool = BIG ? 180 : 127;     // most rows whose cosine matrix goes through the tile
    static constexpr uint32_t kCols = BIG ? 256u : 128u;  // tensor-memory columns (a power of two >= the matrix's columns)
    static constexpr int kCpl = BIG ? 6 : 4;             // candidates per lane of the one-warp loop
};

// Layout after the 1024-byte aligned base. `key` (score keys) and `r` (reciprocal norms) share storage.
__host__ __device__ inline TriSmem plan_tri_smem(int N, int budget, bool big) {
    TriSmem p;
    const unsigned np = (unsigned)((N + 3) & ~3);
    unsigned o = 0;
    p.tile = o;   o += big ? TriCfg<true>::kTileBytes : TriCfg<false>::kTileBytes;
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

// Shared memory -> global memory as one bulk copy (16-byte aligned, a multiple of 16 bytes), and the wait that
// must precede leaving the CTA or reusing the source: until the copies issued by this thread have read it.
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// BOUNDED: the P rows are only the best-scored part of the pool, and every candidate left out scores at most
// `bound_key` (as an order-preserving key), so its Eq. 2 value can never exceed that. The loop is exact as long
// as the winning value stays above the bound; at the first pick that does not, it stops and returns false.
template <int CPL, bool BOUNDED = false>
__device__ __forceinline__ bool picks_bounded(int lane, int P, int picks, bool with_sims, const float* s,
                                                  const unsigned short* bypool, const float* r, float lam, const float* tri,
                                                  uint32_t* park_key, int* park_row, uint32_t bound_key = 0u) {
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
            if (BOUNDED && bk <= bound_key) return false;
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
    return true;
}

// FUSED: score + select + compact; otherwise selection only (scores are read from a.scores and
// nothing is rewritten).
template <bool FUSED, bool BIG>
__global__ void __launch_bounds__(kTcThreads, BIG ? 3 : 7) event_pool_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab) {
    using Cfg = TriCfg<BIG>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int N = lay.N;
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);
    const TriSmem sp = plan_tri_smem(N, a.budget, BIG);
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
    uint32_t* bound_holder = reinterpret_cast<uint32_t*>(smem + sp.misc + 28);  // large size: key no left-out candidate exceeds
    float* thr_holder = reinterpret_cast<float*>(smem + sp.misc + 56);          // large size: the pool's score threshold
    const uint32_t tile_u32 = smem_u32(tile);
    const uint32_t half_bytes = Cfg::kTileBytes / 2048u * 1024u;  // the operand's two 128-byte column halves

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
    // shared signatures (Eq. 1, or its per-layer variant): the cosines come from the matrix formed once per
    // sequence (or per sequence and layer) instead of from this head's V rows
    const float* G = a.gram ? a.gram + id.b * a.gram_sb + id.l * a.gram_sl : nullptr;

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
    const int n_late = FUSED && n > Cfg::kKRows ? n - Cfg::kKRows : 0;  // rows that wait for a free slot
    if (tid == 0) {
        mbar_init(barK, 1);
        mbar_init(barM, 1);
        mbar_init(barL, 1);
        mbar_init_fence();
        // the K rows are asked for before anything else: the wait for tensor memory below overlaps their flight
        if (FUSED) request_k_rows(0, n - n_late, 0, barK);
    }
    if (FUSED && warp == 1) fill_sector_table(sect, lane);
    // (the large size claims half of the SM's columns: two of the three resident CTAs hold theirs at a time, the
    // third waits in the allocation until one has moved its triangle out; claiming late instead measured 2 % slower)
    if (!BIG && use_tc && warp == 0) tmem_alloc(smem_u32(tmem_holder), Cfg::kCols);
    if (BIG && (G || !similarity) && warp == 0) tmem_relinquish();  // this event takes no tensor memory
    if (BIG && !(G || !similarity) && warp == 0) tmem_alloc(smem_u32(tmem_holder), Cfg::kCols);
    tc_fence_before();
    const bool have_tmem = BIG ? (similarity && !G) : use_tc;
    // The address of the columns is read after the next block-wide barrier: in the fused kernel that is the one
    // that follows the position and statistic loads, so that warps 1..3 do those while warp 0 may still be
    // waiting for columns.
    uint32_t tbase = 0u;
    if (!FUSED) {
        __syncthreads();
        tc_fence_after();
        tbase = have_tmem ? *tmem_holder : 0u;
    }

    phase_stamp(id.e, 1);
    // ---- scores ---------------------------------------------------------------------------------
    int bad = 0;
    int timeout = 0;
    if (FUSED) {
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
        fill_statistic_tables(a.qstat + ((long long)id.l * lay.H + id.h) * kTcD, tab, tid, gtab, phitab);
        if (rotate) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pmax = max(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, off));
            if (lane == 0) redi[warp] = pmax;
        }
        __syncthreads();
        tc_fence_after();
        tbase = have_tmem ? *tmem_holder : 0u;
        long long pref = 0;
        if (rotate) pref = a.p_ref ? (long long)a.p_ref[id.b] : (long long)max(max(redi[0], redi[1]), max(redi[2], redi[3])) + 1;
        // lane covers frequencies f0..f0+7 of the row handled by its group of eight lanes
        const int grp = lane >> 3, f0 = (lane & 7) * 8;
        // spacing of rows 16 slots apart at the newest end of the event: what a token-by-token cache has everywhere
        const long long D16 = n > 16 ? (long long)spos[n - 1] - (long long)spos[n - 17] : 0;
        ChainScore cs;
        cs.set_step(D16, phitab + f0, sect);
        // whether every row sits D16 after the row 16 slots before it (found once; the chains then need no look at
        // the positions)
        bool uniform = false;
        if (BIG) {
            bool uni = true;
            for (int j = 16 + tid; j < n; j += kTcThreads) uni &= (long long)spos[j] - (long long)spos[j - 16] == D16;
            uniform = __syncthreads_and(uni);
        }
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
                if (!fresh && !uniform) fresh = !__all_sync(0xFFFFFFFFu, !live || (long long)spos[j] - (long long)spos[j - 16] == D16);
                if (fresh) {
                    if (live) cs.anchor(pref - (long long)spos[j], gtab + f0, phitab + f0, sect);
                } else {
                    cs.advance();
                }
                float acc = 0.f;
                if (live) {
                    const unsigned char* krow = tile + (j & (Cfg::kKRows - 1)) * 256 + (lane & 7) * 16;
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
        timeout = !mbar_wait_bounded(barK, 0, a.wait_polls);
        phase_stamp(id.e, 10);  // (K rows have arrived)
        if (BIG) {
            // The tile holds the whole event. A lane group scores two rows side by side, row j of the first half
            // of the rounds and row j + 16 * half of the second: two independent chains that share the turn S, so
            // that one chain's dependent arithmetic fills the other's latency.
            const int half = (rounds + 1) >> 1;
            ChainScore cb;
            AKV_PHASE_ACC_DECL(cyc_anchor);
#pragma unroll 1
            for (int round = 0; round < half; ++round) {
                const int ja = 16 * round + 4 * warp + grp, jb = ja + 16 * half;
                const bool la = ja < n, lb = jb < n;
                // each chain on its own: after an event the kept rows' positions are irregular (fresh rotation every
                // round) while the rows appended since are consecutive (chained)
                bool fa = round == 0 || a.no_chain, fb = fa;
                if (!fa && !uniform) {
                    fa = !__all_sync(0xFFFFFFFFu, !la || (long long)spos[ja] - (long long)spos[ja - 16] == D16);
                    fb = !__all_sync(0xFFFFFFFFu, !lb || (long long)spos[jb] - (long long)spos[jb - 16] == D16);
                }
                AKV_PHASE_ACC_BEGIN(cyc_anchor);
                if (fa) {
                    if (la) cs.anchor(pref - (long long)spos[ja], gtab + f0, phitab + f0, sect);
                } else {
                    cs.advance();
                }
                if (fb) {
                    if (lb) cb.anchor(pref - (long long)spos[jb], gtab + f0, phitab + f0, sect);
                } else {
                    cb.advance_by(cs);
                }
                AKV_PHASE_ACC_END(cyc_anchor);
                float acca = 0.f, accb = 0.f;
                if (la) {
                    const unsigned char* krow = tile + ja * 256 + (lane & 7) * 16;
                    acca = cs.dot(*reinterpret_cast<const uint4*>(krow), *reinterpret_cast<const uint4*>(krow + 128));
                }
                if (lb) {
                    const unsigned char* krow = tile + jb * 256 + (lane & 7) * 16;
                    accb = cb.dot(*reinterpret_cast<const uint4*>(krow), *reinterpret_cast<const uint4*>(krow + 128));
                }
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) {
                    acca += __shfl_xor_sync(0xFFFFFFFFu, acca, off);
                    accb += __shfl_xor_sync(0xFFFFFFFFu, accb, off);
                }
                if ((lane & 7) == 0) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int j = h ? jb : ja;
                        const float acc = h ? accb : acca;
                        if (j < n) {
                            if (a.scores) a.scores[(long long)id.e * N + j] = acc;
                            const bool fin = isfinite(acc);
                            bad |= !fin;
                            const float sj = fin ? acc : -INFINITY;
                            s[j] = sj;
                            key[j] = orderable(sj);
                        }
                    }
                }
            }
            AKV_PHASE_ACC_STORE(id.e, 11, cyc_anchor);
            phase_stamp(id.e, 12);  // (scoring loop left)
        }
#pragma unroll 1
        for (int pass = 0; !BIG && pass < 2; ++pass) {
            // first and third stretch share one copy of the loop (the kernel's code should stay small)
            if (pass && n_late > 0) timeout |= !mbar_wait_bounded(barL, 0, a.wait_polls);
            score_rounds(pass ? Cfg::kKRows / 16 : 0, pass ? rounds : late_round);
            if (!pass) {
                if (n_late > 0) {
                    __syncthreads();
                    if (tid == 0) request_k_rows(Cfg::kKRows, n, 0, barL);
                }
                score_rounds(late_round, min(rounds, Cfg::kKRows / 16));
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
        mbar_wait_bounded(barK, 0, a.wait_polls);  // give copies still in flight another bounded chance to land
        if (n_late > 0) mbar_wait_bounded(barL, 0, a.wait_polls);
        if (have_tmem && warp == 0) tmem_dealloc(tbase, Cfg::kCols);
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
        // Large size: the cosine matrix is formed for an active set of at most kMaxPool rows, the best-scored part
        // of the pool. Every candidate left out scores at most `bound`, the (kMaxPool + 1)-th largest key, and its
        // Eq. 2 value never exceeds its score: the loop over the active set is exact as long as its winning
        // value stays above that (it nearly always does: with lambda = 0.5 the picks reach a few ranks beyond
        // the budget; the rare event where it does not is redone over the whole pool).
        uint32_t bound = 0u;
        if constexpr (BIG) if (similarity) {
            int pool_size = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) pool_size += kk[k] != 0u && !(from_orderable(kk[k]) < thr);
            pool_size = __reduce_add_sync(0xFFFFFFFFu, pool_size);
            if (pool_size > Cfg::kMaxPool) {
                for (int lo = 30; lo >= 0; lo -= 2) {
                    const uint32_t v1 = bound | (1u << lo), v2 = bound | (2u << lo), v3 = bound | (3u << lo);
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
                    bound = c3 > Cfg::kMaxPool ? v3 : (c2 > Cfg::kMaxPool ? v2 : (c1 > Cfg::kMaxPool ? v1 : bound));
                }
            }
        }
        int base = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool in = kk[k] != 0u && (similarity ? (!(from_orderable(kk[k]) < thr) && (!BIG || kk[k] > bound)) : kk[k] >= kb);
            const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
            if (in) bypool[base + __popc(mask & ((1u << lane) - 1u))] = (unsigned short)(lane + 32 * k);
            base += __popc(mask);
        }
        if (lane == 0) {
            *pool_holder = base;
            if (BIG) {
                *bound_holder = bound;
                *thr_holder = thr;
            }
        }
    }
    __syncthreads();  // every key has been read: its storage becomes r below
    int P = *pool_holder;
    const uint32_t bound_key = BIG ? *bound_holder : 0u;
    const bool fast = similarity && P <= Cfg::kMaxPool && picks > 1;
    bool slow = similarity && P > Cfg::kMaxPool;  // (small size only; the large size may set it after its loop)
    int cont_from = -1;                           // large size: picks already made when the bound was reached

    phase_stamp(id.e, 3);
    // ---- V rows of the pool as the swizzled operand tile ---------------------------------------------
    if (similarity && !slow && G) {
        // the active set's cosine matrix, gathered from the shared one: row a of the triangle holds the shared
        // matrix's row of slot a at the slots of rows 0..a; the signatures are unit rows, so there are no norms
        // (a warp per row, its lanes across the row's columns: a lane's columns are the same for every row, so it
        // keeps their slots in registers, and the loads of a row, all from one 1 KB row of the shared matrix, are
        // in flight together)
        int col[Cfg::kCpl];
#pragma unroll
        for (int k = 0; k < Cfg::kCpl; ++k) col[k] = lane + 32 * k < P ? bypool[lane + 32 * k] : 0;
        // four rows of a warp at a time: their loads are issued before any of them is stored
        for (int ra0 = warp; ra0 < P; ra0 += 4 * (kTcThreads / 32)) {
            float x[4][Cfg::kCpl];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ra = ra0 + i * (kTcThreads / 32);
                const float* grow = G + (long long)bypool[min(ra, P - 1)] * N;
#pragma unroll
                for (int k = 0; k < Cfg::kCpl; ++k) x[i][k] = (ra < P && lane + 32 * k <= ra) ? __ldg(grow + col[k]) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ra = ra0 + i * (kTcThreads / 32);
                const int trow = tri_row(ra);
#pragma unroll
                for (int k = 0; k < Cfg::kCpl; ++k)
                    if (ra < P && lane + 32 * k <= ra) tri[trow + lane + 32 * k] = x[i][k];
            }
        }
        for (int ra = tid; ra < P; ra += kTcThreads) r[ra] = 1.f;
    } else if (similarity && !slow) {
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
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    phase_stamp(id.e, 4);
    // large size, rows from 128 on (nb of them): a second product, the last 128 rows of the operand against those
    // rows, gives their cosines against one another; what lies left of column 128 comes from the first product
    // by symmetry
    const bool product = fast && !G;  // the cosine matrix comes off the tensor core
    const int nb = (BIG && product && P > 128) ? P - 128 : 0;
    const int ncols = (P + 15) & ~15, base2 = ncols - 128;
    if (product) {
        if (tid == 0) {
            tc_fence_after();
            const uint32_t idesc = umma_idesc_bf16(128, ncols);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                umma_bf16(tbase, umma_desc_sw128(tile_u32 + koff), umma_desc_sw128(tile_u32 + koff), idesc, kk > 0 ? 1u : 0u);
            }
            if (BIG && nb > 0) {
                const uint32_t idesc2 = umma_idesc_bf16(128, ncols - 128);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                    umma_bf16(tbase + (uint32_t)ncols, umma_desc_sw128(tile_u32 + (uint32_t)base2 * 128u + koff),
                              umma_desc_sw128(tile_u32 + 128u * 128u + koff), idesc2, kk > 0 ? 1u : 0u);
                }
            }
            umma_commit(barM);
        }
        timeout = !mbar_wait_bounded(barM, 0, a.wait_polls);
        tc_fence_after();
    }
    timeout = __syncthreads_or(timeout);  // also: the product has read the whole tile before the triangle lands on it
    if (timeout) {
        if (tid == 0 && a.status) a.status[id.e] = 3;
        if (have_tmem && warp == 0) tmem_dealloc(tbase, Cfg::kCols);
        return;
    }
    phase_stamp(id.e, 5);
    if (product) {
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
        if (BIG && nb > 0) {
            // rows from 128 on. Left of column 128: row a's entry in column b is row b's entry in column a (every
            // thread moves its own row's columns 128..). From column 128 on: the second product, whose lane L holds
            // row base2 + L against rows 128.. in the columns after the first product's.
            const uint32_t lanes = tbase + ((uint32_t)(warp * 32) << 16);
            for (int cb = 0; cb < (nb + 31) >> 5; ++cb) {
                uint32_t v[32];
                tmem_ld32(lanes + 128u + (uint32_t)(32 * cb), v);
                tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 32; ++k)
                    if (32 * cb + k < nb) tri[tri_row(128 + 32 * cb + k) + rho] = __uint_as_float(v[k]);
            }
            const int ra = base2 + rho - 128;  // this thread's row of the second product, counted from row 128
            float diag = 0.f;                  // its squared norm (one square root and one division per thread, after the loop)
            for (int cb = 0; cb < (nb + 31) >> 5; ++cb) {
                uint32_t v[32];
                tmem_ld32(lanes + (uint32_t)ncols + (uint32_t)(32 * cb), v);
                tmem_ld_wait();
                if (ra >= 0 && ra < nb) {
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        if (32 * cb + k <= ra) tri[tri_row(128 + ra) + 128 + 32 * cb + k] = __uint_as_float(v[k]);
                        diag = (32 * cb + k == ra) ? __uint_as_float(v[k]) : diag;
                    }
                }
            }
            if (ra >= 0 && ra < nb) r[128 + ra] = 1.f / (sqrtf(diag) + a.eps);
        }
    } else if (slow) {
        // reciprocal norms (Eq. 1); this pool does not fit the tile, its V rows are read in place
        for (int rho = tid; rho < P; rho += kTcThreads) {
            if (G) { r[rho] = 1.f; continue; }
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
    if (have_tmem && warp == 0) tmem_dealloc(tbase, Cfg::kCols);

    phase_stamp(id.e, 6);
    // ---- Algorithm 1 in warp 0 -------------------------------------------------------------------------
    // The winning key of every pick is parked in gain[] and its pool row in order[]; both are decoded
    // after the loop.
    uint32_t* park_key = reinterpret_cast<uint32_t*>(gain);
    if (!slow) {
        if (warp == 0) {
            if (BIG) {
                const bool ok = fast ? picks_cosine<Cfg::kCpl, true>(lane, P, picks, s, bypool, r, a.lam, tri, park_key, order, bound_key,
                                                                     reinterpret_cast<float*>(tile + kContMact), redi)
                                     : picks_bounded<8>(lane, P, picks, false, s, bypool, r, a.lam, tri, park_key, order);
                if (lane == 0) *pick_holder = ok ? 0 : -2;
            } else if (P <= 128) {
                picks_in_one_warp<4>(lane, P, picks, fast, s, bypool, r, a.lam, tri, park_key, order);
            } else {
                picks_in_one_warp<8>(lane, P, picks, false, s, bypool, r, a.lam, tri, park_key, order);
            }
        }
        if (BIG) {
            __syncthreads();
            if (*pick_holder == -2) {
                // A winning value fell to the bound with `done` picks made. Those stand (no left-out candidate could
                // have won them). The rest of the picks, a few as a rule, are taken over the whole pool with rows of
                // the cosine matrix as plain dot products (below), from the state the loop left: its running maxima
                // for the rows it had, and for the rows it had left out the maximum over the picks made, formed here.
                slow = true;
                cont_from = redi[0];
                const int done = cont_from;
                float* m_act = reinterpret_cast<float*>(tile + kContMact);                  // by old pool row (from the loop)
                float* m_slot = reinterpret_cast<float*>(tile + kContScratch);              // by slot
                float* m_init = m_slot + 256;                                               // by new pool row
                unsigned short* inv = reinterpret_cast<unsigned short*>(m_init + 256);      // slot -> new pool row
                unsigned short* left = inv + 256;                                           // new pool rows the loop had left out
                int* chosen = reinterpret_cast<int*>(left + 256);                           // slots of the picks made
                unsigned char* state = reinterpret_cast<unsigned char*>(chosen + 128);      // by slot: 1 in the old active set
                int* n_left = reinterpret_cast<int*>(state + 256);
                for (int j = tid; j < 256; j += kTcThreads) state[j] = 0;
                if (tid == 0) *n_left = 0;
                __syncthreads();
                for (int rho = tid; rho < P; rho += kTcThreads) {
                    const int j = bypool[rho];
                    state[j] = 1;
                    m_slot[j] = m_act[rho];
                }
                for (int t = tid; t < done; t += kTcThreads) chosen[t] = bypool[order[t]];
                __syncthreads();
                if (warp == 0) {
                    const float thr = *thr_holder;
                    int base = 0;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int j = lane + 32 * k;
                        const bool in = j < n && !(s[j] < thr);
                        const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
                        if (in) bypool[base + __popc(mask & ((1u << lane) - 1u))] = (unsigned short)j;
                        base += __popc(mask);
                    }
                    if (lane == 0) *pool_holder = base;
                }
                __syncthreads();
                P = *pool_holder;
                for (int rho = tid; rho < P; rho += kTcThreads) {
                    const int j = bypool[rho];
                    inv[j] = (unsigned short)rho;
                    if (state[j]) {
                        m_init[rho] = m_slot[j];
                    } else {
                        m_init[rho] = 0.f;
                        left[atomicAdd(n_left, 1)] = (unsigned short)rho;
                    }
                    if (G) { r[rho] = 1.f; continue; }
                    const __nv_bfloat16* vrow = Vg + rowoff(j);
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
                __syncthreads();
                for (int t = tid; t < done; t += kTcThreads) order[t] = inv[chosen[t]];
                __syncthreads();
                // left-out rows against the picks made: m = max(0, max_t r_t <V_c, V_t>), every (row, pick) pair its own
                // dot product, the maximum by an integer atomic (the values are non-negative floats)
                const int pairs = *n_left * done;
                for (int x = tid; x < pairs; x += kTcThreads) {
                    const int c = left[x / done], i = order[x % done];
                    float acc;
                    if (G) {
                        acc = G[(long long)bypool[i] * N + bypool[c]];
                    } else {
                        const __nv_bfloat16* vi = Vg + rowoff(bypool[i]);
                        const __nv_bfloat16* vc = Vg + rowoff(bypool[c]);
                        acc = 0.f;
#pragma unroll 4
                        for (int q = 0; q < 16; ++q) {
                            float xi[8], xc[8];
                            load8(vi + q * 8, xi);
                            load8(vc + q * 8, xc);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc = fmaf(xi[e], xc[e], acc);
                        }
                    }
                    const float v = fmaxf(r[i] * acc, 0.f);
                    atomicMax(reinterpret_cast<int*>(m_init) + c, __float_as_int(v));
                }
                __syncthreads();
            }
        }
    }
    if (slow) {
        GreedyLane<8> g;
        if (warp == 0) {
            g.init(lane, P, s, bypool, r, a.lam, true);
            if (BIG && cont_from >= 0) {
                // continue after the picks the bounded loop made: its maxima, and those picks out of the running
                // (rowbuf, the first 1 KB of the tile, is written by the loop below; the scratch lies behind it)
                const float* m_init = reinterpret_cast<const float*>(tile + kContScratch) + 256;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int rho = lane + 32 * k;
                    if (rho < P) {
                        const float m0 = m_init[rho];
                        g.M[k] = m0;
                        if (m0 == __int_as_float(0x7f800000)) g.am[k] = 0u;  // picked already (the loop's +inf)
                    }
                }
            }
        }
        for (int t = BIG && cont_from > 0 ? cont_from : 0; t < picks; ++t) {
            if (warp == 0) {
                uint32_t bk;
                const int irho = g.pick(lane, bk);
                if (lane == 0) { park_key[t] = bk; order[t] = irho; *pick_holder = irho; }
            }
            if (t + 1 == picks) break;
            __syncthreads();
            const int irho = *pick_holder;
            // row irho of the cosine matrix: from the shared matrix, else by plain dot products
            const __nv_bfloat16* vpick = Vg + rowoff(bypool[irho]);
            for (int rho = tid; rho < P; rho += kTcThreads) {
                if (G) { rowbuf[rho] = G[(long long)bypool[irho] * N + bypool[rho]]; continue; }
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
    } else if ((unsigned)picks * 512u <= Cfg::kTileBytes) {
        // The tile holds the kept rows of K and of V side by side: one round of 16-byte gathers, one barrier.
        // Stores: slots 0..picks-1 are contiguous in a dense cache (and page by page in a paged one), so one
        // thread writes them back with a few bulk copies. (Gathering by one bulk copy per row measured slower.)
        const uint32_t vhalf = Cfg::kTileBytes / 2u;
        for (int x = tid; x < picks * 16; x += kTcThreads) {
            const long long off = rowoff(idx[x >> 4]) + (x & 15) * 8;
            cp_async16(tile_u32 + (uint32_t)x * 16u, Kg + off);
            cp_async16(tile_u32 + vhalf + (uint32_t)x * 16u, Vg + off);
        }
        cp_async_wait_all();
        fence_proxy_async();  // the bulk stores below read what these copies wrote
        __syncthreads();      // every kept row is on chip before the first store
        const bool runs = dense ? lay.sn == kTcD : lay.s_page_n == kTcD;
        if (runs) {
            if (tid == 0) {
                for (int row = 0; row < picks;) {
                    const int run = dense ? picks - row : min(picks - row, lay.page_size - row % lay.page_size);
                    const long long off = rowoff(row);
                    bulk_s2g(Kg + off, tile_u32 + (uint32_t)row * 256u, (uint32_t)run * 256u);
                    bulk_s2g(Vg + off, tile_u32 + vhalf + (uint32_t)row * 256u, (uint32_t)run * 256u);
                    row += run;
                }
                bulk_store_wait_read();  // shared memory is read out before the CTA may leave
            }
        } else {
            for (int x = tid; x < picks * 16; x += kTcThreads) {
                const long long off = rowoff(x >> 4) + (x & 15) * 8;
                copy16(reinterpret_cast<char*>(Kg + off), tile + x * 16);
                copy16(reinterpret_cast<char*>(Vg + off), tile + vhalf + x * 16);
            }
        }
    } else {
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            __nv_bfloat16* X = pass ? Vg : Kg;
            __syncthreads();  // the tile is free (greedy loop, or the previous pass, is done with it)
            for (int x = tid; x < picks * 16; x += kTcThreads)
                cp_async16(tile_u32 + (uint32_t)x * 16u, X + rowoff(idx[x >> 4]) + (x & 15) * 8);
            cp_async_wait_all();
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
