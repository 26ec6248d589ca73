// One-launch event kernel for large candidate pools (bf16, d = 128, per-head signatures, N beyond the
// 256 rows that the other tensor-memory kernels hold): prefill compression, N = 4096 -> budget 128.
// One CTA of nine warps per event.
//
//   1. K streams through a ring of eight 64-row stages (cp.async.bulk + full/empty mbarriers, one
//      producer warp, eight scoring warps); every row is scored as it lands and only its score stays
//      on chip. K is read from HBM exactly once.
//   2. s_(b) by a radix-4 bisection over the score keys (all eight warps), then either the top-k
//      flags (lambda = 0) or the pool of candidates that can ever be an arg-max of Eq. 2
//      (s_i >= s_(b) - lambda (1 + slack), see akv_select_pool.cuh), in slot order.
//   3. Only the pool's V rows are read (about 350 of 4096 at lambda = 0.5), into a K-major,
//      128-byte-swizzled operand tile in shared memory.
//   4. Algorithm 1 over the pool, every thread owning up to four candidates (score, norm and running
//      maximum in registers). After a pick, the cosines of the picked row against the whole pool are
//      one thin tensor-core product per block of 128 pool rows: tcgen05.mma with the block as one
//      operand and, as the other, the 16 tile rows around the picked one (no data moves), results
//      in tensor memory, one tcgen05.ld per candidate. Pool rows beyond the tile (rare) take plain
//      dot products from global memory; a pool that exceeds even that takes a plain-dot loop.
//   5. Kept K and V rows are staged on chip and written to slots 0..b-1 of the same buffers.
#pragma once
#include "akv_event_pool.cuh"

namespace akv {

constexpr int kStWarps = 8;                        // scoring / selection warps
constexpr int kStWork = kStWarps * 32;             // their threads
constexpr int kStThreads = kStWork + 32;           // plus the producer warp
constexpr int kStStageRows = 64;                   // K rows per ring stage
constexpr int kStMaxStages = 8;                    // ring depth: 8 stages (128 KB in flight per SM) when they fit, else 4
constexpr unsigned kStStageBytes = kStStageRows * 256u;
constexpr unsigned kStStageChunk = 4u * kStStageBytes;  // kept rows of K and of V (128 each) staged on their way out
constexpr int kStRoundRows = kStWarps * 4;         // rows scored per round (4 per warp)
constexpr int kStCpl = 4;                          // candidates per thread: pools of up to 1024 rows on the tensor-core route
constexpr int kStExtra = 256;                      // pool rows beyond the tile that the tensor-core route still takes
constexpr int kStActive = 248;                     // rows of the active set whose cosine matrix goes to shared memory as a triangle
constexpr int kStWin = 64;                         // pool rows whose cosine columns one product pass yields
constexpr int kStSpare = kStWin;                   // tile rows after the last pool row (reach of a window; scratch row)
constexpr uint32_t kStTmemCols = 512;              // 8 blocks of 128 pool rows x 64 columns

struct StSmem {
    unsigned tile, pool, taken, xs, order, gain, idx, gtab, sect, slot, misc, total;
    unsigned tile_bytes, s, spos, rall, ptaken;  // offsets inside the tile region (valid until the V rows arrive)
    int cap_rows;                                // pool rows the operand tile holds
    int stages;                                  // ring depth
};
// The tile region holds, in turn: the ring + scores + positions (scoring), the pool's V rows (selection), the
// kept rows on their way out. The plain-dot route keeps its per-candidate arrays where the V rows would be.
__host__ __device__ inline StSmem plan_st_smem(int N, int budget, int smem_limit) {
    StSmem p;
    const unsigned np = (unsigned)((N + 3) & ~3);
    unsigned fixed = 0;
    fixed += align16(np * 2);                     // pool
    fixed += align16(np);                         // taken
    fixed += 4u * kStExtra * 4u;                  // xs, xlr, xM, xr: state of the rows beyond the tile
    fixed += 3 * align16((unsigned)budget * 4);   // order, gain, idx
    fixed += 1024 + 256 + 256 + 256;              // gtab + phitab, sect, slot, misc
    fixed += 1024;                                // room to align the base to 1024 bytes
    const unsigned arrays = 3 * align16(np * 4) + align16(np);  // s, spos, rall, ptaken
    unsigned tile_bytes = (unsigned)smem_limit > fixed ? ((unsigned)smem_limit - fixed) / 2048u * 2048u : 0u;
    const unsigned max_tile = (1024u + kStSpare) * 256u;
    if (tile_bytes > max_tile) tile_bytes = max_tile;
    // whole blocks of 128 rows (a block's product reads all 128 of its rows), as long as the scoring phase still fits
    if (tile_bytes / 32768u * 32768u >= 4u * kStStageBytes + arrays) tile_bytes = tile_bytes / 32768u * 32768u;
    p.stages = tile_bytes >= (unsigned)kStMaxStages * kStStageBytes + arrays ? kStMaxStages : 4;
    const unsigned ring = (unsigned)p.stages * kStStageBytes;
    p.cap_rows = tile_bytes >= ring + arrays ? (int)(tile_bytes / 256u) - kStSpare : 0;  // 0: the shape does not fit
    p.tile_bytes = tile_bytes;
    unsigned o = 0;
    p.tile = o;   o += tile_bytes;
    p.pool = o;   o += align16(np * 2);
    p.taken = o;  o += align16(np);
    p.xs = o;     o += 4u * kStExtra * 4u;
    p.order = o;  o += align16((unsigned)budget * 4);
    p.gain = o;   o += align16((unsigned)budget * 4);
    p.idx = o;    o += align16((unsigned)budget * 4);
    p.gtab = o;   o += 1024;   // folded statistic (64 x 8 bytes) and phase steps (64 x 8 bytes)
    p.sect = o;   o += 256;
    p.slot = o;   o += 256;    // 2 x 8 arg-max keys of 8 bytes, 2 x 8 norms
    p.misc = o;   o += 256;    // mbarriers (full, empty, product), tensor-memory base, counters
    p.total = o + 1024;
    p.s = ring;
    p.spos = p.s + align16(np * 4);
    p.rall = p.spos + align16(np * 4);
    p.ptaken = p.rall + align16(np * 4);
    return p;
}

// barrier of the eight work warps (the producer warp has left by the time it is used)
__device__ __forceinline__ void work_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kStWork) : "memory"); }

// eight bf16 of a row against eight of another, accumulated in fp32 (exact products)
__device__ __forceinline__ void dot8_bf16(const uint4& a, const uint4& b, float2& acc) {
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        acc = __ffma2_rn(make_float2(bf16lo(aw[i]), bf16hi(aw[i])), make_float2(bf16lo(bw[i]), bf16hi(bw[i])), acc);
}

__global__ void __launch_bounds__(kStThreads, 1) event_stream_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab,
                                                                    int smem_limit) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ int radix_part[2][kStWarps][3];
    __shared__ int scan_part[2][kStWarps];
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int N = lay.N;
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);
    const StSmem sp = plan_st_smem(N, a.budget, smem_limit);
    unsigned char* tile = smem + sp.tile;
    float* s = reinterpret_cast<float*>(tile + sp.s);
    int* spos = reinterpret_cast<int*>(tile + sp.spos);
    unsigned short* pool = reinterpret_cast<unsigned short*>(smem + sp.pool);
    unsigned char* taken = smem + sp.taken;
    float* xs = reinterpret_cast<float*>(smem + sp.xs);  // rows beyond the tile: score, lambda / norm, running maximum, 1 / norm
    float* xlr = xs + kStExtra;
    float* xM = xlr + kStExtra;
    float* xr = xM + kStExtra;
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    float2* gtab = reinterpret_cast<float2*>(smem + sp.gtab);
    unsigned long long* phitab = reinterpret_cast<unsigned long long*>(gtab + 64);
    float2* sect = reinterpret_cast<float2*>(smem + sp.sect);
    unsigned long long* slot = reinterpret_cast<unsigned long long*>(smem + sp.slot);  // [2][8] keys
    float* slot_r = reinterpret_cast<float*>(smem + sp.slot + 128);                    // [2][8] norms of the warps' best
    const uint32_t bar_full = smem_u32(smem + sp.misc);  // up to 8 barriers
    const uint32_t bar_empty = bar_full + 64;            // up to 8 barriers
    const uint32_t barM = bar_full + 128;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sp.misc + 136);
    int* cnt = reinterpret_cast<int*>(smem + sp.misc + 144);  // [0] a wait ran out, [1] newest position
    const int nst = sp.stages;              // 8 or 4
    const int nsh = nst == 8 ? 3 : 2;       // its logarithm: stage index and round of the ring by mask and shift
    const uint32_t tile_u32 = smem_u32(tile);
    const int cap = sp.cap_rows;
    const uint32_t half_bytes = (uint32_t)(cap + kStSpare) * 128u;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool worker = warp < kStWarps;
    const bool similarity = a.greedy != 0;
    const bool dense = lay.page_size == 0;
    const long long ev_off = dense ? id.b * lay.sb + id.l * lay.sl + id.h * lay.sh : 0;
    auto rowoff = [&](int j) -> long long {
        return dense ? ev_off + (long long)j * lay.sn : row_offset(lay, id.b, id.l, id.h, j);
    };
    __nv_bfloat16* Kg = reinterpret_cast<__nv_bfloat16*>(a.K);
    __nv_bfloat16* Vg = reinterpret_cast<__nv_bfloat16*>(a.V);
    const int* gpos = event_pos(a.pos, id);
    const bool rotate = gpos != nullptr;

    phase_stamp(id.e, 0);  // phases: 0 start, 1 tables + positions, 2 K scored, 3 s_(b), 4 pool / top-k, 5 V rows + norms, 6 picks, 7 outputs, 8 end
    // ---- set-up: barriers, tables, positions on chip --------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < nst; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, kStWarps);
        }
        mbar_init_fence();
        cnt[0] = 0;
        cnt[1] = INT_MIN;
    }
    if (warp == 1) fill_sector_table(sect, lane);
    fill_statistic_tables(a.qstat + ((long long)id.l * lay.H + id.h) * kTcD, tab, tid, gtab, phitab);
    __syncthreads();
    {
        int pmax = INT_MIN;
        for (int j = tid; j < n; j += kStThreads) {
            const int p = rotate ? gpos[j] : 0;
            spos[j] = p;
            pmax = max(pmax, p);
        }
        pmax = __reduce_max_sync(0xFFFFFFFFu, pmax);
        if (lane == 0) atomicMax(&cnt[1], pmax);
    }
    __syncthreads();
    long long pref = 0;
    if (rotate) pref = a.p_ref ? (long long)a.p_ref[id.b] : (long long)cnt[1] + 1;
    // D: the spacing of rows one stage (64 slots) apart at the newest end, which a cache filled token by token has
    // everywhere. Whether it does is found once, here; the scoring loop then chains without looking at positions.
    const long long D = n > kStStageRows ? (long long)spos[n - 1] - (long long)spos[n - 1 - kStStageRows] : 0;
    bool uniform;
    {
        bool uni = true;
        for (int j = kStStageRows + tid; j < n; j += kStThreads) uni &= (long long)spos[j] - (long long)spos[j - kStStageRows] == D;
        uniform = __syncthreads_and(uni);
    }

    phase_stamp(id.e, 1);
    // ---- K through the ring, scored as it lands ---------------------------------------------------------------
    const int stages = (n + kStStageRows - 1) / kStStageRows;
    int bad = 0;
    if (!worker) {
        if (lane == 0) {
            for (int st = 0; st < stages; ++st) {
                const int sl = st & (nst - 1);
                if (st >= nst && !mbar_wait_bounded(bar_empty + 8 * sl, (uint32_t)(((st >> nsh) - 1) & 1), a.wait_polls)) {
                    atomicExch(&cnt[0], 1);
                    break;
                }
                const int r0 = st * kStStageRows, r1 = min(n, r0 + kStStageRows);
                mbar_expect_tx(bar_full + 8 * sl, (uint32_t)(r1 - r0) * 256u);
                // as few copies as the layout allows: the whole stage when its rows are contiguous, whole pages
                // when pages are, else row by row (starve, a testing aid: none at all, the scoring warps' wait runs out)
                for (int row = r0; row < r1 && !a.starve;) {
                    int run = 1;
                    if (dense && lay.sn == kTcD) run = r1 - row;
                    else if (!dense && lay.s_page_n == kTcD) run = min(r1 - row, lay.page_size - row % lay.page_size);
                    bulk_g2s(tile_u32 + (uint32_t)sl * kStStageBytes + (uint32_t)(row - r0) * 256u, Kg + rowoff(row),
                             (uint32_t)run * 256u, bar_full + 8 * sl);
                    row += run;
                }
            }
        }
    } else {
        const int grp = lane >> 3, f0 = (lane & 7) * 8;
        // A lane group scores two rows of every stage, 32 slots apart, as two independent chains (the second
        // hides the first one's latencies); each chain steps by one stage = 64 slots.
        const int D32 = (int)D;
        const bool d_fits = (long long)D32 == D;
        ChainScore ca, cb;  // cb uses ca's S
        ca.set_step(D, phitab + f0, sect);
        AKV_PHASE_ACC_DECL(cyc_kwait);
        for (int st = 0; st < stages; ++st) {
            const int sl = st & (nst - 1);
            AKV_PHASE_ACC_BEGIN(cyc_kwait);
            const bool landed = mbar_wait_bounded(bar_full + 8 * sl, (uint32_t)((st >> nsh) & 1), a.wait_polls);
            AKV_PHASE_ACC_END(cyc_kwait);
            if (!landed) {
                atomicExch(&cnt[0], 1);
                break;
            }
            const int ja = st * kStStageRows + 4 * warp + grp, jb = ja + kStRoundRows;
            const bool la = ja < n, lb = jb < n;
            bool fresh = (st & (kChainRounds - 1)) == 0 || a.no_chain || !d_fits;
            int pa = 0, pb = 0;
            if (fresh || !uniform) {
                pa = la ? spos[ja] : 0;
                pb = lb ? spos[jb] : 0;
            }
            if (!fresh && !uniform)
                fresh = !__all_sync(0xFFFFFFFFu, (!la || pa - spos[ja - kStStageRows] == D32) && (!lb || pb - spos[jb - kStStageRows] == D32));
            if (fresh) {
                if (la) ca.anchor(pref - (long long)pa, gtab + f0, phitab + f0, sect);
                if (lb) cb.anchor(pref - (long long)pb, gtab + f0, phitab + f0, sect);
            } else {
                ca.advance();
                cb.advance_by(ca);
            }
            float acca = 0.f, accb = 0.f;
            const unsigned char* krow = tile + sl * kStStageBytes + (4 * warp + grp) * 256 + (lane & 7) * 16;
            if (la) acca = ca.dot(*reinterpret_cast<const uint4*>(krow), *reinterpret_cast<const uint4*>(krow + 128));
            if (lb) accb = cb.dot(*reinterpret_cast<const uint4*>(krow + kStRoundRows * 256), *reinterpret_cast<const uint4*>(krow + kStRoundRows * 256 + 128));
#pragma unroll
            for (int off = 4; off > 0; off >>= 1) {
                acca += __shfl_xor_sync(0xFFFFFFFFu, acca, off);
                accb += __shfl_xor_sync(0xFFFFFFFFu, accb, off);
            }
            if ((lane & 7) == 0) {
                if (la) {
                    if (a.scores) a.scores[(long long)id.e * N + ja] = acca;
                    const bool fin = isfinite(acca);
                    bad |= !fin;
                    s[ja] = fin ? acca : -INFINITY;
                }
                if (lb) {
                    if (a.scores) a.scores[(long long)id.e * N + jb] = accb;
                    const bool fin = isfinite(accb);
                    bad |= !fin;
                    s[jb] = fin ? accb : -INFINITY;
                }
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_empty + 8 * sl) : "memory");
        }
        AKV_PHASE_ACC_STORE(id.e, 13, cyc_kwait);
    }
    __syncthreads();
    if (cnt[0]) {
        // a wait ran out: report it, give copies that may still be in flight a bounded chance to land, leave
        if (tid == 0) {
            if (a.status) a.status[id.e] = 3;
            for (int sl = 0; sl < nst; ++sl) {
                mbar_wait_bounded(bar_full + 8 * sl, 0, a.wait_polls);
                mbar_wait_bounded(bar_full + 8 * sl, 1, a.wait_polls);
            }
        }
        return;
    }
    bad = __syncthreads_or(bad);
    if (!worker) return;  // the producer warp is done; the work warps meet at their own barrier from here on

    phase_stamp(id.e, 2);
    const int np4 = (N + 3) & ~3;
    for (int j = tid; j < np4; j += kStWork) taken[j] = 0;

    // ---- s_(b): the picks-th largest score key, two bits per round ---------------------------------------------
    uint32_t kb = 0u;
    if (picks > 0) {
        // up to 16 keys per thread stay in registers (N <= 4096); longer events read theirs from shared memory
        constexpr int kRegKeys = 16;
        const bool in_regs = n <= kRegKeys * kStWork;
        uint32_t kreg[kRegKeys];
#pragma unroll
        for (int i = 0; i < kRegKeys; ++i) {
            const int j = tid + i * kStWork;
            kreg[i] = (in_regs && j < n) ? orderable(s[j]) : 0u;
        }
        for (int lo = 30; lo >= 0; lo -= 2) {
            const uint32_t v1 = kb | (1u << lo), v2 = kb | (2u << lo), v3 = kb | (3u << lo);
            // the three counts of a warp (at most 512 each when the keys sit in registers) travel in one word
            uint32_t c = 0u;
            int c1 = 0, c2 = 0, c3 = 0;
            if (in_regs) {
#pragma unroll
                for (int i = 0; i < kRegKeys; ++i) c += (kreg[i] >= v1) + ((kreg[i] >= v2) << 10) + ((kreg[i] >= v3) << 20);
                c = __reduce_add_sync(0xFFFFFFFFu, c);
                c1 = c & 1023; c2 = (c >> 10) & 1023; c3 = c >> 20;
            } else {
                for (int j = tid; j < n; j += kStWork) {
                    const uint32_t k = orderable(s[j]);
                    c1 += k >= v1;
                    c2 += k >= v2;
                    c3 += k >= v3;
                }
                c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
                c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
                c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
            }
            int (*rp)[3] = radix_part[(lo >> 1) & 1];  // per-warp partial counts, double-buffered by round
            if (lane == 0) { rp[warp][0] = c1; rp[warp][1] = c2; rp[warp][2] = c3; }
            work_barrier();
            int t1 = 0, t2 = 0, t3 = 0;
#pragma unroll
            for (int w = 0; w < kStWarps; ++w) { t1 += rp[w][0]; t2 += rp[w][1]; t3 += rp[w][2]; }
            kb = t3 >= picks ? v3 : (t2 >= picks ? v2 : (t1 >= picks ? v1 : kb));
        }
    }
    phase_stamp(id.e, 3);
    const float sb = from_orderable(kb);

    // block-wide ordered compaction over the slots: calls emit(j, position) for every flagged slot, in slot
    // order; returns the number of flagged slots
    auto ordered_scan = [&](auto&& flag, auto&& emit) -> int {
        int base = 0;
        int it = 0;
        for (int j0 = 0; j0 < n; j0 += kStWork, ++it) {
            const int j = j0 + tid;
            const bool in = j < n && flag(j);
            const uint32_t mask = __ballot_sync(0xFFFFFFFFu, in);
            int* spart = scan_part[it & 1];
            if (lane == 0) spart[warp] = __popc(mask);
            work_barrier();
            int before = 0, total = 0;
#pragma unroll
            for (int w = 0; w < kStWarps; ++w) {
                before += w < warp ? spart[w] : 0;
                total += spart[w];
            }
            if (in) emit(j, base + before + __popc(mask & ((1u << lane) - 1u)));
            base += total;
        }
        work_barrier();
        return base;
    };

    // the winning key of every pick: value in the high word, 0xFFFFFFFF - pool row in the low word
    // (a thread whose wait on the tensor core ran out offers the all-ones key: every thread then sees it win)
    auto exchange_best = [&](int t, unsigned long long best, float best_r, float& ri) -> unsigned long long {
        const uint32_t hi = (uint32_t)(best >> 32), lo = (uint32_t)best;
        const uint32_t whi = __reduce_max_sync(0xFFFFFFFFu, hi);
        const uint32_t wlo = __reduce_max_sync(0xFFFFFFFFu, hi == whi ? lo : 0u);
        unsigned long long* sl = slot + (t & 1) * kStWarps;
        float* slr = slot_r + (t & 1) * kStWarps;
        if (hi == whi && lo == wlo) {  // one lane per warp, unless the warp has no candidate left (all keys 0)
            sl[warp] = best;
            slr[warp] = best_r;
        }
        work_barrier();
        unsigned long long top = sl[0];
        int wtop = 0;
#pragma unroll
        for (int w = 1; w < kStWarps; ++w)
            if (sl[w] > top) { top = sl[w]; wtop = w; }
        ri = slr[wtop];
        if (tid == 0) gain[t] = from_orderable((uint32_t)(top >> 32));
        return top;
    };
    auto key_row = [](unsigned long long key) -> int { return (int)(0xFFFFFFFFu - (uint32_t)key); };

    int P = 0;
    if (!similarity) {
        // top-k: every key above the picks-th one, and the lowest slots among those equal to it
        float* ps = reinterpret_cast<float*>(spos);  // positions are no longer needed
        const int above = ordered_scan([&](int j) { return orderable(s[j]) > kb; }, [&](int j, int) { taken[j] = 1; });
        ordered_scan([&](int j) { return orderable(s[j]) == kb; }, [&](int j, int pos) { if (pos < picks - above) taken[j] = 1; });
        // the chosen slots as a pool in slot order, then the pick order: by score, equal scores by slot
        P = ordered_scan([&](int j) { return taken[j] != 0; }, [&](int j, int pos) { pool[pos] = (unsigned short)j; ps[pos] = s[j]; });
        for (int rho = tid; rho < P; rho += kStWork) {
            const uint32_t k = orderable(ps[rho]);
            int rank = 0;
            for (int o = 0; o < P; ++o) {
                const uint32_t ko = orderable(ps[o]);
                rank += ko > k || (ko == k && o < rho);
            }
            order[rank] = pool[rho];
            gain[rank] = ps[rho];
        }
        work_barrier();
    } else {
        const float thr = a.no_prune ? -INFINITY : fmaf(-1.001f, a.lam, sb) - 1e-6f * fabsf(sb);  // -inf keeps everyone
        P = ordered_scan([&](int j) { return !(s[j] < thr); }, [&](int j, int pos) { pool[pos] = (unsigned short)j; });

        phase_stamp(id.e, 4);
        // ======== active-set route ===============================================================================
        // The picks hardly ever reach beyond the best-scored few dozen rows past the budget. So: the cosine matrix
        // of the pool's kStActive best-scored rows only (one tcgen05 product per block of 128 rows, lower triangle
        // to shared memory), and Algorithm 1 as a one-warp loop over that triangle. Every candidate left out
        // scores at most `bound` and its Eq. 2 value never exceeds its score, so the loop is exact as long as the
        // winning value stays above the bound; if it ever does not, the event is redone by the routes below.
        bool done = false;
        if (picks > 1 && cap >= 256) {
            // the (kStActive + 1)-th largest key of the pool (0: the pool is no larger than the active set)
            uint32_t bound = 0u;
            if (P > kStActive) {
                uint32_t pk[kStCpl + 1];
#pragma unroll
                for (int k = 0; k <= kStCpl; ++k) {
                    const int rho = tid + k * kStWork;
                    pk[k] = rho < P ? orderable(s[pool[rho]]) : 0u;
                }
                const bool in_regs = P <= (kStCpl + 1) * kStWork;
                for (int lo = 30; lo >= 0; lo -= 2) {
                    const uint32_t v1 = bound | (1u << lo), v2 = bound | (2u << lo), v3 = bound | (3u << lo);
                    int c1 = 0, c2 = 0, c3 = 0;
                    if (in_regs) {
#pragma unroll
                        for (int k = 0; k <= kStCpl; ++k) { c1 += pk[k] >= v1; c2 += pk[k] >= v2; c3 += pk[k] >= v3; }
                    } else {
                        for (int rho = tid; rho < P; rho += kStWork) {
                            const uint32_t k = orderable(s[pool[rho]]);
                            c1 += k >= v1; c2 += k >= v2; c3 += k >= v3;
                        }
                    }
                    c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
                    c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
                    c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
                    int (*rp)[3] = radix_part[(lo >> 1) & 1];
                    if (lane == 0) { rp[warp][0] = c1; rp[warp][1] = c2; rp[warp][2] = c3; }
                    work_barrier();
                    int t1 = 0, t2 = 0, t3 = 0;
#pragma unroll
                    for (int w = 0; w < kStWarps; ++w) { t1 += rp[w][0]; t2 += rp[w][1]; t3 += rp[w][2]; }
                    bound = t3 > kStActive ? v3 : (t2 > kStActive ? v2 : (t1 > kStActive ? v1 : bound));
                }
            }
            // the active rows, in slot order (ties in the loop then go to the lower row = the lower slot)
            unsigned short* act = reinterpret_cast<unsigned short*>(xs);  // 256 entries
            float* ar = xs + 128;                                          // their reciprocal norms: 256 floats
            const int R = ordered_scan([&](int j) { return !(s[j] < thr) && orderable(s[j]) > bound; },
                                       [&](int j, int pos) { act[pos] = (unsigned short)j; });
            if (warp == 0) tmem_alloc(smem_u32(tmem_holder), kStTmemCols);
            for (int x = tid; x < R * 16; x += kStWork) {
                const int rho = x >> 4, c = x & 15;
                cp_async16(tile_u32 + tile_chunk(rho, c, half_bytes), Vg + rowoff(act[rho]) + c * 8);
            }
            if (tid == 0) {
                mbar_init(barM, 1);
                mbar_init_fence();
            }
            cp_async_wait_all();
            fence_proxy_async();
            tc_fence_before();
            work_barrier();
            tc_fence_after();
            const uint32_t tbase = *tmem_holder;
            const int nblk = (R + 127) >> 7, ncol = (R + 15) & ~15;
            if (tid == 0) {
                const uint32_t idesc = umma_idesc_bf16(128, ncol);
                for (int blk = 0; blk < nblk; ++blk) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                        umma_bf16(tbase + (uint32_t)(256 * blk), umma_desc_sw128(tile_u32 + (uint32_t)blk * 16384u + koff),
                                  umma_desc_sw128(tile_u32 + koff), idesc, kk > 0 ? 1u : 0u);
                    }
                }
                umma_commit(barM);
            }
            int timeout = !mbar_wait_bounded(barM, 0, a.wait_polls);
            tc_fence_after();
            // every thread has seen the product complete (it has read the whole tile) before the triangle lands on the tile
            timeout = __reduce_or_sync(0xFFFFFFFFu, timeout);
            if (lane == 0 && timeout) atomicExch(&cnt[0], 1);
            work_barrier();
            if (!cnt[0]) {
                // lower triangle -> shared memory: warp w holds rows 128 (w / 4) + 32 (w % 4) + lane of the matrix
                float* tri = reinterpret_cast<float*>(tile);
                const int blk = warp >> 2, row = 128 * blk + 32 * (warp & 3) + lane;
                if (128 * blk + 32 * (warp & 3) < R) {
                    const uint32_t lanes = tbase + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(256 * blk);
                    const int trow = tri_row(row), last_cb = (128 * blk + 32 * (warp & 3) + 31) >> 5;
                    float diag = 0.f;  // the diagonal entry: squared norm
                    for (int cb = 0; cb <= last_cb; ++cb) {
                        uint32_t v[32];
                        tmem_ld32(lanes + (uint32_t)(32 * cb), v);
                        tmem_ld_wait();
                        if (row < R) {
#pragma unroll
                            for (int k = 0; k < 32; ++k) {
                                if (32 * cb + k <= row) tri[trow + 32 * cb + k] = __uint_as_float(v[k]);
                                diag = (32 * cb + k == row) ? __uint_as_float(v[k]) : diag;
                            }
                        }
                    }
                    if (row < R) ar[row] = 1.f / (sqrtf(diag) + a.eps);
                }
            }
            tc_fence_before();
            work_barrier();
            if (warp == 0) tmem_dealloc(tbase, kStTmemCols);
            if (cnt[0]) {
                if (tid == 0 && a.status) a.status[id.e] = 3;
                return;
            }
            phase_stamp(id.e, 5);
            if (warp == 0) {
                const bool ok = picks_cosine<8, true>(lane, R, picks, s, act, ar, a.lam, reinterpret_cast<float*>(tile),
                                                           reinterpret_cast<uint32_t*>(gain), order, bound);
                if (lane == 0) cnt[2] = ok ? 1 : 0;
            }
            work_barrier();
            done = cnt[2] != 0;
            if (done) {
                for (int t = tid; t < picks; t += kStWork) {
                    const int j = act[order[t]];
                    gain[t] = from_orderable(reinterpret_cast<uint32_t*>(gain)[t]);
                    order[t] = j;
                }
            }
            work_barrier();
        }
        if (done) {
            // picks are in order[] / gain[]
        } else if (P <= cap + kStExtra && picks > 1) {
            // ======== tensor-core route: any pool that fits the tile (a few rows may stay outside) ================
            // thread (warp w, lane l) owns pool rows 128 (2 k + w / 4) + 32 (w % 4) + l, k < 4: row r of a block of 128
            // is lane r of tensor memory, and a warp reads the lanes of its own quarter
            const int quarter = warp & 3, blk0 = warp >> 2;
            const int resident = min(P, cap), extras = P - resident;
            // The pool goes into the tile by descending score (equal scores by slot): picks then come roughly in
            // tile order, and one product pass, which yields the cosine columns of the 64 tile rows from the picked
            // one on, serves the picks that follow until one falls outside that window.
            {
                unsigned long long* skey = reinterpret_cast<unsigned long long*>(spos);  // positions and the plain-dot arrays are dead
                unsigned short* sorted = reinterpret_cast<unsigned short*>(xs);
                for (int rho = tid; rho < P; rho += kStWork)
                    skey[rho] = ((unsigned long long)orderable(s[pool[rho]]) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)rho);
                work_barrier();
                unsigned long long mine[kStCpl + 1];
                int rank[kStCpl + 1];
#pragma unroll
                for (int k = 0; k <= kStCpl; ++k) {
                    const int rho = tid + k * kStWork;
                    mine[k] = rho < P ? skey[rho] : ~0ull;
                    rank[k] = 0;
                }
                for (int o = 0; o < P; ++o) {
                    const unsigned long long ko = skey[o];
#pragma unroll
                    for (int k = 0; k <= kStCpl; ++k) rank[k] += ko > mine[k];
                }
#pragma unroll
                for (int k = 0; k <= kStCpl; ++k) {
                    const int rho = tid + k * kStWork;
                    if (rho < P) sorted[rank[k]] = pool[rho];
                }
                work_barrier();
                for (int rho = tid; rho < P; rho += kStWork) pool[rho] = sorted[rho];
                work_barrier();
            }
            float sv[kStCpl], lr[kStCpl], rr[kStCpl], M[kStCpl];
            uint32_t klow[kStCpl];  // low key word: 0xFFFF - slot (ties go to the lower slot), then the pool row
            uint32_t alive = 0u;
#pragma unroll
            for (int k = 0; k < kStCpl; ++k) {
                const int rho = 128 * (2 * k + blk0) + 32 * quarter + lane;
                sv[k] = 0.f; lr[k] = 0.f; rr[k] = 0.f; M[k] = 0.f; klow[k] = 0u;
                if (rho < resident) {
                    const int j = pool[rho];
                    sv[k] = s[j];
                    klow[k] = ((0xFFFFu - (uint32_t)j) << 16) | (uint32_t)rho;
                    alive |= 1u << k;
                }
            }
            uint32_t xklow = 0u;
            if (tid < extras) {
                const int j = pool[resident + tid];
                xs[tid] = s[j];
                xM[tid] = 0.f;
                xklow = ((0xFFFFu - (uint32_t)j) << 16) | (uint32_t)(resident + tid);
            }
            bool xalive = tid < extras;
            if (warp == 0) tmem_alloc(smem_u32(tmem_holder), kStTmemCols);
            work_barrier();  // every score has been read: the V rows may land on them
            for (int x = tid; x < resident * 16; x += kStWork) {
                const int rho = x >> 4, c = x & 15;
                cp_async16(tile_u32 + tile_chunk(rho, c, half_bytes), Vg + rowoff(pool[rho]) + c * 8);
            }
            cp_async_wait_all();
            fence_proxy_async();
            tc_fence_before();
            work_barrier();
            tc_fence_after();
            const uint32_t tbase = *tmem_holder;
            // reciprocal norms (Eq. 1)
#pragma unroll
            for (int k = 0; k < kStCpl; ++k) {
                if (alive & (1u << k)) {
                    const int rho = 128 * (2 * k + blk0) + 32 * quarter + lane;
                    float2 acc = make_float2(0.f, 0.f);
#pragma unroll 4
                    for (int c = 0; c < 16; ++c) {
                        const uint4 v = *reinterpret_cast<const uint4*>(tile + tile_chunk(rho, c, half_bytes));
                        dot8_bf16(v, v, acc);
                    }
                    rr[k] = 1.f / (sqrtf(acc.x + acc.y) + a.eps);
                    lr[k] = a.lam * rr[k];
                }
            }
            // a row beyond the tile stays in its thread's registers for the whole loop (256 bytes)
            uint4 own[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) own[c] = make_uint4(0u, 0u, 0u, 0u);
            if (xalive) {
                const __nv_bfloat16* vrow = Vg + rowoff(pool[resident + tid]);
                float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    own[c] = *reinterpret_cast<const uint4*>(vrow + c * 8);
                    dot8_bf16(own[c], own[c], acc);
                }
                xr[tid] = 1.f / (sqrtf(acc.x + acc.y) + a.eps);
                xlr[tid] = a.lam * xr[tid];
            }
            const int nblk = (resident + 127) >> 7;
            // window: 128 tile rows when the pool has at most four blocks (4 x 128 columns of tensor memory), else 64;
            // it starts a little before the picked row, because a candidate that an earlier pick's penalty held back
            // is picked later, behind the front of the sequence
            const int win = nblk <= 4 ? 2 * kStWin : kStWin, back = nblk <= 4 ? 40 : 24;
            const uint32_t idesc = umma_idesc_bf16(128, win);
            int cbase = -1;  // first tile row of the window whose columns tensor memory holds (-1: none)
            // block w's product is issued by lane 0 of warp w (blocks are independent: own rows, own columns), each
            // with its own commit; the barrier completes when all nblk of them have arrived
            if (tid == 0) {
                mbar_init(barM, (uint32_t)nblk);
                mbar_init_fence();
            }
            work_barrier();
            int timeout = 0;
            uint32_t mround = 0;
            AKV_PHASE_ACC_DECL(cyc_argmax);
            AKV_PHASE_ACC_DECL(cyc_product);
            AKV_PHASE_ACC_DECL(cyc_update);
            phase_stamp(id.e, 5);
            for (int t = 0; t < picks; ++t) {
                AKV_PHASE_ACC_BEGIN(cyc_argmax);
                // Eq. 2 for the candidates still competing, Eq. 3's arg-max (ties to the lower pool row = lower slot)
                unsigned long long best = 0ull;
                float best_r = 0.f;
#pragma unroll
                for (int k = 0; k < kStCpl; ++k) {
                    if (alive & (1u << k)) {
                        const unsigned long long key = ((unsigned long long)orderable(fmaf(-lr[k], M[k], sv[k])) << 32) | klow[k];
                        if (key > best) { best = key; best_r = rr[k]; }
                    }
                }
                if (xalive) {
                    const unsigned long long key = ((unsigned long long)orderable(fmaf(-xlr[tid], xM[tid], xs[tid])) << 32) | xklow;
                    if (key > best) { best = key; best_r = xr[tid]; }
                }
                if (timeout) best = ~0ull;
                float ri;
                const unsigned long long top = exchange_best(t, best, best_r, ri);
                if (top == ~0ull) {  // some thread's wait ran out in the previous pick
                    timeout = 1;
                    break;
                }
                AKV_PHASE_ACC_END(cyc_argmax);
                const int irho = (int)((uint32_t)top & 0xFFFFu);
                if (tid == 0) order[t] = pool[irho];
#pragma unroll
                for (int k = 0; k < kStCpl; ++k)
                    if (128 * (2 * k + blk0) + 32 * quarter + lane == irho) alive &= ~(1u << k);
                if (resident + tid == irho) xalive = false;
                if (t + 1 == picks) break;
                // cosines of the picked row against the pool: already in tensor memory when the row lies in the current
                // window; else one product per block of 128 rows, block x (the 64 tile rows from the picked one on)^T
                const bool hit = irho < resident && cbase >= 0 && irho >= cbase && irho < cbase + win;
                AKV_PHASE_ACC_BEGIN(cyc_product);
                if (!hit) {
                    cbase = max(irho - back, 0) & ~7;
                    if (irho >= resident) {
                        // the picked row lies beyond the tile: it becomes the scratch row after the last pool row
                        cbase = cap;
                        if (tid < 16) cp_async16(tile_u32 + tile_chunk(cap, tid, half_bytes), Vg + rowoff(pool[irho]) + tid * 8);
                        cp_async_wait_all();
                        fence_proxy_async();
                        work_barrier();
                    }
                    if (lane == 0 && warp < nblk) {
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                            umma_bf16(tbase + (uint32_t)(win * warp), umma_desc_sw128(tile_u32 + (uint32_t)warp * 16384u + koff),
                                      umma_desc_sw128(tile_u32 + (uint32_t)cbase * 128u + koff), idesc, kk > 0 ? 1u : 0u);
                        }
                        umma_commit(barM);
                    }
                }
                const int col = irho >= resident ? 0 : irho - cbase;
                // rows beyond the tile: plain dot products, both rows read in place, while the tensor core works
                if (xalive) {
                    const int prow = irho >= resident ? cap : irho;  // the picked row sits in the tile (as the scratch row if need be)
                    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        dot8_bf16(own[c], *reinterpret_cast<const uint4*>(tile + tile_chunk(prow, c, half_bytes)), acc);
                    xM[tid] = fmaxf(xM[tid], ri * (acc.x + acc.y));
                }
                if (!hit) {
                    if (!mbar_wait_bounded(barM, mround & 1u, a.wait_polls)) timeout = 1;  // offered to everyone at the next exchange
                    ++mround;
                    if (irho >= resident) cbase = -1;  // the scratch row's window serves this pick only
                }
                AKV_PHASE_ACC_END(cyc_product);
                AKV_PHASE_ACC_BEGIN(cyc_update);
                tc_fence_after();
                {
                    // tcgen05.ld is a warp-wide instruction: every lane issues it, for every block the pool has
                    // (a warp-uniform test); what a retired candidate reads is not used
                    float dv[kStCpl];
#pragma unroll
                    for (int k = 0; k < kStCpl; ++k)
                        dv[k] = (2 * k + blk0 < nblk)
                                    ? tmem_ld1(tbase + ((uint32_t)(32 * quarter) << 16) + (uint32_t)(win * (2 * k + blk0) + col))
                                    : 0.f;
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < kStCpl; ++k)
                        if (alive & (1u << k)) M[k] = fmaxf(M[k], ri * dv[k]);
                }
                tc_fence_before();
                AKV_PHASE_ACC_END(cyc_update);
            }
            AKV_PHASE_ACC_STORE(id.e, 10, cyc_argmax);
            AKV_PHASE_ACC_STORE(id.e, 11, cyc_product);
            AKV_PHASE_ACC_STORE(id.e, 12, cyc_update);
            tc_fence_before();
            work_barrier();
            if (warp == 0) tmem_dealloc(tbase, kStTmemCols);
            if (timeout) {  // uniform: it comes out of an exchange
                if (tid == 0 && a.status) a.status[id.e] = 3;
                return;
            }
        } else {
            // ======== plain-dot route: any pool size; V rows read in place, state where the V rows would be ======
            float* ps = reinterpret_cast<float*>(spos);
            float* m = s;
            float* r = reinterpret_cast<float*>(tile + sp.rall);
            unsigned char* ptaken = tile + sp.ptaken;
            for (int rho = tid; rho < P; rho += kStWork) ps[rho] = s[pool[rho]];
            work_barrier();  // s is dead: every pool score sits in ps
            for (int rho = tid; rho < P; rho += kStWork) {
                m[rho] = 0.f;
                ptaken[rho] = 0;
            }
            // Work items: (pool row, half) with the halves taking alternate 16-byte chunks; neighbouring lanes hold
            // the two halves of one row and combine them with one shuffle.
            const int items = 2 * P, items_up = (items + 31) & ~31;
            auto vchunk = [&](int rho, int c) -> uint4 { return *reinterpret_cast<const uint4*>(Vg + rowoff(pool[rho]) + c * 8); };
            for (int i = tid; i < items_up; i += kStWork) {
                const int rho = i >> 1, half = i & 1;
                float2 acc = make_float2(0.f, 0.f);
                if (rho < P) {
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) {
                        const uint4 v = vchunk(rho, 2 * cc + half);
                        dot8_bf16(v, v, acc);
                    }
                }
                float ss = acc.x + acc.y;
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
                if (rho < P && half == 0) r[rho] = 1.f / (sqrtf(ss) + a.eps);
            }
            work_barrier();
            // Pass t folds the cosines of pick t - 1 into every candidate's running maximum and, in the same sweep,
            // finds the arg-max of Eq. 2 for pick t. The first pass (no pick yet) is the plain arg-max of the scores.
            int irho = -1;
            float ri = 0.f;
            for (int t = 0; t < picks; ++t) {
                unsigned long long best = 0ull;
                float best_r = 0.f;
                for (int i = tid; i < items_up; i += kStWork) {
                    const int rho = i >> 1, half = i & 1;
                    const bool live = rho < P && !ptaken[rho] && rho != irho;  // (the last pick's flag may not be visible yet)
                    float dotv = 0.f;
                    if (irho >= 0) {
                        float2 acc = make_float2(0.f, 0.f);
                        if (live) {
#pragma unroll
                            for (int cc = 0; cc < 8; ++cc) dot8_bf16(vchunk(rho, 2 * cc + half), vchunk(irho, 2 * cc + half), acc);
                        }
                        dotv = acc.x + acc.y;
                        dotv += __shfl_xor_sync(0xFFFFFFFFu, dotv, 1);
                    }
                    if (live && half == 0) {
                        float mm = m[rho];
                        if (irho >= 0) {
                            mm = fmaxf(mm, dotv * (ri * r[rho]));
                            m[rho] = mm;
                        }
                        const unsigned long long key = ((unsigned long long)orderable(fmaf(-a.lam, mm, ps[rho])) << 32) |
                                                       (unsigned long long)(0xFFFFFFFFu - (uint32_t)rho);
                        if (key > best) { best = key; best_r = r[rho]; }
                    }
                }
                irho = key_row(exchange_best(t, best, best_r, ri));
                if (tid == 0) {
                    order[t] = pool[irho];
                    ptaken[irho] = 1;
                }
            }
        }
        work_barrier();
        for (int t = tid; t < picks; t += kStWork) taken[order[t]] = 1;
        work_barrier();
    }

    phase_stamp(id.e, 6);
    // ---- sort(S) and outputs -------------------------------------------------------------------------
    const int kept = ordered_scan([&](int j) { return taken[j] != 0; }, [&](int j, int pos) { idx[pos] = j; });
    for (int t = kept + tid; t < a.budget; t += kStWork) idx[t] = -1;
    work_barrier();
    const long long ob = (long long)id.e * a.budget;
    for (int t = tid; t < a.budget; t += kStWork) {
        a.idx_sorted[ob + t] = idx[t];
        if (a.pick_order) a.pick_order[ob + t] = t < picks ? order[t] : -1;
        if (a.pick_gain) a.pick_gain[ob + t] = t < picks ? gain[t] : 0.f;
    }
    if (tid == 0) {
        if (a.n_kept) a.n_kept[id.e] = picks;
        if (a.status) a.status[id.e] = n < bud ? 2 : (bad ? 1 : 0);
    }

    phase_stamp(id.e, 7);
    // ---- compaction in place: every kept row of a chunk is on chip before the chunk's first store --------
    // (a chunk's destinations [c0, c1) can only be sources of the same or of later chunks: idx is ascending
    // and idx[t] >= t; later chunks' sources lie at or beyond their own destinations)
    int* wpos = a.pos.p ? a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh : nullptr;
    const int chunk = (int)(kStStageChunk / 512u);  // rows of K and of V staged per round
    const int moved = min(picks, kept);  // (equal by construction; the smaller one keeps every index read below valid)
    for (int c0 = 0; c0 < moved; c0 += chunk) {
        const int cn = min(chunk, moved - c0);
        work_barrier();
        for (int x = tid; x < cn * 16; x += kStWork) {
            const long long off = rowoff(idx[c0 + (x >> 4)]) + (x & 15) * 8;
            cp_async16(tile_u32 + (uint32_t)x * 16u, Kg + off);
            cp_async16(tile_u32 + (uint32_t)(chunk * 256) + (uint32_t)x * 16u, Vg + off);
        }
        int pv = 0;
        if (wpos && tid < cn) pv = gpos[idx[c0 + tid]];
        cp_async_wait_all();
        work_barrier();
        for (int x = tid; x < cn * 16; x += kStWork) {
            const long long off = rowoff(c0 + (x >> 4)) + (x & 15) * 8;
            *reinterpret_cast<uint4*>(Kg + off) = *reinterpret_cast<const uint4*>(tile + x * 16);
            *reinterpret_cast<uint4*>(Vg + off) = *reinterpret_cast<const uint4*>(tile + chunk * 256 + x * 16);
        }
        if (wpos && tid < cn) wpos[c0 + tid] = pv;
    }
    phase_stamp(id.e, 8);
}

}  // namespace akv
