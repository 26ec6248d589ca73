// Tensor-memory path for bf16, d = 128, per-head signatures, N <= 256: one CTA of four warps per
// event, several CTAs resident per SM.
//
//   1. K rows arrive in shared memory by per-row bulk copies (cp.async.bulk + mbarrier) and are
//      scored there (fused RoPE rotate-and-dot against the folded query statistic).
//   2. Candidates are ranked by score (ties to the lower slot). Only candidates with
//        s_i >= s_(b) - lambda * (1 + slack)
//      can ever be an argmax of Eq. 2 (the running maximum m never exceeds 1, so every still
//      unchosen member of the top-b scores beats them): that pool of P rows, in rank order, is
//      the only part of V that is read.
//   3. The pool's V rows are laid out as a K-major, 128-byte-swizzled operand tile and ONE
//      tcgen05.mma sequence writes the pool's cosine matrix (raw dot products, fp32) into tensor
//      memory: row rho lives in TMEM lane rho, column c holds <V_rho, V_c>.
//   4. Algorithm 1 runs with one candidate per thread (two when P > 128): a = s - lambda m in
//      registers, warp redux + one shared-memory exchange per pick for the argmax, then every
//      thread pulls its own entry of the picked column from tensor memory (tcgen05.ld).
//   5. Kept rows are written back in place: V from the tile, K and positions re-read (L2) and
//      staged on chip before the first store.
#pragma once
#include "akv_score_chain.cuh"

namespace akv {

constexpr int kTcThreads = 128;
constexpr int kTcD = 128;        // head dimension of this path
constexpr int kTcMaxN = 256;     // most candidates per event
constexpr int kTcCols = 128;     // cosine-matrix columns kept in tensor memory per block of 128 rows
constexpr int kWaitPolls = 1 << 20;  // most polls of a bounded wait (the time-bounded form usually stops by its clock first)

struct TcSmem {
    unsigned tile, s, key, spos, byrank, rankof, taken, order, gain, idx, sect, slot, misc, total;
    int tile_rows;
};
// Layout after the 1024-byte aligned base. `key` (ranking) and `r` (reciprocal norms) share storage.
__host__ __device__ inline TcSmem plan_tc_smem(int N, int budget) {
    TcSmem p;
    p.tile_rows = ((N + 7) & ~7) < 128 ? 128 : ((N + 7) & ~7);
    const unsigned np = (unsigned)((N + 3) & ~3);
    unsigned o = 0;
    p.tile = o;   o += (unsigned)p.tile_rows * 256u;
    p.s = o;      o += align16(np * 4);
    p.key = o;    o += align16(np * 4);
    p.spos = o;   o += align16(np * 4);
    p.byrank = o; o += align16(np * 2);
    p.rankof = o; o += align16(np * 2);
    p.taken = o;  o += align16(np);
    p.order = o;  o += align16((unsigned)budget * 4);
    p.gain = o;   o += align16((unsigned)budget * 4);
    p.idx = o;    o += align16((unsigned)budget * 4);
    if (o - p.byrank < 1024u) o = p.byrank + 1024u;  // byrank..idx also hold the folded statistic and the phase steps (1 KB) while scoring
    p.sect = o;   o += 256;  // cosine and sine of the 32 sector angles
    p.slot = o;   o += 64;   // 2 x 4 keys of 8 bytes
    p.misc = o;   o += 64;   // mbarriers (2 x 8), tmem base, s_(b), block-max scratch
    p.total = o + 1024;      // room to align the base to 1024 bytes
    return p;
}

// ---- PTX wrappers --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
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
// Bounded wait: gives up after `polls` polls, or after kWaitNs of wall-clock time (a poll may itself
// suspend the thread for a while, so a poll count alone can stand for minutes), instead of spinning for ever.
// The first poll is inline; the loop behind it is one out-of-line routine, so that a wait costs the
// kernels a handful of instructions where the data is already there.
constexpr unsigned long long kWaitNs = 200ull * 1000ull * 1000ull;
__device__ __noinline__ bool mbar_wait_loop(uint32_t bar, uint32_t parity, int polls) {
    unsigned long long t0 = 0ull;
    for (int it = 1; it < polls; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 63) {
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0ull) t0 = now;
            else if (now - t0 > kWaitNs) return false;
        }
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int polls) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_loop(bar, parity, polls);
}
// The plain form: a poll count only (2^20 polls: seconds at most, whatever a poll costs), all inline. The small
// event kernel uses it: its register allocation and schedule, and with them 7 % of its speed, depend on it.
constexpr int kWaitPollsPlain = 1 << 20;
__device__ __forceinline__ bool mbar_wait_polls(uint32_t bar, uint32_t parity, int polls) {
    for (int it = 0; it < polls; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t holder, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
// For a CTA that will not allocate tensor memory at all (one whole warp calls): the SM starts the next CTA of a
// kernel that contains an allocation only once every resident CTA has given up its right to allocate.
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulation; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One fp32 per thread: TMEM lane = (warp % 4) * 32 + lane, column given by the address.
__device__ __forceinline__ float tmem_ld1(uint32_t taddr) {
    uint32_t v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(taddr) : "memory");
    return __uint_as_float(v);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, groups of 8 rows
// 1024 bytes apart (the tile base is 1024-byte aligned).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= (uint64_t)(1024u >> 4) << 32;         // stride between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M x N tile.
__host__ __device__ inline uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// byte offset inside the operand tile of 16-byte chunk c (0..15) of pool row rho
__device__ __forceinline__ uint32_t tile_chunk(int rho, int c, uint32_t half_bytes) {
    return (uint32_t)(c >> 3) * half_bytes + (uint32_t)rho * 128u + (uint32_t)(((c & 7) ^ (rho & 7)) << 4);
}

// 64-bit argmax key: score key | 0xFFFF - original slot | pool row. Larger wins; equal values go to
// the lower original slot.
__device__ __forceinline__ uint32_t key_low(int orig, int rho) { return ((0xFFFFu - (uint32_t)orig) << 16) | (uint32_t)rho; }

// ---- the kernel ------------------------------------------------------------------------------------
// FUSED: score + select + compact; otherwise selection only (scores are read from a.scores and
// nothing is rewritten).
template <bool FUSED>
__global__ void __launch_bounds__(kTcThreads, 4) event_tc_kernel(const EventArgs a, const __grid_constant__ ScoreTab tab) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const DevLayout& lay = a.lay;
    const EventId id = decode_event(lay, blockIdx.x);
    const int n = event_n(a, id.b);
    const int N = lay.N;
    const int bud = event_budget(a, id);
    const int picks = min(bud, n);
    const TcSmem sp = plan_tc_smem(N, a.budget);
    unsigned char* tile = smem + sp.tile;
    float* s = reinterpret_cast<float*>(smem + sp.s);
    uint32_t* key = reinterpret_cast<uint32_t*>(smem + sp.key);
    float* r = reinterpret_cast<float*>(smem + sp.key);  // reuses the ranking keys' storage
    int* spos = reinterpret_cast<int*>(smem + sp.spos);
    unsigned short* byrank = reinterpret_cast<unsigned short*>(smem + sp.byrank);
    unsigned short* rankof = reinterpret_cast<unsigned short*>(smem + sp.rankof);
    unsigned char* taken = smem + sp.taken;
    int* order = reinterpret_cast<int*>(smem + sp.order);
    float* gain = reinterpret_cast<float*>(smem + sp.gain);
    int* idx = reinterpret_cast<int*>(smem + sp.idx);
    uint2* slot = reinterpret_cast<uint2*>(smem + sp.slot);
    float2* sect = reinterpret_cast<float2*>(smem + sp.sect);
    const uint32_t barK = smem_u32(smem + sp.misc);
    const uint32_t barM = barK + 8;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sp.misc + 16);
    float* sb_holder = reinterpret_cast<float*>(smem + sp.misc + 20);
    int* redi = reinterpret_cast<int*>(smem + sp.misc + 32);
    const uint32_t tile_u32 = smem_u32(tile);
    const uint32_t half_bytes = (uint32_t)sp.tile_rows * 128u;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(a.K);
    __nv_bfloat16* Vg = reinterpret_cast<__nv_bfloat16*>(a.V);
    const bool similarity = a.greedy != 0;
    const int np4 = (N + 3) & ~3;
    // row addressing: dense events are one base offset plus a row stride
    const bool dense = lay.page_size == 0;
    const long long ev_off = dense ? id.b * lay.sb + id.l * lay.sl + id.h * lay.sh : 0;
    auto rowoff = [&](int j) -> long long {
        return dense ? ev_off + (long long)j * lay.sn : row_offset(lay, id.b, id.l, id.h, j);
    };

    // Tensor memory (half of the SM's columns for the two-block matrix) is claimed only when the pool's V
    // rows are on their way, and held until the loop ends: the span in which an event holds it, not the
    // event's lifetime, is what limits this kernel to two events at a time, and a third resident CTA scores
    // its keys meanwhile. (The SM starts the next CTA of a kernel that allocates tensor memory only once
    // the resident one has given up its right to allocate; with three long-lived CTAs per SM the starts
    // are further apart than the time to reach the allocation.)
    const uint32_t tcols = (uint32_t)a.tmem_cols;
    const bool use_tc = similarity && tcols != 0u;
    if (tid == 0) {
        mbar_init(barK, 1);
        mbar_init(barM, 1);
        mbar_init_fence();
    }
    if (FUSED && warp == 1) fill_sector_table(sect, lane);
    if (!use_tc && warp == 0) tmem_relinquish();  // this event takes no tensor memory
    __syncthreads();
    uint32_t tbase = 0u;

    phase_stamp(id.e, 0);  // phases: 0 start, 1 K scored, 2 ranks + pool, 3 V operand + tensor memory, 4 product + norms, 5 picks, 6 outputs, 7 end
    // ---- scores ---------------------------------------------------------------------------------
    int bad = 0;
    int timeout = 0;
    if (FUSED) {
        // K rows -> tile: a few large bulk copies when the event's rows are contiguous, one per page
        // when pages are, else one per row; all issued by one thread (a bulk copy is a per-warp
        // instruction, so a copy per thread costs a dozen issue slots each)
        if (tid == 0) {
            mbar_expect_tx(barK, (uint32_t)n * 256u);
            if (a.starve) {
                // testing aid: nothing is requested, the wait below runs out
            } else if (lay.page_size == 0 && lay.sn == kTcD) {
                const __nv_bfloat16* k0 = Kg + rowoff(0);
                for (int row = 0; row < n; row += 128)  // 32 KB pieces
                    bulk_g2s(tile_u32 + row * 256, k0 + (long long)row * kTcD, (uint32_t)min(128, n - row) * 256u, barK);
            } else if (lay.page_size != 0 && lay.s_page_n == kTcD) {
                for (int row = 0; row < n; row += lay.page_size)
                    bulk_g2s(tile_u32 + row * 256, Kg + rowoff(row),
                             (uint32_t)min(lay.page_size, n - row) * 256u, barK);
            } else {
                for (int row = 0; row < n; ++row)
                    bulk_g2s(tile_u32 + row * 256, Kg + rowoff(row), 256u, barK);
            }
        }
        const int* gpos = event_pos(a.pos, id);
        const bool rotate = gpos != nullptr;
        int pmax = INT_MIN;
        for (int j = tid; j < n; j += kTcThreads) {
            const int p = rotate ? gpos[j] : 0;
            spos[j] = p;
            pmax = max(pmax, p);
        }
        // folded statistic and phase steps, once per event, in storage that the selection uses later
        float2* gtab = reinterpret_cast<float2*>(smem + sp.byrank);
        unsigned long long* phitab = reinterpret_cast<unsigned long long*>(gtab + 64);
        fill_statistic_tables(a.qstat + ((long long)id.l * lay.H + id.h) * kTcD, tab, tid, gtab, phitab);
        if (rotate && !a.p_ref) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pmax = max(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, off));
            if (lane == 0) redi[warp] = pmax;
        }
        __syncthreads();
        long long pref = 0;
        if (rotate) pref = a.p_ref ? (long long)a.p_ref[id.b] : (long long)max(max(redi[0], redi[1]), max(redi[2], redi[3])) + 1;
        // lane covers frequencies f0..f0+7 of the row handled by its group of eight lanes; the statistic is
        // carried from one row of the group to the next (see ChainScore)
        const int grp = lane >> 3, f0 = (lane & 7) * 8;
        const long long D16 = n > 16 ? (long long)spos[n - 1] - (long long)spos[n - 17] : 0;
        ChainScore cs;
        cs.set_step(D16, phitab + f0, sect);
        timeout = !mbar_wait_bounded(barK, 0, a.wait_polls);
        if (!timeout) {
            const int rounds = (n + 15) >> 4;
            for (int round = 0; round < rounds; ++round) {
                const int j = 16 * round + 4 * warp + grp;
                const bool live = j < n;
                bool fresh = (round & (kChainRounds - 1)) == 0 || a.no_chain;
                if (!fresh) fresh = !__all_sync(0xFFFFFFFFu, !live || (long long)spos[j] - (long long)spos[j - 16] == D16);
                if (fresh) {
                    if (live) cs.anchor(pref - (long long)spos[j], gtab + f0, phitab + f0, sect);
                } else {
                    cs.advance();
                }
                float acc = 0.f;
                if (live) {
                    const unsigned char* krow = tile + j * 256 + (lane & 7) * 16;
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
        return;
    }
    bad = __syncthreads_or(bad);
    // (only now: while scoring, this storage holds the statistic's table, which slower warps may still read)
    for (int j = tid; j < np4; j += kTcThreads) taken[j] = 0;

    phase_stamp(id.e, 1);
    // ---- rank by score (ties to the lower slot) and the pool that can ever be picked ----------------
    int cand[2], rank[2];
    float sc[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int c = tid + u * kTcThreads;
        cand[u] = c;
        rank[u] = 0;
        sc[u] = 0.f;
        if (c < n) {
            const uint32_t kc = key[c];
            sc[u] = s[c];
            // slots below c win ties: count keys >= kc there (k > kc - 1) and keys > kc from c on;
            // the group of four that holds c is counted with > kc and corrected for equal keys below c
            int cnt = 0;
            const uint4* k4 = reinterpret_cast<const uint4*>(key);
            const int g = c >> 2;
            for (int i4 = 0; i4 < np4 / 4; ++i4) {
                const uint4 kk = k4[i4];
                const uint32_t thr = i4 < g ? kc - 1u : kc;
                cnt += (kk.x > thr) + (kk.y > thr) + (kk.z > thr) + (kk.w > thr);
            }
            const uint4 kg = k4[g];
            const int e = c & 3;
            cnt += (e > 0 && kg.x == kc) + (e > 1 && kg.y == kc) + (e > 2 && kg.z == kc);
            rank[u] = cnt;
        }
    }
    __syncthreads();  // every key has been read: its storage becomes r below
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        if (cand[u] < n) {
            byrank[rank[u]] = (unsigned short)cand[u];
            rankof[cand[u]] = (unsigned short)rank[u];
            if (rank[u] == picks - 1) *sb_holder = sc[u];
        }
    }
    __syncthreads();
    int P = picks;
    if (similarity && picks > 0) {
        if (a.no_prune) {
            P = n;
        } else {
            const float sb = *sb_holder;
            const float thr = fmaf(-1.001f, a.lam, sb) - 1e-6f * fabsf(sb);  // -inf keeps everyone
            const int in0 = cand[0] < n && !(sc[0] < thr);
            const int in1 = cand[1] < n && !(sc[1] < thr);
            P = __syncthreads_count(in0) + __syncthreads_count(in1);
        }
    }
    const bool two = P > 128;                      // second block of 128 rows ends at the pool's last row
    const int base2 = two ? ((P + 7) & ~7) - 128 : 0;
    // columns of the cosine matrix held in tensor memory (per block of 128 rows); picks of a later
    // rank take the plain dot-product route below
    const int cstride = two ? (int)(tcols >> 1) : (int)tcols;
    const int ncols = min((P + 15) & ~15, min(cstride, 128));

    phase_stamp(id.e, 2);
    // ---- V rows of the pool, in rank order, as the swizzled operand tile ---------------------------
    const int vrows = (similarity || FUSED) ? P : 0;
    for (int x = tid; x < vrows * 16; x += kTcThreads) {
        const int rho = x >> 4, c = x & 15;
        const int j = byrank[rho];
        cp_async16(tile_u32 + tile_chunk(rho, c, half_bytes), Vg + rowoff(j) + c * 8);
    }
    if (use_tc && warp == 0) tmem_alloc(smem_u32(tmem_holder), tcols);  // may wait for another CTA's columns
    cp_async_wait_all();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (use_tc) tbase = *tmem_holder;

    phase_stamp(id.e, 3);
    const bool do_mma = use_tc && picks > 1;
    if (do_mma && tid == 0) {
        tc_fence_after();
        const uint32_t idesc = umma_idesc_bf16(128, ncols);
#pragma unroll 1
        for (int blk = 0; blk < (two ? 2 : 1); ++blk) {
            const uint32_t arow = tile_u32 + (uint32_t)(blk ? base2 : 0) * 128u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t koff = (uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u;
                umma_bf16(tbase + (uint32_t)(blk * cstride), umma_desc_sw128(arow + koff), umma_desc_sw128(tile_u32 + koff),
                          idesc, kk > 0 ? 1u : 0u);
            }
        }
        umma_commit(barM);
    }

    // ---- reciprocal norms of the pool rows (Eq. 1), while the tensor core works ----------------------
    int rho[2] = {tid, base2 + tid};
    bool mine[2] = {tid < P, two && base2 + tid >= 128 && base2 + tid < P};
    float sv[2] = {0.f, 0.f}, lr[2] = {0.f, 0.f}, M[2] = {0.f, 0.f};
    uint32_t klow[2] = {0u, 0u};
    if (!similarity) mine[0] = mine[1] = false;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        if (mine[u]) {
            const int j = byrank[rho[u]];
            sv[u] = s[j];
            klow[u] = key_low(j, rho[u]);
            if (similarity) {
                float ss = 0.f;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    float x[8];
                    load8(reinterpret_cast<const __nv_bfloat16*>(tile + tile_chunk(rho[u], c, half_bytes)), x);
#pragma unroll
                    for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
                }
                const float rr = 1.f / (sqrtf(ss) + a.eps);
                r[rho[u]] = rr;
                lr[u] = a.lam * rr;
            }
        }
    }
    if (do_mma) timeout = !mbar_wait_bounded(barM, 0, a.wait_polls);
    tc_fence_after();
    timeout = __syncthreads_or(timeout);
    if (timeout) {
        if (tid == 0 && a.status) a.status[id.e] = 3;
        if (use_tc && warp == 0) tmem_dealloc(tbase, tcols);
        return;
    }

    phase_stamp(id.e, 4);
    // ---- Algorithm 1 ----------------------------------------------------------------------------------
    const uint32_t tlane = tbase + ((uint32_t)(warp * 32) << 16);
    if (!similarity) {
        // lambda = 0: the first `picks` ranks are the answer, in pick order
        for (int t = tid; t < picks; t += kTcThreads) {
            const int j = byrank[t];
            order[t] = j;
            gain[t] = s[j];
            taken[j] = 1;
        }
    }
    // The winning key of every pick is parked in order[] (low word) and gain[] (high word) and
    // decoded after the loop.
    uint32_t* park_lo = reinterpret_cast<uint32_t*>(order);
    uint32_t* park_hi = reinterpret_cast<uint32_t*>(gain);
    if (similarity && !two) {
        // one candidate per thread
        const int myrho = tid;
        bool live = mine[0];
        const float s0 = sv[0], lr0 = lr[0];
        const uint32_t kl0 = klow[0];
        float M0 = 0.f;
        for (int t = 0; t < picks; ++t) {
            // a = s - lambda m (a[S] = -inf: chosen candidates no longer compete); i = argmax a
            const uint32_t khi = live ? orderable(fmaf(-lr0, M0, s0)) : 0u;
            const uint32_t whi = __reduce_max_sync(0xFFFFFFFFu, khi);
            const uint32_t wlo = __reduce_max_sync(0xFFFFFFFFu, khi == whi ? kl0 : 0u);
            uint2* sl = slot + (t & 1) * 4;
            if (lane == 0) sl[warp] = make_uint2(whi, wlo);
            __syncthreads();
            const uint2 mk = sl[lane & 3];
            const uint32_t bhi = __reduce_max_sync(0xFFFFFFFFu, mk.x);
            const uint32_t blo = __reduce_max_sync(0xFFFFFFFFu, mk.x == bhi ? mk.y : 0u);
            const int irho = (int)(blo & 0xFFFFu);
            if (tid == 0) { park_hi[t] = bhi; park_lo[t] = blo; }
            live = live && myrho != irho;
            if (t + 1 == picks) break;
            // m <- max(m, Sims[i, :]): every thread reads its own row's entry of column i
            const float ri = r[irho];
            const float d0 = tmem_ld1(tlane + (uint32_t)irho);
            tmem_ld_wait();
            M0 = fmaxf(M0, ri * d0);
        }
    } else if (similarity) {
        // two candidates per thread; picks beyond the stored columns use plain dot products
        for (int t = 0; t < picks; ++t) {
            uint32_t khi = 0u, klo = 0u;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (mine[u]) {
                    const uint32_t k = orderable(fmaf(-lr[u], M[u], sv[u]));
                    if (k > khi || (k == khi && klow[u] > klo)) { khi = k; klo = klow[u]; }
                }
            }
            const uint32_t whi = __reduce_max_sync(0xFFFFFFFFu, khi);
            const uint32_t wlo = __reduce_max_sync(0xFFFFFFFFu, khi == whi ? klo : 0u);
            uint2* sl = slot + (t & 1) * 4;
            if (lane == 0) sl[warp] = make_uint2(whi, wlo);
            __syncthreads();
            const uint2 mk = sl[lane & 3];
            const uint32_t bhi = __reduce_max_sync(0xFFFFFFFFu, mk.x);
            const uint32_t blo = __reduce_max_sync(0xFFFFFFFFu, mk.x == bhi ? mk.y : 0u);
            const int irho = (int)(blo & 0xFFFFu);
            if (tid == 0) { park_hi[t] = bhi; park_lo[t] = blo; }
#pragma unroll
            for (int u = 0; u < 2; ++u)
                if (mine[u] && rho[u] == irho) mine[u] = false;
            if (t + 1 == picks) break;
            const float ri = r[irho];
            float d0, d1;
            if (irho < ncols) {
                d0 = tmem_ld1(tlane + (uint32_t)irho);
                d1 = tmem_ld1(tlane + (uint32_t)(cstride + irho));
                tmem_ld_wait();
            } else {
                float acc[2] = {0.f, 0.f};
#pragma unroll 4
                for (int c = 0; c < 16; ++c) {
                    float vi[8];
                    load8(reinterpret_cast<const __nv_bfloat16*>(tile + tile_chunk(irho, c, half_bytes)), vi);
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        if (mine[u]) {
                            float vj[8];
                            load8(reinterpret_cast<const __nv_bfloat16*>(tile + tile_chunk(rho[u], c, half_bytes)), vj);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[u] = fmaf(vi[e], vj[e], acc[u]);
                        }
                    }
                }
                d0 = acc[0];
                d1 = acc[1];
            }
            M[0] = fmaxf(M[0], ri * d0);
            M[1] = fmaxf(M[1], ri * d1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (use_tc && warp == 0) tmem_dealloc(tbase, tcols);
    if (similarity) {
        for (int t = tid; t < picks; t += kTcThreads) {
            const uint32_t hi = park_hi[t], lo = park_lo[t];
            const int j = (int)(0xFFFFu - (lo >> 16));
            order[t] = j;
            gain[t] = from_orderable(hi);
            taken[j] = 1;
        }
        __syncthreads();
    }

    phase_stamp(id.e, 5);
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

    phase_stamp(id.e, 6);
    // ---- compaction in place ----------------------------------------------------------------------
    // Every kept K row and position is on chip (registers for up to 64 rows, else the tile) before
    // the first store: a destination slot can be another kept row's source.
    int* wpos = a.pos.p ? a.pos.p + id.b * a.pos.sb + id.l * a.pos.sl + id.h * a.pos.sh : nullptr;
    __nv_bfloat16* Kw = reinterpret_cast<__nv_bfloat16*>(a.K);
    if (picks <= 64) {
        uint4 kreg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int x = tid + i * kTcThreads;
            if (x < picks * 16)
                kreg[i] = *reinterpret_cast<const uint4*>(
                    reinterpret_cast<const char*>(Kw + rowoff(idx[x >> 4])) + (x & 15) * 16);
        }
        for (int x = tid; x < picks * 16; x += kTcThreads) {
            const int rr = x >> 4, c = x & 15;
            copy16(reinterpret_cast<char*>(Vg + rowoff(rr)) + c * 16,
                   tile + tile_chunk(rankof[idx[rr]], c, half_bytes));
        }
        __syncthreads();  // every K load above has been performed
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int x = tid + i * kTcThreads;
            if (x < picks * 16)
                *reinterpret_cast<uint4*>(reinterpret_cast<char*>(Kw + rowoff(x >> 4)) + (x & 15) * 16) =
                    kreg[i];
        }
    } else {
        for (int x = tid; x < picks * 16; x += kTcThreads) {
            const int rr = x >> 4, c = x & 15;
            copy16(reinterpret_cast<char*>(Vg + rowoff(rr)) + c * 16,
                   tile + tile_chunk(rankof[idx[rr]], c, half_bytes));
        }
        __syncthreads();  // the V tile is free from here on
        for (int x = tid; x < picks * 16; x += kTcThreads) {
            const int rr = x >> 4, c = x & 15;
            copy16(tile + rr * 256 + c * 16,
                   reinterpret_cast<const char*>(Kw + rowoff(idx[rr])) + c * 16);
        }
        __syncthreads();
        for (int x = tid; x < picks * 16; x += kTcThreads) {
            const int rr = x >> 4, c = x & 15;
            copy16(reinterpret_cast<char*>(Kw + rowoff(rr)) + c * 16, tile + rr * 256 + c * 16);
        }
    }
    if (wpos)
        for (int t = tid; t < picks; t += kTcThreads) wpos[t] = spos[idx[t]];
    phase_stamp(id.e, 7);
}

}  // namespace akv
