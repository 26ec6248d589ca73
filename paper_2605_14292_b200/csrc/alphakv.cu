// C ABI of the alphakv library: argument validation, table set-up and kernel launches.
#include "../../include/alphakv.h"

#include <atomic>
#include <climits>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "akv_event_general.cuh"
#include "akv_event_pool.cuh"
#include "akv_event_stream.cuh"
#include "akv_gram.cuh"
#include "akv_select_pool.cuh"

using namespace akv;

struct akv_handle {
    int device;
    int smem_optin;    // largest dynamic shared memory per CTA
    int sm_count;
    void* ws;          // grow-only scratch
    size_t ws_bytes;
    // cached score tables
    ScoreTab tab;
    float tab_base;
    int tab_d, tab_W;
    char err[512];     // message of the last failed call on this handle
};

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};

static akv_status_t fail(akv_status_t s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}
#define CUDA_TRY(expr)                                                                             \
    do {                                                                                           \
        cudaError_t e_ = (expr);                                                                   \
        if (e_ != cudaSuccess) return fail(AKV_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

// Failures are formatted into a thread-local buffer (a failure can precede any handle: akv_create
// itself, a NULL handle); calls that have a handle also leave the message there.
extern "C" const char* akv_last_error(const akv_handle_t* h) { return h ? h->err : g_err; }
static akv_status_t finish(akv_handle* h, akv_status_t s) {
    if (h && s != AKV_OK) {
        strncpy(h->err, g_err, sizeof(h->err) - 1);
        h->err[sizeof(h->err) - 1] = 0;
    }
    return s;
}
extern "C" uint64_t akv_launch_count(void) { return g_launches.load(); }
extern "C" const char* akv_status_string(akv_status_t s) {
    switch (s) {
        case AKV_OK: return "ok";
        case AKV_ERR_INVALID_ARG: return "invalid argument";
        case AKV_ERR_UNSUPPORTED: return "unsupported";
        case AKV_ERR_BUDGET: return "budget out of range";
        case AKV_ERR_ALIGNMENT: return "alignment";
        case AKV_ERR_WORKSPACE: return "workspace";
        case AKV_ERR_CUDA: return "cuda error";
    }
    return "unknown";
}

extern "C" void akv_default_options(akv_options_t* o) {
    if (!o) return;
    o->lambda = 0.5f;
    o->eps = 1e-8f;
    o->rope_base = 10000.f;
    o->future_window = 1;
    o->sig_mode = AKV_SIG_PER_HEAD;
    o->flags = 0;
    o->head_budgets = nullptr;
    o->shared_gram = nullptr;
    o->gqa_group = 1;
    o->gqa_reduce = 0;
}

extern "C" akv_status_t akv_create(akv_handle_t** out, int device) {
    if (!out) return fail(AKV_ERR_INVALID_ARG, "akv_create: out is NULL");
    *out = nullptr;
    int count = 0;
    CUDA_TRY(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return fail(AKV_ERR_INVALID_ARG, "akv_create: device %d of %d", device, count);
    akv_handle* h = new akv_handle();
    memset(h, 0, sizeof(*h));
    h->device = device;
    cudaError_t e = cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) {
        delete h;
        return fail(AKV_ERR_CUDA, "akv_create: %s", cudaGetErrorString(e));
    }
    h->tab_d = -1;
    *out = h;
    return AKV_OK;
}

extern "C" akv_status_t akv_destroy(akv_handle_t* h) {
    if (!h) return AKV_OK;
    if (h->ws) {
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(h->device);
        cudaFree(h->ws);
        cudaSetDevice(prev);
    }
    delete h;
    return AKV_OK;
}

static akv_status_t workspace(akv_handle* h, size_t bytes, void** out) {
    if (bytes > h->ws_bytes) {
        if (h->ws) {
            CUDA_TRY(cudaDeviceSynchronize());  // earlier launches may still use the old buffer
            CUDA_TRY(cudaFree(h->ws));
            h->ws = nullptr;
            h->ws_bytes = 0;
        }
        size_t want = (bytes + (size_t(1) << 20) - 1) & ~((size_t(1) << 20) - 1);
        if (cudaMalloc(&h->ws, want) != cudaSuccess) {
            cudaGetLastError();
            return fail(AKV_ERR_WORKSPACE, "cannot allocate %zu bytes of scratch", want);
        }
        h->ws_bytes = want;
    }
    *out = h->ws;
    return AKV_OK;
}

// ------------------------------------------------------------------------------------------------
// validation
// ------------------------------------------------------------------------------------------------
static bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static akv_status_t check_layout(const akv_layout_t* y, DevLayout* out) {
    if (!y) return fail(AKV_ERR_INVALID_ARG, "layout is NULL");
    if (y->B < 1 || y->L < 1 || y->H < 1 || y->N < 1 || y->d < 1)
        return fail(AKV_ERR_INVALID_ARG, "layout: B, L, H, N, d must be positive (got %d %d %d %d %d)", y->B, y->L, y->H,
                    y->N, y->d);
    if (y->dtype != AKV_F32 && y->dtype != AKV_BF16) return fail(AKV_ERR_UNSUPPORTED, "layout: dtype %d", (int)y->dtype);
    if (y->d % 8 != 0 || y->d > kMaxD) return fail(AKV_ERR_UNSUPPORTED, "layout: d = %d must be a multiple of 8, <= %d", y->d, kMaxD);
    if ((long long)y->B * y->L * y->H > INT_MAX) return fail(AKV_ERR_UNSUPPORTED, "layout: too many events");
    const long long es = y->dtype == AKV_BF16 ? 2 : 4;
    DevLayout o;
    memset(&o, 0, sizeof(o));
    o.B = y->B; o.L = y->L; o.H = y->H; o.N = y->N; o.d = y->d;
    o.dtype = (int)y->dtype;
    o.sl = y->stride_l;
    if (y->page_size == 0) {
        o.sb = y->stride_b; o.sh = y->stride_h; o.sn = y->stride_n;
        if (o.sn < y->d) return fail(AKV_ERR_INVALID_ARG, "layout: stride_n %lld < d", o.sn);
        const long long st[4] = {o.sb, o.sl, o.sh, o.sn};
        for (long long s : st)
            if (s < 0 || (s * es) % 16 != 0) return fail(AKV_ERR_ALIGNMENT, "layout: stride %lld elements is not a multiple of 16 bytes", s);
    } else {
        if (!is_pow2(y->page_size)) return fail(AKV_ERR_INVALID_ARG, "layout: page_size %d is not a power of two", y->page_size);
        if (!y->block_table) return fail(AKV_ERR_INVALID_ARG, "layout: paged but block_table is NULL");
        if (y->pages_per_seq < 1 || (long long)y->pages_per_seq * y->page_size < y->N)
            return fail(AKV_ERR_INVALID_ARG, "layout: N = %d exceeds pages_per_seq * page_size", y->N);
        o.page_size = y->page_size;
        o.page_shift = 0;
        while ((1 << o.page_shift) < y->page_size) ++o.page_shift;
        o.table = y->block_table;
        o.pps = y->pages_per_seq;
        o.s_page = y->stride_page; o.s_page_h = y->stride_page_h; o.s_page_n = y->stride_page_n;
        if (o.s_page_n < y->d) return fail(AKV_ERR_INVALID_ARG, "layout: stride_page_n %lld < d", o.s_page_n);
        const long long st[4] = {o.sl, o.s_page, o.s_page_h, o.s_page_n};
        for (long long s : st)
            if (s < 0 || (s * es) % 16 != 0) return fail(AKV_ERR_ALIGNMENT, "layout: stride %lld elements is not a multiple of 16 bytes", s);
    }
    *out = o;
    return AKV_OK;
}

static akv_status_t check_options(const akv_options_t* o) {
    if (!o) return fail(AKV_ERR_INVALID_ARG, "options is NULL");
    if (!(o->lambda >= 0.f) || !std::isfinite(o->lambda)) return fail(AKV_ERR_INVALID_ARG, "lambda must be finite and >= 0");
    if (!(o->eps >= 0.f) || !std::isfinite(o->eps)) return fail(AKV_ERR_INVALID_ARG, "eps must be finite and >= 0");
    if (!(o->rope_base > 0.f) || !std::isfinite(o->rope_base)) return fail(AKV_ERR_INVALID_ARG, "rope_base must be positive");
    if (o->future_window < 1 || o->future_window > 65536) return fail(AKV_ERR_INVALID_ARG, "future_window must be in 1..65536");
    if (o->gqa_group < 0 || o->gqa_group > kMaxGroup) return fail(AKV_ERR_INVALID_ARG, "gqa_group must be in 0..%d", kMaxGroup);
    if (o->gqa_reduce != 0 && o->gqa_reduce != 1) return fail(AKV_ERR_INVALID_ARG, "gqa_reduce must be 0 (mean) or 1 (max)");
    if (o->sig_mode != AKV_SIG_PER_HEAD && o->sig_mode != AKV_SIG_FLAT && o->sig_mode != AKV_SIG_PER_LAYER)
        return fail(AKV_ERR_UNSUPPORTED, "sig_mode %d", (int)o->sig_mode);
    return AKV_OK;
}

static akv_status_t check_budget(int budget, int N) {
    if (budget < 1 || budget > N) return fail(AKV_ERR_BUDGET, "budget %d outside 1..N (N = %d)", budget, N);
    return AKV_OK;
}

static akv_status_t check_pos_written(const DevLayout& y, const int32_t* pos, int64_t sb, int64_t sl, int64_t sh) {
    if (!pos) return AKV_OK;
    if ((y.B > 1 && sb == 0) || (y.L > 1 && sl == 0) || (y.H > 1 && sh == 0))
        return fail(AKV_ERR_INVALID_ARG, "pos is rewritten per event: its (b, l, h) strides must not broadcast");
    return AKV_OK;
}

// phi[f] = frac(theta_f / 2 pi) in 0.64 fixed point; cw[f] = mean_w exp(i w theta_f)
static void build_tables(akv_handle* h, int d, float base, int W) {
    if (h->tab_d == d && h->tab_base == base && h->tab_W == W) return;
    const long double two_pi = 6.283185307179586476925286766559L;
    for (int f = 0; f < d / 2; ++f) {
        const long double theta = powl((long double)base, -2.0L * f / d);
        long double turns = theta / two_pi;
        turns -= floorl(turns);
        h->tab.phi[f] = (unsigned long long)ldexpl(turns, 64);
        double cr = 0.0, ci = 0.0;
        for (int w = 0; w < W; ++w) {
            cr += cos((double)(w * theta));
            ci += sin((double)(w * theta));
        }
        h->tab.cw[f] = make_float2((float)(cr / W), (float)(ci / W));
    }
    for (int f = d / 2; f < kMaxHalf; ++f) {
        h->tab.phi[f] = 0;
        h->tab.cw[f] = make_float2(0.f, 0.f);
    }
    h->tab_d = d; h->tab_base = base; h->tab_W = W;
}

template <typename K>
static akv_status_t set_smem(K kernel, unsigned bytes) {
    if (bytes > 48 * 1024) CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    return AKV_OK;
}

static akv_status_t launched(const char* what) {
    g_launches.fetch_add(1);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(AKV_ERR_CUDA, "%s launch: %s", what, cudaGetErrorString(e));
    return AKV_OK;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

static void fill_score_args(EventArgs& a, const akv_options_t* opt) {
    a.gqa_group = opt->gqa_group < 1 ? 1 : opt->gqa_group;
    a.gqa_max = opt->gqa_reduce == 1 && a.gqa_group > 1;
}

// ------------------------------------------------------------------------------------------------
// launch helpers
// ------------------------------------------------------------------------------------------------
// Every launch helper takes `dry`: with it set, the helper performs its checks and one-time kernel
// attribute calls and returns before launching, so that a call made of several launches can be
// refused as a whole before its first kernel is enqueued.
static akv_status_t launch_score(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry = false) {
    const int E = a.lay.B * a.lay.L * a.lay.H;
    const long long blocks = (long long)((a.lay.N + kScoreRows - 1) / kScoreRows) * E;
    if (blocks > INT_MAX) return fail(AKV_ERR_UNSUPPORTED, "alpha_score: %lld row blocks exceed the grid limit", blocks);
    if (dry) return AKV_OK;
    if (a.status) {
        fill_int_kernel<<<(E + 255) / 256, 256, 0, st>>>(a.status, E, 0);
        akv_status_t s = launched("fill");
        if (s != AKV_OK) return s;
    }
    const unsigned grid = (unsigned)blocks;
    if (a.lay.dtype == AKV_BF16) score_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(a, h->tab);
    else score_kernel<float><<<grid, kThreads, 0, st>>>(a, h->tab);
    return launched("score");
}

// General selection: pool-restricted Algorithm 1; the pool's signature rows stay in shared memory
// when they fit (tile sized to what the device allows).
template <typename T, bool FLAT>
static akv_status_t launch_select_pool(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry) {
    const int E = a.lay.B * a.lay.L * a.lay.H;
    const int row_bytes = a.lay.d * (int)sizeof(T);
    const PoolSmem fixed = plan_pool_smem(a.lay.N, a.budget, row_bytes, 0);
    if ((int)fixed.total > h->smem_optin) return fail(AKV_ERR_UNSUPPORTED, "N = %d is too large for the selection kernel", a.lay.N);
    int tile_rows = (h->smem_optin - (int)fixed.total) / row_bytes;
    if (tile_rows > a.lay.N) tile_rows = a.lay.N;
    if (!a.greedy) tile_rows = 0;
    const PoolSmem sp = plan_pool_smem(a.lay.N, a.budget, row_bytes, tile_rows);
    akv_status_t s = set_smem(select_pool_kernel<T, FLAT>, sp.total);
    if (s != AKV_OK || dry) return s;
    select_pool_kernel<T, FLAT><<<E, kThreads, sp.total, st>>>(a, tile_rows);
    return launched("select_pool");
}
template <typename T>
static akv_status_t launch_select_t(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry) {
    if (a.flat_sig) return launch_select_pool<float, true>(h, a, st, dry);
    return launch_select_pool<T, false>(h, a, st, dry);
}

// Tensor-memory path (bf16, d = 128, per-head signatures, N <= 256): one CTA of four warps per event.
static bool tc_path_ok(const EventArgs& a) {
    return a.lay.dtype == AKV_BF16 && a.lay.d == kTcD && a.lay.N <= kTcMaxN && a.flat_sig == nullptr && a.gqa_group <= 1;
}
template <bool FUSED>
static akv_status_t launch_tc(akv_handle* h, const EventArgs& a0, cudaStream_t st, bool dry = false) {
    EventArgs a = a0;
    const int E = a.lay.B * a.lay.L * a.lay.H;
    const TcSmem sp = plan_tc_smem(a.lay.N, a.budget);
    // 512 columns per SM are shared by the resident CTAs. A pool of more than 128 rows needs two
    // row blocks; with a small budget 64 columns per block hold nearly every pick.
    a.tmem_cols = !a.greedy ? 0 : (a.lay.N <= 128 || a.budget <= 64) ? 128 : 256;
    if ((int)sp.total > h->smem_optin) return fail(AKV_ERR_UNSUPPORTED, "budget %d needs too much shared memory", a.budget);
    akv_status_t s;
    if ((s = set_smem(event_tc_kernel<FUSED>, sp.total)) != AKV_OK) return s;
    CUDA_TRY(cudaFuncSetAttribute(event_tc_kernel<FUSED>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                  (int)cudaSharedmemCarveoutMaxShared));
    if (dry) return AKV_OK;
    event_tc_kernel<FUSED><<<E, kTcThreads, sp.total, st>>>(a, h->tab);
    return launched(FUSED ? "event_tc" : "select_tc");
}

// Single-warp greedy loop over a triangle of the cosine matrix in shared memory. Small size: the shapes whose
// pruned pool normally stays within 127 rows (N <= 128 or budget <= 64). Large size: budgets up to 128 with
// N <= 256, over an active set of the pool's 152 best-scored rows.
static bool tri_path_ok(const EventArgs& a) { return tc_path_ok(a) && (a.lay.N <= 128 || a.budget <= 64); }
static bool tri_big_ok(const EventArgs& a) { return tc_path_ok(a) && !tri_path_ok(a) && a.budget <= 128; }
// shared signatures with their cosine matrix at hand: the large size, which gathers its triangle from that matrix
static bool pool_shared_ok(const EventArgs& a) {
    return a.gram != nullptr && a.lay.dtype == AKV_BF16 && a.lay.d == kTcD && a.lay.N <= kTcMaxN && a.budget <= 128 && a.gqa_group <= 1;
}
template <bool FUSED, bool BIG>
static akv_status_t launch_tri(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry = false) {
    const int E = a.lay.B * a.lay.L * a.lay.H;
    const TriSmem sp = BIG ? plan_tri_smem(a.lay.N, a.budget, true) : plan_tri_smem(a.lay.N, a.budget);
    if ((int)sp.total > h->smem_optin) return fail(AKV_ERR_UNSUPPORTED, "budget %d needs too much shared memory", a.budget);
    akv_status_t s;
    if (BIG) {
        if ((s = set_smem(event_pool_kernel<FUSED, true>, sp.total)) != AKV_OK) return s;
        CUDA_TRY(cudaFuncSetAttribute(event_pool_kernel<FUSED, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
        if (dry) return AKV_OK;
        event_pool_kernel<FUSED, true><<<E, kTcThreads, sp.total, st>>>(a, h->tab);
        return launched(FUSED ? "event_pool" : "select_pool_active");
    }
    if ((s = set_smem(event_tri_kernel<FUSED>, sp.total)) != AKV_OK) return s;
    CUDA_TRY(cudaFuncSetAttribute(event_tri_kernel<FUSED>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                  (int)cudaSharedmemCarveoutMaxShared));
    if (dry) return AKV_OK;
    event_tri_kernel<FUSED><<<E, kTcThreads, sp.total, st>>>(a, h->tab);
    return launched(FUSED ? "event_tri" : "select_tri");
}

static akv_status_t launch_select(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry = false) {
    if (pool_shared_ok(a)) return launch_tri<false, true>(h, a, st, dry);
    if (tri_path_ok(a) && a.V) return launch_tri<false, false>(h, a, st, dry);
    if (tri_big_ok(a) && a.V) return launch_tri<false, true>(h, a, st, dry);
    if (tc_path_ok(a) && a.V) return launch_tc<false>(h, a, st, dry);
    return a.lay.dtype == AKV_BF16 ? launch_select_t<__nv_bfloat16>(h, a, st, dry) : launch_select_t<float>(h, a, st, dry);
}

static akv_status_t launch_compact(akv_handle* h, const CompactArgs& a0, cudaStream_t st, bool dry = false) {
    CompactArgs a = a0;
    const int E = a.lay.B * a.lay.L * a.lay.H;
    const int rowB = a.lay.d * (a.lay.dtype == AKV_BF16 ? 2 : 4);
    int rows = (64 * 1024) / (2 * rowB + 8);
    if (rows > a.budget) rows = a.budget;
    if (rows < 1) rows = 1;
    a.chunk_rows = rows;
    const unsigned bytes = (unsigned)rows * (2 * rowB + 8);
    if (a.lay.dtype == AKV_BF16) {
        akv_status_t s = set_smem(compact_kernel<__nv_bfloat16>, bytes);
        if (s != AKV_OK || dry) return s;
        compact_kernel<__nv_bfloat16><<<E, kThreads, bytes, st>>>(a);
    } else {
        akv_status_t s = set_smem(compact_kernel<float>, bytes);
        if (s != AKV_OK || dry) return s;
        compact_kernel<float><<<E, kThreads, bytes, st>>>(a);
    }
    (void)h;
    return launched("compact");
}

// ------------------------------------------------------------------------------------------------
// entry points
// ------------------------------------------------------------------------------------------------
static akv_status_t alpha_score_impl(akv_handle_t* h, const akv_layout_t* lay, const void* K, const int32_t* pos,
                                    int64_t psb, int64_t psl, int64_t psh, const int32_t* n_cand, const float* qstat,
                                    const int32_t* p_ref, const akv_options_t* opt, float* scores, int32_t* status,
                                    void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_score: handle is NULL");
    EventArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if (!K || !qstat || !scores) return fail(AKV_ERR_INVALID_ARG, "alpha_score: K, qstat and scores must not be NULL");
    if (!aligned16(K)) return fail(AKV_ERR_ALIGNMENT, "alpha_score: K is not 16-byte aligned");
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    build_tables(h, lay->d, opt->rope_base, opt->future_window);
    a.K = const_cast<void*>(K);
    a.pos = PosDesc{const_cast<int*>(pos), psb, psl, psh};
    a.n_cand = n_cand; a.qstat = qstat; a.p_ref = p_ref;
    a.scores = scores; a.status = status;
    fill_score_args(a, opt);
    return launch_score(h, a, (cudaStream_t)stream);
}

static akv_status_t fill_select_args(EventArgs& a, const akv_options_t* opt, const void* V, const float* flat_sig) {
    a.lam = opt->lambda;
    a.eps = opt->eps;
    a.greedy = (opt->lambda > 0.f || (opt->flags & AKV_FLAG_FORCE_GREEDY)) ? 1 : 0;
    a.no_prune = (opt->flags & AKV_FLAG_NO_PRUNE) ? 1 : 0;
    a.starve = (opt->flags & AKV_FLAG_TEST_STARVE_WAIT) ? 1 : 0;
    a.no_chain = (opt->flags & AKV_FLAG_NO_CHAIN) ? 1 : 0;
    a.wait_polls = a.starve ? 64 : kWaitPolls;
    a.head_budgets = opt->head_budgets;
    if (opt->sig_mode != AKV_SIG_PER_HEAD) {
        if (!flat_sig) return fail(AKV_ERR_INVALID_ARG, "shared signature modes need flat_sig");
        if (!aligned16(flat_sig)) return fail(AKV_ERR_ALIGNMENT, "flat_sig is not 16-byte aligned");
        a.flat_sig = flat_sig;
        const long long nd = (long long)a.lay.N * a.lay.d;
        a.sig_sb = opt->sig_mode == AKV_SIG_PER_LAYER ? nd * a.lay.L : nd;
        a.sig_sl = opt->sig_mode == AKV_SIG_PER_LAYER ? nd : 0;
        if (opt->shared_gram) {
            if (!aligned16(opt->shared_gram)) return fail(AKV_ERR_ALIGNMENT, "shared_gram is not 16-byte aligned");
            const long long nn = (long long)a.lay.N * a.lay.N;
            a.gram = opt->shared_gram;
            a.gram_sb = opt->sig_mode == AKV_SIG_PER_LAYER ? nn * a.lay.L : nn;
            a.gram_sl = opt->sig_mode == AKV_SIG_PER_LAYER ? nn : 0;
        }
    } else {
        if (flat_sig || opt->shared_gram) return fail(AKV_ERR_INVALID_ARG, "flat_sig / shared_gram given but sig_mode is per-head");
        if (a.greedy && !V) return fail(AKV_ERR_INVALID_ARG, "V must not be NULL in per-head signature mode");
    }
    return AKV_OK;
}

static akv_status_t alpha_select_impl(akv_handle_t* h, const akv_layout_t* lay, const float* scores, const void* V,
                                     const float* flat_sig, const int32_t* n_cand, int32_t budget,
                                     const akv_options_t* opt, int32_t* idx_sorted, int32_t* pick_order,
                                     float* pick_gain, int32_t* n_kept, int32_t* status, void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_select: handle is NULL");
    EventArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if ((s = check_budget(budget, lay->N)) != AKV_OK) return s;
    if (!scores || !idx_sorted) return fail(AKV_ERR_INVALID_ARG, "alpha_select: scores and idx_sorted must not be NULL");
    if (V && !aligned16(V)) return fail(AKV_ERR_ALIGNMENT, "alpha_select: V is not 16-byte aligned");
    if ((s = fill_select_args(a, opt, V, flat_sig)) != AKV_OK) return s;
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    a.V = const_cast<void*>(V);
    a.n_cand = n_cand;
    a.budget = budget;
    a.scores = const_cast<float*>(scores);
    a.idx_sorted = idx_sorted; a.pick_order = pick_order; a.pick_gain = pick_gain;
    a.n_kept = n_kept; a.status = status;
    return launch_select(h, a, (cudaStream_t)stream);
}

static akv_status_t alpha_signature_flat_impl(akv_handle_t* h, const akv_layout_t* lay, const void* V,
                                             const int32_t* n_cand, const akv_options_t* opt, float* flat_sig,
                                             void* stream, int per_layer) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_signature: handle is NULL");
    DevLayout y;
    akv_status_t s = check_layout(lay, &y);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if (!V || !flat_sig) return fail(AKV_ERR_INVALID_ARG, "alpha_signature_flat: V and flat_sig must not be NULL");
    if (!aligned16(V) || !aligned16(flat_sig)) return fail(AKV_ERR_ALIGNMENT, "alpha_signature_flat: pointers must be 16-byte aligned");
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    const int G = pow2_ceil(y.d >> 3) > 32 ? 32 : pow2_ceil(y.d >> 3);
    const int rpw = 32 / G;                                              // slots per CTA
    const long long blocks = (long long)y.B * (per_layer ? y.L : 1) * ((y.N + rpw - 1) / rpw);
    if (blocks > INT_MAX) return fail(AKV_ERR_UNSUPPORTED, "alpha_signature: %lld blocks exceed the grid limit", blocks);
    const unsigned grid = (unsigned)blocks;
    cudaStream_t st = (cudaStream_t)stream;
    if (y.dtype == AKV_BF16) flat_signature_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(y, V, n_cand, opt->eps, flat_sig, per_layer);
    else flat_signature_kernel<float><<<grid, kThreads, 0, st>>>(y, V, n_cand, opt->eps, flat_sig, per_layer);
    return launched(per_layer ? "layer_signature" : "flat_signature");
}

static akv_status_t kv_compact_impl(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                   int64_t psb, int64_t psl, int64_t psh, const int32_t* idx_sorted, int32_t budget,
                                   void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "kv_compact: handle is NULL");
    CompactArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_budget(budget, lay->N)) != AKV_OK) return s;
    if (!idx_sorted) return fail(AKV_ERR_INVALID_ARG, "kv_compact: idx_sorted is NULL");
    if ((K && !aligned16(K)) || (V && !aligned16(V))) return fail(AKV_ERR_ALIGNMENT, "kv_compact: K/V must be 16-byte aligned");
    if ((s = check_pos_written(a.lay, pos, psb, psl, psh)) != AKV_OK) return s;
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    a.K = K; a.V = V;
    a.pos = PosDesc{pos, psb, psl, psh};
    a.idx_sorted = idx_sorted;
    a.budget = budget;
    return launch_compact(h, a, (cudaStream_t)stream);
}

// Which kernels the fused call runs for a shape: the two tensor-memory kernels (bf16, d = 128, N <= 256,
// per-head signatures), the resident kernel when an event's K and V tiles fit in shared memory, else
// three launches with the scores in global memory.
enum EventRoute { ROUTE_TRI, ROUTE_TRI_BIG, ROUTE_TC, ROUTE_STREAM, ROUTE_RESIDENT, ROUTE_THREE };
// shared memory the streaming kernel may plan with: what the device allows minus its static arrays
static int stream_smem_limit(int smem_optin) { return smem_optin - 1024; }
static bool stream_path_ok(const EventArgs& a, int smem_optin) {
    if (!(a.lay.dtype == AKV_BF16 && a.lay.d == kTcD && a.lay.N > kTcMaxN && a.lay.N <= 65535 && a.flat_sig == nullptr && a.gqa_group <= 1)) return false;
    const StSmem sp = plan_st_smem(a.lay.N, a.budget, stream_smem_limit(smem_optin));
    return sp.cap_rows > 0 && (int)sp.total <= stream_smem_limit(smem_optin);
}
static EventRoute event_route(const EventArgs& a, int smem_optin) {
    if (pool_shared_ok(a)) return ROUTE_TRI_BIG;
    if (tri_path_ok(a)) return ROUTE_TRI;
    if (tri_big_ok(a)) return ROUTE_TRI_BIG;
    if (tc_path_ok(a)) return ROUTE_TC;
    if (stream_path_ok(a, smem_optin)) return ROUTE_STREAM;
    const int es = a.lay.dtype == AKV_BF16 ? 2 : 4;
    const SmemPlan res = plan_smem(a.lay.N, a.lay.d, es, a.budget, true, true);
    return (int)res.total <= smem_optin ? ROUTE_RESIDENT : ROUTE_THREE;
}

extern "C" akv_status_t akv_workspace_bytes(const akv_layout_t* lay, int32_t budget, const akv_options_t* opt, size_t* bytes) {
    if (!bytes) return fail(AKV_ERR_INVALID_ARG, "akv_workspace_bytes: bytes is NULL");
    *bytes = 0;
    EventArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if ((s = check_budget(budget, lay->N)) != AKV_OK) return s;
    a.budget = budget;
    a.greedy = (opt->lambda > 0.f || (opt->flags & AKV_FLAG_FORCE_GREEDY)) ? 1 : 0;
    // only whether shared signatures are in use matters for the route, not where they live
    a.flat_sig = opt->sig_mode != AKV_SIG_PER_HEAD ? reinterpret_cast<const float*>(bytes) : nullptr;
    a.gram = opt->sig_mode != AKV_SIG_PER_HEAD ? opt->shared_gram : nullptr;
    fill_score_args(a, opt);
    int dev = 0, smem_optin = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (event_route(a, smem_optin) == ROUTE_THREE)
        *bytes = (size_t)lay->B * lay->L * lay->H * lay->N * sizeof(float);
    return AKV_OK;
}

// score -> select -> compact on one stream, the scores passing through a.scores. With `dry` set only
// the checks of the three launches run (see launch_score).
static akv_status_t three_launches(akv_handle* h, const EventArgs& a, cudaStream_t st, bool dry) {
    akv_status_t s;
    EventArgs sa = a;
    sa.status = nullptr;  // the selection kernel writes the final status word
    if ((s = launch_score(h, sa, st, dry)) != AKV_OK) return s;
    if ((s = launch_select(h, a, st, dry)) != AKV_OK) return s;
    CompactArgs c;
    memset(&c, 0, sizeof(c));
    c.lay = a.lay; c.K = a.K; c.V = a.V; c.pos = a.pos; c.idx_sorted = a.idx_sorted; c.budget = a.budget;
    return launch_compact(h, c, st, dry);
}

static akv_status_t alpha_compress_event_impl(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                             int64_t psb, int64_t psl, int64_t psh, const int32_t* n_cand,
                                             const float* qstat, const int32_t* p_ref, const float* flat_sig,
                                             int32_t budget, const akv_options_t* opt, int32_t* idx_sorted,
                                             int32_t* pick_order, float* pick_gain, float* scores, int32_t* n_kept,
                                             int32_t* status, void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_compress_event: handle is NULL");
    EventArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if ((s = check_budget(budget, lay->N)) != AKV_OK) return s;
    if (!K || !V || !qstat || !idx_sorted)
        return fail(AKV_ERR_INVALID_ARG, "alpha_compress_event: K, V, qstat and idx_sorted must not be NULL");
    if (!aligned16(K) || !aligned16(V)) return fail(AKV_ERR_ALIGNMENT, "alpha_compress_event: K/V must be 16-byte aligned");
    if ((s = check_pos_written(a.lay, pos, psb, psl, psh)) != AKV_OK) return s;
    if ((s = fill_select_args(a, opt, V, flat_sig)) != AKV_OK) return s;
    fill_score_args(a, opt);
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    build_tables(h, lay->d, opt->rope_base, opt->future_window);
    cudaStream_t st = (cudaStream_t)stream;
    a.K = K; a.V = V;
    a.pos = PosDesc{pos, psb, psl, psh};
    a.n_cand = n_cand; a.qstat = qstat; a.p_ref = p_ref;
    a.budget = budget;
    a.idx_sorted = idx_sorted; a.pick_order = pick_order; a.pick_gain = pick_gain;
    a.scores = scores; a.n_kept = n_kept; a.status = status;

    const EventRoute route = event_route(a, h->smem_optin);
    if (route == ROUTE_TRI) return launch_tri<true, false>(h, a, st);
    if (route == ROUTE_TRI_BIG) return launch_tri<true, true>(h, a, st);
    if (route == ROUTE_TC) return launch_tc<true>(h, a, st);
    if (route == ROUTE_STREAM) {
        const int limit = stream_smem_limit(h->smem_optin);
        const StSmem sp = plan_st_smem(a.lay.N, a.budget, limit);
        if ((s = set_smem(event_stream_kernel, sp.total)) != AKV_OK) return s;
        event_stream_kernel<<<a.lay.B * a.lay.L * a.lay.H, kStThreads, sp.total, st>>>(a, h->tab, limit);
        return launched("event_stream");
    }
    if (route == ROUTE_RESIDENT) {
        const int es = lay->dtype == AKV_BF16 ? 2 : 4;
        const SmemPlan res = plan_smem(lay->N, lay->d, es, budget, true, true);
        const int E = a.lay.B * a.lay.L * a.lay.H;
        // beside the tiles: the pool's list and norms and as much of a cosine triangle as the SM's shared memory
        // leaves room for (at most the whole event's)
        const long long whole = (long long)align16((unsigned)lay->N * 2u) + align16((unsigned)lay->N * 4u) +
                                (long long)lay->N * (lay->N + 1) / 2 * 4;
        const long long room = (long long)h->smem_optin - (long long)res.total;
        const int extra = (int)((room < whole ? room : whole) & ~15ll);
        const unsigned total = res.total + (unsigned)(extra > 0 ? extra : 0);
        if (lay->dtype == AKV_BF16) {
            if ((s = set_smem(event_resident_kernel<__nv_bfloat16>, total)) != AKV_OK) return s;
            event_resident_kernel<__nv_bfloat16><<<E, kThreads, total, st>>>(a, h->tab, extra > 0 ? extra : 0);
        } else {
            if ((s = set_smem(event_resident_kernel<float>, total)) != AKV_OK) return s;
            event_resident_kernel<float><<<E, kThreads, total, st>>>(a, h->tab, extra > 0 ? extra : 0);
        }
        return launched("event");
    }
    // The event does not fit on chip: score -> select -> compact as three launches, scores held in
    // the caller's buffer or in the handle's scratch.
    if ((s = three_launches(h, a, st, /*dry=*/true)) != AKV_OK) return s;
    if (!a.scores) {
        void* ws = nullptr;
        const size_t bytes = (size_t)a.lay.B * a.lay.L * a.lay.H * a.lay.N * sizeof(float);
        if ((s = workspace(h, bytes, &ws)) != AKV_OK) return s;
        a.scores = static_cast<float*>(ws);
    }
    return three_launches(h, a, st, false);
}

// ------------------------------------------------------------------------------------------------
// Three-launch event with the intermediate scores in library-owned static device memory.
// ------------------------------------------------------------------------------------------------
#include <mutex>

static __device__ __align__(256) float g_static_scores[AKV_STATIC_SCORES_MAX];

// In host code `g_static_scores` is only a stand-in for the symbol; the device address comes from
// the runtime, once per device, with that device current.
static akv_status_t static_scores_address(int device, float** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static float* addr[kMaxDevices] = {};
    if (device < 0 || device >= kMaxDevices) return fail(AKV_ERR_UNSUPPORTED, "device %d: at most %d devices", device, kMaxDevices);
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[device]) {
        void* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scores));
        addr[device] = static_cast<float*>(p);
    }
    *out = addr[device];
    return AKV_OK;
}

static akv_status_t alpha_compress_event_static_impl(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V,
                                                    int32_t* pos, int64_t psb, int64_t psl, int64_t psh,
                                                    const int32_t* n_cand, const float* qstat, const int32_t* p_ref,
                                                    const float* flat_sig, int32_t budget, const akv_options_t* opt,
                                                    int32_t* idx_sorted, int32_t* pick_order, float* pick_gain,
                                                    int32_t* n_kept, int32_t* status, void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_compress_event_static: handle is NULL");
    EventArgs a;
    memset(&a, 0, sizeof(a));
    akv_status_t s = check_layout(lay, &a.lay);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if ((s = check_budget(budget, lay->N)) != AKV_OK) return s;
    if (!K || !V || !qstat || !idx_sorted)
        return fail(AKV_ERR_INVALID_ARG, "alpha_compress_event_static: K, V, qstat and idx_sorted must not be NULL");
    if (!aligned16(K) || !aligned16(V)) return fail(AKV_ERR_ALIGNMENT, "alpha_compress_event_static: K/V must be 16-byte aligned");
    const unsigned long long need = (unsigned long long)lay->B * lay->L * lay->H * lay->N;
    if (need > AKV_STATIC_SCORES_MAX)
        return fail(AKV_ERR_WORKSPACE, "alpha_compress_event_static: B*L*H*N = %llu scores exceed the static scratch of %llu",
                    need, (unsigned long long)AKV_STATIC_SCORES_MAX);
    if ((s = check_pos_written(a.lay, pos, psb, psl, psh)) != AKV_OK) return s;
    if ((s = fill_select_args(a, opt, V, flat_sig)) != AKV_OK) return s;
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    fill_score_args(a, opt);
    float* scratch = nullptr;
    if ((s = static_scores_address(h->device, &scratch)) != AKV_OK) return s;
    build_tables(h, lay->d, opt->rope_base, opt->future_window);
    cudaStream_t st = (cudaStream_t)stream;
    a.K = K; a.V = V;
    a.pos = PosDesc{pos, psb, psl, psh};
    a.n_cand = n_cand; a.qstat = qstat; a.p_ref = p_ref;
    a.budget = budget;
    a.idx_sorted = idx_sorted; a.pick_order = pick_order; a.pick_gain = pick_gain;
    a.scores = scratch; a.n_kept = n_kept; a.status = status;
    // Every score the selection reads (slots below n_cand) is written by the scoring launch of this
    // same call, so nothing left in the array by an earlier call needs clearing.
    if ((s = three_launches(h, a, st, /*dry=*/true)) != AKV_OK) return s;
    return three_launches(h, a, st, false);
}


static akv_status_t alpha_gram_shared_impl(akv_handle_t* h, const akv_layout_t* lay, const float* sig, const int32_t* n_cand,
                                           const akv_options_t* opt, float* gram, int32_t* status, void* stream) {
    if (!h) return fail(AKV_ERR_INVALID_ARG, "alpha_gram_shared: handle is NULL");
    DevLayout y;
    akv_status_t s = check_layout(lay, &y);
    if (s != AKV_OK) return s;
    if ((s = check_options(opt)) != AKV_OK) return s;
    if (opt->sig_mode == AKV_SIG_PER_HEAD) return fail(AKV_ERR_INVALID_ARG, "alpha_gram_shared: sig_mode must be FLAT or PER_LAYER");
    if (y.d != kTcD) return fail(AKV_ERR_UNSUPPORTED, "alpha_gram_shared: d = %d (only 128 is built)", y.d);
    if (!sig || !gram) return fail(AKV_ERR_INVALID_ARG, "alpha_gram_shared: sig and gram must not be NULL");
    if (!aligned16(sig) || !aligned16(gram)) return fail(AKV_ERR_ALIGNMENT, "alpha_gram_shared: pointers must be 16-byte aligned");
    DeviceGuard guard(h->device);
    if (!guard.ok) return fail(AKV_ERR_CUDA, "cannot select device %d", h->device);
    const int seq_div = opt->sig_mode == AKV_SIG_PER_LAYER ? y.L : 1;
    const long long groups = (long long)y.B * seq_div;
    const int tiles = (y.N + 127) / 128;
    const long long blocks = groups * tiles * tiles;
    if (blocks > INT_MAX) return fail(AKV_ERR_UNSUPPORTED, "alpha_gram_shared: %lld tiles exceed the grid limit", blocks);
    if ((s = set_smem(gram_shared_kernel, kGramSmem)) != AKV_OK) return s;
    gram_shared_kernel<<<(unsigned)blocks, kGramThreads, kGramSmem, (cudaStream_t)stream>>>(sig, n_cand, seq_div, y.N, gram, status);
    return launched("gram_shared");
}

// ------------------------------------------------------------------------------------------------
// C entry points: each forwards to its implementation above and leaves a failure's message in the handle.
// ------------------------------------------------------------------------------------------------
extern "C" akv_status_t alpha_score(akv_handle_t* h, const akv_layout_t* lay, const void* K, const int32_t* pos,
                                    int64_t psb, int64_t psl, int64_t psh, const int32_t* n_cand, const float* qstat,
                                    const int32_t* p_ref, const akv_options_t* opt, float* scores, int32_t* status,
                                    void* stream) {
    return finish(h, alpha_score_impl(h, lay, K, pos, psb, psl, psh, n_cand, qstat, p_ref, opt, scores, status, stream));
}
extern "C" akv_status_t alpha_select(akv_handle_t* h, const akv_layout_t* lay, const float* scores, const void* V,
                                     const float* flat_sig, const int32_t* n_cand, int32_t budget,
                                     const akv_options_t* opt, int32_t* idx_sorted, int32_t* pick_order,
                                     float* pick_gain, int32_t* n_kept, int32_t* status, void* stream) {
    return finish(h, alpha_select_impl(h, lay, scores, V, flat_sig, n_cand, budget, opt, idx_sorted, pick_order, pick_gain,
                                       n_kept, status, stream));
}
extern "C" akv_status_t alpha_signature_flat(akv_handle_t* h, const akv_layout_t* lay, const void* V,
                                             const int32_t* n_cand, const akv_options_t* opt, float* flat_sig,
                                             void* stream) {
    return finish(h, alpha_signature_flat_impl(h, lay, V, n_cand, opt, flat_sig, stream, 0));
}
extern "C" akv_status_t alpha_signature_layer(akv_handle_t* h, const akv_layout_t* lay, const void* V,
                                              const int32_t* n_cand, const akv_options_t* opt, float* layer_sig,
                                              void* stream) {
    return finish(h, alpha_signature_flat_impl(h, lay, V, n_cand, opt, layer_sig, stream, 1));
}
extern "C" akv_status_t alpha_gram_shared(akv_handle_t* h, const akv_layout_t* lay, const float* sig, const int32_t* n_cand,
                                          const akv_options_t* opt, float* gram, int32_t* status, void* stream) {
    return finish(h, alpha_gram_shared_impl(h, lay, sig, n_cand, opt, gram, status, stream));
}
extern "C" akv_status_t kv_compact(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                   int64_t psb, int64_t psl, int64_t psh, const int32_t* idx_sorted, int32_t budget,
                                   void* stream) {
    return finish(h, kv_compact_impl(h, lay, K, V, pos, psb, psl, psh, idx_sorted, budget, stream));
}
extern "C" akv_status_t alpha_compress_event(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                             int64_t psb, int64_t psl, int64_t psh, const int32_t* n_cand,
                                             const float* qstat, const int32_t* p_ref, const float* flat_sig,
                                             int32_t budget, const akv_options_t* opt, int32_t* idx_sorted,
                                             int32_t* pick_order, float* pick_gain, float* scores, int32_t* n_kept,
                                             int32_t* status, void* stream) {
    return finish(h, alpha_compress_event_impl(h, lay, K, V, pos, psb, psl, psh, n_cand, qstat, p_ref, flat_sig, budget, opt,
                                               idx_sorted, pick_order, pick_gain, scores, n_kept, status, stream));
}
extern "C" akv_status_t alpha_compress_event_static(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V,
                                                    int32_t* pos, int64_t psb, int64_t psl, int64_t psh,
                                                    const int32_t* n_cand, const float* qstat, const int32_t* p_ref,
                                                    const float* flat_sig, int32_t budget, const akv_options_t* opt,
                                                    int32_t* idx_sorted, int32_t* pick_order, float* pick_gain,
                                                    int32_t* n_kept, int32_t* status, void* stream) {
    return finish(h, alpha_compress_event_static_impl(h, lay, K, V, pos, psb, psl, psh, n_cand, qstat, p_ref, flat_sig, budget,
                                                      opt, idx_sorted, pick_order, pick_gain, n_kept, status, stream));
}

#ifdef AKV_PHASE_CLOCKS
// Profiling builds only: registers a device buffer of kPhaseSlots int64 per event for the kernels' phase
// stamps (NULL switches them off again).
extern "C" int akv_debug_phase_buffer(long long* device_buffer) {
    return (int)cudaMemcpyToSymbol(akv::g_phase_buf, &device_buffer, sizeof(device_buffer));
}
extern "C" int akv_debug_phase_slots(void) { return akv::kPhaseSlots; }
#endif
