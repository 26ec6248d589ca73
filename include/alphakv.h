/*
 * alphakv -- KV-cache compression event of the alpha retainer, CUDA (sm_100a).
 *
 * One *event* is one (sequence, layer, KV head). For every event the library
 *   1. scores each cached token (alpha_score),
 *   2. picks `budget` tokens with the greedy set-conditioned rule
 *        Delta(i | S) = s_i - lambda * max(0, max_{j in S} cos(v_i, v_j))      (Eq. 2)
 *        i_{t+1} = argmax_{i not in S_t} Delta(i | S_t),  i_1 = argmax s       (Eq. 3)
 *      which at lambda = 0 is exactly top-k (Section 4.1, Algorithm 1)         (alpha_select),
 *   3. moves the kept K/V rows to slots 0..budget-1 of the same buffer         (kv_compact),
 * or does all three in one call (alpha_compress_event).
 *
 * Conventions that hold for every entry point
 *   - Plain C linkage; no C++/torch types. Every tensor pointer is DEVICE memory
 *     owned by the caller and is not retained after the call. Scalars, the
 *     layout and the options are HOST structs read during the call.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream). The return code reports host-side validation
 *     and launch errors only; nothing is launched when it is not AKV_OK.
 *   - No exceptions, aborts or exits. akv_last_error() gives a message for the
 *     last failure.
 *   - Tensors are addressed [B, L, H, N, d]: B sequences, L layers, H KV heads,
 *     N slots per (sequence, layer, head), d head dimension (contiguous).
 *     d must be a multiple of 8 and at most 256; row starts must be 16-byte
 *     aligned (base pointers 16-byte aligned, strides multiples of 16 bytes).
 *   - Per-event status words (device, int32 [B, L, H], optional):
 *       0 ok; 1 a non-finite score was seen (such a token is never preferred);
 *       2 fewer candidates than the budget (all are kept, n_kept < budget,
 *         unused idx entries are -1); 3 an internal bounded wait gave up.
 *   - Ties in any argmax go to the lower slot index.
 */
#ifndef ALPHAKV_H
#define ALPHAKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct akv_handle akv_handle_t; /* opaque; owns only its own scratch workspace */

typedef enum {
    AKV_OK = 0,
    AKV_ERR_INVALID_ARG = 1, /* null pointer, bad shape, negative lambda, ... */
    AKV_ERR_UNSUPPORTED = 2, /* d, dtype or mode outside what is built */
    AKV_ERR_BUDGET = 3,      /* budget < 1 or budget > N */
    AKV_ERR_ALIGNMENT = 4,   /* pointer or stride breaks the 16-byte rule */
    AKV_ERR_WORKSPACE = 5,   /* scratch could not be provided */
    AKV_ERR_CUDA = 6         /* a CUDA runtime call failed (see akv_last_error) */
} akv_status_t;

typedef enum { AKV_F32 = 0, AKV_BF16 = 1 } akv_dtype_t;

/* What V-space the cosine of Eq. 2 is taken in (Section 6 names the per-head and the
 * per-layer variant of Eq. 1). PER_HEAD: the event's own V rows (the sums of Eq. 1
 * reduced to the one head). FLAT: Eq. 1 literally, one signature per (sequence, slot)
 * shared by all layers and heads, produced by alpha_signature_flat. PER_LAYER: the
 * sum of Eq. 1 taken over the KV heads of one layer only, one signature per
 * (sequence, layer, slot), produced by alpha_signature_layer. */
typedef enum { AKV_SIG_PER_HEAD = 0, AKV_SIG_FLAT = 1, AKV_SIG_PER_LAYER = 2 } akv_sig_mode_t;

/* Layout of K and of V (both use the same one). Strides are in ELEMENTS.
 * Dense (page_size == 0): row (b,l,h,n) starts at
 *     b*stride_b + l*stride_l + h*stride_h + n*stride_n.
 * Paged (page_size > 0, a power of two): slot n of sequence b lives in page
 *     p = block_table[b*pages_per_seq + n/page_size] and row (b,l,h,n) starts at
 *     l*stride_l + p*stride_page + h*stride_page_h + (n % page_size)*stride_page_n.
 *   (stride_b, stride_h, stride_n are ignored.) N must be <= pages_per_seq*page_size.
 */
typedef struct {
    int32_t B, L, H, N, d;
    akv_dtype_t dtype;
    int64_t stride_b, stride_l, stride_h, stride_n;
    int32_t page_size;
    const int32_t* block_table; /* device, int32 [B, pages_per_seq]; paged only */
    int32_t pages_per_seq;
    int64_t stride_page, stride_page_h, stride_page_n;
} akv_layout_t;

#define AKV_FLAG_FORCE_GREEDY 1u /* run the greedy loop even at lambda == 0 (testing aid) */
#define AKV_FLAG_NO_PRUNE 2u     /* never shrink the candidate pool before the loop (testing aid) */
/* Testing aid for the bounded waits of the fused on-chip kernels: no K row is requested and the
 * waits poll only a few times, so every wait runs out with nothing in flight; each event then
 * reports status 3 and K, V and pos are left as they were. */
#define AKV_FLAG_TEST_STARVE_WAIT 4u
/* Testing aid: when an event's positions are an arithmetic progression the fused on-chip kernels turn
 * the query statistic from row to row by one constant complex factor per frequency instead of taking
 * every row's sines and cosines afresh; this flag switches that off. Scores agree to rounding. */
#define AKV_FLAG_NO_CHAIN 8u

typedef struct {
    float lambda;          /* >= 0; 0 takes the top-k branch of Algorithm 1 */
    float eps;             /* epsilon of Eq. 1: v = u / (||u||_2 + eps); default 1e-8 */
    float rope_base;       /* RoPE base, default 10000 */
    int32_t future_window; /* W >= 1 future query positions averaged by the score; default 1 */
    akv_sig_mode_t sig_mode;
    uint32_t flags;
    /* Per-(layer, head) budgets (Section 2 "Budget-allocation compression", Section 6: alpha as the
     * scorer inside a per-head or per-layer budget allocator): device int32 [L, H], or NULL for the
     * same budget everywhere. Event (b, l, h) keeps min(head_budgets[l*H + h], n_cand) rows; every
     * entry must lie in 1..budget, where the call's `budget` argument is the largest of them and
     * stays the row length of idx_sorted / pick_order / pick_gain (unused entries -1 / -1 / 0). */
    const int32_t* head_budgets;
    /* Cosine matrix of the shared signatures (FLAT and PER_LAYER modes), from alpha_gram_shared: device fp32
     * [B, N, N] (FLAT) or [B, L, N, N] (PER_LAYER), or NULL. With it, every event of a sequence (of a sequence
     * and layer) reads its cosines from the one matrix, Algorithm 1's "Sims", instead of forming dot products
     * of signature rows pick by pick; bf16 caches with d = 128, N <= 256 and budget <= 128 then run as one
     * launch. Other shapes ignore it and use flat_sig. */
    const float* shared_gram;
    /* Grouped-query attention: qstat holds gqa_group statistics per KV head, [L, H * gqa_group, d] (0 and 1 both
     * mean one). The score of a key is the mean over the group's query heads of their scores (gqa_reduce = 0;
     * the same as scoring with the averaged statistic, the score being linear in it) or the largest of them
     * (gqa_reduce = 1: a key that any query head of the group wants is kept). At most 8 per group. Groups
     * larger than one run on the general kernels (the resident one or three launches). */
    int32_t gqa_group;
    int32_t gqa_reduce;
} akv_options_t;

/* Fills *opt with the defaults named above (lambda = 0.5, the value the paper settles on). */
void akv_default_options(akv_options_t* opt);

/* Creates a handle bound to CUDA device `device`. The handle keeps a grow-only
 * scratch buffer (cudaMalloc on first need, freed by akv_destroy; akv_workspace_bytes
 * tells how large a call needs it). One handle must not be used from two host threads
 * at once, and every call on one handle shares that scratch: two calls that use it and
 * whose kernels overlap on the GPU (different streams, no ordering between them) race
 * on it -- order such calls, or give each stream its own handle. */
akv_status_t akv_create(akv_handle_t** out, int device);
akv_status_t akv_destroy(akv_handle_t* h);
/* Message of the most recent failed call on handle `h` (storage inside the handle, valid
 * until the next failure or akv_destroy). With h == NULL: the most recent failure on the
 * calling thread, whichever handle it was on -- the only way to read why akv_create
 * failed or what a call given a NULL handle complained about. */
const char* akv_last_error(const akv_handle_t* h);
/* Bytes of handle scratch that alpha_compress_event needs for this layout, budget and
 * options when its `scores` argument is NULL: 0 when the event runs in one launch with
 * everything on chip, else the B*L*H*N fp32 scores that pass from the scoring launch to
 * the selection launch. The answer depends on the current device's shared-memory size.
 * Callers that cannot tolerate a cudaMalloc inside the call can pass their own `scores`
 * buffer (then no scratch is used) or use alpha_compress_event_static. */
akv_status_t akv_workspace_bytes(const akv_layout_t* lay, int32_t budget, const akv_options_t* opt, size_t* bytes);
const char* akv_status_string(akv_status_t s);
/* Number of kernels this library has launched so far in this process. */
uint64_t akv_launch_count(void);

/*
 * alpha_score -- per-token retention score s (Section 4.1 takes it from the TriAttention
 * scorer and does not print the formula; the library uses the following reading:
 * keys are stored pre-RoPE, coordinate f pairs with f + d/2,
 *   s_i = (1/sqrt d) Re sum_f c_f z(q)_f conj(z(k_i)_f) exp(i (p_ref - p_i) theta_f),
 *   theta_f = rope_base^(-2f/d), c_f = (1/W) sum_{w<W} exp(i w theta_f),
 *   z(x)_f = x_f + i x_{f+d/2},
 * the mean RoPE attention logit of the head's query statistic at positions
 * p_ref..p_ref+W-1 against key i at p_i).
 *   K       device, layout `lay`, read only.
 *   pos     device int32, slot positions; element (b,l,h,n) at
 *           b*pos_stride_b + l*pos_stride_l + h*pos_stride_h + n (a stride of 0
 *           broadcasts). NULL: keys are already rotated, s_i = q . k_i / sqrt d.
 *   n_cand  device int32 [B] valid slots per sequence, or NULL for N.
 *   qstat   device fp32 [L, H, d] query statistic per KV head; with opt->gqa_group = G > 1,
 *           [L, H * G, d]: G statistics per KV head, reduced by opt->gqa_reduce.
 *   p_ref   device int32 [B], or NULL for (largest position of the event) + 1.
 *   scores  device fp32 [B, L, H, N] out; slots >= n_cand are left untouched.
 *   status  device int32 [B, L, H] out or NULL.
 */
akv_status_t alpha_score(akv_handle_t* h, const akv_layout_t* lay, const void* K, const int32_t* pos,
                         int64_t pos_stride_b, int64_t pos_stride_l, int64_t pos_stride_h,
                         const int32_t* n_cand, const float* qstat, const int32_t* p_ref,
                         const akv_options_t* opt, float* scores, int32_t* status, void* stream);

/*
 * alpha_select -- Algorithm 1: greedy fill of the budget under Eq. 2 / Eq. 3, or
 * top-k when lambda == 0. fp32 accumulation; cos(v_i, v_j) = <V_i, V_j> r_i r_j
 * with r = 1 / (||V||_2 + eps) (Eq. 1's normalisation).
 *   scores     device fp32 [B, L, H, N] in.
 *   V          device, layout `lay`, read only (PER_HEAD mode); may be NULL in the other modes.
 *   flat_sig   device fp32 signatures: [B, N, d] in FLAT mode (from alpha_signature_flat),
 *              [B, L, N, d] in PER_LAYER mode (from alpha_signature_layer), NULL in PER_HEAD mode.
 *   Limits: the general selection kernel keeps per-candidate state in shared memory, which bounds
 *   N at about 10 000 (AKV_ERR_UNSUPPORTED beyond).
 *   budget     1 <= budget <= N (the paper's k).
 *   idx_sorted device int32 [B, L, H, budget] out: sort(S), ascending slot index.
 *   pick_order device int32 [B, L, H, budget] out or NULL: i_1, i_2, ... in pick order.
 *   pick_gain  device fp32  [B, L, H, budget] out or NULL: Delta(i_t | S_{t-1}) at each pick.
 *   n_kept     device int32 [B, L, H] out or NULL: min(budget, n_cand).
 */
akv_status_t alpha_select(akv_handle_t* h, const akv_layout_t* lay, const float* scores, const void* V,
                          const float* flat_sig, const int32_t* n_cand, int32_t budget,
                          const akv_options_t* opt, int32_t* idx_sorted, int32_t* pick_order,
                          float* pick_gain, int32_t* n_kept, int32_t* status, void* stream);

/*
 * alpha_signature_flat -- Eq. 1: u_i = (1/(L H)) sum_l sum_h V_i^(l,h), v_i = u_i / (||u_i||_2 + eps),
 * one signature per (sequence, slot); slots must mean the same token in every head.
 *   flat_sig  device fp32 [B, N, d] out (unit-normalised rows).
 */
akv_status_t alpha_signature_flat(akv_handle_t* h, const akv_layout_t* lay, const void* V,
                                  const int32_t* n_cand, const akv_options_t* opt, float* flat_sig,
                                  void* stream);

/*
 * alpha_signature_layer -- the per-layer variant of Eq. 1 that Section 6 names: the sum runs over the
 * KV heads of one layer, u_i^(l) = (1/H) sum_h V_i^(l,h), v_i^(l) = u_i^(l) / (||u_i^(l)||_2 + eps).
 *   layer_sig  device fp32 [B, L, N, d] out (unit-normalised rows); pass it as `flat_sig` with
 *              sig_mode = AKV_SIG_PER_LAYER.
 */
akv_status_t alpha_signature_layer(akv_handle_t* h, const akv_layout_t* lay, const void* V,
                                   const int32_t* n_cand, const akv_options_t* opt, float* layer_sig,
                                   void* stream);

/*
 * alpha_gram_shared -- the cosine matrix of shared signatures, formed once per sequence (FLAT) or per sequence
 * and layer (PER_LAYER): Algorithm 1's "Sims <- V V^T" for the unit rows of Eq. 1, gram[g][i][j] = <v_i, v_j>.
 * Accuracy: each fp32 signature row is split into three bf16 parts and the product runs on the tensor cores
 * with fp32 accumulation; entries are within 5e-7 of the float64 value (the fp32 signatures themselves carry
 * most of that). Needs d = 128 (AKV_ERR_UNSUPPORTED
 * otherwise).
 *   sig     device fp32 [B, N, d] (FLAT, from alpha_signature_flat) or [B, L, N, d] (PER_LAYER), per opt->sig_mode.
 *   gram    device fp32 [B, N, N] or [B, L, N, N] out; rows and columns >= n_cand are left untouched.
 *   status  device int32, one word, or NULL: set to 3 if an internal bounded wait gave up (else untouched).
 */
akv_status_t alpha_gram_shared(akv_handle_t* h, const akv_layout_t* lay, const float* sig, const int32_t* n_cand,
                               const akv_options_t* opt, float* gram, int32_t* status, void* stream);

/*
 * kv_compact -- the retained rows become the new cache of at most `budget` rows
 * (Section 1; Section 4.1): for r = 0..budget-1, row idx_sorted[r]
 * of K, of V and of pos moves to slot r of the SAME buffer (bit copies). Entries
 * idx_sorted[r] < 0 end the list. idx_sorted must be ascending and distinct (as
 * alpha_select writes it); rows at slots >= the kept count are unspecified afterwards.
 *   K, V  device, layout `lay`, rewritten in place (either may be NULL to skip it).
 *   pos   device int32 with the strides above, rewritten in place, or NULL. When given,
 *         its strides must address a distinct row per event (no broadcast).
 */
akv_status_t kv_compact(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                        int64_t pos_stride_b, int64_t pos_stride_l, int64_t pos_stride_h,
                        const int32_t* idx_sorted, int32_t budget, void* stream);

/*
 * alpha_compress_event -- score, select, order and compact in one call; K and V
 * cross HBM once when an event's tiles fit on chip. Arguments as in the three
 * calls above. K, V and pos are rewritten in place (pos may be NULL: already-rotated
 * keys, nothing to carry). Outputs other than idx_sorted are optional (NULL skips).
 *   scores  device fp32 [B, L, H, N] out or NULL.
 */
akv_status_t alpha_compress_event(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                  int64_t pos_stride_b, int64_t pos_stride_l, int64_t pos_stride_h,
                                  const int32_t* n_cand, const float* qstat, const int32_t* p_ref,
                                  const float* flat_sig, int32_t budget, const akv_options_t* opt,
                                  int32_t* idx_sorted, int32_t* pick_order, float* pick_gain,
                                  float* scores, int32_t* n_kept, int32_t* status, void* stream);

/*
 * alpha_compress_event_static -- the same event as alpha_compress_event, for callers that must not
 * allocate device memory. (The paper has no counterpart: this is a deployment variant, not a step
 * of the method.)
 *
 * Who needs it: alpha_compress_event keeps the intermediate scores of an event that does not fit
 * on chip in the handle's scratch, which it grows with cudaMalloc (plus a device-wide synchronise
 * when it regrows). A serving process whose memory pool has already reserved the whole device
 * cannot afford that call failing, and a latency-critical decode thread cannot afford its implicit
 * synchronisation. This entry point calls no cudaMalloc, cudaFree or other allocating routine: the
 * scores go to an array of AKV_STATIC_SCORES_MAX floats (4 MiB) that is part of the library image,
 * so every GPU that loads the library holds those 4 MiB until the process exits.
 *
 *   - It always runs as three launches (score, select, compact) on `stream`; results are those
 *     of alpha_compress_event on the same route.
 *   - Limit: B*L*H*N <= AKV_STATIC_SCORES_MAX, otherwise AKV_ERR_WORKSPACE and nothing is launched.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current). Make that first call before starting any stream capture.
 *   - All calls on one device share the array and it keeps the previous call's scores. Nothing in
 *     it has to start at zero (each call writes every score it later reads), but two calls whose
 *     kernels overlap on the GPU (different streams, no ordering between them) race on it: order
 *     such calls yourself.
 * Arguments as alpha_compress_event, without the `scores` output.
 */
#define AKV_STATIC_SCORES_MAX (1u << 20)
akv_status_t alpha_compress_event_static(akv_handle_t* h, const akv_layout_t* lay, void* K, void* V, int32_t* pos,
                                         int64_t pos_stride_b, int64_t pos_stride_l, int64_t pos_stride_h,
                                         const int32_t* n_cand, const float* qstat, const int32_t* p_ref,
                                         const float* flat_sig, int32_t budget, const akv_options_t* opt,
                                         int32_t* idx_sorted, int32_t* pick_order, float* pick_gain,
                                         int32_t* n_kept, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ALPHAKV_H */
