/*
 * CPU oracle, C twin of alpha_oracle.py -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, double-precision statement of one KV-cache compression event of
 * the alpha retainer, written so that it can be read against the paper:
 *   - score:      reading of the scorer that Section 4.1 inherits from TriAttention
 *                 (formula not printed in the paper; PARITY UNPINNED against the
 *                 real scorer, pinned to closed forms in the tests);
 *   - signature:  Eq. 1 reduced to one head, v_i = V_i / (||V_i||_2 + eps);
 *   - selection:  Eq. 2 evaluated for every candidate from a per-candidate redundancy term
 *                 (largest cosine against the members chosen so far, never below zero), Eq. 3's
 *                 arg-max over the candidates outside the set, then the new member's cosines are
 *                 folded into that term -- what Algorithm 1 computes; lambda = 0 is plain top-k;
 *   - compaction: retained rows become the new cache, ascending index order.
 * No blocking, no pruning, no reordering. It shares no code with the CUDA path
 * and is only called by tests, the smoke check and the benchmark's CPU leg.
 *
 * Build: gcc -O2 -fPIC -shared -o liborc.so alpha_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

static double load_elem(const void* base, int dtype, int64_t i) {
    if (dtype == ORC_BF16) {
        uint32_t u = ((uint32_t)((const uint16_t*)base)[i]) << 16;
        float f;
        memcpy(&f, &u, 4);
        return (double)f;
    }
    return (double)((const float*)base)[i];
}

/* s_i = (1/sqrt d) Re sum_f c_f z(q)_f conj(z(k_i)_f) exp(i (p_ref - p_i) theta_f),
 * theta_f = base^(-2f/d), c_f = mean_{w<W} exp(i w theta_f), z(x)_f = x_f + i x_{f+d/2}.
 * pos == NULL: s_i = q . k_i / sqrt d. */
void orc_score(const void* K, int dtype, int n, int d, const int32_t* pos, const float* q,
               int64_t p_ref, int W, double base, double* s) {
    const int half = d / 2;
    const double inv = 1.0 / sqrt((double)d);
    if (!pos) {
        for (int i = 0; i < n; ++i) {
            double acc = 0.0;
            for (int j = 0; j < d; ++j) acc += (double)q[j] * load_elem(K, dtype, (int64_t)i * d + j);
            s[i] = acc * inv;
        }
        return;
    }
    double* theta = (double*)malloc(sizeof(double) * half);
    double* gr = (double*)malloc(sizeof(double) * half); /* c_f z(q)_f, real and imaginary part */
    double* gi = (double*)malloc(sizeof(double) * half);
    for (int f = 0; f < half; ++f) {
        theta[f] = pow(base, -2.0 * (double)f / (double)d);
        double cr = 0.0, ci = 0.0;
        for (int w = 0; w < W; ++w) {
            cr += cos((double)w * theta[f]);
            ci += sin((double)w * theta[f]);
        }
        cr /= (double)W;
        ci /= (double)W;
        double qr = (double)q[f], qi = (double)q[f + half];
        gr[f] = cr * qr - ci * qi;
        gi[f] = cr * qi + ci * qr;
    }
    for (int i = 0; i < n; ++i) {
        double dist = (double)(p_ref - (int64_t)pos[i]);
        double acc = 0.0;
        for (int f = 0; f < half; ++f) {
            double kr = load_elem(K, dtype, (int64_t)i * d + f);
            double ki = load_elem(K, dtype, (int64_t)i * d + f + half);
            /* g * conj(k) */
            double tr = gr[f] * kr + gi[f] * ki;
            double ti = gi[f] * kr - gr[f] * ki;
            double ang = dist * theta[f];
            acc += tr * cos(ang) - ti * sin(ang);
        }
        s[i] = acc * inv;
    }
    free(theta);
    free(gr);
    free(gi);
}

/* v_i = V_i / (||V_i||_2 + eps), written to sig [n, d] */
void orc_signature(const void* V, int dtype, int n, int d, double eps, double* sig) {
    for (int i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int j = 0; j < d; ++j) {
            double x = load_elem(V, dtype, (int64_t)i * d + j);
            ss += x * x;
        }
        double r = 1.0 / (sqrt(ss) + eps);
        for (int j = 0; j < d; ++j) sig[(int64_t)i * d + j] = load_elem(V, dtype, (int64_t)i * d + j) * r;
    }
}

/* argmax over candidates not yet in S, ties to the lowest index; a candidate at
 * -inf can still be taken when nothing better is left, so picks stay distinct */
static int argmax_lowest(const double* a, const char* inS, int n) {
    int best = -1;
    for (int i = 0; i < n; ++i) {
        if (inS[i]) continue;
        if (best < 0 || a[i] > a[best]) best = i;
    }
    return best;
}

static double second_best(const double* a, int n, int skip) {
    double v = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (i != skip && a[i] > v) v = a[i];
    return v;
}

/* Greedy fill (Eq. 2, Eq. 3). order/gain/margin have k entries; returns the number of picks
 * (min(k, n)); *status: 0 ok, 1 non-finite score seen, 2 n < k. */
int orc_select(const double* s_in, const double* sig, int n, int d, int k, double lam,
               int force_greedy, int64_t* order, double* gain, double* margin, int* status) {
    double* s = (double*)malloc(sizeof(double) * n);
    double* a = (double*)malloc(sizeof(double) * n);
    double* m = (double*)calloc(n, sizeof(double));
    char* inS = (char*)calloc(n, 1);
    int st = 0;
    for (int i = 0; i < n; ++i) {
        s[i] = s_in[i];
        if (!isfinite(s[i])) {
            s[i] = -INFINITY;
            st = 1;
        }
    }
    if (n < k) {
        k = n;
        st = 2;
    }
    const int topk_branch = (lam == 0.0 && !force_greedy);
    for (int t = 0; t < k; ++t) {
        for (int i = 0; i < n; ++i) {
            double pen = (t == 0 || topk_branch) ? 0.0 : lam * m[i];
            a[i] = inS[i] ? -INFINITY : s[i] - pen;
        }
        int i = argmax_lowest(a, inS, n);
        double sec = second_best(a, n, i);
        order[t] = i;
        gain[t] = a[i];
        margin[t] = (isfinite(a[i]) && isfinite(sec)) ? a[i] - sec : (isfinite(a[i]) ? INFINITY : 0.0);
        inS[i] = 1;
        if (!topk_branch) {
            const double* vi = sig + (int64_t)i * d;
            for (int j = 0; j < n; ++j) {
                const double* vj = sig + (int64_t)j * d;
                double c = 0.0;
                for (int x = 0; x < d; ++x) c += vj[x] * vi[x];
                if (c > m[j]) m[j] = c;
            }
        }
    }
    free(s);
    free(a);
    free(m);
    free(inS);
    if (status) *status = st;
    return k;
}

static int cmp_i64(const void* x, const void* y) {
    int64_t a = *(const int64_t*)x, b = *(const int64_t*)y;
    return (a > b) - (a < b);
}

/* Whole events over a dense batch [E, n, d] (E = B*L*H, event e = (b*L + l)*H + h),
 * events e0 <= e < e1. pos is [E, n] or NULL; qstat [L*H, d]; p_ref [B] or NULL
 * (then max position + 1 of the event). Outputs (any may be NULL): scores [E, n],
 * idx_sorted [E, k] (int32, -1 padded), order [E, k], Kout/Vout [E, k, d] raw
 * copies, posout [E, k]. budgets: NULL, or [L*H] per-(layer, head) budgets (each <= k, the
 * row length of the outputs): event (b, l, h) then keeps budgets[l*H + h] rows (Section 6: the
 * selector used inside a per-head or per-layer budget allocator). */
void orc_event_batch(const void* K, const void* V, int dtype, int B, int L, int H, int n, int d,
                     const int32_t* pos, const float* qstat, const int32_t* p_ref, int W, double base,
                     double eps, int k, double lam, int force_greedy, int e0, int e1, double* scores,
                     int32_t* idx_sorted, int32_t* order_out, void* Kout, void* Vout, int32_t* posout,
                     int32_t* status_out, const int32_t* budgets) {
    (void)B;
    const size_t es = dtype == ORC_BF16 ? 2 : 4;
    double* s = (double*)malloc(sizeof(double) * n);
    double* sig = (double*)malloc(sizeof(double) * (size_t)n * d);
    int64_t* order = (int64_t*)malloc(sizeof(int64_t) * k);
    double* gain = (double*)malloc(sizeof(double) * k);
    double* margin = (double*)malloc(sizeof(double) * k);
    for (int e = e0; e < e1; ++e) {
        const int b = e / (L * H);
        const int lh = e % (L * H);
        const char* Ke = (const char*)K + (size_t)e * n * d * es;
        const char* Ve = (const char*)V + (size_t)e * n * d * es;
        const int32_t* pe = pos ? pos + (size_t)e * n : NULL;
        int64_t pr = 0;
        if (pe) {
            if (p_ref) pr = p_ref[b];
            else {
                int32_t mx = pe[0];
                for (int i = 1; i < n; ++i) if (pe[i] > mx) mx = pe[i];
                pr = (int64_t)mx + 1;
            }
        }
        orc_score(Ke, dtype, n, d, pe, qstat + (size_t)lh * d, pr, W, base, s);
        orc_signature(Ve, dtype, n, d, eps, sig);
        int st = 0;
        const int k_event = budgets ? (budgets[lh] < k ? budgets[lh] : k) : k;
        int kk = orc_select(s, sig, n, d, k_event, lam, force_greedy, order, gain, margin, &st);
        if (scores) memcpy(scores + (size_t)e * n, s, sizeof(double) * n);
        if (order_out)
            for (int t = 0; t < k; ++t) order_out[(size_t)e * k + t] = t < kk ? (int32_t)order[t] : -1;
        qsort(order, kk, sizeof(int64_t), cmp_i64);
        for (int t = 0; t < k; ++t) {
            if (idx_sorted) idx_sorted[(size_t)e * k + t] = t < kk ? (int32_t)order[t] : -1;
            if (t < kk) {
                if (Kout) memcpy((char*)Kout + ((size_t)e * k + t) * d * es, Ke + (size_t)order[t] * d * es, d * es);
                if (Vout) memcpy((char*)Vout + ((size_t)e * k + t) * d * es, Ve + (size_t)order[t] * d * es, d * es);
                if (posout && pe) posout[(size_t)e * k + t] = pe[order[t]];
            }
        }
        if (status_out) status_out[e] = st;
    }
    free(s);
    free(sig);
    free(order);
    free(gain);
    free(margin);
}
