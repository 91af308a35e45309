// CPU oracle for the HiViS drafter step.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, loop-by-loop statement of what the drafter computes, written
// from the paper (Algorithm 1; Sec. 3.2 "The overall framework"; Sec. 3.3
// "Step-dependent bias-correction residuals", Eq. 1-2; Sec. 2.1 for greedy
// verification; "Training Setup" for the residual reuse rule).  It shares no
// code with the CUDA library and must never be linked, imported or executed by
// the product path: only the tests, the smoke check and the benchmark's CPU
// baseline leg may use it.
//
// Arithmetic type: `real`, fixed at compile time (-DHVO_REAL=float or double).
// Inputs that come from storage (weights, target hidden states, residual rows,
// target logits) are always fp32 arrays (holding bf16-representable values for
// a bf16 workload); everything computed is `real`.
//
// Conventions (readings of the paper where it is silent):
//   * every weight is row-major [out, in];  y = W x.
//   * fc is [d, 2d]: columns [0,d) act on the hidden feature (the paper's w1,
//     transposed), columns [d,2d) on the token embedding (w2, transposed).
//   * RoPE pairs element i with i + dh/2 inside each head ("rotate half"),
//     angle = pos * base^(-2i/dh).
//   * the drafter layer is pre-norm: RMSNorm -> attention -> +residual ->
//     RMSNorm -> SwiGLU MLP -> +residual;  no norm in front of the LM head.
//   * argmax returns the lowest index among equal maxima; a NaN never wins.
//
// The only liberties taken for speed: OpenMP over independent output rows of a
// matrix-vector product, and a vectorisable (reassociated) inner dot product.
// No blocking, no fusion, no caching beyond the KV cache that the incremental
// form is defined by.

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef HVO_REAL
#define HVO_REAL double
#endif
typedef HVO_REAL real;

extern "C" {

typedef struct {
    int d, hq, hkv, dh, ffn, vocab;
    double eps, rope_base;
} hvo_dims;

typedef struct {
    const float *embed, *lm_head, *fc, *norm1, *wq, *wk, *wv, *bq, *bk, *bv, *wo, *norm2,
        *w_gate, *w_up, *w_down;
} hvo_weights;

// Optional copies of the intermediates of one position (any pointer may be null).
typedef struct {
    real *u, *q, *k, *v, *attn, *y, *act, *g;
} hvo_taps;

int hvo_real_bytes(void) { return (int)sizeof(real); }

int hvo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"

// ------------------------------------------------------------------ primitives
static real dot(const float* w, const real* x, int n) {
    real acc = 0;
#pragma omp simd reduction(+ : acc)
    for (int i = 0; i < n; ++i) acc += (real)w[i] * x[i];
    return acc;
}

// y[r] = sum_c W[r][c] x[c]   (+ bias[r] if bias)
static void matvec(const float* W, const float* bias, int rows, int cols, const real* x, real* y) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r) {
        real s = dot(W + (size_t)r * cols, x, cols);
        if (bias) s += (real)bias[r];
        y[r] = s;
    }
}

extern "C" {

// Semantic fusion (Algorithm 1, the fusion of the prefix and of every drafted position; Sec. 3.2):
//   u = fc * [f ; E[id]]  (+ rho)          rho = the projected residual r^i w, may be null
void hvo_fuse(const hvo_dims* D, const hvo_weights* W, const real* f, int id, const real* rho,
              real* u) {
    const int d = D->d;
    std::vector<real> cat(2 * (size_t)d);
    for (int i = 0; i < d; ++i) cat[i] = f[i];
    for (int i = 0; i < d; ++i) cat[d + i] = (real)W->embed[(size_t)id * d + i];
    matvec(W->fc, nullptr, d, 2 * d, cat.data(), u);
    if (rho)
        for (int i = 0; i < d; ++i) u[i] += rho[i];
}

// rho_i = w r_i   (the paper's r^i w with w stored [out, in]); w == null copies the rows.
void hvo_fold_residuals(int d, int R, const float* r, const float* w, real* rho) {
    for (int i = 0; i < R; ++i) {
        std::vector<real> ri(d);
        for (int j = 0; j < d; ++j) ri[j] = (real)r[(size_t)i * d + j];
        if (w)
            matvec(w, nullptr, d, d, ri.data(), rho + (size_t)i * d);
        else
            for (int j = 0; j < d; ++j) rho[(size_t)i * d + j] = ri[j];
    }
}

// out = gamma * x / sqrt(mean(x^2) + eps)
void hvo_rmsnorm(int n, const real* x, const float* gamma, double eps, real* out) {
    real ss = 0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    const real inv = (real)(1.0 / std::sqrt((double)ss / n + eps));
    for (int i = 0; i < n; ++i) out[i] = (real)gamma[i] * x[i] * inv;
}

// Rotary embedding, in place, on n_heads heads of width dh at position pos.
void hvo_rope(int n_heads, int dh, double base, int pos, real* x) {
    const int half = dh / 2;
    for (int h = 0; h < n_heads; ++h) {
        real* xh = x + (size_t)h * dh;
        for (int i = 0; i < half; ++i) {
            const double theta = (double)pos * std::pow(base, -2.0 * i / dh);
            const real c = (real)std::cos(theta), s = (real)std::sin(theta);
            const real a = xh[i], b = xh[i + half];
            xh[i] = a * c - b * s;
            xh[i + half] = b * c + a * s;
        }
    }
}

void hvo_qkv(const hvo_dims* D, const hvo_weights* W, const real* a, real* q, real* k, real* v) {
    matvec(W->wq, W->bq, D->hq * D->dh, D->d, a, q);
    matvec(W->wk, W->bk, D->hkv * D->dh, D->d, a, k);
    matvec(W->wv, W->bv, D->hkv * D->dh, D->d, a, v);
}

// Attention of one query position over cache rows [0, len): for every query head h
// (sharing KV head h / (hq/hkv)):  softmax_t(q_h . K_t / sqrt(dh)) weighted sum of V_t.
// Kc, Vc: [len][hkv*dh], K already rotated.
void hvo_attend(const hvo_dims* D, const real* q, const real* Kc, const real* Vc, int len,
                real* out) {
    const int dh = D->dh, G = D->hq / D->hkv, kvw = D->hkv * D->dh;
    const real scale = (real)(1.0 / std::sqrt((double)dh));
    for (int h = 0; h < D->hq; ++h) {
        const int hk = h / G;
        std::vector<real> sc(len);
        real mx = -INFINITY;
        for (int t = 0; t < len; ++t) {
            real s = 0;
            for (int i = 0; i < dh; ++i) s += q[(size_t)h * dh + i] * Kc[(size_t)t * kvw + hk * dh + i];
            sc[t] = s * scale;
            if (sc[t] > mx) mx = sc[t];
        }
        real den = 0;
        for (int t = 0; t < len; ++t) {
            sc[t] = std::exp(sc[t] - mx);
            den += sc[t];
        }
        for (int i = 0; i < dh; ++i) {
            real acc = 0;
            for (int t = 0; t < len; ++t) acc += sc[t] * Vc[(size_t)t * kvw + hk * dh + i];
            out[(size_t)h * dh + i] = acc / den;
        }
    }
}

// g = y + w_down * ( silu(w_gate m) * (w_up m) ),  m = RMSNorm(y; norm2)
void hvo_mlp(const hvo_dims* D, const hvo_weights* W, const real* y, real* act_out, real* g) {
    const int d = D->d, F = D->ffn;
    std::vector<real> m(d), gate(F), up(F), act(F), down(d);
    hvo_rmsnorm(d, y, W->norm2, D->eps, m.data());
    matvec(W->w_gate, nullptr, F, d, m.data(), gate.data());
    matvec(W->w_up, nullptr, F, d, m.data(), up.data());
    for (int i = 0; i < F; ++i) act[i] = gate[i] / ((real)1 + std::exp(-gate[i])) * up[i];
    matvec(W->w_down, nullptr, d, F, act.data(), down.data());
    for (int i = 0; i < d; ++i) g[i] = y[i] + down[i];
    if (act_out) std::memcpy(act_out, act.data(), sizeof(real) * F);
}

// First maximum; *gap (if given) = best - second best (0 for a tie, +inf for n == 1).
int hvo_argmax(int n, const real* x, real* gap) {
    int best = 0;
    real bv = -INFINITY, second = -INFINITY;
    for (int i = 0; i < n; ++i) {
        const real v = x[i];
        if (v > bv) {
            second = bv;
            bv = v;
            best = i;
        } else if (v > second) {
            second = v;
        }
    }
    if (gap) *gap = bv - second;
    return best;
}

int hvo_argmax_f32(int n, const float* x) {
    int best = 0;
    float bv = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (x[i] > bv) {
            bv = x[i];
            best = i;
        }
    return best;
}

static void copy_tap(real* dst, const real* src, int n) {
    if (dst) std::memcpy(dst, src, sizeof(real) * n);
}

// Steps 1-3 for one position, K/V only: fuse, +rho, RMSNorm, K and V projections,
// RoPE on K, store row `pos` of the cache.  What the drafter keeps of a prefix position.
void hvo_position_kv(const hvo_dims* D, const hvo_weights* W, const real* f, int id,
                     const real* rho, int pos, real* Kc, real* Vc) {
    const int d = D->d, kvw = D->hkv * D->dh;
    std::vector<real> u(d), a(d);
    hvo_fuse(D, W, f, id, rho, u.data());
    hvo_rmsnorm(d, u.data(), W->norm1, D->eps, a.data());
    real* k = Kc + (size_t)pos * kvw;
    real* v = Vc + (size_t)pos * kvw;
    matvec(W->wk, W->bk, kvw, d, a.data(), k);
    matvec(W->wv, W->bv, kvw, d, a.data(), v);
    hvo_rope(D->hkv, D->dh, D->rope_base, pos, k);
}

// One position through the whole drafter layer with a KV cache (incremental form):
// input pair (f, id) and residual rho at position pos; rows [0,pos) of the cache must
// be filled; writes row pos; returns g = the layer output (the drafter's f').
void hvo_position(const hvo_dims* D, const hvo_weights* W, const real* f, int id, const real* rho,
                  int pos, real* Kc, real* Vc, real* g, const hvo_taps* taps) {
    const int d = D->d, qw = D->hq * D->dh, kvw = D->hkv * D->dh;
    std::vector<real> u(d), a(d), q(qw), attn(qw), o(d), y(d), act(D->ffn);
    hvo_fuse(D, W, f, id, rho, u.data());
    hvo_rmsnorm(d, u.data(), W->norm1, D->eps, a.data());
    real* k = Kc + (size_t)pos * kvw;
    real* v = Vc + (size_t)pos * kvw;
    hvo_qkv(D, W, a.data(), q.data(), k, v);
    hvo_rope(D->hq, D->dh, D->rope_base, pos, q.data());
    hvo_rope(D->hkv, D->dh, D->rope_base, pos, k);
    hvo_attend(D, q.data(), Kc, Vc, pos + 1, attn.data());
    matvec(W->wo, nullptr, d, qw, attn.data(), o.data());
    for (int i = 0; i < d; ++i) y[i] = u[i] + o[i];
    hvo_mlp(D, W, y.data(), act.data(), g);
    if (taps) {
        copy_tap(taps->u, u.data(), d);
        copy_tap(taps->q, q.data(), qw);
        copy_tap(taps->k, k, kvw);
        copy_tap(taps->v, v, kvw);
        copy_tap(taps->attn, attn.data(), qw);
        copy_tap(taps->y, y.data(), d);
        copy_tap(taps->act, act.data(), D->ffn);
        copy_tap(taps->g, g, d);
    }
}

// Prefix build (Algorithm 1, the prefix build; Eq. 1): positions 0..T-2 carry target features and
// the initial residual rho0; only their K/V are ever consumed by a one-layer drafter.
// Pair T-1 is left for draft step 0.  Kc, Vc: [>= T+k-1][hkv*dh].
void hvo_prefill(const hvo_dims* D, const hvo_weights* W, int T, const int* ids,
                 const float* hidden, const real* rho0, int start_pos, real* Kc, real* Vc) {
    std::vector<real> f(D->d);
    for (int p = 0; p + 1 < T; ++p) {
        for (int i = 0; i < D->d; ++i) f[i] = (real)hidden[(size_t)p * D->d + i];
        hvo_position_kv(D, W, f.data(), ids[p], rho0, start_pos + p, Kc, Vc);
    }
}

// Chained drafting (Algorithm 1, the drafting loop; Eq. 2).  The cache holds n_cached rows; step 0
// consumes the pending pair (pend_hidden, pend_id) at position n_cached with residual row 0;
// step s >= 1 consumes (g of step s-1, token chosen at step s-1) at position n_cached + s
// with residual row min(s, R-1).  rho: [R][d] projected residuals.
// forced_ids (nullable): the token fed forward after step s is forced_ids[s] instead of the
// argmax (teacher forcing); out_ids always records the argmax.
// out_logits [k][V], out_gaps [k] (top-2 gap), out_g [k][d]: nullable.
void hvo_draft(const hvo_dims* D, const hvo_weights* W, int n_cached, int pend_id,
               const float* pend_hidden, int k, const real* rho, int R, real* Kc, real* Vc,
               const int* forced_ids, int* out_ids, real* out_logits, real* out_gaps, real* out_g) {
    const int d = D->d, V = D->vocab;
    std::vector<real> f(d), g(d), logits(V);
    for (int i = 0; i < d; ++i) f[i] = (real)pend_hidden[i];
    int id = pend_id;
    for (int s = 0; s < k; ++s) {
        const int row = s < R - 1 ? s : R - 1;
        hvo_position(D, W, f.data(), id, rho + (size_t)row * d, n_cached + s, Kc, Vc, g.data(),
                     nullptr);
        matvec(W->lm_head, nullptr, V, d, g.data(), logits.data());
        real gap;
        const int best = hvo_argmax(V, logits.data(), &gap);
        out_ids[s] = best;
        if (out_logits) std::memcpy(out_logits + (size_t)s * V, logits.data(), sizeof(real) * V);
        if (out_gaps) out_gaps[s] = gap;
        if (out_g) std::memcpy(out_g + (size_t)s * d, g.data(), sizeof(real) * d);
        id = forced_ids ? forced_ids[s] : best;
        f = g;
    }
}

// The same k steps with NO cache: at every step the whole sequence (T true-feature pairs
// followed by the self-fed pairs so far) is pushed through the layer from scratch with an
// L x L causal mask, exactly as the drafting loop of Algorithm 1 writes M_q(prefix, ...).  Brute force
// for small sizes; must agree with hvo_prefill + hvo_draft.
void hvo_draft_bruteforce(const hvo_dims* D, const hvo_weights* W, int T, const int* ids,
                          const float* hidden, int k, const real* rho, int R,
                          const int* forced_ids, int* out_ids, real* out_logits, real* out_g) {
    const int d = D->d, V = D->vocab, qw = D->hq * D->dh, kvw = D->hkv * D->dh;
    const int G = D->hq / D->hkv, dh = D->dh;
    const int Lmax = T + k - 1;
    // inputs of every position: feature, token id, residual row
    std::vector<real> feat((size_t)Lmax * d);
    std::vector<int> tok(Lmax), rrow(Lmax);
    for (int p = 0; p < T; ++p) {
        for (int i = 0; i < d; ++i) feat[(size_t)p * d + i] = (real)hidden[(size_t)p * d + i];
        tok[p] = ids[p];
        rrow[p] = 0;
    }
    const real scale = (real)(1.0 / std::sqrt((double)dh));
    for (int s = 0; s < k; ++s) {
        const int L = T + s;
        std::vector<real> U((size_t)L * d), Q((size_t)L * qw), K((size_t)L * kvw), Vv((size_t)L * kvw);
        std::vector<real> a(d);
        for (int p = 0; p < L; ++p) {
            hvo_fuse(D, W, &feat[(size_t)p * d], tok[p], rho + (size_t)rrow[p] * d, &U[(size_t)p * d]);
            hvo_rmsnorm(d, &U[(size_t)p * d], W->norm1, D->eps, a.data());
            hvo_qkv(D, W, a.data(), &Q[(size_t)p * qw], &K[(size_t)p * kvw], &Vv[(size_t)p * kvw]);
            hvo_rope(D->hq, dh, D->rope_base, p, &Q[(size_t)p * qw]);
            hvo_rope(D->hkv, dh, D->rope_base, p, &K[(size_t)p * kvw]);
        }
        // masked L x L attention, all positions
        std::vector<real> A((size_t)L * qw), g_all((size_t)L * d);
        for (int h = 0; h < D->hq; ++h) {
            const int hk = h / G;
            std::vector<real> S((size_t)L * L);
            for (int p = 0; p < L; ++p)
                for (int t = 0; t < L; ++t) {
                    real sc = 0;
                    for (int i = 0; i < dh; ++i)
                        sc += Q[(size_t)p * qw + h * dh + i] * K[(size_t)t * kvw + hk * dh + i];
                    S[(size_t)p * L + t] = (t <= p) ? sc * scale : -INFINITY;
                }
            for (int p = 0; p < L; ++p) {
                real mx = -INFINITY, den = 0;
                for (int t = 0; t < L; ++t) mx = S[(size_t)p * L + t] > mx ? S[(size_t)p * L + t] : mx;
                for (int t = 0; t < L; ++t) {
                    S[(size_t)p * L + t] = std::exp(S[(size_t)p * L + t] - mx);
                    den += S[(size_t)p * L + t];
                }
                for (int i = 0; i < dh; ++i) {
                    real acc = 0;
                    for (int t = 0; t < L; ++t) acc += S[(size_t)p * L + t] * Vv[(size_t)t * kvw + hk * dh + i];
                    A[(size_t)p * qw + h * dh + i] = acc / den;
                }
            }
        }
        std::vector<real> o(d), y(d);
        for (int p = 0; p < L; ++p) {
            matvec(W->wo, nullptr, d, qw, &A[(size_t)p * qw], o.data());
            for (int i = 0; i < d; ++i) y[i] = U[(size_t)p * d + i] + o[i];
            hvo_mlp(D, W, y.data(), nullptr, &g_all[(size_t)p * d]);
        }
        const real* g = &g_all[(size_t)(L - 1) * d];
        std::vector<real> logits(V);
        matvec(W->lm_head, nullptr, V, d, g, logits.data());
        const int best = hvo_argmax(V, logits.data(), nullptr);
        out_ids[s] = best;
        if (out_logits) std::memcpy(out_logits + (size_t)s * V, logits.data(), sizeof(real) * V);
        if (out_g) std::memcpy(out_g + (size_t)s * d, g, sizeof(real) * d);
        if (s + 1 < k) {   // the self-fed pair of the next step (Algorithm 1, the drafting loop)
            const int p = L;
            std::memcpy(&feat[(size_t)p * d], g, sizeof(real) * d);
            tok[p] = forced_ids ? forced_ids[s] : best;
            rrow[p] = (s + 1) < R - 1 ? (s + 1) : R - 1;
        }
    }
}

// Greedy verification (Sec. 2.1; Algorithm 1, the verification step).  Row j of logits [(k+1)][V] is the
// target's prediction after the root token and j draft tokens.  Draft token j (0-based) is
// accepted iff it equals argmax(row j) and every earlier one was accepted.  n = number
// accepted; next = argmax(row n) (the correction, or the bonus token when n == k);
// the drafter cache keeps base_len + min(n, k-1) rows (the row of the last draft token
// was never written).
void hvo_verify(int k, int V, const int* draft_ids, const float* logits, int base_len, int* n_out,
                int* next_out, int* kv_len_out) {
    int n = 0;
    while (n < k && hvo_argmax_f32(V, logits + (size_t)n * V) == draft_ids[n]) ++n;
    *n_out = n;
    *next_out = hvo_argmax_f32(V, logits + (size_t)n * V);
    *kv_len_out = base_len + (n < k - 1 ? n : k - 1);
}

}  // extern "C"
