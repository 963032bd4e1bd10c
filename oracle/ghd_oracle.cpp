// CPU oracle for the tree-verification step of speculative decoding.
//
// THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It is a plain, slow,
// double-precision restatement of what the verify step computes, written from
// the paper's problem statement, and it shares no code with the CUDA path.
// Only the tests, the smoke check and the benchmark's CPU-baseline leg may
// load it.
//
// What it follows (paper sections):
//   * Sec. II-C, "Predict-then-Verify": all drafted tokens are verified in one
//     forward of the target model and the longest validated prefix is kept.
//   * Sec. II-C, Fig. 3: under a verification tree a token is related only to
//     certain tokens - the whole KV cache plus, among the drafted tokens, its
//     own root-to-node ancestors.
//   * Sec. II-B, Eq. (1): X = Q K^T, A = softmax(X), O = A V per head; heads are
//     concatenated and fed to the next linear layer; an MLP block follows.
//   * Sec. II-A: decode processes only new tokens against cached K/V and
//     appends the new K/V.
//   * Sec. IV-A: the model is LLaMA-7B shaped (Vicuna-7B), hence RMSNorm,
//     rotary position embedding, SwiGLU MLP and no biases.
//   * Sec. IV-A "Metrics" and Table I (width 1 gives acceptance length 1):
//     the acceptance length counts the tokens a step produces.
//
// Readings where the paper is silent (softmax scale 1/sqrt(d_head), rotate-half
// RoPE with position = kv_len + depth, first-index argmax ties, deepest-valid-
// node acceptance with lowest-index ties) are listed in the design notes.
//
// Pins: every function below is pinned by tests/test_oracle_*.py against brute
// force, closed forms and the invariants named there.  Nothing about real
// acceptance rates (Table I, Fig. 8/9) is reproduced: parity unpinned for those.
//
// Precision: inputs of storage type f16/f32 are converted exactly to double;
// all arithmetic is double; nothing is re-rounded between operations except
// the K/V rows written back to the cache (rounded to the cache's type).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_F16 = 1, DT_F64 = 2 };

inline double load_el(const void* p, int dt, size_t i) {
    if (dt == DT_F32) return (double)static_cast<const float*>(p)[i];
    if (dt == DT_F16) return (double)static_cast<const _Float16*>(p)[i];
    return static_cast<const double*>(p)[i];
}

inline void store_el(void* p, int dt, size_t i, double v) {
    if (dt == DT_F32) static_cast<float*>(p)[i] = (float)v;
    else if (dt == DT_F16) static_cast<_Float16*>(p)[i] = (_Float16)v;
    else static_cast<double*>(p)[i] = v;
}

// y[i][o] = sum_k x[i][k] * w[o][k], each sum accumulated in increasing k.
// The node loop is innermost only so that the row of w is converted once.
void linear(const double* x, const void* w, int wdt, int n, int k, int m, double* y) {
    std::vector<double> xt((size_t)k * n);
    for (int i = 0; i < n; ++i)
        for (int c = 0; c < k; ++c) xt[(size_t)c * n + i] = x[(size_t)i * k + c];
#pragma omp parallel
    {
        std::vector<double> wrow(k), acc(n);
#pragma omp for schedule(static)
        for (int o = 0; o < m; ++o) {
            for (int c = 0; c < k; ++c) wrow[c] = load_el(w, wdt, (size_t)o * k + c);
            for (int i = 0; i < n; ++i) acc[i] = 0.0;
            for (int c = 0; c < k; ++c) {
                const double wv = wrow[c];
                const double* xc = &xt[(size_t)c * n];
                for (int i = 0; i < n; ++i) acc[i] += wv * xc[i];
            }
            for (int i = 0; i < n; ++i) y[(size_t)i * m + o] = acc[i];
        }
    }
}

void rmsnorm(const double* x, const void* g, int gdt, int n, int d, double eps, double* out) {
    for (int i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int c = 0; c < d; ++c) ss += x[(size_t)i * d + c] * x[(size_t)i * d + c];
        const double r = 1.0 / std::sqrt(ss / d + eps);
        for (int c = 0; c < d; ++c) out[(size_t)i * d + c] = x[(size_t)i * d + c] * r * load_el(g, gdt, c);
    }
}

// Rotary embedding, rotate-half pairing (t, t + dh/2), angle pos * theta^(-2t/dh).
void rope(double* u, const int32_t* pos, int n, int heads, int dh, double theta) {
    const int half = dh / 2;
    for (int i = 0; i < n; ++i)
        for (int h = 0; h < heads; ++h) {
            double* s = u + ((size_t)i * heads + h) * dh;
            for (int t = 0; t < half; ++t) {
                const double ang = (double)pos[i] * std::pow(theta, -2.0 * t / dh);
                const double c = std::cos(ang), sn = std::sin(ang);
                const double a = s[t], b = s[t + half];
                s[t] = a * c - b * sn;
                s[t + half] = b * c + a * sn;
            }
        }
}

// Eq. (1) restricted to the visible pairs: node i sees cache rows 0..L-1 and the
// new rows j with vis[i][j] != 0.  Two-pass softmax, scale 1/sqrt(dh).
void tree_attention(const double* q, const double* kn, const double* vn,
                    const void* kc, const void* vc, int cdt,
                    int n, int heads, int dh, int L, int Lmax,
                    const uint8_t* vis, double* out) {
    const double scale = 1.0 / std::sqrt((double)dh);
#pragma omp parallel for collapse(2) schedule(static)
    for (int h = 0; h < heads; ++h)
        for (int i = 0; i < n; ++i) {
            std::vector<double> s((size_t)L + n);
            std::vector<char> on((size_t)L + n, 0);
            const double* qi = q + ((size_t)i * heads + h) * dh;
            for (int j = 0; j < L; ++j) {
                double a = 0.0;
                for (int c = 0; c < dh; ++c) a += qi[c] * load_el(kc, cdt, ((size_t)h * Lmax + j) * dh + c);
                s[j] = a * scale;
                on[j] = 1;
            }
            for (int j = 0; j < n; ++j) {
                if (!vis[(size_t)i * n + j]) continue;
                const double* kj = kn + ((size_t)j * heads + h) * dh;
                double a = 0.0;
                for (int c = 0; c < dh; ++c) a += qi[c] * kj[c];
                s[L + j] = a * scale;
                on[L + j] = 1;
            }
            double mx = -INFINITY;
            for (int j = 0; j < L + n; ++j) if (on[j] && s[j] > mx) mx = s[j];
            double den = 0.0;
            for (int j = 0; j < L + n; ++j) if (on[j]) { s[j] = std::exp(s[j] - mx); den += s[j]; }
            double* oi = out + ((size_t)i * heads + h) * dh;
            for (int c = 0; c < dh; ++c) oi[c] = 0.0;
            for (int j = 0; j < L; ++j) {
                const double p = s[j] / den;
                for (int c = 0; c < dh; ++c) oi[c] += p * load_el(vc, cdt, ((size_t)h * Lmax + j) * dh + c);
            }
            for (int j = 0; j < n; ++j) {
                if (!on[L + j]) continue;
                const double p = s[L + j] / den;
                const double* vj = vn + ((size_t)j * heads + h) * dh;
                for (int c = 0; c < dh; ++c) oi[c] += p * vj[c];
            }
        }
}

}  // namespace

extern "C" {

struct orc_cfg {
    int32_t d_model, n_heads, d_head, d_ffn, vocab, n_layers, max_kv_len;
    int32_t dtype;  // storage type of weights and caches: 0 = f32, 1 = f16
    double rms_eps, rope_theta;
};

struct orc_layer_w {
    const void *wqkv, *wo, *w_gate_up, *w_down, *rms1, *rms2;
};

struct orc_kv {
    void *k, *v;  // [n_heads][max_kv_len][d_head], storage type cfg.dtype
};

// Ancestor-or-self relation by walking parent[] from every node (no bit tricks).
// vis[i][j] = 1 iff j lies on the root-to-i path; depth = number of edges to the
// root; pos = kv_len + depth.  Returns 0, or -1 for an invalid parent array.
int orc_tree_build(const int32_t* parent, int n, int kv_len, uint8_t* vis, int32_t* depth, int32_t* pos) {
    if (n < 1 || parent[0] != -1) return -1;
    for (int i = 1; i < n; ++i)
        if (parent[i] < 0 || parent[i] >= i) return -1;
    std::memset(vis, 0, (size_t)n * n);
    for (int i = 0; i < n; ++i) {
        int steps = 0;
        for (int a = i; a != -1; a = parent[a]) { vis[(size_t)i * n + a] = 1; ++steps; }
        depth[i] = steps - 1;
        pos[i] = kv_len + depth[i];
    }
    return 0;
}

void orc_rmsnorm(const double* x, const void* g, int gdt, int n, int d, double eps, double* out) {
    rmsnorm(x, g, gdt, n, d, eps, out);
}

void orc_linear(const double* x, const void* w, int wdt, int n, int k, int m, double* y) {
    linear(x, w, wdt, n, k, m, y);
}

void orc_rope(double* u, const int32_t* pos, int n, int heads, int dh, double theta) {
    rope(u, pos, n, heads, dh, theta);
}

void orc_tree_attention(const double* q, const double* kn, const double* vn, const void* kc, const void* vc,
                        int cdt, int n, int heads, int dh, int L, int Lmax, const uint8_t* vis, double* out) {
    tree_attention(q, kn, vn, kc, vc, cdt, n, heads, dh, L, Lmax, vis, out);
}

// One decoder layer for all n tree nodes.  x, y: double [n][d_model].  The new
// (rotated) keys and the new values are written to cache rows kv_len + i, rounded
// to the cache's storage type; the attention itself uses the unrounded values.
// attn_dbg (optional, may be null): concatenated head outputs [n][d_model].
void orc_layer(const orc_cfg* cfg, const orc_layer_w* w, orc_kv* kv, int kv_len,
               int n, const uint8_t* vis, const int32_t* pos,
               const double* x, double* y, double* attn_dbg) {
    const int d = cfg->d_model, H = cfg->n_heads, dh = cfg->d_head, f = cfg->d_ffn, dt = cfg->dtype;
    const int Lmax = cfg->max_kv_len;
    std::vector<double> h((size_t)n * d), qkv((size_t)n * 3 * d);
    rmsnorm(x, w->rms1, dt, n, d, cfg->rms_eps, h.data());
    linear(h.data(), w->wqkv, dt, n, d, 3 * d, qkv.data());
    std::vector<double> q((size_t)n * d), k((size_t)n * d), v((size_t)n * d);
    for (int i = 0; i < n; ++i)
        for (int c = 0; c < d; ++c) {
            q[(size_t)i * d + c] = qkv[(size_t)i * 3 * d + c];
            k[(size_t)i * d + c] = qkv[(size_t)i * 3 * d + d + c];
            v[(size_t)i * d + c] = qkv[(size_t)i * 3 * d + 2 * d + c];
        }
    rope(q.data(), pos, n, H, dh, cfg->rope_theta);
    rope(k.data(), pos, n, H, dh, cfg->rope_theta);
    std::vector<double> att((size_t)n * d);
    tree_attention(q.data(), k.data(), v.data(), kv->k, kv->v, dt, n, H, dh, kv_len, Lmax, vis, att.data());
    for (int i = 0; i < n; ++i)
        for (int hh = 0; hh < H; ++hh)
            for (int c = 0; c < dh; ++c) {
                const size_t dst = ((size_t)hh * Lmax + kv_len + i) * dh + c;
                store_el(kv->k, dt, dst, k[((size_t)i * H + hh) * dh + c]);
                store_el(kv->v, dt, dst, v[((size_t)i * H + hh) * dh + c]);
            }
    if (attn_dbg) std::memcpy(attn_dbg, att.data(), sizeof(double) * n * d);
    std::vector<double> y1((size_t)n * d), proj((size_t)n * d);
    linear(att.data(), w->wo, dt, n, d, d, proj.data());
    for (size_t e = 0; e < (size_t)n * d; ++e) y1[e] = x[e] + proj[e];
    std::vector<double> h2((size_t)n * d), gu((size_t)n * 2 * f), u((size_t)n * f);
    rmsnorm(y1.data(), w->rms2, dt, n, d, cfg->rms_eps, h2.data());
    linear(h2.data(), w->w_gate_up, dt, n, d, 2 * f, gu.data());
    for (int i = 0; i < n; ++i)
        for (int c = 0; c < f; ++c) {
            const double g = gu[(size_t)i * 2 * f + c], up = gu[(size_t)i * 2 * f + f + c];
            u[(size_t)i * f + c] = g / (1.0 + std::exp(-g)) * up;
        }
    linear(u.data(), w->w_down, dt, n, f, d, proj.data());
    for (size_t e = 0; e < (size_t)n * d; ++e) y[e] = y1[e] + proj[e];
}

// First index of the row maximum.
void orc_argmax(const double* logits, int n, int v, int32_t* out) {
    for (int i = 0; i < n; ++i) {
        int best = 0;
        for (int c = 1; c < v; ++c)
            if (logits[(size_t)i * v + c] > logits[(size_t)i * v + best]) best = c;
        out[i] = best;
    }
}

// Whole step: embedding rows of the draft tokens, all layers, final norm,
// lm_head, row argmax.  logits: double [n][vocab] (required); hidden (optional):
// double [n][d_model], the last layer's output before the final norm.
void orc_step(const orc_cfg* cfg, const void* embed, const orc_layer_w* layers, const void* rms_final,
              const void* lm_head, orc_kv* kv, int kv_len, int n, const uint8_t* vis, const int32_t* pos,
              const int32_t* tokens, double* logits, int32_t* amax, double* hidden) {
    const int d = cfg->d_model, dt = cfg->dtype;
    std::vector<double> x((size_t)n * d), y((size_t)n * d);
    for (int i = 0; i < n; ++i)
        for (int c = 0; c < d; ++c) x[(size_t)i * d + c] = load_el(embed, dt, (size_t)tokens[i] * d + c);
    for (int l = 0; l < cfg->n_layers; ++l) {
        orc_layer(cfg, &layers[l], &kv[l], kv_len, n, vis, pos, x.data(), y.data(), nullptr);
        x.swap(y);
    }
    if (hidden) std::memcpy(hidden, x.data(), sizeof(double) * n * d);
    rmsnorm(x.data(), rms_final, dt, n, d, cfg->rms_eps, y.data());
    linear(y.data(), lm_head, dt, n, d, cfg->vocab, logits);
    orc_argmax(logits, n, cfg->vocab, amax);
}

// Greedy acceptance by brute force.  Node i is valid when every edge (p -> c) on
// the root-to-i path has tokens[c] == amax[p]; the root is always valid.  The
// winner is the valid node of greatest depth (lowest index among equals).
// n_matched = depth of the winner, nodes = root..winner (n_matched + 1 entries),
// out_tokens[j] = amax[nodes[j]] (n_matched + 1 entries; the last is the token
// the target model itself adds).  Returns n_matched.
int orc_accept(const int32_t* parent, const int32_t* tokens, const int32_t* amax, int n,
               int32_t* nodes, int32_t* out_tokens) {
    int win = 0, win_depth = 0;
    for (int i = 0; i < n; ++i) {
        bool ok = true;
        int dep = 0;
        for (int c = i; parent[c] != -1; c = parent[c]) {
            if (tokens[c] != amax[parent[c]]) ok = false;
            ++dep;
        }
        if (ok && dep > win_depth) { win = i; win_depth = dep; }
    }
    int c = win;
    for (int j = win_depth; j >= 0; --j) { nodes[j] = c; c = parent[c]; }
    for (int j = 0; j <= win_depth; ++j) out_tokens[j] = amax[nodes[j]];
    return win_depth;
}

}  // extern "C"
