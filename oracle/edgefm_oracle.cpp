// CPU oracle for one batch-1 decode step of a Qwen2.5-style decoder (Eq. 4 of the paper:
// y_t <- DecodeStep(y_{t-1}, KV; theta_d), KV <- UpdateKV(KV, y_t)).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA path is checked
// against.  It shares no code with the CUDA path, and nothing in the product path may call it.
//
// Conventions (the paper names the operators of the step in its hotspot list of Sec. 3.4 --
// QKV, RoPE, KV-cache write, decode attention, OProj, GateUp, DownProj, normalisation,
// activation, sampling -- but prints no formula for them; the formulas are the public Qwen2.5
// block):
//   * weights, biases, norm weights, embedding and the KV cache are bf16; read exactly as fp32.
//   * every vector between operators (x, q, k, v, scores, a, logits) is stored as fp32;
//     every sum, exp, sqrt, sin, cos is evaluated in fp64 and rounded to fp32 once.
//   * RMSNorm: x_i * rsqrt(mean(x^2) + eps) * w_i   (eps inside the root, no "+1" on w).
//   * RoPE: rotate-half pairs (i, i + d/2), angle pos * theta^(-2i/d)  (the "slice, negate,
//     concat" form the paper's App. B mentions for its BPU port).
//   * GQA: query head h reads kv head h / (n_q / n_kv).
//   * attention: scores / sqrt(d), max-subtracted softmax over slots 0 .. cur_len (the slot just
//     written included, as rounded to bf16), no mask.
//   * new k (after RoPE) and v are rounded to bf16 (round to nearest even) when appended.
//   * greedy sampling (Sec. 4.2: temperature 0, top_k = 1): lowest index among the maxima.
//   * compressed cache (Sec. 3.9, KV~ = C(KV) with on-demand reconstruction; the paper fixes no C): every cached
//     row (one position of one kv head, d values) of K and of V is stored as d signed 8-bit codes and one fp32 scale,
//     scale = amax / 127, code_j = clamp(rint(x_j * (127 / amax)), -127, 127), both evaluated in fp32 (a
//     floating-point value decides an integer here, so the decision is taken in the precision the CUDA path uses);
//     an all-zero row has scale 0.  Attention reads code * scale (fp32 product) wherever the uncompressed path reads
//     the bf16 value, the row appended by the step itself included; the appended row is compressed from the fp32 k
//     (after RoPE) and v, not from a bf16 rounding of them.
//
// Parity pins: every function below is pinned by tests/test_oracle_pins.py (closed forms,
// brute force, invariants) and the whole step by an independent numpy fp64 uncached forward
// (oracle/tiny_ref.py).  Parity unpinned: agreement with real Qwen2.5 checkpoints (no weights
// are available offline).
#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

namespace {

inline float bf16_to_f32(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// Round to nearest, ties to even; NaN stays NaN (quiet), infinities are preserved.
inline uint16_t f32_to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

// y[r] = sum_k W[r][k] * x[k] (+ b[r]);  W row-major [rows][cols].
void gemv(const uint16_t *W, const float *x, const uint16_t *bias, int64_t rows, int64_t cols, float *y) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const uint16_t *w = W + r * cols;
        double acc = 0.0;
        for (int64_t k = 0; k < cols; ++k) acc += static_cast<double>(bf16_to_f32(w[k])) * static_cast<double>(x[k]);
        if (bias) acc += static_cast<double>(bf16_to_f32(bias[r]));
        y[r] = static_cast<float>(acc);
    }
}

void rmsnorm(const float *x, const uint16_t *w, int64_t n, double eps, float *out) {
    double ss = 0.0;
    for (int64_t i = 0; i < n; ++i) ss += static_cast<double>(x[i]) * static_cast<double>(x[i]);
    const double r = 1.0 / std::sqrt(ss / static_cast<double>(n) + eps);
    for (int64_t i = 0; i < n; ++i)
        out[i] = static_cast<float>(static_cast<double>(x[i]) * r * static_cast<double>(bf16_to_f32(w[i])));
}

// In-place rotate-half RoPE of one head vector u[0:d] at integer position pos.
void rope(float *u, int64_t d, int64_t pos, double theta) {
    const int64_t half = d / 2;
    for (int64_t i = 0; i < half; ++i) {
        const double inv_freq = std::pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(d));
        const double phi = static_cast<double>(pos) * inv_freq;
        const double c = std::cos(phi), s = std::sin(phi);
        const double a = u[i], b = u[i + half];
        u[i] = static_cast<float>(a * c - b * s);
        u[i + half] = static_cast<float>(b * c + a * s);
    }
}

// p_t = exp(s_t - max s) / sum; in place.
void softmax(float *s, int64_t n) {
    double m = -INFINITY;
    for (int64_t t = 0; t < n; ++t) m = s[t] > m ? s[t] : m;
    double z = 0.0;
    std::vector<double> p(n);
    for (int64_t t = 0; t < n; ++t) { p[t] = std::exp(static_cast<double>(s[t]) - m); z += p[t]; }
    for (int64_t t = 0; t < n; ++t) s[t] = static_cast<float>(p[t] / z);
}

double silu(double g) { return g / (1.0 + std::exp(-g)); }

// Lowest index among the maxima; NaN never wins.
int64_t argmax(const float *v, int64_t n) {
    int64_t best = 0;
    float bv = v[0];
    for (int64_t i = 1; i < n; ++i)
        if (v[i] > bv || (bv != bv && v[i] == v[i])) { bv = v[i]; best = i; }
    return best;
}

// Attention of n_q query heads over n cached positions of one layer.
// K, V: bf16, element (g, t, j) at g * stride_head + t * stride_pos + j.
void attention(const float *q, const uint16_t *K, const uint16_t *V, int64_t n_q, int64_t n_kv, int64_t d,
               int64_t n, int64_t stride_head, int64_t stride_pos, float *out) {
    const int64_t group = n_q / n_kv;
    const double scale = 1.0 / std::sqrt(static_cast<double>(d));
#pragma omp parallel for schedule(static)
    for (int64_t h = 0; h < n_q; ++h) {
        const int64_t g = h / group;
        const float *qh = q + h * d;
        std::vector<float> s(n);
        for (int64_t t = 0; t < n; ++t) {
            const uint16_t *kt = K + g * stride_head + t * stride_pos;
            double acc = 0.0;
            for (int64_t j = 0; j < d; ++j) acc += static_cast<double>(qh[j]) * static_cast<double>(bf16_to_f32(kt[j]));
            s[t] = static_cast<float>(acc * scale);
        }
        softmax(s.data(), n);
        for (int64_t j = 0; j < d; ++j) {
            double acc = 0.0;
            for (int64_t t = 0; t < n; ++t)
                acc += static_cast<double>(s[t]) * static_cast<double>(bf16_to_f32(V[g * stride_head + t * stride_pos + j]));
            out[h * d + j] = static_cast<float>(acc);
        }
    }
}

// C of Sec. 3.9 for one cache row: d values -> d codes and a scale.  fp32 arithmetic on purpose (see the header).
void quantize_row(const float *x, int64_t d, int8_t *codes, float *scale) {
    float amax = 0.f;
    for (int64_t j = 0; j < d; ++j) amax = std::fabs(x[j]) > amax ? std::fabs(x[j]) : amax;
    if (!(amax > 0.f)) {
        for (int64_t j = 0; j < d; ++j) codes[j] = 0;
        *scale = 0.f;
        return;
    }
    const float inv = 127.0f / amax;
    for (int64_t j = 0; j < d; ++j) {
        float c = std::nearbyintf(x[j] * inv);   // round to nearest, ties to even (default rounding mode)
        c = c > 127.f ? 127.f : (c < -127.f ? -127.f : c);
        codes[j] = static_cast<int8_t>(c);
    }
    *scale = amax / 127.0f;
}

// Attention over a compressed cache: as attention(), every K / V value reconstructed as code * scale (fp32).
// K8, V8: element (g, t, j) at g * stride_head + t * stride_pos + j;  scales: (g, t) at g * stride_head_s + t.
void attention_q8(const float *q, const int8_t *K8, const float *Ks, const int8_t *V8, const float *Vs, int64_t n_q, int64_t n_kv,
                  int64_t d, int64_t n, int64_t stride_head, int64_t stride_pos, int64_t stride_head_s, float *out) {
    const int64_t group = n_q / n_kv;
    const double scale = 1.0 / std::sqrt(static_cast<double>(d));
#pragma omp parallel for schedule(static)
    for (int64_t h = 0; h < n_q; ++h) {
        const int64_t g = h / group;
        const float *qh = q + h * d;
        std::vector<float> s(n);
        for (int64_t t = 0; t < n; ++t) {
            const int8_t *kt = K8 + g * stride_head + t * stride_pos;
            const float ks = Ks[g * stride_head_s + t];
            double acc = 0.0;
            for (int64_t j = 0; j < d; ++j) acc += static_cast<double>(qh[j]) * static_cast<double>(static_cast<float>(kt[j]) * ks);
            s[t] = static_cast<float>(acc * scale);
        }
        softmax(s.data(), n);
        for (int64_t j = 0; j < d; ++j) {
            double acc = 0.0;
            for (int64_t t = 0; t < n; ++t)
                acc += static_cast<double>(s[t]) *
                       static_cast<double>(static_cast<float>(V8[g * stride_head + t * stride_pos + j]) * Vs[g * stride_head_s + t]);
            out[h * d + j] = static_cast<float>(acc);
        }
    }
}

struct LayerW {
    const uint16_t *input_norm, *wqkv, *bqkv, *wo, *post_norm, *w_gate_up, *w_down;
};

struct Model {
    int64_t L, H, nq, nkv, d, F, V, Tmax;
    double eps, theta;
    std::vector<LayerW> layers;
    const uint16_t *embed, *final_norm, *lm_head;
    std::vector<uint16_t> K, Vc;  // [L][nkv][Tmax][d]
    bool q8 = false;              // compressed cache: codes [L][nkv][Tmax][d] and scales [L][nkv][Tmax] instead of K, Vc
    std::vector<int8_t> K8, V8;
    std::vector<float> Ks, Vs;
    int64_t cur_len = 0;
    int64_t kv_index(int64_t l, int64_t g, int64_t t) const { return ((l * nkv + g) * Tmax + t) * d; }
    int64_t sc_index(int64_t l, int64_t g, int64_t t) const { return (l * nkv + g) * Tmax + t; }
};

}  // namespace

extern "C" {

// ---- operator-level entry points (used by the pins and by per-kernel parity tests) -------------
float oracle_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }
uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16(f); }
void oracle_gemv(const uint16_t *W, const float *x, const uint16_t *bias, int64_t rows, int64_t cols, float *y) {
    gemv(W, x, bias, rows, cols, y);
}
void oracle_rmsnorm(const float *x, const uint16_t *w, int64_t n, double eps, float *out) { rmsnorm(x, w, n, eps, out); }
void oracle_rope(float *u, int64_t d, int64_t pos, double theta) { rope(u, d, pos, theta); }
void oracle_softmax(float *s, int64_t n) { softmax(s, n); }
double oracle_silu(double g) { return silu(g); }
int64_t oracle_argmax(const float *v, int64_t n) { return argmax(v, n); }
void oracle_attention(const float *q, const uint16_t *K, const uint16_t *V, int64_t n_q, int64_t n_kv, int64_t d,
                      int64_t n, int64_t stride_head, int64_t stride_pos, float *out) {
    attention(q, K, V, n_q, n_kv, d, n, stride_head, stride_pos, out);
}

// ---- whole-model entry points ---------------------------------------------------------------
// Weight pointers are borrowed host bf16 buffers (see include/edgefm.h for the same layouts);
// layer_ptrs is an array of 7 pointers per layer in the order of struct LayerW (bqkv may be null).
void *oracle_model_create(int64_t n_layers, int64_t hidden, int64_t n_q, int64_t n_kv, int64_t head_dim, int64_t ffn,
                          int64_t vocab, double eps, double theta, const uint16_t *const *layer_ptrs,
                          const uint16_t *embed, const uint16_t *final_norm, const uint16_t *lm_head,
                          int64_t max_context) {
    Model *m = new (std::nothrow) Model();
    if (!m) return nullptr;
    m->L = n_layers; m->H = hidden; m->nq = n_q; m->nkv = n_kv; m->d = head_dim; m->F = ffn; m->V = vocab;
    m->Tmax = max_context; m->eps = eps; m->theta = theta;
    for (int64_t l = 0; l < n_layers; ++l) {
        const uint16_t *const *p = layer_ptrs + 7 * l;
        m->layers.push_back(LayerW{p[0], p[1], p[2], p[3], p[4], p[5], p[6]});
    }
    m->embed = embed; m->final_norm = final_norm; m->lm_head = lm_head;
    m->K.assign(static_cast<size_t>(n_layers * n_kv * max_context * head_dim), 0);
    m->Vc.assign(m->K.size(), 0);
    return m;
}

void oracle_model_destroy(void *h) { delete static_cast<Model *>(h); }

// Switch an empty model to the compressed cache of Sec. 3.9 (before any load or step).
int oracle_model_use_int8_kv(void *h) {
    Model *m = static_cast<Model *>(h);
    if (m->cur_len != 0) return 1;
    m->q8 = true;
    m->K8.assign(m->K.size(), 0);
    m->V8.assign(m->K.size(), 0);
    m->Ks.assign(static_cast<size_t>(m->L * m->nkv * m->Tmax), 0.f);
    m->Vs.assign(m->Ks.size(), 0.f);
    return 0;
}

void oracle_quantize_row(const float *x, int64_t d, int8_t *codes, float *scale) { quantize_row(x, d, codes, scale); }
void oracle_attention_q8(const float *q, const int8_t *K8, const float *Ks, const int8_t *V8, const float *Vs, int64_t n_q, int64_t n_kv,
                         int64_t d, int64_t n, float *out) {
    attention_q8(q, K8, Ks, V8, Vs, n_q, n_kv, d, n, n * d, d, n, out);
}

// Codes and scales of the compressed cache in its internal layout: [L][n_kv][max_context][d] and [L][n_kv][max_context].
void oracle_model_export_kv_q8(void *h, int8_t *k8, int8_t *v8, float *ks, float *vs) {
    Model *m = static_cast<Model *>(h);
    std::memcpy(k8, m->K8.data(), m->K8.size());
    std::memcpy(v8, m->V8.data(), m->V8.size());
    std::memcpy(ks, m->Ks.data(), m->Ks.size() * 4);
    std::memcpy(vs, m->Vs.data(), m->Vs.size() * 4);
}

// Load n positions of K/V (bf16, [L][n_kv][n][d] contiguous, keys already rotated) into slots 0..n-1.
int oracle_model_load_kv(void *h, const uint16_t *k, const uint16_t *v, int64_t n) {
    Model *m = static_cast<Model *>(h);
    if (n > m->Tmax || n < 0) return 1;
    for (int64_t l = 0; l < m->L; ++l)
        for (int64_t g = 0; g < m->nkv; ++g) {
            const int64_t src = ((l * m->nkv + g) * n) * m->d;
            if (m->q8) {   // the given rows are compressed one by one
                std::vector<float> row(m->d);
                for (int64_t t = 0; t < n; ++t) {
                    for (int64_t j = 0; j < m->d; ++j) row[j] = bf16_to_f32(k[src + t * m->d + j]);
                    quantize_row(row.data(), m->d, &m->K8[m->kv_index(l, g, t)], &m->Ks[m->sc_index(l, g, t)]);
                    for (int64_t j = 0; j < m->d; ++j) row[j] = bf16_to_f32(v[src + t * m->d + j]);
                    quantize_row(row.data(), m->d, &m->V8[m->kv_index(l, g, t)], &m->Vs[m->sc_index(l, g, t)]);
                }
                continue;
            }
            std::memcpy(&m->K[m->kv_index(l, g, 0)], k + src, static_cast<size_t>(n * m->d) * 2);
            std::memcpy(&m->Vc[m->kv_index(l, g, 0)], v + src, static_cast<size_t>(n * m->d) * 2);
        }
    m->cur_len = n;
    return 0;
}

int64_t oracle_model_cur_len(void *h) { return static_cast<Model *>(h)->cur_len; }

// Drop the cache rows from slot n on (n <= cache length): the "Commit" of block verification (Sec. 3.11) keeps only the
// rows of the accepted tokens.
int oracle_model_truncate(void *h, int64_t n) {
    Model *m = static_cast<Model *>(h);
    if (n < 0 || n > m->cur_len) return 1;
    m->cur_len = n;
    return 0;
}

// Copy the whole cache out in its internal layout [L][n_kv][max_context][d].
void oracle_model_export_kv(void *h, uint16_t *k_out, uint16_t *v_out) {
    Model *m = static_cast<Model *>(h);
    std::memcpy(k_out, m->K.data(), m->K.size() * 2);
    std::memcpy(v_out, m->Vc.data(), m->Vc.size() * 2);
}

// One decode step: consumes `token` at RoPE position `pos`, appends its K/V at slot cur_len,
// writes fp32 logits[V] (if non-null) and returns the greedy next token (-1 on a full cache).
int64_t oracle_model_step(void *h, int64_t token, int64_t pos, float *logits_out) {
    Model *m = static_cast<Model *>(h);
    if (m->cur_len >= m->Tmax || token < 0 || token >= m->V) return -1;
    const int64_t H = m->H, d = m->d, nq = m->nq, nkv = m->nkv, F = m->F;
    const int64_t R = (nq + 2 * nkv) * d;
    std::vector<float> x(H), xn(H), qkv(R), attn(nq * d), proj(H), gu(2 * F), a(F), logits(m->V);
    for (int64_t i = 0; i < H; ++i) x[i] = bf16_to_f32(m->embed[token * H + i]);
    const int64_t slot = m->cur_len;
    for (int64_t l = 0; l < m->L; ++l) {
        const LayerW &w = m->layers[l];
        rmsnorm(x.data(), w.input_norm, H, m->eps, xn.data());
        gemv(w.wqkv, xn.data(), w.bqkv, R, H, qkv.data());
        float *q = qkv.data(), *k = q + nq * d, *v = k + nkv * d;
        for (int64_t hh = 0; hh < nq; ++hh) rope(q + hh * d, d, pos, m->theta);
        for (int64_t g = 0; g < nkv; ++g) rope(k + g * d, d, pos, m->theta);
        if (m->q8) {
            for (int64_t g = 0; g < nkv; ++g) {
                quantize_row(k + g * d, d, &m->K8[m->kv_index(l, g, slot)], &m->Ks[m->sc_index(l, g, slot)]);
                quantize_row(v + g * d, d, &m->V8[m->kv_index(l, g, slot)], &m->Vs[m->sc_index(l, g, slot)]);
            }
            attention_q8(q, &m->K8[m->kv_index(l, 0, 0)], &m->Ks[m->sc_index(l, 0, 0)], &m->V8[m->kv_index(l, 0, 0)],
                         &m->Vs[m->sc_index(l, 0, 0)], nq, nkv, d, slot + 1, m->Tmax * d, d, m->Tmax, attn.data());
        } else {
            for (int64_t g = 0; g < nkv; ++g)
                for (int64_t j = 0; j < d; ++j) {
                    m->K[m->kv_index(l, g, slot) + j] = f32_to_bf16(k[g * d + j]);
                    m->Vc[m->kv_index(l, g, slot) + j] = f32_to_bf16(v[g * d + j]);
                }
            attention(q, &m->K[m->kv_index(l, 0, 0)], &m->Vc[m->kv_index(l, 0, 0)], nq, nkv, d, slot + 1, m->Tmax * d, d,
                      attn.data());
        }
        gemv(w.wo, attn.data(), nullptr, H, nq * d, proj.data());
        for (int64_t i = 0; i < H; ++i) x[i] = static_cast<float>(static_cast<double>(x[i]) + static_cast<double>(proj[i]));
        rmsnorm(x.data(), w.post_norm, H, m->eps, xn.data());
        gemv(w.w_gate_up, xn.data(), nullptr, 2 * F, H, gu.data());
        for (int64_t i = 0; i < F; ++i)
            a[i] = static_cast<float>(silu(static_cast<double>(gu[i])) * static_cast<double>(gu[F + i]));
        gemv(w.w_down, a.data(), nullptr, H, F, proj.data());
        for (int64_t i = 0; i < H; ++i) x[i] = static_cast<float>(static_cast<double>(x[i]) + static_cast<double>(proj[i]));
    }
    rmsnorm(x.data(), m->final_norm, H, m->eps, xn.data());
    gemv(m->lm_head, xn.data(), nullptr, m->V, H, logits.data());
    if (logits_out) std::memcpy(logits_out, logits.data(), static_cast<size_t>(m->V) * 4);
    m->cur_len += 1;
    return argmax(logits.data(), m->V);
}

}  // extern "C"
