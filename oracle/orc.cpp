// CPU oracle for adaptive self-speculative decoding (arXiv 2410.01028).
//
// THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It is a plain, slow,
// obviously-correct restatement of what the CUDA library computes, used only
// by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
// It shares no code, header, table or constant generator with the CUDA
// library and neither includes the other.
//
// What it computes, and the passage each part follows:
//   * cosine similarity of a hidden-state row before and after a sublayer and
//     its average over the prompt (ACS, C_l)            -- Section 3.1, Section 3.2 (definition of C_l)
//   * the Adaptive Draft Model Generator                 -- Algorithm 1, rules 1 and 2 of Section 3.2,
//                                                           rule subsets of Table 5
//   * greedy self-speculative decoding: draft with the sub-network D, verify
//     k+1 tokens with M, accept the matching prefix, replace the first
//     rejected token with M's                           -- Section 1 (paragraphs 2 and 3)
//   * the Llama-style dense decoder those run on.  The paper treats the model
//     as given; the architecture (RMSNorm, rotary embedding with half-split
//     pairing, SwiGLU, untied LM head, bf16 weights) and the points where
//     activations are rounded are a reading fixed by this build and listed
//     in the design notes (roundings R1..R8 below).
//
// Arithmetic: every sum is accumulated in double; values are rounded to float
// or bfloat16 only at the stated points:
//   R1 residual stream is float                R5 attention output -> bf16
//   R2 RMSNorm output -> bf16                  R6 o, y = x + o are float
//   R3 q,k (after RoPE), v -> bf16; cache bf16 R7 silu(g)*u -> bf16; z = y + dn float
//   R4 scores, softmax: no rounding            R8 logits float; argmax = lowest index of the maximum
// With ORC_FLAG_NO_ROUNDING the bf16 roundings (R2,R3,R5,R7) are skipped,
// which gives the "exact arithmetic" variant used to bound the rounding error.
//
// Pins (tests/test_oracle_*.py): closed forms of the cosine; hand-derived ADMG
// sets; brute force over all masks on L=2; prefill == sequential decode;
// zeroed output projections => identity sublayer, cosine exactly 1; S=1 =>
// attention output equals the value row; rotation at position 0 is the
// identity; a numpy restatement of single sublayers; speculative == greedy
// autoregressive output for every mask and draft length.
// Two opt-in extensions that the paper does not have (off by default): MLP sublayers removed by their own
// similarity (orc_admg_ext; pinned by brute force over all masks on L=2), and C_l kept running over the rows
// committed after the prompt, with Algorithm 1 run again every few rounds (pinned: the running C_l after a
// generation equals the C_l of one prefill over prompt + emitted tokens, for both decoding modes).
//   * verification when sampling is used: drafted tokens are sampled from D's distribution q and accepted
//     with probability min(1, p/q) under M's distribution p, a rejected token is resampled from the
//     normalised max(0, p - q), so that every emitted token is distributed as if M had sampled it
//                                                       -- Section 1 (third paragraph; the rule of the two
//                                                          speculative-sampling papers cited there), used for
//                                                          the T > 0 columns of Tables 3 and 4
//     Random numbers come from one counter-based generator, Philox4x32-10 (Salmon et al., SC'11), keyed
//     by the seed and indexed by (position of the token being chosen, kind of draw).  Pins: the generator's
//     published known-answer vectors; softmax and inverse-CDF sampling against scipy / numpy; T -> 0 gives
//     the greedy loop; q = p accepts everything; the emitted-token histogram over 10^5 rounds equals p for a
//     deliberately wrong q (chi-square).
// Parity unpinned: absolute token ids / logits of the random synthetic models
// (the paper prints no worked example).
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------- number formats
inline float bf16_bits_to_float(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// round a float to the nearest bfloat16 (ties to even); result returned as float
inline float round_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return f;  // inf / nan unchanged
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    std::memcpy(&f, &u, 4);
    return f;
}

// ---------------------------------------------------------------- dot product
// sum_k w[k]*x[k] in index order: bf16 weights, float activations, one double accumulator.
// The product of two floats is exact in double, so the only rounding is in the running sum.
double dot_bf16_f32(const uint16_t* w, const float* x, int64_t n) {
    double acc = 0;
    for (int64_t k = 0; k < n; ++k) acc += (double)bf16_bits_to_float(w[k]) * (double)x[k];
    return acc;
}

// out[m][r] = sum_k W[r][k] * x[m][k]     W: [n_out, n_in] bf16 row-major, x: [M, n_in]
// (output rows are shared among threads; every element is one independent dot product)
void matvec_rows(const uint16_t* W, int64_t n_out, int64_t n_in, const float* x, int M, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_out; ++r)
        for (int m = 0; m < M; ++m) out[(int64_t)m * n_out + r] = dot_bf16_f32(W + r * n_in, x + (int64_t)m * n_in, n_in);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------- public structs
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, max_seq;
    float rms_eps, rope_theta;
    uint32_t flags;
} orc_config;

typedef struct {  // bf16 bit patterns, row-major [out,in], stacked over layers; borrowed, never copied
    const uint16_t *embed, *lm_head, *final_norm;
    const uint16_t *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *wg, *wu, *wd;
} orc_weights;

typedef struct { float alpha; int32_t m, n; uint32_t flags; float alpha_mlp; int32_t refresh; } orc_admg_params;
typedef struct { int32_t mode, draft_len, max_new, eos_id; orc_admg_params admg; float draft_exit_margin; float temperature; uint64_t seed; } orc_gen_params;
typedef struct {
    int64_t full_passes, draft_passes, verify_passes, rounds, drafted, accepted, prefill_rows;
    double ms_prefill, ms_full, ms_draft, ms_verify, ms_total;
} orc_stats;

enum { ORC_FLAG_NO_ROUNDING = 1u };
enum { ORC_USE_CS = 1u, ORC_USE_RULE1 = 2u, ORC_USE_RULE2 = 4u, ORC_USE_CS_MLP = 8u, ORC_RUNNING_C = 16u };
enum { ORC_MODE_AR = 0, ORC_MODE_SPEC = 1, ORC_MODE_SPEC_MANUAL_MASK = 2 };
enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_STATE = -2, ORC_ERR_OVERFLOW = -4 };

// ---------------------------------------------------------------- cosine (Section 3.2, summand of C_l)
// <x,y> / (||x||_2 ||y||_2); the denominator is clamped at 1e-30 so that two
// zero rows do not divide by zero (the paper is silent on that case).
double orc_cosine(const float* x, const float* y, int64_t n) {
    double sxy = 0, sxx = 0, syy = 0;
    for (int64_t i = 0; i < n; ++i) {
        sxy += (double)x[i] * (double)y[i];
        sxx += (double)x[i] * (double)x[i];
        syy += (double)y[i] * (double)y[i];
    }
    return sxy / std::max(std::sqrt(sxx) * std::sqrt(syy), 1e-30);
}

// ---------------------------------------------------------------- ADMG (Algorithm 1)
// Layers are numbered l = 1..L as in the paper; array index is l-1.
//   remove_MLP  = { l : l is a positive multiple of m, l <= L-n }          (rule 1, guarded by rule 2)
//   remove_ATTN = { l : C_l >= alpha, l <= L-n }  union  remove_MLP         (CS thresholding, rule 2)
// flags choose the rule subsets of Table 5: without ORC_USE_RULE2 n is taken
// as 0; without ORC_USE_RULE1 remove_MLP is empty; without ORC_USE_CS the
// threshold test is dropped.  The comparison is done in float, inclusive.
int orc_admg(const float* C, int32_t L, float alpha, int32_t m, int32_t n, uint32_t flags, uint8_t* remove_attn,
             uint8_t* remove_mlp) {
    if (!C || L < 0 || n < 0 || m < 0 || !remove_attn || !remove_mlp) return ORC_ERR_ARG;
    const int32_t n_eff = (flags & ORC_USE_RULE2) ? n : 0;
    for (int32_t l = 1; l <= L; ++l) {
        const bool removable = l <= L - n_eff;
        const bool by_rule1 = (flags & ORC_USE_RULE1) && m >= 1 && (l % m == 0) && removable;
        const bool by_cs = (flags & ORC_USE_CS) && (C[l - 1] >= alpha) && removable;
        remove_mlp[l - 1] = by_rule1 ? 1 : 0;
        remove_attn[l - 1] = (by_cs || by_rule1) ? 1 : 0;
    }
    return ORC_OK;
}

// Extension beyond Algorithm 1 (the paper measures the MLP similarities, Table 1, but its rule never looks at
// them): with ORC_USE_CS_MLP an MLP sublayer is also removed when its own similarity reaches alpha_mlp, under
// the same protection of the last n layers.  remove_ATTN stays exactly Algorithm 1's set.
//   remove_MLP' = remove_MLP  union  { l : Cmlp_l >= alpha_mlp, l <= L-n }
int orc_admg_ext(const float* C_attn, const float* C_mlp, int32_t L, float alpha, float alpha_mlp, int32_t m, int32_t n,
                 uint32_t flags, uint8_t* remove_attn, uint8_t* remove_mlp) {
    const int rc = orc_admg(C_attn, L, alpha, m, n, flags, remove_attn, remove_mlp);
    if (rc) return rc;
    if (!(flags & ORC_USE_CS_MLP)) return ORC_OK;
    if (!C_mlp) return ORC_ERR_ARG;
    const int32_t n_eff = (flags & ORC_USE_RULE2) ? n : 0;
    for (int32_t l = 1; l <= L - n_eff; ++l)
        if (C_mlp[l - 1] >= alpha_mlp) remove_mlp[l - 1] = 1;
    return ORC_OK;
}

// ---------------------------------------------------------------- random numbers (sampling-based verification)
// Philox4x32-10: ten rounds of  (c0,c1,c2,c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
// with the key bumped by the Weyl constants after every round (Salmon, Moraes, Dror, Shaw, SC'11).
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0, c1 = n1, c2 = n2, c3 = n3;
        k0 += W0, k1 += W1;
    }
    out[0] = c0, out[1] = c1, out[2] = c2, out[3] = c3;
}

// kinds of draw at one position of the sequence
enum { ORC_DRAW_DRAFT = 0, ORC_DRAW_ACCEPT = 1, ORC_DRAW_TARGET = 2 };

// The uniform number in (0,1) for (seed, position of the token being chosen, kind of draw): first output word of
// the generator with key = seed and counter = (position, kind, 0, 0), mapped to (x + 1/2) / 2^32.
double orc_uniform(uint64_t seed, uint32_t position, uint32_t kind) {
    const uint32_t ctr[4] = {position, kind, 0u, 0u}, key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return ((double)out[0] + 0.5) * (1.0 / 4294967296.0);
}

// p_i = exp(l_i / T) / sum_j exp(l_j / T), evaluated with the maximum subtracted
void orc_softmax_t(const float* logits, int32_t V, double T, double* p) {
    double mx = -INFINITY;
    for (int32_t i = 0; i < V; ++i) mx = std::max(mx, (double)logits[i] / T);
    double sum = 0;
    for (int32_t i = 0; i < V; ++i) {
        p[i] = std::exp((double)logits[i] / T - mx);
        sum += p[i];
    }
    for (int32_t i = 0; i < V; ++i) p[i] /= sum;
}

// Inverse-CDF sampling from non-negative weights w (not necessarily normalised): the smallest i with
// w_0 + ... + w_i > u * (w_0 + ... + w_{V-1}); if rounding leaves none, the last index with w_i > 0.
int32_t orc_sample_cdf(const double* w, int32_t V, double u) {
    double total = 0;
    for (int32_t i = 0; i < V; ++i) total += w[i];
    const double target = u * total;
    double run = 0;
    int32_t last = 0;
    for (int32_t i = 0; i < V; ++i) {
        if (w[i] > 0) last = i;
        run += w[i];
        if (run > target) return i;
    }
    return last;
}

// Verification of k drafted tokens when sampling is used (Section 1; speculative sampling).  p has k+1 rows (M's
// distribution for the token after each verify row), q has k rows (D's distribution each draft was sampled from),
// drafts[j] is the token at position pos0 + 1 + j.  Draft j is accepted when its ACCEPT draw is below
// min(1, p_j(x)/q_j(x)); the first rejected one is replaced by a token sampled from max(0, p_j - q_j) (normalised)
// with the TARGET draw of that position; if all k are accepted one more token is sampled from p_k.  out receives
// the accepted drafts followed by that last token (a+1 tokens); returns a.
int32_t orc_spec_accept(const double* p, const double* q, const int32_t* drafts, int32_t k, int32_t V, uint64_t seed,
                        int32_t pos0, int32_t* out) {
    std::vector<double> res(V);
    for (int32_t j = 0; j < k; ++j) {
        const int32_t x = drafts[j];
        const double pj = p[(size_t)j * V + x], qj = q[(size_t)j * V + x];
        const double r = orc_uniform(seed, (uint32_t)(pos0 + 1 + j), ORC_DRAW_ACCEPT);
        if (r * qj < pj) {  // r < min(1, p/q), written without the division
            out[j] = x;
            continue;
        }
        double mass = 0;
        for (int32_t i = 0; i < V; ++i) {
            res[i] = std::max(0.0, p[(size_t)j * V + i] - q[(size_t)j * V + i]);
            mass += res[i];
        }
        const double u = orc_uniform(seed, (uint32_t)(pos0 + 1 + j), ORC_DRAW_TARGET);
        // (a rejection implies p != q, so the residual has mass; should rounding leave none, fall back to p)
        out[j] = mass > 0 ? orc_sample_cdf(res.data(), V, u) : orc_sample_cdf(p + (size_t)j * V, V, u);
        return j;
    }
    out[k] = orc_sample_cdf(p + (size_t)k * V, V, orc_uniform(seed, (uint32_t)(pos0 + 1 + k), ORC_DRAW_TARGET));
    return k;
}

// ---------------------------------------------------------------- decoder state
struct orc_ctx {
    orc_config c;
    orc_weights w;
    bool round;                      // apply the bf16 roundings R2,R3,R5,R7
    int32_t kv_dim;
    std::vector<float> rope_cos, rope_sin;  // [max_seq][head_dim/2]
    std::vector<float> kcache, vcache;      // [L][max_seq][kv_dim]
    int32_t n_committed = 0;         // positions whose K/V belong to the accepted sequence
    int32_t draft_cursor = 0;        // next position a draft step writes
    std::vector<uint8_t> skip_attn, skip_mlp;
    std::vector<double> sumcos_attn, sumcos_mlp;  // running sums over prompt rows
    int64_t n_sim_rows = 0;
    bool running_c = false;          // fold the rows committed after the prompt into the sums as well (opt-in)
    // sampling (temperature > 0): every token is drawn instead of taken as the argmax
    double temperature = 0.0;
    uint64_t seed = 0;
    std::vector<double> q_rows;      // [drafts of this round][V]: D's distribution each drafted token was sampled from
    std::vector<int32_t> drafted;    // the tokens sampled by the draft steps of this round
    // results of the last pass
    int32_t last_M = 0;
    std::vector<float> last_logits;              // [M][V]
    std::vector<float> last_cos_attn, last_cos_mlp;  // [L][M]; NaN where the sublayer was skipped
    std::vector<int32_t> last_argmax;            // [M]
    std::vector<float> last_margin;              // [M] top1 - top2
    orc_stats stats{};
    std::string err;
};

static double now_ms() {
    return std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

int orc_create(const orc_config* cfg, const orc_weights* w, orc_ctx** out) {
    if (!cfg || !w || !out) return ORC_ERR_ARG;
    const orc_config& c = *cfg;
    if (c.n_layers < 0 || c.d_model <= 0 || c.n_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 || c.head_dim % 2 ||
        c.n_heads * c.head_dim != c.d_model || c.n_heads % c.n_kv_heads || c.d_ffn <= 0 || c.vocab <= 0 || c.max_seq <= 0)
        return ORC_ERR_ARG;
    orc_ctx* x = new orc_ctx();
    x->c = c;
    x->w = *w;
    x->round = !(c.flags & ORC_FLAG_NO_ROUNDING);
    x->kv_dim = c.n_kv_heads * c.head_dim;
    const int half = c.head_dim / 2;
    x->rope_cos.resize((size_t)c.max_seq * half);
    x->rope_sin.resize((size_t)c.max_seq * half);
    // rotary embedding: pair (j, j+hd/2) of a head is rotated by angle p * theta^(-2j/hd)
    for (int p = 0; p < c.max_seq; ++p)
        for (int j = 0; j < half; ++j) {
            const double ang = (double)p * std::pow((double)c.rope_theta, -2.0 * j / (double)c.head_dim);
            x->rope_cos[(size_t)p * half + j] = (float)std::cos(ang);
            x->rope_sin[(size_t)p * half + j] = (float)std::sin(ang);
        }
    x->kcache.assign((size_t)c.n_layers * c.max_seq * x->kv_dim, 0.f);
    x->vcache.assign((size_t)c.n_layers * c.max_seq * x->kv_dim, 0.f);
    x->skip_attn.assign(c.n_layers, 0);
    x->skip_mlp.assign(c.n_layers, 0);
    x->sumcos_attn.assign(c.n_layers, 0.0);
    x->sumcos_mlp.assign(c.n_layers, 0.0);
    *out = x;
    return ORC_OK;
}

int orc_destroy(orc_ctx* x) {
    delete x;
    return ORC_OK;
}

const char* orc_last_error(orc_ctx* x) { return x ? x->err.c_str() : "null context"; }

// new context: nothing cached, no similarities, empty skip mask
int orc_reset(orc_ctx* x) {
    if (!x) return ORC_ERR_ARG;
    x->n_committed = x->draft_cursor = 0;
    std::fill(x->skip_attn.begin(), x->skip_attn.end(), 0);
    std::fill(x->skip_mlp.begin(), x->skip_mlp.end(), 0);
    std::fill(x->sumcos_attn.begin(), x->sumcos_attn.end(), 0.0);
    std::fill(x->sumcos_mlp.begin(), x->sumcos_mlp.end(), 0.0);
    x->n_sim_rows = 0;
    x->last_M = 0;
    x->drafted.clear();
    x->stats = orc_stats{};
    return ORC_OK;
}

// RMSNorm of each row, R2:  xn_i = x_i * (mean(x^2)+eps)^(-1/2) * gain_i   (rounded to bf16)
static void rmsnorm_rows(const orc_ctx* x, const float* in, int M, const uint16_t* gain, float* out) {
    const int d = x->c.d_model;
    for (int m = 0; m < M; ++m) {
        double ss = 0;
        for (int i = 0; i < d; ++i) ss += (double)in[(size_t)m * d + i] * (double)in[(size_t)m * d + i];
        const double inv = 1.0 / std::sqrt(ss / d + (double)x->c.rms_eps);
        for (int i = 0; i < d; ++i) {
            const float v = (float)((double)in[(size_t)m * d + i] * inv * (double)bf16_bits_to_float(gain[i]));
            out[(size_t)m * d + i] = x->round ? round_bf16(v) : v;
        }
    }
}

// One pass of M rows (tokens at positions pos0..pos0+M-1) through the decoder.
//   use_mask : sublayers in the context's skip sets are the identity (the draft model D, Section 1 / 3.2);
//              a skipped attention sublayer neither reads nor writes its K/V.
//   acc_sim  : add each row's cosines to the running sums that define C_l (prefill only).
// Rows are causal among themselves: the row at position p attends to keys 0..p.
static int forward_rows(orc_ctx* x, const int32_t* tokens, int M, int pos0, bool use_mask, bool acc_sim) {
    const orc_config& c = x->c;
    const int d = c.d_model, hd = c.head_dim, half = hd / 2, f = c.d_ffn, V = c.vocab, kvd = x->kv_dim, L = c.n_layers;
    const int group = c.n_heads / c.n_kv_heads;
    if (M <= 0 || pos0 < 0) return ORC_ERR_ARG;
    if ((int64_t)pos0 + M > c.max_seq) return ORC_ERR_OVERFLOW;
    for (int m = 0; m < M; ++m)
        if (tokens[m] < 0 || tokens[m] >= V) return ORC_ERR_ARG;

    std::vector<float> h((size_t)M * d), hn((size_t)M * d), y((size_t)M * d), att((size_t)M * d), t((size_t)M * f);
    std::vector<double> q((size_t)M * d), kk((size_t)M * kvd), vv((size_t)M * kvd), o((size_t)M * d), g((size_t)M * f),
        u((size_t)M * f);
    std::vector<float> qf((size_t)M * d);
    const float nanv = std::nanf("");
    x->last_M = M;
    x->last_cos_attn.assign((size_t)L * M, nanv);
    x->last_cos_mlp.assign((size_t)L * M, nanv);

    // R1: the residual stream starts as the embedding row, widened exactly
    for (int m = 0; m < M; ++m)
        for (int i = 0; i < d; ++i) h[(size_t)m * d + i] = bf16_bits_to_float(x->w.embed[(size_t)tokens[m] * d + i]);

    for (int l = 0; l < L; ++l) {
        // ------------------------------------------------ attention sublayer
        if (!(use_mask && x->skip_attn[l])) {
            rmsnorm_rows(x, h.data(), M, x->w.attn_norm + (size_t)l * d, hn.data());
            matvec_rows(x->w.wq + (size_t)l * d * d, d, d, hn.data(), M, q.data());
            matvec_rows(x->w.wk + (size_t)l * kvd * d, kvd, d, hn.data(), M, kk.data());
            matvec_rows(x->w.wv + (size_t)l * kvd * d, kvd, d, hn.data(), M, vv.data());
            float* kc = x->kcache.data() + (size_t)l * c.max_seq * kvd;
            float* vc = x->vcache.data() + (size_t)l * c.max_seq * kvd;
            for (int m = 0; m < M; ++m) {
                const int p = pos0 + m;
                const float* rc = x->rope_cos.data() + (size_t)p * half;
                const float* rs = x->rope_sin.data() + (size_t)p * half;
                // R3: rotate q and k pairwise, then round; v is only rounded
                for (int hh = 0; hh < c.n_heads; ++hh)
                    for (int j = 0; j < half; ++j) {
                        const float a = (float)q[(size_t)m * d + hh * hd + j], b = (float)q[(size_t)m * d + hh * hd + j + half];
                        const float ra = (float)((double)a * rc[j] - (double)b * rs[j]);
                        const float rb = (float)((double)b * rc[j] + (double)a * rs[j]);
                        qf[(size_t)m * d + hh * hd + j] = x->round ? round_bf16(ra) : ra;
                        qf[(size_t)m * d + hh * hd + j + half] = x->round ? round_bf16(rb) : rb;
                    }
                for (int hh = 0; hh < c.n_kv_heads; ++hh)
                    for (int j = 0; j < half; ++j) {
                        const float a = (float)kk[(size_t)m * kvd + hh * hd + j], b = (float)kk[(size_t)m * kvd + hh * hd + j + half];
                        const float ra = (float)((double)a * rc[j] - (double)b * rs[j]);
                        const float rb = (float)((double)b * rc[j] + (double)a * rs[j]);
                        kc[(size_t)p * kvd + hh * hd + j] = x->round ? round_bf16(ra) : ra;
                        kc[(size_t)p * kvd + hh * hd + j + half] = x->round ? round_bf16(rb) : rb;
                    }
                for (int i = 0; i < kvd; ++i) {
                    const float v = (float)vv[(size_t)m * kvd + i];
                    vc[(size_t)p * kvd + i] = x->round ? round_bf16(v) : v;
                }
            }
            // R4: softmax(q.k / sqrt(hd)) over keys 0..p, times V
            const double inv_sqrt_hd = 1.0 / std::sqrt((double)hd);
#pragma omp parallel for collapse(2) schedule(static)
            for (int m = 0; m < M; ++m)
                for (int hh = 0; hh < c.n_heads; ++hh) {
                    const int p = pos0 + m, kvh = hh / group;
                    std::vector<double> s(p + 1);
                    double smax = -INFINITY;
                    for (int j = 0; j <= p; ++j) {
                        double acc = 0;
                        for (int e = 0; e < hd; ++e)
                            acc += (double)qf[(size_t)m * d + hh * hd + e] * (double)kc[(size_t)j * kvd + kvh * hd + e];
                        s[j] = acc * inv_sqrt_hd;
                        smax = std::max(smax, s[j]);
                    }
                    double denom = 0;
                    for (int j = 0; j <= p; ++j) {
                        s[j] = std::exp(s[j] - smax);
                        denom += s[j];
                    }
                    for (int e = 0; e < hd; ++e) {
                        double acc = 0;
                        for (int j = 0; j <= p; ++j) acc += s[j] * (double)vc[(size_t)j * kvd + kvh * hd + e];
                        const float a = (float)(acc / denom);
                        att[(size_t)m * d + hh * hd + e] = x->round ? round_bf16(a) : a;  // R5
                    }
                }
            matvec_rows(x->w.wo + (size_t)l * d * d, d, d, att.data(), M, o.data());
            for (int m = 0; m < M; ++m) {
                for (int i = 0; i < d; ++i) y[(size_t)m * d + i] = (float)((double)h[(size_t)m * d + i] + o[(size_t)m * d + i]);  // R6
                const double cs = orc_cosine(h.data() + (size_t)m * d, y.data() + (size_t)m * d, d);
                x->last_cos_attn[(size_t)l * M + m] = (float)cs;
                if (acc_sim) x->sumcos_attn[l] += cs;
            }
            h.swap(y);
        }
        // ------------------------------------------------ MLP sublayer
        if (!(use_mask && x->skip_mlp[l])) {
            rmsnorm_rows(x, h.data(), M, x->w.mlp_norm + (size_t)l * d, hn.data());
            matvec_rows(x->w.wg + (size_t)l * f * d, f, d, hn.data(), M, g.data());
            matvec_rows(x->w.wu + (size_t)l * f * d, f, d, hn.data(), M, u.data());
            for (size_t i = 0; i < (size_t)M * f; ++i) {  // R7: silu(g) * u
                const double gv = (double)(float)g[i], uv = (double)(float)u[i];
                const float tv = (float)(gv / (1.0 + std::exp(-gv)) * uv);
                t[i] = x->round ? round_bf16(tv) : tv;
            }
            matvec_rows(x->w.wd + (size_t)l * d * f, d, f, t.data(), M, o.data());
            for (int m = 0; m < M; ++m) {
                for (int i = 0; i < d; ++i) y[(size_t)m * d + i] = (float)((double)h[(size_t)m * d + i] + o[(size_t)m * d + i]);
                const double cs = orc_cosine(h.data() + (size_t)m * d, y.data() + (size_t)m * d, d);
                x->last_cos_mlp[(size_t)l * M + m] = (float)cs;
                if (acc_sim) x->sumcos_mlp[l] += cs;
            }
            h.swap(y);
        }
    }
    if (acc_sim) x->n_sim_rows += M;

    // R8: final norm, LM head, argmax (lowest index among equal maxima)
    rmsnorm_rows(x, h.data(), M, x->w.final_norm, hn.data());
    std::vector<double> lg((size_t)M * V);
    matvec_rows(x->w.lm_head, V, d, hn.data(), M, lg.data());
    x->last_logits.resize((size_t)M * V);
    x->last_argmax.resize(M);
    x->last_margin.resize(M);
    for (int m = 0; m < M; ++m) {
        int best = 0;
        float bestv = -INFINITY, second = -INFINITY;
        for (int v = 0; v < V; ++v) {
            const float z = (float)lg[(size_t)m * V + v];
            x->last_logits[(size_t)m * V + v] = z;
            if (z > bestv) {
                second = bestv;
                bestv = z;
                best = v;
            } else if (z > second) {
                second = z;
            }
        }
        x->last_argmax[m] = best;
        x->last_margin[m] = bestv - second;
    }
    return ORC_OK;
}

// Opt-in extension (the paper computes C_l over the prompt only): the first n rows of the last full-model pass,
// which the caller has just committed, join the mean.  C_l then is the mean over every committed row.
static void fold_committed_rows(orc_ctx* x, int n) {
    const int M = x->last_M;
    for (int l = 0; l < x->c.n_layers; ++l)
        for (int m = 0; m < n; ++m) {
            x->sumcos_attn[l] += (double)x->last_cos_attn[(size_t)l * M + m];
            x->sumcos_mlp[l] += (double)x->last_cos_mlp[(size_t)l * M + m];
        }
    x->n_sim_rows += n;
}

int orc_set_running_similarity(orc_ctx* x, int32_t on) {
    if (!x) return ORC_ERR_ARG;
    x->running_c = on != 0;
    return ORC_OK;
}

int orc_set_sampling(orc_ctx* x, float temperature, uint64_t seed) {
    if (!x || !(temperature >= 0.f)) return ORC_ERR_ARG;
    x->temperature = (double)temperature;
    x->seed = seed;
    return ORC_OK;
}

// The token that row m of the last pass chooses for position pos: M's (or D's) argmax when decoding greedily, else a
// draw of the given kind from softmax(logits / T).  dist, when given, receives that distribution.
static int32_t choose_token(orc_ctx* x, int m, int32_t pos, uint32_t kind, double* dist) {
    if (x->temperature <= 0.0) return x->last_argmax[m];
    const int V = x->c.vocab;
    std::vector<double> local;
    if (!dist) {
        local.resize(V);
        dist = local.data();
    }
    orc_softmax_t(x->last_logits.data() + (size_t)m * V, V, x->temperature, dist);
    return orc_sample_cdf(dist, V, orc_uniform(x->seed, (uint32_t)pos, kind));
}

// Section 3.2: the whole input context goes through M, fills the KV cache, yields t_1 and the
// per-layer similarity sums.  May be called repeatedly to feed the prompt in pieces.
int orc_prefill(orc_ctx* x, const int32_t* tokens, int32_t n, int32_t* first_token) {
    if (!x || !tokens || n <= 0) return ORC_ERR_ARG;
    const double t0 = now_ms();
    const int rc = forward_rows(x, tokens, n, x->n_committed, false, true);
    if (rc) return rc;
    x->n_committed += n;
    x->draft_cursor = x->n_committed;
    x->stats.prefill_rows += n;
    x->stats.ms_prefill += now_ms() - t0;
    x->drafted.clear();
    if (first_token) *first_token = choose_token(x, n - 1, x->n_committed, ORC_DRAW_TARGET, nullptr);
    return ORC_OK;
}

// C_l = (1/S) sum_s cos(X_s^l, Y_s^l), for the attention and the MLP sublayers
int orc_get_similarity(orc_ctx* x, float* c_attn, float* c_mlp, int32_t* n_rows) {
    if (!x) return ORC_ERR_ARG;
    if (n_rows) *n_rows = (int32_t)x->n_sim_rows;
    if (x->n_sim_rows == 0) return ORC_ERR_STATE;
    for (int l = 0; l < x->c.n_layers; ++l) {
        if (c_attn) c_attn[l] = (float)(x->sumcos_attn[l] / (double)x->n_sim_rows);
        if (c_mlp) c_mlp[l] = (float)(x->sumcos_mlp[l] / (double)x->n_sim_rows);
    }
    return ORC_OK;
}

int orc_set_skip_mask(orc_ctx* x, const uint8_t* skip_attn, const uint8_t* skip_mlp) {
    if (!x || !skip_attn || !skip_mlp) return ORC_ERR_ARG;
    for (int l = 0; l < x->c.n_layers; ++l) {
        x->skip_attn[l] = skip_attn[l] ? 1 : 0;
        x->skip_mlp[l] = skip_mlp[l] ? 1 : 0;
    }
    x->draft_cursor = x->n_committed;
    x->drafted.clear();
    return ORC_OK;
}

// Algorithm 1 on the attention similarities of the prompt; installs the result as the draft model's mask
int orc_admg_update(orc_ctx* x, const orc_admg_params* p, uint8_t* skip_attn, uint8_t* skip_mlp) {
    if (!x || !p) return ORC_ERR_ARG;
    std::vector<float> C(x->c.n_layers), Cm(x->c.n_layers);
    int rc = orc_get_similarity(x, C.data(), Cm.data(), nullptr);
    if (rc) return rc;
    std::vector<uint8_t> a(x->c.n_layers), b(x->c.n_layers);
    rc = orc_admg_ext(C.data(), Cm.data(), x->c.n_layers, p->alpha, p->alpha_mlp, p->m, p->n, p->flags, a.data(), b.data());
    if (rc) return rc;
    orc_set_skip_mask(x, a.data(), b.data());
    if (skip_attn) std::memcpy(skip_attn, a.data(), a.size());
    if (skip_mlp) std::memcpy(skip_mlp, b.data(), b.size());
    return ORC_OK;
}

// one autoregressive step of M: consumes token_in at the next position, commits it, returns the argmax
int orc_decode_step(orc_ctx* x, int32_t token_in, int32_t* token_out) {
    if (!x) return ORC_ERR_ARG;
    const double t0 = now_ms();
    const int rc = forward_rows(x, &token_in, 1, x->n_committed, false, false);
    if (rc) return rc;
    x->n_committed += 1;
    x->draft_cursor = x->n_committed;
    if (x->running_c) fold_committed_rows(x, 1);
    x->stats.full_passes += 1;
    x->stats.ms_full += now_ms() - t0;
    x->drafted.clear();
    if (token_out) *token_out = choose_token(x, 0, x->n_committed, ORC_DRAW_TARGET, nullptr);
    return ORC_OK;
}

// one step of the draft model D (M without the masked sublayers) at the draft cursor; commits nothing
int orc_draft_step(orc_ctx* x, int32_t token_in, int32_t* token_out) {
    if (!x) return ORC_ERR_ARG;
    const double t0 = now_ms();
    const int rc = forward_rows(x, &token_in, 1, x->draft_cursor, true, false);
    if (rc) return rc;
    x->draft_cursor += 1;
    x->stats.draft_passes += 1;
    x->stats.ms_draft += now_ms() - t0;
    // when sampling, the drafted token is a DRAFT draw from D's distribution q, which the verification needs again
    const size_t j = x->drafted.size(), V = x->c.vocab;
    int32_t tok;
    if (x->temperature > 0.0) {
        x->q_rows.resize((j + 1) * V);
        tok = choose_token(x, 0, x->draft_cursor, ORC_DRAW_DRAFT, x->q_rows.data() + j * V);
    } else {
        tok = x->last_argmax[0];
    }
    x->drafted.push_back(tok);
    if (token_out) *token_out = tok;
    return ORC_OK;
}

// Section 1: M processes [t_last, d_1..d_k] in parallel at positions n..n+k; d_{j+1} is accepted while it
// equals M's prediction g_j; the first rejected draft is replaced by M's token.  out_tokens receives the
// accepted drafts followed by g_a (a+1 tokens); a+1 positions are committed.
int orc_verify(orc_ctx* x, const int32_t* tokens, int32_t k, int32_t* n_accepted, int32_t* out_tokens) {
    if (!x || !tokens || k < 0) return ORC_ERR_ARG;
    const double t0 = now_ms();
    if (x->temperature > 0.0) {
        // the k tokens to verify must be the ones the last k draft steps sampled: their distributions q are needed
        if ((int32_t)x->drafted.size() != k) return ORC_ERR_STATE;
        for (int j = 0; j < k; ++j)
            if (x->drafted[j] != tokens[j + 1]) return ORC_ERR_STATE;
    }
    const int rc = forward_rows(x, tokens, k + 1, x->n_committed, false, false);
    if (rc) return rc;
    int a = 0;
    std::vector<int32_t> emitted(k + 1);
    if (x->temperature > 0.0) {
        const int V = x->c.vocab;
        std::vector<double> p((size_t)(k + 1) * V);
        for (int j = 0; j <= k; ++j) orc_softmax_t(x->last_logits.data() + (size_t)j * V, V, x->temperature, p.data() + (size_t)j * V);
        a = orc_spec_accept(p.data(), x->q_rows.data(), tokens + 1, k, V, x->seed, x->n_committed, emitted.data());
    } else {
        while (a < k && tokens[a + 1] == x->last_argmax[a]) ++a;
        for (int j = 0; j < a; ++j) emitted[j] = tokens[j + 1];
        emitted[a] = x->last_argmax[a];
    }
    x->drafted.clear();
    if (out_tokens)
        for (int j = 0; j <= a; ++j) out_tokens[j] = emitted[j];
    if (n_accepted) *n_accepted = a;
    x->n_committed += a + 1;
    x->draft_cursor = x->n_committed;
    if (x->running_c) fold_committed_rows(x, a + 1);
    x->stats.verify_passes += 1;
    x->stats.drafted += k;
    x->stats.accepted += a;
    x->stats.ms_verify += now_ms() - t0;
    return ORC_OK;
}

// Whole method: prefill -> t_1 -> (ADMG) -> repeat { k draft steps, verify } until max_new tokens.
// out receives max_new tokens, out[0] = t_1.  margins (optional) receives, for each emitted token, the
// top1-top2 logit gap of the full-model row that produced it.
int orc_generate(orc_ctx* x, const int32_t* prompt, int32_t n_prompt, const orc_gen_params* gp, int32_t* out,
                 int32_t* n_out, orc_stats* stats, float* margins) {
    if (!x || !prompt || n_prompt <= 0 || !gp || !out || !n_out || gp->max_new <= 0 || gp->draft_len < 0)
        return ORC_ERR_ARG;
    std::vector<uint8_t> ka = x->skip_attn, km = x->skip_mlp;
    orc_reset(x);
    if (gp->mode == ORC_MODE_SPEC_MANUAL_MASK) orc_set_skip_mask(x, ka.data(), km.data());
    x->running_c = (gp->admg.flags & ORC_RUNNING_C) != 0;
    if (!(gp->temperature >= 0.f)) return ORC_ERR_ARG;
    x->temperature = (double)gp->temperature;
    x->seed = gp->seed;
    const double t0 = now_ms();
    int32_t last;
    int rc = orc_prefill(x, prompt, n_prompt, &last);
    if (rc) return rc;
    int32_t produced = 0;
    auto emit = [&](int32_t tok, float margin) {
        if (produced < gp->max_new) {
            if (margins) margins[produced] = margin;
            out[produced++] = tok;
        }
    };
    emit(last, x->last_margin[n_prompt - 1]);
    bool stop = (gp->eos_id >= 0 && last == gp->eos_id);
    if (gp->mode == ORC_MODE_SPEC) {
        rc = orc_admg_update(x, &gp->admg, nullptr, nullptr);
        if (rc) return rc;
    }
    std::vector<int32_t> row(gp->draft_len + 1), acc(gp->draft_len + 1);
    while (produced < gp->max_new && !stop) {
        if (gp->mode == ORC_MODE_AR) {
            int32_t nxt;
            rc = orc_decode_step(x, last, &nxt);
            if (rc) return rc;
            emit(nxt, x->last_margin[0]);
            last = nxt;
            stop = (gp->eos_id >= 0 && nxt == gp->eos_id);
            continue;
        }
        int32_t k = std::min<int32_t>(gp->draft_len, gp->max_new - produced - 1);
        k = std::min<int32_t>(k, x->c.max_seq - x->n_committed - 1);
        if (k < 0) return ORC_ERR_OVERFLOW;
        row[0] = last;
        for (int j = 0; j < k; ++j) {
            rc = orc_draft_step(x, row[j], &row[j + 1]);
            if (rc) return rc;
            // draft exiting (fixed-threshold form of the mechanism Section 4 takes from Draft & Verify): the first draft
            // token whose top-2 logit gap in D is below the threshold ends the run; it is still verified
            if (gp->draft_exit_margin > 0.f && j + 1 < k && x->last_margin[0] < gp->draft_exit_margin) k = j + 1;
        }
        int32_t a = 0;
        rc = orc_verify(x, row.data(), k, &a, acc.data());
        if (rc) return rc;
        x->stats.rounds += 1;
        for (int j = 0; j <= a && !stop; ++j) {
            emit(acc[j], x->last_margin[j]);
            stop = (gp->eos_id >= 0 && acc[j] == gp->eos_id);
        }
        last = acc[a];
        // running similarities: Algorithm 1 is run again on the refreshed C_l every `refresh` rounds
        if (gp->mode == ORC_MODE_SPEC && x->running_c && gp->admg.refresh > 0 && x->stats.rounds % gp->admg.refresh == 0) {
            rc = orc_admg_update(x, &gp->admg, nullptr, nullptr);
            if (rc) return rc;
        }
    }
    *n_out = produced;
    x->stats.ms_total = now_ms() - t0;
    if (stats) *stats = x->stats;
    return ORC_OK;
}

int orc_get_stats(orc_ctx* x, orc_stats* s) {
    if (!x || !s) return ORC_ERR_ARG;
    *s = x->stats;
    return ORC_OK;
}

int orc_get_positions(orc_ctx* x, int32_t* n_committed, int32_t* draft_cursor) {
    if (!x) return ORC_ERR_ARG;
    if (n_committed) *n_committed = x->n_committed;
    if (draft_cursor) *draft_cursor = x->draft_cursor;
    return ORC_OK;
}

// per-row results of the last pass.  cos arrays are [L][M], NaN where the sublayer was skipped.
int orc_get_last(orc_ctx* x, int32_t* M, float* logits, float* cos_attn, float* cos_mlp, int32_t* argmax, float* margin) {
    if (!x || x->last_M == 0) return ORC_ERR_STATE;
    const int m = x->last_M;
    if (M) *M = m;
    if (logits) std::memcpy(logits, x->last_logits.data(), sizeof(float) * (size_t)m * x->c.vocab);
    if (cos_attn) std::memcpy(cos_attn, x->last_cos_attn.data(), sizeof(float) * (size_t)m * x->c.n_layers);
    if (cos_mlp) std::memcpy(cos_mlp, x->last_cos_mlp.data(), sizeof(float) * (size_t)m * x->c.n_layers);
    if (argmax) std::memcpy(argmax, x->last_argmax.data(), sizeof(int32_t) * m);
    if (margin) std::memcpy(margin, x->last_margin.data(), sizeof(float) * m);
    return ORC_OK;
}

// K and V rows of one layer at one position, as floats (tests of the cache logic)
int orc_get_kv(orc_ctx* x, int32_t layer, int32_t pos, float* k, float* v) {
    if (!x || layer < 0 || layer >= x->c.n_layers || pos < 0 || pos >= x->c.max_seq) return ORC_ERR_ARG;
    const size_t off = ((size_t)layer * x->c.max_seq + pos) * x->kv_dim;
    if (k) std::memcpy(k, x->kcache.data() + off, sizeof(float) * x->kv_dim);
    if (v) std::memcpy(v, x->vcache.data() + off, sizeof(float) * x->kv_dim);
    return ORC_OK;
}

// ---------------------------------------------------------------- single fused sublayer product
// The building block of every sublayer, for kernel-level comparisons:
//   xin = has_norm ? bf16(RMSNorm(x; gain, eps)) : x          x: [M, n_in] float
//   a   = W  xin                                              W: [n_out, n_in] bf16
//   epilogue 0 (plain)    : out[M, n_out] = float(a)
//   epilogue 1 (SwiGLU)   : b = W2 xin;  out = bf16(silu(float(a)) * float(b))
//   epilogue 2 (residual) : out = float(res + a);  cos[m] = cosine(res[m], out[m])
int orc_fused_matvec(const float* x, int32_t M, int32_t n_in, const uint16_t* gain, float eps, const uint16_t* W,
                     const uint16_t* W2, int32_t n_out, int32_t epilogue, const float* res, float* out, float* cosv) {
    if (!x || !W || !out || M <= 0 || n_in <= 0 || n_out <= 0) return ORC_ERR_ARG;
    std::vector<float> xin((size_t)M * n_in);
    if (gain) {
        for (int m = 0; m < M; ++m) {
            double ss = 0;
            for (int i = 0; i < n_in; ++i) ss += (double)x[(size_t)m * n_in + i] * (double)x[(size_t)m * n_in + i];
            const double inv = 1.0 / std::sqrt(ss / n_in + (double)eps);
            for (int i = 0; i < n_in; ++i)
                xin[(size_t)m * n_in + i] =
                    round_bf16((float)((double)x[(size_t)m * n_in + i] * inv * (double)bf16_bits_to_float(gain[i])));
        }
    } else {
        std::memcpy(xin.data(), x, sizeof(float) * xin.size());
    }
    std::vector<double> a((size_t)M * n_out), b;
    matvec_rows(W, n_out, n_in, xin.data(), M, a.data());
    if (epilogue == 0) {
        for (size_t i = 0; i < a.size(); ++i) out[i] = (float)a[i];
    } else if (epilogue == 1) {
        if (!W2) return ORC_ERR_ARG;
        b.resize(a.size());
        matvec_rows(W2, n_out, n_in, xin.data(), M, b.data());
        for (size_t i = 0; i < a.size(); ++i) {
            const double gv = (double)(float)a[i], uv = (double)(float)b[i];
            out[i] = round_bf16((float)(gv / (1.0 + std::exp(-gv)) * uv));
        }
    } else if (epilogue == 2) {
        if (!res) return ORC_ERR_ARG;
        for (int m = 0; m < M; ++m) {
            for (int i = 0; i < n_out; ++i) out[(size_t)m * n_out + i] = (float)((double)res[(size_t)m * n_out + i] + a[(size_t)m * n_out + i]);
            if (cosv) cosv[m] = (float)orc_cosine(res + (size_t)m * n_out, out + (size_t)m * n_out, n_out);
        }
    } else {
        return ORC_ERR_ARG;
    }
    return ORC_OK;
}

int orc_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"
