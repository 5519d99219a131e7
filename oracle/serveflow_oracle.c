/*
 * CPU oracle for the fast-slow serving path.  TEST INFRASTRUCTURE ONLY: it exists
 * so that the CUDA library can be checked against a plain, slow, independent
 * statement of what each stage computes.  Only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it; the serving library never does,
 * and the two share no code.
 *
 * Every function is the stage's definition evaluated flow by flow, with no
 * blocking, fusion or reordering.  The paper fixes the cascade (Sec. 3.1, Fig. 4:
 * every flow goes through the fast model, only uncertain ones go on to the slow
 * model, which sees more packets of the same flow), the least-confidence score
 * LC(x) = 1 - max_y P(y|x) and the entropy score (Sec. 3.2), and the threshold
 * rule of Algorithm 1.  It is silent on the concrete features and model shapes of
 * the synthetic stand-in workload; those readings are stated beside each function.
 *
 * Parity status: every function below is pinned by tests that do not re-use its
 * own formula (hand-computed values, closed forms, brute force, invariants).
 * sfo_sigmoid is a derived convenience output (closed-form pins: 0 -> 1/2, ln 3 -> 3/4,
 * symmetry); routing never uses it.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (no FMA
 * contraction, so every fp32 operation rounds once).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

/* ------------------------------------------------------------------------- */
/* Number formats                                                            */
/* ------------------------------------------------------------------------- */

/* Exact unsigned integer -> fp32, round to nearest, ties to even: the one
 * conversion every feature slot uses.  Keep the 24 leading bits, look at the
 * discarded remainder, round, scale back (the scaling is exact). */
float sfo_u128_to_f32(uint64_t hi, uint64_t lo)
{
    u128 v = ((u128)hi << 64) | lo;
    if (v == 0) return 0.0f;
    int len = 0;
    for (u128 t = v; t; t >>= 1) len++;
    if (len <= 24) return (float)(uint32_t)v;
    int s = len - 24;
    u128 q = v >> s;
    u128 rem = v - (q << s);
    u128 half = (u128)1 << (s - 1);
    if (rem > half || (rem == half && (q & 1))) q += 1;
    return ldexpf((float)(uint32_t)q, s);
}

static float u128f(u128 v) { return sfo_u128_to_f32((uint64_t)(v >> 64), (uint64_t)v); }

/* fp32 -> bfloat16 (1 sign, 8 exponent, 7 fraction bits = the upper half of an
 * fp32), round to nearest even, returned as the fp32 holding that value.  Inputs
 * here are always finite. */
float sfo_bf16_round(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    uint32_t low = u & 0xFFFFu;
    uint32_t up = u >> 16;
    if (low > 0x8000u || (low == 0x8000u && (up & 1u))) up += 1;
    u = up << 16;
    memcpy(&x, &u, 4);
    return x;
}

/* ------------------------------------------------------------------------- */
/* S1: statistical features of the first N packets                           */
/* ------------------------------------------------------------------------- */
/* Reading (the paper's pipeline has a "feature computation" step, Fig. 1, but
 * its features are nPrint bits; the stand-in workload asks for count, sum, min,
 * max, mean, variance of sizes and inter-arrival times plus direction counts,
 * from integer sums with one fixed fp32 division order):
 *   feature 8g+k, group g = (quantity, subset):
 *     g0 size/all  g1 iat/all  g2 size/fwd  g3 size/bwd  g4 iat/fwd  g5 iat/bwd
 *     g6 size/turn g7 iat/turn          (fwd: dir bit 0, bwd: dir bit 1,
 *     turn: packets i >= 1 whose direction differs from packet i-1)
 *   slot k: 0 cnt, 1 sum, 2 min, 3 max, 4 mean, 5 var, 6 first, 7 last.
 *   Window: packets 0..m-1, m = min(N, n_valid[f]).
 *   cnt, sum S1, sum of squares S2, min, max, first, last are exact integers;
 *   each is converted to fp32 once (RNE).  mean = fp32(S1) / fp32(cnt).
 *   var = fp32(V) / fp32(cnt*cnt) with V = cnt*S2 - S1*S1 exact (population
 *   variance).  An empty subset gives eight zeros.
 */
static int in_subset(uint32_t g, uint32_t i, const uint32_t* dirw)
{
    uint32_t d = (dirw[i >> 5] >> (i & 31)) & 1u;
    switch (g) {
    case 0: case 1: return 1;
    case 2: case 4: return d == 0;
    case 3: case 5: return d == 1;
    default: {
        if (i == 0) return 0;
        uint32_t p = (dirw[(i - 1) >> 5] >> ((i - 1) & 31)) & 1u;
        return d != p;
    }
    }
}

void sfo_extract_features(const uint16_t* size, const uint32_t* iat_us, const uint32_t* dir_bits,
                          const uint8_t* n_valid, uint64_t n, uint32_t pitch, uint32_t N, uint32_t F,
                          float* feat)
{
    uint32_t words = (pitch + 31) / 32;
    uint32_t G = F / 8;
    for (uint64_t f = 0; f < n; f++) {
        uint32_t m = N;
        if (n_valid && n_valid[f] < m) m = n_valid[f];
        const uint32_t* dw = dir_bits + f * words;
        for (uint32_t g = 0; g < G; g++) {
            int use_size = (g == 0 || g == 2 || g == 3 || g == 6);
            uint32_t cnt = 0, mn = 0, mx = 0, first = 0, last = 0;
            u128 s1 = 0, s2 = 0;
            for (uint32_t i = 0; i < m; i++) {
                if (!in_subset(g, i, dw)) continue;
                uint32_t x = use_size ? (uint32_t)size[f * pitch + i] : iat_us[f * pitch + i];
                if (cnt == 0) { mn = x; mx = x; first = x; }
                if (x < mn) mn = x;
                if (x > mx) mx = x;
                last = x;
                s1 += x;
                s2 += (u128)x * x;
                cnt++;
            }
            float* o = feat + f * F + 8 * g;
            if (cnt == 0) { for (int k = 0; k < 8; k++) o[k] = 0.0f; continue; }
            u128 V = (u128)cnt * s2 - s1 * s1;
            float fc = u128f(cnt);
            float fs = u128f(s1);
            o[0] = fc;
            o[1] = fs;
            o[2] = u128f(mn);
            o[3] = u128f(mx);
            o[4] = fs / fc;
            o[5] = u128f(V) / u128f((u128)cnt * cnt);
            o[6] = u128f(first);
            o[7] = u128f(last);
        }
    }
}

/* First-packet header-bit features (Sec. 4.1, Sec. 4.4: 1024 header bits per packet from the
 * IPv4, TCP and UDP headers, with a subscription to a subset of the columns).
 * Reading (the bit layout is re-derived from the header sizes, not taken from any tool): a
 * packet row holds 128 bytes = IPv4 header bytes 0..59, TCP header bytes 0..59, UDP header
 * bytes 0..7; column i of the 1024 is bit (7 - i%8) of byte i/8 (network bit order).  A column
 * whose byte lies at or beyond the number of bytes present in its section (sec_len[3]: a
 * 20-byte IPv4 header has no option bytes, a UDP packet has no TCP section) is -1; otherwise
 * it is 0 or 1.  Only the subscribed columns are written: out[f][j] = column sub[j]. */
void sfo_header_bits(const uint8_t* bytes, const uint8_t* sec_len, uint64_t n, const uint16_t* sub, uint32_t m,
                     float* out)
{
    static const uint32_t sec_start[3] = {0, 60, 120};
    for (uint64_t f = 0; f < n; f++)
        for (uint32_t j = 0; j < m; j++) {
            uint32_t col = sub[j], byte = col / 8, bit = 7 - col % 8;
            uint32_t sec = byte < 60 ? 0 : (byte < 120 ? 1 : 2);
            if (byte - sec_start[sec] >= sec_len[f * 3 + sec]) out[f * m + j] = -1.0f;
            else out[f * m + j] = (float)((bytes[f * 128 + byte] >> bit) & 1u);
        }
}

/* ------------------------------------------------------------------------- */
/* S2: tree ensembles                                                        */
/* ------------------------------------------------------------------------- */
/* Reading: complete binary trees of depth d in heap order (children of node i
 * are 2i+1 and 2i+2); at a node go LEFT iff x[fid] <= thr; the leaf index is the
 * final heap position minus (2^d - 1). */
static uint32_t walk(const float* x, const uint16_t* fid, const float* thr, uint32_t depth)
{
    uint32_t i = 0;
    for (uint32_t l = 0; l < depth; l++)
        i = (x[fid[i]] <= thr[i]) ? 2 * i + 1 : 2 * i + 2;
    return i - ((1u << depth) - 1u);
}

/* Random forest with soft voting: class probabilities are the mean over trees of
 * the leaves' class vectors, summed in tree order t = 0..T-1 in fp32 starting
 * from 0, then one division by fp32(T). */
void sfo_forest_rf(const float* feat, uint64_t n, uint32_t F, uint32_t T, uint32_t depth, uint32_t C,
                   const uint16_t* fid, const float* thr, const float* leaf,
                   float* prob, uint16_t* leaf_idx)
{
    uint32_t n_int = (1u << depth) - 1u, n_leaf = 1u << depth;
    float* acc = (float*)malloc(sizeof(float) * C);
    for (uint64_t f = 0; f < n; f++) {
        const float* x = feat + f * F;
        for (uint32_t c = 0; c < C; c++) acc[c] = 0.0f;
        for (uint32_t t = 0; t < T; t++) {
            uint32_t l = walk(x, fid + (uint64_t)t * n_int, thr + (uint64_t)t * n_int, depth);
            if (leaf_idx) leaf_idx[f * T + t] = (uint16_t)l;
            const float* lv = leaf + ((uint64_t)t * n_leaf + l) * C;
            for (uint32_t c = 0; c < C; c++) acc[c] = acc[c] + lv[c];
        }
        for (uint32_t c = 0; c < C; c++) prob[f * C + c] = acc[c] / (float)T;
    }
    free(acc);
}

/* Boosted trees, binary logistic: margin = 0 + sum of leaf scalars in tree order
 * (fp32).  The class-1 probability is sigmoid(margin); decisions use the margin. */
void sfo_forest_gbdt(const float* feat, uint64_t n, uint32_t F, uint32_t T, uint32_t depth,
                     const uint16_t* fid, const float* thr, const float* leaf,
                     float* margin, uint16_t* leaf_idx)
{
    uint32_t n_int = (1u << depth) - 1u, n_leaf = 1u << depth;
    for (uint64_t f = 0; f < n; f++) {
        const float* x = feat + f * F;
        float acc = 0.0f;
        for (uint32_t t = 0; t < T; t++) {
            uint32_t l = walk(x, fid + (uint64_t)t * n_int, thr + (uint64_t)t * n_int, depth);
            if (leaf_idx) leaf_idx[f * T + t] = (uint16_t)l;
            acc = acc + leaf[(uint64_t)t * n_leaf + l];
        }
        margin[f] = acc;
    }
}

double sfo_sigmoid(double margin) { return 1.0 / (1.0 + exp(-margin)); }

/* Boosted trees, multi-class (the layout of the gradient-boosting libraries the paper names in
 * Sec. 4.4): one tree per class and boosting round, tree t belongs to class t mod C;
 * margin[c] = 0 + sum of the leaf scalars of class c's trees in tree order (fp32).  The class
 * probabilities are softmax(margin); the label is the largest margin (lowest index on ties). */
void sfo_forest_gbdt_mc(const float* feat, uint64_t n, uint32_t F, uint32_t T, uint32_t depth, uint32_t C,
                        const uint16_t* fid, const float* thr, const float* leaf,
                        float* margin, uint16_t* leaf_idx)
{
    uint32_t n_int = (1u << depth) - 1u, n_leaf = 1u << depth;
    for (uint64_t f = 0; f < n; f++) {
        const float* x = feat + f * F;
        float* m = margin + f * C;
        for (uint32_t c = 0; c < C; c++) m[c] = 0.0f;
        for (uint32_t t = 0; t < T; t++) {
            uint32_t l = walk(x, fid + (uint64_t)t * n_int, thr + (uint64_t)t * n_int, depth);
            if (leaf_idx) leaf_idx[f * T + t] = (uint16_t)l;
            m[t % C] = m[t % C] + leaf[(uint64_t)t * n_leaf + l];
        }
    }
}

/* ------------------------------------------------------------------------- */
/* S3: uncertainty, threshold, assignment                                    */
/* ------------------------------------------------------------------------- */
/* Least confidence, Sec. 3.2: LC(x) = 1 - max_y P(y|x), one fp32 subtraction. */
float sfo_least_confidence(const float* p, uint32_t C)
{
    float mx = p[0];
    for (uint32_t c = 1; c < C; c++) if (p[c] > mx) mx = p[c];
    return 1.0f - mx;
}

/* Entropy, Sec. 3.2: H(x) = - sum_i P(y_i|x) log P(y_i|x) (natural log; terms
 * with P = 0 contribute 0). */
double sfo_entropy(const float* p, uint32_t C)
{
    double h = 0.0;
    for (uint32_t c = 0; c < C; c++) if (p[c] > 0.0f) h -= (double)p[c] * log((double)p[c]);
    return h;
}

/* Forest rule: label = argmax (lowest index on ties), score u = LC, a flow is
 * assigned to the slow model iff u > tau[label] (strict).  Assigned flow ids are
 * listed in ascending order.  Returns the number assigned (the list is written
 * up to `capacity` entries). */
uint64_t sfo_route_lc(const float* prob, uint64_t n, uint32_t C, const float* tau,
                      float* score, uint8_t* label, uint8_t* decision,
                      uint32_t* esc_ids, uint64_t capacity)
{
    uint64_t k = 0;
    for (uint64_t f = 0; f < n; f++) {
        const float* p = prob + f * C;
        uint32_t a = 0;
        for (uint32_t c = 1; c < C; c++) if (p[c] > p[a]) a = c;
        float u = sfo_least_confidence(p, C);
        int esc = u > tau[a];
        if (score) score[f] = u;
        if (label) label[f] = (uint8_t)a;
        if (decision) decision[f] = (uint8_t)esc;
        if (esc) { if (esc_ids && k < capacity) esc_ids[k] = (uint32_t)f; k++; }
    }
    return k;
}

/* Entropy rule (Sec. 3.2): score H(x) = -sum_i P(y_i|x) log P(y_i|x), evaluated in double and
 * stored as fp32; label = argmax; assigned iff H > tau[label] (strict). */
uint64_t sfo_route_entropy(const float* prob, uint64_t n, uint32_t C, const float* tau,
                           float* score, uint8_t* label, uint8_t* decision,
                           uint32_t* esc_ids, uint64_t capacity)
{
    uint64_t k = 0;
    for (uint64_t f = 0; f < n; f++) {
        const float* p = prob + f * C;
        uint32_t a = 0;
        for (uint32_t c = 1; c < C; c++) if (p[c] > p[a]) a = c;
        float h = (float)sfo_entropy(p, C);
        int esc = h > tau[a];
        if (score) score[f] = h;
        if (label) label[f] = (uint8_t)a;
        if (decision) decision[f] = (uint8_t)esc;
        if (esc) { if (esc_ids && k < capacity) esc_ids[k] = (uint32_t)f; k++; }
    }
    return k;
}

/* Least confidence of a softmax over margins (Sec. 3.2 applied to a multi-class boosted model):
 * LC = 1 - max_c softmax(m)_c = 1 - 1 / sum_j exp(m_j - m_max), in double precision. */
double sfo_softmax_lc(const float* m, uint32_t C)
{
    float mx = m[0];
    for (uint32_t c = 1; c < C; c++) if (m[c] > mx) mx = m[c];
    double s = 0.0;
    for (uint32_t c = 0; c < C; c++) s += exp((double)m[c] - (double)mx);
    return 1.0 - 1.0 / s;
}

uint64_t sfo_route_softmax_lc(const float* margin, uint64_t n, uint32_t C, const float* tau,
                              float* score, uint8_t* label, uint8_t* decision,
                              uint32_t* esc_ids, uint64_t capacity)
{
    uint64_t k = 0;
    for (uint64_t f = 0; f < n; f++) {
        const float* m = margin + f * C;
        uint32_t a = 0;
        for (uint32_t c = 1; c < C; c++) if (m[c] > m[a]) a = c;
        float u = (float)sfo_softmax_lc(m, C);
        int esc = u > tau[a];
        if (score) score[f] = u;
        if (label) label[f] = (uint8_t)a;
        if (decision) decision[f] = (uint8_t)esc;
        if (esc) { if (esc_ids && k < capacity) esc_ids[k] = (uint32_t)f; k++; }
    }
    return k;
}

/* Binary boosted rule, taken in margin space: |p - 0.5| < 0.2 with p =
 * sigmoid(margin) is the same set as |margin| < ln(0.7/0.3) because the sigmoid
 * is monotone and odd about (0, 0.5).  score = |margin|, label = margin > 0,
 * assigned iff score < tau_m (strict). */
uint64_t sfo_route_absmargin(const float* margin, uint64_t n, float tau_m,
                             float* score, uint8_t* label, uint8_t* decision,
                             uint32_t* esc_ids, uint64_t capacity)
{
    uint64_t k = 0;
    for (uint64_t f = 0; f < n; f++) {
        float m = fabsf(margin[f]);
        int esc = m < tau_m;
        if (score) score[f] = m;
        if (label) label[f] = (uint8_t)(margin[f] > 0.0f);
        if (decision) decision[f] = (uint8_t)esc;
        if (esc) { if (esc_ids && k < capacity) esc_ids[k] = (uint32_t)f; k++; }
    }
    return k;
}

/* Algorithm 1 (universal uncertainty thresholds): sort the validation scores in
 * ascending order; for a quantile q the index is ceil(q * len(U)) and the
 * threshold is U[index].  Reading: the index is 1-based (U = {.1,.2,.3,.4},
 * q = .5 gives .2, so that the share of scores above the threshold is 1 - q);
 * q is the rational q_num/q_den so the ceiling is taken in integers. */
static int cmp_float(const void* a, const void* b)
{
    float x = *(const float*)a, y = *(const float*)b;
    return (x > y) - (x < y);
}

void sfo_universal_thresholds(const float* U, uint64_t len, const uint32_t* q_num, uint32_t q_den,
                              uint32_t n_q, float* T_out)
{
    float* s = (float*)malloc(sizeof(float) * (len ? len : 1));
    memcpy(s, U, sizeof(float) * len);
    qsort(s, len, sizeof(float), cmp_float);
    for (uint32_t j = 0; j < n_q; j++) {
        uint64_t idx = ((uint64_t)q_num[j] * len + q_den - 1) / q_den;   /* ceil */
        if (idx < 1) idx = 1;
        if (idx > len) idx = len;
        T_out[j] = s[idx - 1];
    }
    free(s);
}

/* Wide rows of the assigned flows (input of the slow model).
 * Reading: per packet 16 fields (layout 0, P x 16, packet-major):
 *   0: size * 2^-11   1: L(iat) * 2^-7   2: direction as 0/1   3..15: header byte * 2^-8
 * or 8 channels (layout 1, [position][channel]): size, L(iat), dir, header bytes 0..4.
 * L is an integer piecewise-linear log2: v = iat + 1, e = floor(log2 v), the two
 * bits below the leading one give the fraction: L = 4e + (bits), in [0, 128].
 * Packets at or beyond n_valid (or beyond P_real) are zero.  With to_bf16 the
 * values are rounded to bfloat16 (and returned as fp32). */
uint32_t sfo_ilog(uint32_t a)
{
    uint64_t v = (uint64_t)a + 1;
    uint32_t e = 0;
    while ((v >> (e + 1)) != 0) e++;
    uint64_t two = (e >= 2) ? (v >> (e - 2)) : (v << (2 - e));
    return 4 * e + (uint32_t)(two & 3);
}

void sfo_wide_rows(int layout, const uint32_t* esc_ids, uint64_t n_esc,
                   const uint16_t* size, const uint32_t* iat_us, const uint32_t* dir_bits,
                   const uint8_t* hdr, const uint8_t* n_valid, uint32_t pitch, uint32_t hdr_bytes,
                   uint32_t P, uint32_t P_real, int to_bf16, float* rows)
{
    uint32_t words = (pitch + 31) / 32;
    uint32_t W = layout == 0 ? 16 : 8;
    uint32_t nh = layout == 0 ? 13 : 5;
    for (uint64_t r = 0; r < n_esc; r++) {
        uint64_t f = esc_ids[r];
        uint32_t m = P_real;
        if (n_valid && n_valid[f] < m) m = n_valid[f];
        float* o = rows + r * (uint64_t)P * W;
        for (uint32_t i = 0; i < P; i++) {
            float* q = o + (uint64_t)i * W;
            if (i >= m) { for (uint32_t k = 0; k < W; k++) q[k] = 0.0f; continue; }
            q[0] = (float)size[f * pitch + i] * 0x1p-11f;
            q[1] = (float)sfo_ilog(iat_us[f * pitch + i]) * 0x1p-7f;
            q[2] = (float)((dir_bits[f * words + (i >> 5)] >> (i & 31)) & 1u);
            for (uint32_t k = 0; k < nh; k++)
                q[3 + k] = (float)hdr[(f * pitch + i) * hdr_bytes + k] * 0x1p-8f;
            if (to_bf16) for (uint32_t k = 0; k < W; k++) q[k] = sfo_bf16_round(q[k]);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* S4: slow models                                                           */
/* ------------------------------------------------------------------------- */
/* Multi-layer perceptron: h0 = row; h_{k+1} = ReLU(W_k h_k + b_k); logits =
 * W_L h_L + b_L; label = argmax (lowest index on ties).  Sums in double.  In bf16
 * mode the weights are rounded to bf16 once and every hidden activation is
 * rounded to bf16 after the ReLU; biases and logits stay fp32. */
void sfo_mlp(const float* rows, uint64_t n_rows, uint32_t n_layers, const uint32_t* dims,
             const float* const* W, const float* const* b, int bf16,
             float* logits, uint8_t* label)
{
    uint32_t maxd = 0;
    for (uint32_t l = 0; l <= n_layers; l++) if (dims[l] > maxd) maxd = dims[l];
    float** Wr = (float**)malloc(sizeof(float*) * n_layers);
    for (uint32_t l = 0; l < n_layers; l++) {
        uint64_t cnt = (uint64_t)dims[l] * dims[l + 1];
        Wr[l] = (float*)malloc(sizeof(float) * cnt);
        for (uint64_t i = 0; i < cnt; i++) Wr[l][i] = bf16 ? sfo_bf16_round(W[l][i]) : W[l][i];
    }
    float* h = (float*)malloc(sizeof(float) * maxd);
    float* g = (float*)malloc(sizeof(float) * maxd);
    for (uint64_t r = 0; r < n_rows; r++) {
        for (uint32_t k = 0; k < dims[0]; k++) h[k] = bf16 ? sfo_bf16_round(rows[r * dims[0] + k]) : rows[r * dims[0] + k];
        for (uint32_t l = 0; l < n_layers; l++) {
            uint32_t K = dims[l], O = dims[l + 1];
            for (uint32_t o = 0; o < O; o++) {
                double acc = 0.0;
                for (uint32_t k = 0; k < K; k++) acc += (double)Wr[l][(uint64_t)o * K + k] * (double)h[k];
                float v = (float)(acc + (double)b[l][o]);
                if (l + 1 < n_layers) {
                    if (v < 0.0f) v = 0.0f;
                    if (bf16) v = sfo_bf16_round(v);
                }
                g[o] = v;
            }
            float* t = h; h = g; g = t;
        }
        uint32_t Cn = dims[n_layers], a = 0;
        for (uint32_t c = 0; c < Cn; c++) {
            logits[r * Cn + c] = h[c];
            if (h[c] > h[a]) a = c;
        }
        if (label) label[r] = (uint8_t)a;
    }
    for (uint32_t l = 0; l < n_layers; l++) free(Wr[l]);
    free(Wr); free(h); free(g);
}

/* 1-D CNN over a sequence of L positions x Cin channels (channels last):
 * conv(k, Cin->C1) + bias + ReLU, conv(k, C1->C2) + bias + ReLU, mean over the L
 * positions, linear C2 -> n_cls + bias.  Reading (the paper lists convolution,
 * pooling and fully connected layers without shapes): stride 1, zero padding of
 * (k-1)/2 on both sides so the length stays L; activations rounded to bf16 in
 * bf16 mode; the pooled mean and the logits are not rounded.
 * w1[C1][k][Cin], w2[C2][k][C1], w3[n_cls][C2]. */
void sfo_cnn(const float* rows, uint64_t n_rows, uint32_t L, uint32_t Cin, uint32_t C1, uint32_t C2,
             uint32_t k, uint32_t n_cls, const float* w1, const float* b1, const float* w2,
             const float* b2, const float* w3, const float* b3, int bf16,
             float* logits, uint8_t* label)
{
    int pad = (int)(k - 1) / 2;
    uint64_t n1 = (uint64_t)C1 * k * Cin, n2 = (uint64_t)C2 * k * C1, n3 = (uint64_t)n_cls * C2;
    float* v1 = (float*)malloc(sizeof(float) * n1);
    float* v2 = (float*)malloc(sizeof(float) * n2);
    float* v3 = (float*)malloc(sizeof(float) * n3);
    for (uint64_t i = 0; i < n1; i++) v1[i] = bf16 ? sfo_bf16_round(w1[i]) : w1[i];
    for (uint64_t i = 0; i < n2; i++) v2[i] = bf16 ? sfo_bf16_round(w2[i]) : w2[i];
    for (uint64_t i = 0; i < n3; i++) v3[i] = bf16 ? sfo_bf16_round(w3[i]) : w3[i];
    float* h1 = (float*)malloc(sizeof(float) * L * C1);
    float* h2 = (float*)malloc(sizeof(float) * L * C2);
    double* pool = (double*)malloc(sizeof(double) * C2);
    for (uint64_t r = 0; r < n_rows; r++) {
        const float* x = rows + r * (uint64_t)L * Cin;
        for (uint32_t p = 0; p < L; p++)
            for (uint32_t o = 0; o < C1; o++) {
                double acc = 0.0;
                for (uint32_t t = 0; t < k; t++) {
                    int q = (int)p + (int)t - pad;
                    if (q < 0 || q >= (int)L) continue;
                    for (uint32_t c = 0; c < Cin; c++)
                        acc += (double)v1[((uint64_t)o * k + t) * Cin + c] * (double)x[(uint64_t)q * Cin + c];
                }
                float v = (float)(acc + (double)b1[o]);
                if (v < 0.0f) v = 0.0f;
                h1[(uint64_t)p * C1 + o] = bf16 ? sfo_bf16_round(v) : v;
            }
        for (uint32_t p = 0; p < L; p++)
            for (uint32_t o = 0; o < C2; o++) {
                double acc = 0.0;
                for (uint32_t t = 0; t < k; t++) {
                    int q = (int)p + (int)t - pad;
                    if (q < 0 || q >= (int)L) continue;
                    for (uint32_t c = 0; c < C1; c++)
                        acc += (double)v2[((uint64_t)o * k + t) * C1 + c] * (double)h1[(uint64_t)q * C1 + c];
                }
                float v = (float)(acc + (double)b2[o]);
                if (v < 0.0f) v = 0.0f;
                h2[(uint64_t)p * C2 + o] = bf16 ? sfo_bf16_round(v) : v;
            }
        for (uint32_t o = 0; o < C2; o++) {
            double s = 0.0;
            for (uint32_t p = 0; p < L; p++) s += (double)h2[(uint64_t)p * C2 + o];
            pool[o] = s / (double)L;
        }
        uint32_t a = 0;
        for (uint32_t c = 0; c < n_cls; c++) {
            double acc = 0.0;
            for (uint32_t o = 0; o < C2; o++) acc += (double)v3[(uint64_t)c * C2 + o] * pool[o];
            logits[r * n_cls + c] = (float)(acc + (double)b3[c]);
            if (logits[r * n_cls + c] > logits[r * n_cls + a]) a = c;
        }
        if (label) label[r] = (uint8_t)a;
    }
    free(v1); free(v2); free(v3); free(h1); free(h2); free(pool);
}

/* ------------------------------------------------------------------------- */
/* S5: merge                                                                 */
/* ------------------------------------------------------------------------- */
/* The slow model's answer replaces the fast one for assigned flows; all other
 * flows keep the fast answer (Sec. 3.1).  stage = 1 (fast) or 2 (slow). */
void sfo_merge(const uint8_t* label_fast, uint64_t n, const uint32_t* esc_ids, uint64_t n_esc,
               const uint8_t* label_slow, uint8_t* label, uint8_t* stage)
{
    for (uint64_t f = 0; f < n; f++) { label[f] = label_fast[f]; stage[f] = 1; }
    for (uint64_t r = 0; r < n_esc; r++) { label[esc_ids[r]] = label_slow[r]; stage[esc_ids[r]] = 2; }
}
