/*
 * CPU oracle for the batch-1 Llama-family decode step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of what the
 * decode path computes.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the CUDA library never does, and the two share no code.
 *
 * What it follows: the paper defines the model by reference only (a bias-free, full-rotary,
 * SiLU-SwiGLU, RMSNorm, grouped-query-attention Llama-family decoder, Sections 1 and 7
 * "Architecture coverage"), one launch = one forward pass = one decoded token with the KV cache
 * persisting between steps ("Synchronization model", Section 4), and weight-only int8 / int4 variants
 * whose dequantisation is folded into the matrix-vector products while embeddings, scales and all
 * non-GEMV buffers keep their 16-bit types ("Quantized generation", Section 5).  Where the paper is
 * silent the reading taken is stated next to each function.
 *
 * Arithmetic: activations are stored as fp32; every dot product, sum of squares and softmax sum is
 * accumulated in fp64; the KV cache holds bf16 (round to nearest even at append) and attention reads
 * the rounded entries, including the one appended in the same step.
 * Variants beyond the paper's text, each the same step with one storage type changed: grouped int8
 * weights (wdtype 3: the int8 rule per row and group of columns; Section 7 mentions dequantising "per
 * group") and an fp8 e4m3 KV cache (kv_dtype 1: entries rounded to nearest even, saturating at +-448).
 *
 * Parity pins (tests/test_oracle_*.py): RMSNorm closed forms; RoPE pair-norm preservation, the pos=0
 * identity and hand values; softmax rows summing to one; attention at pos 0 returning the cached V;
 * split-K combine equal to the unsplit result; exact-integer GEMVs; integer pack/unpack round trips and
 * hand-worked quantiser rows (per row and per group); the e4m3 conversions against torch's float8_e4m3fn
 * (all codes, all midpoints, saturation); a second, dense, cache-free recomputation of a 2-layer
 * hidden-64 toy (also with every quantised weight type and with the fp8 cache); a library cross-check
 * against a random-init transformers LlamaForCausalLM.
 * Parity unpinned: whether an *untied* LM head stays bf16 in the quantised variants is not fixed by the
 * paper; both readings are implemented (quantize_lm_head 0 / 1) and each is pinned against the dense form,
 * but which of the two the paper's kernels used cannot be pinned from its text.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ----------------------------------------------------------------------------------------------
 * 16-bit float formats (own conversion routines)
 * -------------------------------------------------------------------------------------------- */

static inline float bits_to_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static inline uint32_t f32_to_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

/* bf16 is the top half of an fp32 word: widening is exact. */
float orc_bf16_to_f32(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

/* fp32 -> bf16, round to nearest, ties to even.  NaN stays NaN. */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* IEEE binary16 -> fp32 (exact), subnormals included. */
float orc_f16_to_f32(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1fu;
    uint32_t man = h & 0x3ffu;
    if (exp == 0) {
        if (man == 0) return bits_to_f32(sign);
        float v = (float)man * (1.0f / 16777216.0f);      /* man * 2^-24, exact */
        return sign ? -v : v;
    }
    if (exp == 31) return bits_to_f32(sign | 0x7f800000u | (man << 13));
    return bits_to_f32(sign | ((exp + 112u) << 23) | (man << 13));
}

/* fp32 -> IEEE binary16, round to nearest, ties to even; overflow -> inf; subnormals kept. */
uint16_t orc_f32_to_f16(float f) {
    uint32_t u = f32_to_bits(f);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t a = u & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);          /* NaN */
    if (a >= 0x47800000u) return (uint16_t)(sign | 0x7c00u);         /* >= 65536 -> inf (65520 rounds up below) */
    if (a < 0x33000000u) return sign;                                /* < 2^-25 -> 0 */
    int e = (int)(a >> 23) - 127;                                    /* unbiased exponent */
    uint32_t m = (a & 0x7fffffu) | 0x800000u;                        /* 24-bit significand */
    int shift = (e < -14) ? (13 + (-14 - e)) : 13;                   /* bits dropped */
    uint32_t kept = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (kept & 1u))) kept++;
    uint32_t out;
    if (e < -14) out = kept;                                         /* subnormal (may carry into normal) */
    else out = ((uint32_t)(e + 15) << 10) + (kept - 0x400u);         /* carry propagates into exponent */
    if (out >= 0x7c00u) out = 0x7c00u;
    return (uint16_t)(sign | out);
}

/* ----------------------------------------------------------------------------------------------
 * Elementary pieces
 * -------------------------------------------------------------------------------------------- */

/* RMSNorm.  Reading (paper silent): a_i = x_i * g_i / sqrt(mean_j x_j^2 + eps); eps inside the root,
 * mean over all H entries, weight applied after normalisation. */
void orc_rmsnorm(const float* x, const uint16_t* g_bf16, int H, float eps, float* out) {
    double ss = 0.0;
    for (int i = 0; i < H; i++) ss += (double)x[i] * (double)x[i];
    double r = 1.0 / sqrt(ss / (double)H + (double)eps);
    for (int i = 0; i < H; i++) out[i] = (float)((double)x[i] * r * (double)orc_bf16_to_f32(g_bf16[i]));
}

/* Rotary embedding of one head at position pos, in place.  Reading (paper silent; it requires
 * token-for-token agreement with the HuggingFace Llama forward): half-split pairing (i, i + hd/2),
 * frequency theta^(-2i/hd) for pair i, no scaling, every dimension rotated. */
void orc_rope(float* u, int hd, int pos, double theta) {
    int half = hd / 2;
    for (int i = 0; i < half; i++) {
        double f = pow(theta, -2.0 * (double)i / (double)hd);
        double phi = (double)pos * f;
        double c = cos(phi), s = sin(phi);
        double a = u[i], b = u[i + half];
        u[i] = (float)(a * c - b * s);
        u[i + half] = (float)(b * c + a * s);
    }
}

/* SiLU: z * sigmoid(z). */
float orc_silu(float z) { return (float)((double)z / (1.0 + exp(-(double)z))); }

/* ----------------------------------------------------------------------------------------------
 * fp8 "e4m3" (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; the one NaN is
 * magnitude code 0x7f; largest finite value 448 = code 0x7e): the element type of the optional 8-bit KV
 * cache.  Narrowing is round-to-nearest-even with saturation: every finite value beyond 448 (and either
 * infinity) becomes +-448; NaN stays NaN.
 * -------------------------------------------------------------------------------------------- */
float orc_e4m3_to_f32(uint8_t code) {
    int e = (code >> 3) & 0xf, m = code & 7;
    double v;
    if (e == 0xf && m == 7) return (code & 0x80) ? -NAN : NAN;
    if (e == 0) v = ldexp((double)m, -9);                     /* subnormal: m/8 * 2^-6 */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (float)((code & 0x80) ? -v : v);
}

uint8_t orc_f32_to_e4m3(float x) {
    uint8_t sign = signbit(x) ? 0x80 : 0x00;
    double a = fabs((double)x);
    if (isnan(x)) return (uint8_t)(sign | 0x7f);
    if (a > 448.0) return (uint8_t)(sign | 0x7e);             /* saturate (464 and beyond would need code 0x7f) */
    if (a < ldexp(1.0, -6)) {                                 /* subnormal range: multiples of 2^-9; rint ties to even */
        int q = (int)rint(ldexp(a, 9));                       /* 0..8; 8 is the smallest normal, code 0x08 */
        return (uint8_t)(sign | q);
    }
    int ex;
    double f = frexp(a, &ex);                                 /* a = f * 2^ex, f in [0.5, 1) */
    int E = ex - 1;                                           /* a = (2f) * 2^E, 2f in [1, 2) */
    int m = (int)rint((2.0 * f - 1.0) * 8.0);                 /* 0..8, ties to even */
    if (m == 8) { m = 0; E += 1; }
    int code = ((E + 7) << 3) | m;
    if (code > 0x7e) code = 0x7e;
    return (uint8_t)(sign | code);
}

/* Index of the largest entry; the lowest index wins an exact tie. */
int orc_argmax(const float* v, int n) {
    int best = 0;
    for (int i = 1; i < n; i++) if (v[i] > v[best]) best = i;
    return best;
}

/* ----------------------------------------------------------------------------------------------
 * Weight formats and the matrix-vector product
 *   wdtype 0: bf16 [rows][cols]
 *   wdtype 1: int8 [rows][cols], symmetric, one fp16 scale per output row: w = s * q
 *   wdtype 2: int4 [rows][cols/2], element j in byte j/2 (even j: bits 0-3, odd j: bits 4-7),
 *             asymmetric, per row and group of `group` consecutive columns an fp16 scale and an
 *             integer-valued fp16 zero point: w = s * (q - z)
 *   wdtype 3: int8 [rows][cols], symmetric, per row and group of `group` consecutive columns an fp16
 *             scale: w = s * q  ("dequantize per group", Section 7)
 * The dequantised value is formed in fp32; both products are exact there (11-bit by <=8-bit
 * significands), so dequantised weights are comparable bit for bit.
 * -------------------------------------------------------------------------------------------- */

float orc_dequant(int wdtype, const void* W, const uint16_t* scale, const uint16_t* zero, int group,
                  int cols, int o, int j) {
    size_t idx = (size_t)o * (size_t)cols + (size_t)j;
    if (wdtype == 0) return orc_bf16_to_f32(((const uint16_t*)W)[idx]);
    if (wdtype == 1) return orc_f16_to_f32(scale[o]) * (float)((const int8_t*)W)[idx];
    if (wdtype == 3) {
        size_t gi = (size_t)o * (size_t)(cols / group) + (size_t)(j / group);
        return orc_f16_to_f32(scale[gi]) * (float)((const int8_t*)W)[idx];
    }
    {
        uint8_t byte = ((const uint8_t*)W)[idx >> 1];
        int q = (j & 1) ? (byte >> 4) : (byte & 0x0f);
        size_t gi = (size_t)o * (size_t)(cols / group) + (size_t)(j / group);
        float s = orc_f16_to_f32(scale[gi]);
        float z = orc_f16_to_f32(zero[gi]);
        return s * ((float)q - z);
    }
}

/* y[o] = sum_j deq(W[o][j]) * x[j], accumulated in fp64, for o in [0, rows). */
void orc_gemv(int wdtype, const void* W, const uint16_t* scale, const uint16_t* zero, int group,
              int rows, int cols, const float* x, float* y) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < rows; o++) {
        double acc = 0.0;
        if (wdtype == 0) {
            const uint16_t* w = (const uint16_t*)W + (size_t)o * cols;
            for (int j = 0; j < cols; j++) acc += (double)orc_bf16_to_f32(w[j]) * (double)x[j];
        } else if (wdtype == 1) {
            const int8_t* w = (const int8_t*)W + (size_t)o * cols;
            float s = orc_f16_to_f32(scale[o]);
            for (int j = 0; j < cols; j++) acc += (double)(s * (float)w[j]) * (double)x[j];
        } else {
            for (int j = 0; j < cols; j++)
                acc += (double)orc_dequant(wdtype, W, scale, zero, group, cols, o, j) * (double)x[j];
        }
        y[o] = (float)acc;
    }
}

/* ----------------------------------------------------------------------------------------------
 * Round-to-nearest weight quantisers (the paper's "naive round-to-nearest", Section 5).  Reading:
 * every step is an fp32 IEEE operation (division, rint under the default ties-to-even mode), the
 * scale is rounded to fp16 first and the integer codes are computed with the rounded scale.
 * -------------------------------------------------------------------------------------------- */

/* int8, symmetric, per output row: s = fp16(amax/127) (1 if the row is all zero);
 * q = clamp(rint(w / s), -127, 127). */
void orc_quantize_int8(const uint16_t* W_bf16, int rows, int cols, int8_t* q, uint16_t* scale) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < rows; o++) {
        const uint16_t* w = W_bf16 + (size_t)o * cols;
        float amax = 0.0f;
        for (int j = 0; j < cols; j++) { float a = fabsf(orc_bf16_to_f32(w[j])); if (a > amax) amax = a; }
        uint16_t sh = (amax == 0.0f) ? orc_f32_to_f16(1.0f) : orc_f32_to_f16(amax / 127.0f);
        float s = orc_f16_to_f32(sh);
        if (s == 0.0f) { sh = orc_f32_to_f16(1.0f); s = 1.0f; }
        scale[o] = sh;
        for (int j = 0; j < cols; j++) {
            float r = rintf(orc_bf16_to_f32(w[j]) / s);
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            q[(size_t)o * cols + j] = (int8_t)r;
        }
    }
}

/* int8, symmetric, per output row and group of `group` consecutive columns: the per-row rule applied to
 * each group: s = fp16(amax/127) (1 if the group is all zero); q = clamp(rint(w / s), -127, 127). */
void orc_quantize_int8_grouped(const uint16_t* W_bf16, int rows, int cols, int group, int8_t* q, uint16_t* scale) {
    int ng = cols / group;
#pragma omp parallel for schedule(static)
    for (int o = 0; o < rows; o++) {
        const uint16_t* w = W_bf16 + (size_t)o * cols;
        for (int g = 0; g < ng; g++) {
            float amax = 0.0f;
            for (int j = g * group; j < (g + 1) * group; j++) {
                float a = fabsf(orc_bf16_to_f32(w[j]));
                if (a > amax) amax = a;
            }
            uint16_t sh = (amax == 0.0f) ? orc_f32_to_f16(1.0f) : orc_f32_to_f16(amax / 127.0f);
            float s = orc_f16_to_f32(sh);
            if (s == 0.0f) { sh = orc_f32_to_f16(1.0f); s = 1.0f; }
            scale[(size_t)o * ng + g] = sh;
            for (int j = g * group; j < (g + 1) * group; j++) {
                float r = rintf(orc_bf16_to_f32(w[j]) / s);
                if (r > 127.0f) r = 127.0f;
                if (r < -127.0f) r = -127.0f;
                q[(size_t)o * cols + j] = (int8_t)r;
            }
        }
    }
}

/* int4, asymmetric, per row and group: mn = min(w, 0), mx = max(w, 0) (range always contains zero so
 * the zero point is a code), s = fp16((mx - mn)/15) (1 if mx == mn), z = clamp(rint(-mn / s), 0, 15),
 * q = clamp(rint(w / s) + z, 0, 15). */
void orc_quantize_int4(const uint16_t* W_bf16, int rows, int cols, int group, uint8_t* packed,
                       uint16_t* scale, uint16_t* zero) {
    int ng = cols / group;
#pragma omp parallel for schedule(static)
    for (int o = 0; o < rows; o++) {
        const uint16_t* w = W_bf16 + (size_t)o * cols;
        uint8_t* out = packed + (size_t)o * (cols / 2);
        for (int g = 0; g < ng; g++) {
            float mn = 0.0f, mx = 0.0f;
            for (int j = g * group; j < (g + 1) * group; j++) {
                float v = orc_bf16_to_f32(w[j]);
                if (v < mn) mn = v;
                if (v > mx) mx = v;
            }
            uint16_t sh = (mx == mn) ? orc_f32_to_f16(1.0f) : orc_f32_to_f16((mx - mn) / 15.0f);
            float s = orc_f16_to_f32(sh);
            if (s == 0.0f) { sh = orc_f32_to_f16(1.0f); s = 1.0f; }
            float z = rintf(-mn / s);
            if (!(z > 0.0f)) z = 0.0f;             /* also turns -0 (an all-positive group) into +0 */
            if (z > 15.0f) z = 15.0f;
            scale[(size_t)o * ng + g] = sh;
            zero[(size_t)o * ng + g] = orc_f32_to_f16(z);
            for (int j = g * group; j < (g + 1) * group; j++) {
                float r = rintf(orc_bf16_to_f32(w[j]) / s) + z;
                if (r < 0.0f) r = 0.0f;
                if (r > 15.0f) r = 15.0f;
                uint8_t code = (uint8_t)r;
                if (j & 1) out[j >> 1] = (uint8_t)((out[j >> 1] & 0x0f) | (code << 4));
                else       out[j >> 1] = (uint8_t)((out[j >> 1] & 0xf0) | code);
            }
        }
    }
}

/* ----------------------------------------------------------------------------------------------
 * Attention for one query head over cache positions [j0, j1)
 * -------------------------------------------------------------------------------------------- */

/* One cache element as fp32.  The cache is an array of 16-bit words whatever its element type: a bf16 bit
 * pattern (kv_dtype 0), or an e4m3 code in the low byte (kv_dtype 1). */
static float kv_to_f32(int kv_dtype, uint16_t word) {
    return kv_dtype == 1 ? orc_e4m3_to_f32((uint8_t)word) : orc_bf16_to_f32(word);
}

/* Plain softmax attention.  K, V: [n_pos][hd] rows of one kv head, bf16 (orc_attention_head) or of the given
 * cache element type (orc_attention_head_kv).  Reading (paper silent): scores scaled by 1/sqrt(hd), every
 * position j0 <= j < j1 attended, no other mask.
 * Optionally returns the softmax weights (w_out, length j1-j0, may be NULL). */
void orc_attention_head_kv(int kv_dtype, const float* q, const uint16_t* K, const uint16_t* V, int hd, int j0, int j1,
                           float* o, double* w_out);
void orc_attention_head(const float* q, const uint16_t* K, const uint16_t* V, int hd, int j0, int j1,
                        float* o, double* w_out) {
    orc_attention_head_kv(0, q, K, V, hd, j0, j1, o, w_out);
}
void orc_attention_head_kv(int kv_dtype, const float* q, const uint16_t* K, const uint16_t* V, int hd, int j0, int j1,
                           float* o, double* w_out) {
    int n = j1 - j0;
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    double inv = 1.0 / sqrt((double)hd);
    double M = -INFINITY;
    for (int j = j0; j < j1; j++) {
        double d = 0.0;
        for (int t = 0; t < hd; t++) d += (double)q[t] * (double)kv_to_f32(kv_dtype, K[(size_t)j * hd + t]);
        s[j - j0] = d * inv;
        if (s[j - j0] > M) M = s[j - j0];
    }
    double Z = 0.0;
    for (int j = 0; j < n; j++) { s[j] = exp(s[j] - M); Z += s[j]; }
    for (int t = 0; t < hd; t++) {
        double acc = 0.0;
        for (int j = 0; j < n; j++) acc += (s[j] / Z) * (double)kv_to_f32(kv_dtype, V[(size_t)(j + j0) * hd + t]);
        o[t] = (float)acc;
    }
    if (w_out) for (int j = 0; j < n; j++) w_out[j] = s[j] / Z;
    free(s);
}

/* Split-K partial over [j0, j1): running maximum m, denominator l = sum exp(s - m), and
 * acc[t] = sum exp(s - m) V[j][t].  (Used by tests of the combine identity; the decode step below uses
 * the unsplit definition.) */
void orc_attention_partial(const float* q, const uint16_t* K, const uint16_t* V, int hd, int j0, int j1,
                           double* m_out, double* l_out, double* acc) {
    double inv = 1.0 / sqrt((double)hd);
    double M = -INFINITY;
    for (int j = j0; j < j1; j++) {
        double d = 0.0;
        for (int t = 0; t < hd; t++) d += (double)q[t] * (double)orc_bf16_to_f32(K[(size_t)j * hd + t]);
        d *= inv;
        if (d > M) M = d;
    }
    double l = 0.0;
    for (int t = 0; t < hd; t++) acc[t] = 0.0;
    for (int j = j0; j < j1; j++) {
        double d = 0.0;
        for (int t = 0; t < hd; t++) d += (double)q[t] * (double)orc_bf16_to_f32(K[(size_t)j * hd + t]);
        double w = exp(d * inv - M);
        l += w;
        for (int t = 0; t < hd; t++) acc[t] += w * (double)orc_bf16_to_f32(V[(size_t)j * hd + t]);
    }
    *m_out = M; *l_out = l;
}

/* Combine C partials: o = sum_c e^{m_c - M} acc_c / sum_c e^{m_c - M} l_c, M = max_c m_c. */
void orc_attention_combine(const double* m, const double* l, const double* acc, int C, int hd, float* o) {
    double M = -INFINITY;
    for (int c = 0; c < C; c++) if (m[c] > M) M = m[c];
    double Z = 0.0;
    for (int c = 0; c < C; c++) Z += exp(m[c] - M) * l[c];
    for (int t = 0; t < hd; t++) {
        double a = 0.0;
        for (int c = 0; c < C; c++) a += exp(m[c] - M) * acc[(size_t)c * hd + t];
        o[t] = (float)(a / Z);
    }
}

/* ----------------------------------------------------------------------------------------------
 * The decode step
 * -------------------------------------------------------------------------------------------- */

typedef struct {
    int32_t hidden, n_layers, n_q_heads, n_kv_heads, head_dim, mlp, vocab, max_seq;
    int32_t tied_embeddings;
    float rms_eps;
    float rope_theta;
    int32_t wdtype;        /* 0 bf16, 1 int8, 2 int4, 3 grouped int8: applies to the seven per-layer linears only */
    int32_t group_size;    /* int4 / grouped int8: group length along the input dimension */
    int32_t round_kv;      /* 1: cache entries rounded to the cache element type (the contract); 0: test-only, see below */
    int32_t quantize_lm_head; /* 0: the LM head stays bf16 (the reading taken of the paper); 1: it is quantised like
                                 the per-layer linears (wdtype, group_size) -- the other reading of "linear GEMV
                                 weights move to int8 / int4" for an untied head; the embedding gather stays bf16 */
    int32_t kv_dtype;      /* element type of the KV cache: 0 bf16 (what the paper's kernels keep, Section 5), 1 fp8 e4m3
                              (a variant: the same step with the cache rounded to 8 bits instead of 16) */
} orc_config;

/* Canonical weights.  Per-layer arrays are indexed [layer]; linears are indexed by
 * kind 0..6 = q, k, v, o, gate, up, down, each row-major [out][in]. */
typedef struct {
    const uint16_t* embed;          /* bf16 [V][H] */
    const uint16_t* lm_head;        /* bf16 [V][H]; NULL when tied */
    const uint16_t* final_norm;     /* bf16 [H] */
    const uint16_t* const* attn_norm;
    const uint16_t* const* mlp_norm;
    const void* const* w[7];
    const uint16_t* const* scale[7];
    const uint16_t* const* zero[7];
    const void* lm_head_q;          /* quantize_lm_head: codes of the LM head (of the embedding matrix when tied) */
    const uint16_t* lm_head_scale;  /*   fp16 scales: int8 [V]; int4 [V][H/group]                                */
    const uint16_t* lm_head_zero;   /*   int4: fp16 integer-valued zero points [V][H/group]                      */
} orc_weights;

/* logits = W_lm . y: the bf16 matrix (the embedding matrix when tied), or its quantised form */
static void lm_head(const orc_config* c, const orc_weights* w, const float* y, float* logits) {
    if (c->quantize_lm_head && c->wdtype != 0)
        orc_gemv(c->wdtype, w->lm_head_q, w->lm_head_scale, c->wdtype == 2 ? w->lm_head_zero : NULL, c->group_size,
                 c->vocab, c->hidden, y, logits);
    else
        orc_gemv(0, c->tied_embeddings ? w->embed : w->lm_head, NULL, NULL, 0, c->vocab, c->hidden, y, logits);
}

static void linear(const orc_config* c, const orc_weights* w, int kind, int layer, int rows, int cols,
                   const float* x, float* y) {
    orc_gemv(c->wdtype, w->w[kind][layer],
             c->wdtype ? w->scale[kind][layer] : NULL,
             c->wdtype == 2 ? w->zero[kind][layer] : NULL,
             c->group_size, rows, cols, x, y);
}

/*
 * One decode step for one sequence: token at position pos (0-based); the cache holds positions
 * [0, pos) on entry and [0, pos] on exit.
 *   kv_cache : K then V, each [L][n_kv][max_seq][hd] bf16 (uint16 words), updated in place.
 *   kv_f32   : test-only shadow cache of the same shape in fp32, used instead of kv_cache when
 *              cfg->round_kv == 0 (lets a library forward that keeps fp32 keys/values be compared);
 *              NULL otherwise.
 *   logits   : [V] fp32 out.   next_token : 1 int out.
 *   hidden   : [(L+1)][H] fp32 out, may be NULL: row 0 = embedding, row l+1 = residual stream after layer l.
 * Returns 0, or -1 on a bad argument.
 *
 * Readings where the paper is silent: pre-norm residual blocks without biases; grouped-query mapping
 * q head h -> kv head floor(h / (n_q/n_kv)); K cached after the rotation; LM head = embedding matrix when
 * tied, and it stays bf16 in the quantised variants (tied or not).
 */

/* Distance between two bf16 (or, sign_bit = 0x80, e4m3) values in representable steps (sign-magnitude bit
 * patterns ordered as integers). */
static int steps_apart(uint16_t a, uint16_t b, uint16_t sign_bit) {
    uint16_t mag = (uint16_t)(sign_bit - 1);
    int ia = (a & sign_bit) ? -(int)(a & mag) : (int)(a & mag);
    int ib = (b & sign_bit) ? -(int)(b & mag) : (int)(b & mag);
    return ia > ib ? ia - ib : ib - ia;
}

/* The cache entry appended for one fp32 value.  The contract is round-to-nearest-even to bf16 (to e4m3 with
 * saturation for an fp8 cache; the entry is then the code in a 16-bit word).  Two correct
 * implementations whose fp32 values differ in the last bits (another summation order) may land on either side
 * of a rounding boundary, i.e. on neighbouring bf16 values: both are valid cache entries.  A caller that
 * compares another implementation with this one can pass that implementation's entry as `pref`: it is adopted
 * only if it is this oracle's own rounding or one of its two neighbours, so that everything computed FROM the
 * cache afterwards is compared like with like; otherwise the oracle keeps its own.  `own` always receives the
 * oracle's own rounding. */
static uint16_t cache_entry(int kv_dtype, float value, const uint16_t* pref, uint16_t* own, int* adopted) {
    uint16_t r = kv_dtype == 1 ? (uint16_t)orc_f32_to_e4m3(value) : orc_f32_to_bf16(value);
    if (own) *own = r;
    if (pref && *pref != r && (kv_dtype != 1 || (*pref & 0x7f) != 0x7f) &&
        steps_apart(*pref, r, kv_dtype == 1 ? 0x80 : 0x8000) <= 1) { if (adopted) (*adopted)++; return *pref; }
    return r;
}

int orc_decode_step_rows(const orc_config* c, const orc_weights* w, int token, int pos,
                         uint16_t* kv_cache, float* kv_f32, float* logits, int* next_token, float* hidden,
                         const uint16_t* rows_pref, uint16_t* rows_own, int* n_adopted);

int orc_decode_step(const orc_config* c, const orc_weights* w, int token, int pos,
                    uint16_t* kv_cache, float* kv_f32, float* logits, int* next_token, float* hidden) {
    return orc_decode_step_rows(c, w, token, pos, kv_cache, kv_f32, logits, next_token, hidden, NULL, NULL, NULL);
}

/* The same step with the appended cache rows exposed: rows_pref / rows_own are [2][L][n_kv][hd] bf16 (K rows then
 * V rows of slot `pos`), either may be NULL; see cache_entry.  *n_adopted counts the preferred entries taken. */
int orc_decode_step_rows(const orc_config* c, const orc_weights* w, int token, int pos,
                         uint16_t* kv_cache, float* kv_f32, float* logits, int* next_token, float* hidden,
                         const uint16_t* rows_pref, uint16_t* rows_own, int* n_adopted) {
    const int H = c->hidden, L = c->n_layers, nq = c->n_q_heads, nkv = c->n_kv_heads, hd = c->head_dim;
    const int I = c->mlp, V = c->vocab, S = c->max_seq;
    if (token < 0 || token >= V || pos < 0 || pos >= S || nq % nkv != 0 || (hd & 1)) return -1;
    const int n_rep = nq / nkv;
    const size_t kv_half = (size_t)L * nkv * S * hd;

    float* x = (float*)malloc(sizeof(float) * H);
    float* a = (float*)malloc(sizeof(float) * H);
    float* q = (float*)malloc(sizeof(float) * nq * hd);
    float* k = (float*)malloc(sizeof(float) * nkv * hd);
    float* v = (float*)malloc(sizeof(float) * nkv * hd);
    float* o = (float*)malloc(sizeof(float) * nq * hd);
    float* t = (float*)malloc(sizeof(float) * H);
    float* gt = (float*)malloc(sizeof(float) * I);
    float* up = (float*)malloc(sizeof(float) * I);
    float* m = (float*)malloc(sizeof(float) * I);

    /* step 0: embedding row */
    for (int i = 0; i < H; i++) x[i] = orc_bf16_to_f32(w->embed[(size_t)token * H + i]);
    if (hidden) memcpy(hidden, x, sizeof(float) * H);

    for (int l = 0; l < L; l++) {
        /* 1: attention-side norm;  2: q, k, v projections */
        orc_rmsnorm(x, w->attn_norm[l], H, c->rms_eps, a);
        linear(c, w, 0, l, nq * hd, H, a, q);
        linear(c, w, 1, l, nkv * hd, H, a, k);
        linear(c, w, 2, l, nkv * hd, H, a, v);
        /* 3: rotate every q head and k head at this position */
        for (int h = 0; h < nq; h++) orc_rope(q + (size_t)h * hd, hd, pos, (double)c->rope_theta);
        for (int g = 0; g < nkv; g++) orc_rope(k + (size_t)g * hd, hd, pos, (double)c->rope_theta);
        /* 4: append to the cache (slot pos of this layer) */
        for (int g = 0; g < nkv; g++) {
            size_t base = (((size_t)l * nkv + g) * S + (size_t)pos) * hd;
            const size_t rbase = ((size_t)l * nkv + g) * hd, rhalf = (size_t)L * nkv * hd;
            for (int d = 0; d < hd; d++) {
                if (c->round_kv) {
                    kv_cache[base + d] = cache_entry(c->kv_dtype, k[g * hd + d], rows_pref ? rows_pref + rbase + d : NULL,
                                                     rows_own ? rows_own + rbase + d : NULL, n_adopted);
                    kv_cache[kv_half + base + d] = cache_entry(c->kv_dtype, v[g * hd + d], rows_pref ? rows_pref + rhalf + rbase + d : NULL,
                                                               rows_own ? rows_own + rhalf + rbase + d : NULL, n_adopted);
                } else {
                    kv_f32[base + d] = k[g * hd + d];
                    kv_f32[kv_half + base + d] = v[g * hd + d];
                }
            }
        }
        /* 5: attention of each q head over positions 0..pos of its kv head */
#pragma omp parallel for schedule(static)
        for (int h = 0; h < nq; h++) {
            int g = h / n_rep;
            size_t base = ((size_t)l * nkv + g) * S * hd;
            if (c->round_kv) {
                orc_attention_head_kv(c->kv_dtype, q + (size_t)h * hd, kv_cache + base, kv_cache + kv_half + base, hd, 0, pos + 1,
                                   o + (size_t)h * hd, NULL);
            } else {
                /* same definition on the fp32 shadow cache */
                const float* Kf = kv_f32 + base; const float* Vf = kv_f32 + kv_half + base;
                int n = pos + 1;
                double* s = (double*)malloc(sizeof(double) * (size_t)n);
                double inv = 1.0 / sqrt((double)hd), M = -INFINITY, Z = 0.0;
                for (int j = 0; j < n; j++) {
                    double d = 0.0;
                    for (int e = 0; e < hd; e++) d += (double)q[(size_t)h * hd + e] * (double)Kf[(size_t)j * hd + e];
                    s[j] = d * inv; if (s[j] > M) M = s[j];
                }
                for (int j = 0; j < n; j++) { s[j] = exp(s[j] - M); Z += s[j]; }
                for (int e = 0; e < hd; e++) {
                    double acc = 0.0;
                    for (int j = 0; j < n; j++) acc += (s[j] / Z) * (double)Vf[(size_t)j * hd + e];
                    o[(size_t)h * hd + e] = (float)acc;
                }
                free(s);
            }
        }
        /* 6: output projection and residual */
        linear(c, w, 3, l, H, nq * hd, o, t);
        for (int i = 0; i < H; i++) x[i] = (float)((double)x[i] + (double)t[i]);
        /* 7: MLP-side norm, gate and up projections, SiLU(gate) * up */
        orc_rmsnorm(x, w->mlp_norm[l], H, c->rms_eps, a);
        linear(c, w, 4, l, I, H, a, gt);
        linear(c, w, 5, l, I, H, a, up);
        for (int i = 0; i < I; i++) m[i] = (float)((double)orc_silu(gt[i]) * (double)up[i]);
        /* 8: down projection and residual */
        linear(c, w, 6, l, H, I, m, t);
        for (int i = 0; i < H; i++) x[i] = (float)((double)x[i] + (double)t[i]);
        if (hidden) memcpy(hidden + (size_t)(l + 1) * H, x, sizeof(float) * H);
    }
    /* 9: final norm, LM head (bf16 unless quantize_lm_head), greedy token */
    orc_rmsnorm(x, w->final_norm, H, c->rms_eps, a);
    lm_head(c, w, a, logits);
    if (next_token) *next_token = orc_argmax(logits, V);

    free(x); free(a); free(q); free(k); free(v); free(o); free(t); free(gt); free(up); free(m);
    return 0;
}

/* One decoder layer applied to a given residual stream x_in (fp32 [H]) -> x_out, with the same cache
 * semantics as the full step.  Lets a sampled layer of a large model be checked on its own. */
int orc_layer_step_rows(const orc_config* c, const orc_weights* w, int layer, int pos, const float* x_in,
                        uint16_t* kv_cache, float* x_out, const uint16_t* rows_pref, uint16_t* rows_own, int* n_adopted);

int orc_layer_step(const orc_config* c, const orc_weights* w, int layer, int pos, const float* x_in,
                   uint16_t* kv_cache, float* x_out) {
    return orc_layer_step_rows(c, w, layer, pos, x_in, kv_cache, x_out, NULL, NULL, NULL);
}

/* rows_pref / rows_own: [2][n_kv][hd] bf16, the K row then the V row this layer appends (see cache_entry). */
int orc_layer_step_rows(const orc_config* c, const orc_weights* w, int layer, int pos, const float* x_in,
                        uint16_t* kv_cache, float* x_out, const uint16_t* rows_pref, uint16_t* rows_own, int* n_adopted) {
    const int H = c->hidden, L = c->n_layers, nq = c->n_q_heads, nkv = c->n_kv_heads, hd = c->head_dim;
    const int I = c->mlp, S = c->max_seq;
    if (layer < 0 || layer >= L || pos < 0 || pos >= S || nq % nkv != 0 || (hd & 1)) return -1;
    const int n_rep = nq / nkv, l = layer;
    const size_t kv_half = (size_t)L * nkv * S * hd;
    float* x = (float*)malloc(sizeof(float) * H);
    float* a = (float*)malloc(sizeof(float) * H);
    float* q = (float*)malloc(sizeof(float) * nq * hd);
    float* k = (float*)malloc(sizeof(float) * nkv * hd);
    float* v = (float*)malloc(sizeof(float) * nkv * hd);
    float* o = (float*)malloc(sizeof(float) * nq * hd);
    float* t = (float*)malloc(sizeof(float) * H);
    float* gt = (float*)malloc(sizeof(float) * I);
    float* up = (float*)malloc(sizeof(float) * I);
    float* m = (float*)malloc(sizeof(float) * I);
    memcpy(x, x_in, sizeof(float) * H);
    orc_rmsnorm(x, w->attn_norm[l], H, c->rms_eps, a);
    linear(c, w, 0, l, nq * hd, H, a, q);
    linear(c, w, 1, l, nkv * hd, H, a, k);
    linear(c, w, 2, l, nkv * hd, H, a, v);
    for (int h = 0; h < nq; h++) orc_rope(q + (size_t)h * hd, hd, pos, (double)c->rope_theta);
    for (int g = 0; g < nkv; g++) orc_rope(k + (size_t)g * hd, hd, pos, (double)c->rope_theta);
    for (int g = 0; g < nkv; g++) {
        size_t base = (((size_t)l * nkv + g) * S + (size_t)pos) * hd;
        const size_t rbase = (size_t)g * hd, rhalf = (size_t)nkv * hd;
        for (int d = 0; d < hd; d++) {
            kv_cache[base + d] = cache_entry(c->kv_dtype, k[g * hd + d], rows_pref ? rows_pref + rbase + d : NULL,
                                             rows_own ? rows_own + rbase + d : NULL, n_adopted);
            kv_cache[kv_half + base + d] = cache_entry(c->kv_dtype, v[g * hd + d], rows_pref ? rows_pref + rhalf + rbase + d : NULL,
                                                       rows_own ? rows_own + rhalf + rbase + d : NULL, n_adopted);
        }
    }
#pragma omp parallel for schedule(static)
    for (int h = 0; h < nq; h++) {
        int g = h / n_rep;
        size_t base = ((size_t)l * nkv + g) * S * hd;
        orc_attention_head_kv(c->kv_dtype, q + (size_t)h * hd, kv_cache + base, kv_cache + kv_half + base, hd, 0, pos + 1,
                           o + (size_t)h * hd, NULL);
    }
    linear(c, w, 3, l, H, nq * hd, o, t);
    for (int i = 0; i < H; i++) x[i] = (float)((double)x[i] + (double)t[i]);
    orc_rmsnorm(x, w->mlp_norm[l], H, c->rms_eps, a);
    linear(c, w, 4, l, I, H, a, gt);
    linear(c, w, 5, l, I, H, a, up);
    for (int i = 0; i < I; i++) m[i] = (float)((double)orc_silu(gt[i]) * (double)up[i]);
    linear(c, w, 6, l, H, I, m, t);
    for (int i = 0; i < H; i++) x_out[i] = (float)((double)x[i] + (double)t[i]);
    free(x); free(a); free(q); free(k); free(v); free(o); free(t); free(gt); free(up); free(m);
    return 0;
}

/* Final norm + bf16 LM head + greedy token on a given residual stream. */
int orc_head_step(const orc_config* c, const orc_weights* w, const float* x_in, float* logits, int* next_token) {
    const int H = c->hidden, V = c->vocab;
    float* a = (float*)malloc(sizeof(float) * H);
    orc_rmsnorm(x_in, w->final_norm, H, c->rms_eps, a);
    lm_head(c, w, a, logits);
    if (next_token) *next_token = orc_argmax(logits, V);
    free(a);
    return 0;
}

/* Number of OpenMP threads the loops above will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int orc_num_threads(void) { return omp_get_max_threads(); }
void orc_set_num_threads(int n) { omp_set_num_threads(n); }
#else
int orc_num_threads(void) { return 1; }
void orc_set_num_threads(int n) { (void)n; }
#endif
