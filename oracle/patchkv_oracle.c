/*
 * PatchKV suffix-restore path -- CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, scalar statement of what the hot path computes, written from the paper:
 *   - block scoring, dirty window, top-k, union / block rounding / complement
 *     (Section IV-B Eq. 9; Section IV-C Eqs. 10-12),
 *   - restore of every reused block: dequantise by the block's frozen precision tag
 *     (Section IV-D), correct the RoPE phase of K (Section II-B Eq. 3), place the rows in
 *     their destination KV pages (Section IV-D, last paragraph).
 * It shares no code, header, table or constant with the CUDA library and neither includes
 * the other; the byte layout of a checkpoint is re-declared here from its written description.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Precision: selection is exact integer arithmetic.  Dequantisation forms code * scale in
 * fp32, which is exact (at most 8 + 11 significant bits), and rounds once to bf16 (nearest
 * even).  The K rotation is the fp32 recipe: cos/sin of delta*theta_i evaluated in double and
 * rounded once to fp32, then four fp32 multiplies, one fp32 subtract and one fp32 add, each
 * rounded separately (compile with -ffp-contract=off), then one rounding to bf16.  The same
 * pair is also evaluated in double so that the distance of the recipe from the correctly
 * rounded result can be reported.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py (closed forms,
 * invariants, brute force, numpy/torch conversions).  No value printed in the paper pins a
 * restored element; the record-size formulas are pinned to the payload ratios of Section V-E.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { PKVO_OK = 0, PKVO_E_INVALID = -1, PKVO_E_BOUNDS = -3, PKVO_E_BADINPUT = -7 };
enum { PKVO_TAG_BF16 = 0, PKVO_TAG_INT8 = 1, PKVO_TAG_INT4 = 2, PKVO_TAG_K4V4 = 3 };
enum { PKVO_FMT_BF16 = 0, PKVO_FMT_INT8 = 1, PKVO_FMT_INT4 = 2 };
enum { PKVO_ROPE_HALF = 0, PKVO_ROPE_INTERLEAVED = 1 };
enum { PKVO_LAYERS_INDEPENDENT = 0, PKVO_LAYERS_SHARED = 1 };

/* ------------------------------------------------------------------ number formats */
static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* IEEE binary16 -> binary32, every one of the 65536 patterns exact. */
float pkvo_fp16_to_f32(uint16_t h) {
    uint32_t sign = (uint32_t)(h >> 15) << 31, e = (h >> 10) & 31u, m = h & 1023u;
    if (e == 0) {                       /* zero or subnormal: m * 2^-24 */
        float v = (float)m * (1.0f / 16777216.0f);
        return bits_f32(f32_bits(v) | sign);
    }
    if (e == 31) return bits_f32(sign | 0x7f800000u | (m << 13));
    return bits_f32(sign | ((e + 112u) << 23) | (m << 13));
}

float pkvo_bf16_to_f32(uint16_t b) { return bits_f32((uint32_t)b << 16); }

/* binary32 -> bfloat16, round to nearest, ties to even; NaN stays a (quiet) NaN. */
uint16_t pkvo_f32_to_bf16(float f) {
    uint32_t u = f32_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* binary32 -> binary16, round to nearest even (used by the quantiser of the round-trip pin). */
uint16_t pkvo_f32_to_fp16(float f) {
    uint32_t u = f32_bits(f), sign = (u >> 16) & 0x8000u, a = u & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);
    if (a >= 0x47800000u) return (uint16_t)(sign | 0x7c00u);      /* >= 65536 -> inf (65520.. handled below) */
    if (a < 0x33000000u) return (uint16_t)sign;                   /* < 2^-25 -> 0 */
    int32_t e = (int32_t)(a >> 23) - 127;
    uint32_t m = (a & 0x7fffffu) | 0x800000u;                     /* 24-bit significand */
    int shift = (e < -14) ? (13 + (-14 - e)) : 13;                /* bits dropped */
    uint32_t keep = m >> shift, rem = m & ((1u << shift) - 1u), half = 1u << (shift - 1);
    if (rem > half || (rem == half && (keep & 1u))) keep++;
    uint32_t out;
    if (e < -14) out = keep;                                      /* subnormal (may carry into normal) */
    else out = ((uint32_t)(e + 15) << 10) + (keep - 0x400u);      /* carry propagates into exponent */
    if (out >= 0x7c00u) out = 0x7c00u;
    return (uint16_t)(sign | out);
}

/* ------------------------------------------------------------------ checkpoint format */
static int k_fmt(int tag) { return tag == PKVO_TAG_BF16 ? PKVO_FMT_BF16 : tag == PKVO_TAG_K4V4 ? PKVO_FMT_INT4 : PKVO_FMT_INT8; }
static int v_fmt(int tag) { return tag == PKVO_TAG_BF16 ? PKVO_FMT_BF16 : tag == PKVO_TAG_INT8 ? PKVO_FMT_INT8 : PKVO_FMT_INT4; }

static uint64_t codes_bytes(int fmt, uint64_t elems) {
    return fmt == PKVO_FMT_BF16 ? 2 * elems : fmt == PKVO_FMT_INT8 ? elems : elems / 2;
}
static uint64_t scales_bytes(int fmt, uint64_t elems, int G) {
    return fmt == PKVO_FMT_BF16 ? 0 : 2 * (elems / (uint64_t)G);
}

/* Bytes of one block record [K codes][K scales][V codes][V scales]; 0 for an unknown tag. */
uint64_t pkvo_record_bytes(int tag, int B, int H, int D, int G) {
    if (tag < 0 || tag > PKVO_TAG_K4V4) return 0;
    uint64_t elems = (uint64_t)B * H * D;
    return codes_bytes(k_fmt(tag), elems) + scales_bytes(k_fmt(tag), elems, G) +
           codes_bytes(v_fmt(tag), elems) + scales_bytes(v_fmt(tag), elems, G);
}

/* Dequantise element (t, h, c) of one section to fp32; *raw receives the 16 stored bits of a bf16 code. */
static float dequant_elem(const uint8_t* codes, const uint8_t* scales, int fmt, int H, int D, int G,
                          int t, int h, int c, uint16_t* raw) {
    uint64_t e = ((uint64_t)t * H + h) * D + c;
    if (fmt == PKVO_FMT_BF16) {
        uint16_t b; memcpy(&b, codes + 2 * e, 2);
        *raw = b;
        return pkvo_bf16_to_f32(b);
    }
    uint16_t sb; memcpy(&sb, scales + 2 * (((uint64_t)t * H + h) * (D / G) + c / G), 2);
    float s = pkvo_fp16_to_f32(sb);
    int q;
    if (fmt == PKVO_FMT_INT8) q = (int8_t)codes[e];
    else {
        uint8_t byte = codes[e >> 1];
        int nib = (c & 1) ? (byte >> 4) : (byte & 15);
        q = nib >= 8 ? nib - 16 : nib;
    }
    *raw = 0;
    return (float)q * s;     /* exact: |q| < 2^8, s has 11 significant bits */
}

/* Symmetric quantiser of one group (the inverse direction; used by the round-trip pin only):
 * s = fp16(amax / qmax), q = clamp(rint(x / s), -qmax, qmax) with ties to even, s == 0 -> q = 0. */
void pkvo_quantise_group(const float* x, int G, int qmax, int8_t* q, uint16_t* scale_fp16) {
    float amax = 0.0f;
    for (int i = 0; i < G; i++) { float a = fabsf(x[i]); if (a > amax) amax = a; }
    uint16_t sb = pkvo_f32_to_fp16(amax / (float)qmax);
    float s = pkvo_fp16_to_f32(sb);
    for (int i = 0; i < G; i++) {
        float r = (s > 0.0f) ? nearbyintf(x[i] / s) : 0.0f;
        if (r > (float)qmax) r = (float)qmax;
        if (r < -(float)qmax) r = -(float)qmax;
        q[i] = (int8_t)r;
    }
    *scale_fp16 = sb;
}

/* Dequantise one group of codes (int8 values, also for 4-bit codes) with one fp16 scale. */
void pkvo_dequantise_group(const int8_t* q, int G, uint16_t scale_fp16, float* x) {
    float s = pkvo_fp16_to_f32(scale_fp16);
    for (int i = 0; i < G; i++) x[i] = (float)q[i] * s;
}

/* ------------------------------------------------------------------ RoPE phase correction (Eq. 3) */
/* theta_i = base^(-2i/Dr) unless inv_freq is given; cos/sin(delta * theta_i) in double, rounded to fp32. */
void pkvo_rope_table(int Dr, double base, const float* inv_freq, int delta, float* cos_out, float* sin_out) {
    for (int i = 0; i < Dr / 2; i++) {
        double theta = inv_freq ? (double)inv_freq[i] : pow(base, -2.0 * (double)i / (double)Dr);
        double phi = (double)delta * theta;
        cos_out[i] = (float)cos(phi);
        sin_out[i] = (float)sin(phi);
    }
}

/* One rotary pair in fp32, every operation rounded on its own: (a, b) -> (a c - b s, a s + b c). */
void pkvo_rotate_pair_f32(float a, float b, float c, float s, float* a_out, float* b_out) {
    volatile float ac = a * c, bs = b * s, as = a * s, bc = b * c;
    *a_out = ac - bs;
    *b_out = as + bc;
}

/* Rotate one head vector x[0..D) in fp32 (no bf16 rounding): the Dr/2 rotary pairs are (i, i+Dr/2) in the
 * HALF style and (2i, 2i+1) in the INTERLEAVED style; channels >= Dr pass through. */
void pkvo_rotate_head_f32(const float* x, int D, int Dr, int rope_style, const float* ct, const float* st, float* out) {
    for (int c = 0; c < D; c++) out[c] = x[c];
    for (int i = 0; i < Dr / 2; i++) {
        int ia = rope_style == PKVO_ROPE_HALF ? i : 2 * i;
        int ib = rope_style == PKVO_ROPE_HALF ? i + Dr / 2 : 2 * i + 1;
        pkvo_rotate_pair_f32(x[ia], x[ib], ct[i], st[i], &out[ia], &out[ib]);
    }
}

/* Array forms of the conversions, for the tests that sweep many bit patterns. */
void pkvo_fp16_to_f32_n(const uint16_t* h, int64_t n, float* out) { for (int64_t i = 0; i < n; i++) out[i] = pkvo_fp16_to_f32(h[i]); }
void pkvo_f32_to_bf16_n(const float* x, int64_t n, uint16_t* out) { for (int64_t i = 0; i < n; i++) out[i] = pkvo_f32_to_bf16(x[i]); }
void pkvo_f32_to_fp16_n(const float* x, int64_t n, uint16_t* out) { for (int64_t i = 0; i < n; i++) out[i] = pkvo_f32_to_fp16(x[i]); }

/* ------------------------------------------------------------------ selection */
/* Exact value of a finite non-negative fp16 in units of 2^-24. */
static uint64_t fp16_units(uint16_t h) {
    uint32_t e = (h >> 10) & 31u, m = h & 1023u;
    return e == 0 ? (uint64_t)m : (uint64_t)(1024u + m) << (e - 1);
}

/* Eq. 10 in its block form: mass[l][j] = sum over heads, query positions and the tokens of block j of
 * the stored attention A[l][h][q][s], exactly, in units of 2^-24.  A negative (non-zero), infinite or NaN
 * entry counts as zero and makes the call return PKVO_E_BADINPUT (mass is still filled). */
int pkvo_block_mass(const uint16_t* attn, int L, int Hq, int Q, int n,
                    int64_t stride_layer, int64_t stride_head, int64_t stride_query,
                    int B, uint64_t* mass) {
    if (L < 0 || Hq < 0 || Q < 0 || n < 0 || B <= 0) return PKVO_E_INVALID;
    int NB = (n + B - 1) / B, bad = 0;
    for (int l = 0; l < L; l++)
        for (int j = 0; j < NB; j++) {
            uint64_t acc = 0;
            int s_end = (j + 1) * B < n ? (j + 1) * B : n;
            for (int h = 0; h < Hq; h++)
                for (int q = 0; q < Q; q++) {
                    const uint16_t* row = attn + l * stride_layer + h * stride_head + q * stride_query;
                    for (int s = j * B; s < s_end; s++) {
                        uint16_t x = row[s];
                        if ((x & 0x7fffu) == 0) continue;
                        if ((x & 0x8000u) || ((x >> 10) & 31u) == 31u) { bad = 1; continue; }
                        acc += fp16_units(x);
                    }
                }
            mass[(int64_t)l * NB + j] = acc;
        }
    return bad ? PKVO_E_BADINPUT : PKVO_OK;
}

/* The same sum carried in double (exact below 2^53 units); a cross-check of the integer path. */
int pkvo_block_mass_f64(const uint16_t* attn, int L, int Hq, int Q, int n,
                        int64_t stride_layer, int64_t stride_head, int64_t stride_query,
                        int B, double* mass) {
    if (B <= 0) return PKVO_E_INVALID;
    int NB = (n + B - 1) / B;
    for (int l = 0; l < L; l++)
        for (int j = 0; j < NB; j++) {
            double acc = 0.0;
            for (int h = 0; h < Hq; h++)
                for (int q = 0; q < Q; q++) {
                    const uint16_t* row = attn + l * stride_layer + h * stride_head + q * stride_query;
                    for (int s = j * B; s < (j + 1) * B && s < n; s++) {
                        float v = pkvo_fp16_to_f32(row[s]);
                        if (v > 0.0f && v <= 65504.0f) acc += (double)v;
                    }
                }
            mass[(int64_t)l * NB + j] = acc * 16777216.0;
        }
    return PKVO_OK;
}

/* Norm of Eq. 10, read as division by the total: the importance of unit j (a block, or a token in the token-level
 * form) is its share of the summed mass, I_j = mass_j / sum_j' mass_j' over every unit of the row, the dirty window
 * included.  A positive rescaling leaves the ranking as it is, so selection ranks on the exact masses and this score
 * is reported only.  Masses are exact integers; the quotient is taken in double and rounded once to fp32.  A row
 * whose masses are all zero gets zeros.  LAYERS_SHARED: one row, from the masses summed over the layers.
 * mass u64 [L][NB] -> score fp32 [L][NB] (LAYERS_INDEPENDENT) or [NB] (LAYERS_SHARED). */
int pkvo_normalise(const uint64_t* mass, int L, int NB, int layer_mode, float* score) {
    if (L <= 0 || NB < 0) return PKVO_E_INVALID;
    if (layer_mode != PKVO_LAYERS_INDEPENDENT && layer_mode != PKVO_LAYERS_SHARED) return PKVO_E_INVALID;
    if (layer_mode == PKVO_LAYERS_SHARED) {
        uint64_t total = 0;
        for (int l = 0; l < L; l++) for (int j = 0; j < NB; j++) total += mass[(size_t)l * NB + j];
        for (int j = 0; j < NB; j++) {
            uint64_t m = 0;
            for (int l = 0; l < L; l++) m += mass[(size_t)l * NB + j];
            score[j] = total ? (float)((double)m / (double)total) : 0.0f;
        }
        return PKVO_OK;
    }
    for (int l = 0; l < L; l++) {
        uint64_t total = 0;
        for (int j = 0; j < NB; j++) total += mass[(size_t)l * NB + j];
        for (int j = 0; j < NB; j++)
            score[(size_t)l * NB + j] = total ? (float)((double)mass[(size_t)l * NB + j] / (double)total) : 0.0f;
    }
    return PKVO_OK;
}

typedef struct { uint64_t mass; int32_t idx; } cand_t;
static int cand_cmp(const void* pa, const void* pb) {
    const cand_t* a = (const cand_t*)pa; const cand_t* b = (const cand_t*)pb;
    if (a->mass != b->mass) return a->mass > b->mass ? -1 : 1;     /* larger mass first */
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);       /* ties: lower block index first */
}

/* Eqs. 9, 11, 12 at block granularity.
 *   dirty   = blocks holding a token nearer than min(max(dirty_tokens,0), n) to the edit = [0, ceil(n_d/B))
 *   H_l     = the min(top_k, #candidates) non-dirty blocks of largest mass (ties: lower index)
 *   R_l     = dirty U H_l,  F_l = all other blocks; both ascending.
 * LAYERS_SHARED ranks on the mass summed over layers and gives every layer the same sets.
 * Outputs: mask u8 [L][NB] (1 = repair), repair_idx/reuse_idx i32 [L][NB] (first cnt entries valid,
 * the rest set to -1), repair_cnt/reuse_cnt i32 [L]. */
int pkvo_select(const uint64_t* mass, int L, int n, int B, int dirty_tokens, int top_k, int layer_mode,
                uint8_t* mask, int32_t* repair_idx, int32_t* repair_cnt, int32_t* reuse_idx, int32_t* reuse_cnt) {
    if (L <= 0 || n < 0 || B <= 0 || top_k < 0) return PKVO_E_INVALID;
    if (layer_mode != PKVO_LAYERS_INDEPENDENT && layer_mode != PKVO_LAYERS_SHARED) return PKVO_E_INVALID;
    int NB = (n + B - 1) / B;
    int64_t nd = dirty_tokens < 0 ? 0 : dirty_tokens;
    if (nd > n) nd = n;
    int n_dirty = (int)((nd + B - 1) / B);
    cand_t* cand = (cand_t*)malloc(sizeof(cand_t) * (size_t)(NB > 0 ? NB : 1));
    uint64_t* shared = NULL;
    if (layer_mode == PKVO_LAYERS_SHARED) {
        shared = (uint64_t*)calloc((size_t)(NB > 0 ? NB : 1), sizeof(uint64_t));
        for (int l = 0; l < L; l++) for (int j = 0; j < NB; j++) shared[j] += mass[(int64_t)l * NB + j];
    }
    for (int l = 0; l < L; l++) {
        const uint64_t* m = shared ? shared : mass + (int64_t)l * NB;
        uint8_t* mk = mask + (int64_t)l * NB;
        int nc = 0;
        for (int j = 0; j < NB; j++) {
            mk[j] = j < n_dirty;
            if (j >= n_dirty) { cand[nc].mass = m[j]; cand[nc].idx = j; nc++; }
        }
        qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
        int take = top_k < nc ? top_k : nc;
        for (int i = 0; i < take; i++) mk[cand[i].idx] = 1;
        int nr = 0, nf = 0;
        for (int j = 0; j < NB; j++) {
            if (mk[j]) repair_idx[(int64_t)l * NB + nr++] = j;
            else       reuse_idx[(int64_t)l * NB + nf++] = j;
        }
        for (int i = nr; i < NB; i++) repair_idx[(int64_t)l * NB + i] = -1;
        for (int i = nf; i < NB; i++) reuse_idx[(int64_t)l * NB + i] = -1;
        repair_cnt[l] = nr; reuse_cnt[l] = nf;
    }
    free(cand); free(shared);
    return PKVO_OK;
}

/* ------------------------------------------------------------------ restore */
typedef struct {
    int L, H, D, Dr, rope_style, B, P, G;
    double rope_base;
    const float* inv_freq;               /* optional [Dr/2] */
    uint16_t* k_pool; uint16_t* v_pool;  /* bf16 bit patterns */
    int64_t stride_layer, stride_page, stride_token, stride_head;   /* elements */
    int n_pages;
    int n, delta, dst_shift;
    const int32_t* block_table; int n_table;
    const uint8_t* tags;                 /* [L][NB] */
    const uint64_t* blk_off;             /* [L][NB] byte offset inside the layer payload */
    const uint8_t* const* layer_payload; /* [L] */
    const uint64_t* layer_bytes;         /* [L] */
    const int32_t* reuse_idx;            /* [L][NB] */
    const int32_t* reuse_cnt;            /* [L] */
    int n_threads;                       /* OpenMP threads over (layer, reused block); <= 1 = serial */
    /* optional statistics of the fp32 recipe against the pair evaluated in double (may be NULL):
       [0] max abs difference of the bf16 results, [1] number of K elements whose bf16 differs, [2] K elements */
    double* k_stats;
} pkvo_restore_args;

static int restore_item(const pkvo_restore_args* a, const float* ct, const float* st, int l, int r, double* stats) {
    const int B = a->B, H = a->H, D = a->D, Dr = a->Dr, P = a->P, G = a->G;
    const int NB = (a->n + B - 1) / B;
    int j = a->reuse_idx[(int64_t)l * NB + r];
    if (j < 0 || j >= NB) return PKVO_E_BOUNDS;
    int tag = a->tags[(int64_t)l * NB + j];
    uint64_t rec = pkvo_record_bytes(tag, B, H, D, G);
    if (rec == 0) return PKVO_E_BOUNDS;
    uint64_t off = a->blk_off[(int64_t)l * NB + j];
    if (off > a->layer_bytes[l] || rec > a->layer_bytes[l] - off) return PKVO_E_BOUNDS;
    int valid = a->n - j * B < B ? a->n - j * B : B;
    /* every destination page of the block is validated before anything is written */
    for (int t = 0; t < valid; t++) {
        int64_t u = (int64_t)j * B + t + a->dst_shift;
        if (u / P >= a->n_table) return PKVO_E_BOUNDS;
        int32_t page = a->block_table[u / P];
        if (page < 0 || page >= a->n_pages) return PKVO_E_BOUNDS;
    }
    const uint64_t elems = (uint64_t)B * H * D;
    const int kf = k_fmt(tag), vf = v_fmt(tag);
    const uint8_t* kc = a->layer_payload[l] + off;
    const uint8_t* ks = kc + codes_bytes(kf, elems);
    const uint8_t* vc = ks + scales_bytes(kf, elems, G);
    const uint8_t* vs = vc + codes_bytes(vf, elems);
    float* x = (float*)malloc(sizeof(float) * (size_t)D);
    float* y = (float*)malloc(sizeof(float) * (size_t)D);
    uint16_t* raw = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)D);
    for (int t = 0; t < valid; t++) {
        int64_t u = (int64_t)j * B + t + a->dst_shift;
        int64_t base = (int64_t)l * a->stride_layer + (int64_t)a->block_table[u / P] * a->stride_page +
                       (u % P) * a->stride_token;
        for (int h = 0; h < H; h++) {
            uint16_t* kd = a->k_pool + base + (int64_t)h * a->stride_head;
            uint16_t* vd = a->v_pool + base + (int64_t)h * a->stride_head;
            /* V: dequantise and round once; a bf16 code is copied bit for bit; V gets no rotation (Section IV-C) */
            for (int c = 0; c < D; c++) {
                uint16_t rb; float v = dequant_elem(vc, vs, vf, H, D, G, t, h, c, &rb);
                vd[c] = vf == PKVO_FMT_BF16 ? rb : pkvo_f32_to_bf16(v);
            }
            /* K: dequantise, rotate the rotary pairs by delta, round once */
            for (int c = 0; c < D; c++) x[c] = dequant_elem(kc, ks, kf, H, D, G, t, h, c, &raw[c]);
            for (int c = 0; c < D; c++) kd[c] = kf == PKVO_FMT_BF16 ? raw[c] : pkvo_f32_to_bf16(x[c]);
            if (a->delta != 0) {
                pkvo_rotate_head_f32(x, D, Dr, a->rope_style, ct, st, y);
                for (int i = 0; i < Dr / 2; i++) {
                    int ia = a->rope_style == PKVO_ROPE_HALF ? i : 2 * i;
                    int ib = a->rope_style == PKVO_ROPE_HALF ? i + Dr / 2 : 2 * i + 1;
                    kd[ia] = pkvo_f32_to_bf16(y[ia]);
                    kd[ib] = pkvo_f32_to_bf16(y[ib]);
                    if (stats) {
                        double da = (double)x[ia] * ct[i] - (double)x[ib] * st[i];
                        double db = (double)x[ia] * st[i] + (double)x[ib] * ct[i];
                        uint16_t ia16 = pkvo_f32_to_bf16((float)da), ib16 = pkvo_f32_to_bf16((float)db);
                        double ea = fabs((double)pkvo_bf16_to_f32(ia16) - (double)pkvo_bf16_to_f32(kd[ia]));
                        double eb = fabs((double)pkvo_bf16_to_f32(ib16) - (double)pkvo_bf16_to_f32(kd[ib]));
                        if (ea > stats[0]) stats[0] = ea;
                        if (eb > stats[0]) stats[0] = eb;
                        stats[1] += (ia16 != kd[ia]) + (ib16 != kd[ib]);
                        stats[2] += 2;
                    }
                }
            }
        }
    }
    free(x); free(y); free(raw);
    return PKVO_OK;
}

/* Restore every reused block of every layer of one session.  A block whose directory entry, record
 * extent or destination pages are out of range is skipped whole and the call returns PKVO_E_BOUNDS
 * after finishing the rest.  Blocks of the repair set are never read and never written. */
int pkvo_restore(const pkvo_restore_args* a) {
    if (a->L <= 0 || a->H <= 0 || a->D <= 0 || (a->D & 1) || a->Dr < 0 || (a->Dr & 1) || a->Dr > a->D ||
        a->B <= 0 || a->P <= 0 || a->G <= 0 || a->D % a->G || a->n < 0 || a->dst_shift < 0 || a->dst_shift >= a->P)
        return PKVO_E_INVALID;
    if (a->rope_style != PKVO_ROPE_HALF && a->rope_style != PKVO_ROPE_INTERLEAVED) return PKVO_E_INVALID;
    const int NB = (a->n + a->B - 1) / a->B;
    float* ct = (float*)malloc(sizeof(float) * (size_t)(a->Dr / 2 + 1));
    float* st = (float*)malloc(sizeof(float) * (size_t)(a->Dr / 2 + 1));
    pkvo_rope_table(a->Dr, a->rope_base, a->inv_freq, a->delta, ct, st);
    int status = PKVO_OK;
    double s0 = 0, s1 = 0, s2 = 0;
    const int64_t items = (int64_t)a->L * NB;
#ifdef _OPENMP
    int nt = a->n_threads > 1 ? a->n_threads : 1;
#pragma omp parallel for schedule(dynamic, 8) num_threads(nt) reduction(max : s0) reduction(+ : s1, s2)
#endif
    for (int64_t it = 0; it < items; it++) {
        int l = (int)(it / NB), r = (int)(it % NB);
        if (r >= a->reuse_cnt[l]) continue;
        double st3[3] = {0, 0, 0};
        int rc = restore_item(a, ct, st, l, r, a->k_stats ? st3 : NULL);
        if (rc != PKVO_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            status = rc;
        }
        if (st3[0] > s0) s0 = st3[0];
        s1 += st3[1]; s2 += st3[2];
    }
    if (a->k_stats) { a->k_stats[0] = s0; a->k_stats[1] = s1; a->k_stats[2] = s2; }
    free(ct); free(st);
    return status;
}

int pkvo_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ checkpoint writer (offload side) */
/* Section IV-D, offload: gather the rows of each suffix block from the paged pool, compute per-group scales,
 * pack the block at its precision tag, and cluster blocks of the same representation into contiguous runs.
 * This is the inverse direction of restore; it is outside the resume path and is kept here as the oracle of
 * the library's checkpoint writer. */

/* Directory of the clustered layout: per layer all BF16-tag records, then INT8, INT4, K4V4, each run in
 * ascending block index.  blk_off [L][NB], layer_bytes [L].  An unknown tag makes the call fail. */
int pkvo_plan_checkpoint(const uint8_t* tags, int L, int NB, int B, int H, int D, int G,
                         uint64_t* blk_off, uint64_t* layer_bytes) {
    if (L <= 0 || NB < 0 || B <= 0 || H <= 0 || D <= 0 || G <= 0 || D % G) return PKVO_E_INVALID;
    for (int l = 0; l < L; l++) {
        uint64_t base = 0;
        for (int tag = 0; tag <= PKVO_TAG_K4V4; tag++) {
            uint64_t rec = pkvo_record_bytes(tag, B, H, D, G);
            for (int j = 0; j < NB; j++)
                if (tags[(int64_t)l * NB + j] == tag) { blk_off[(int64_t)l * NB + j] = base; base += rec; }
        }
        for (int j = 0; j < NB; j++) if (tags[(int64_t)l * NB + j] > PKVO_TAG_K4V4) return PKVO_E_INVALID;
        layer_bytes[l] = base;
    }
    return PKVO_OK;
}

typedef struct {
    int L, H, D, B, P, G;
    const uint16_t* k_pool; const uint16_t* v_pool;         /* bf16 bit patterns */
    int64_t stride_layer, stride_page, stride_token, stride_head;
    int n_pages;
    int n, src_shift;                                       /* suffix tokens; slot of the first one in logical page 0 */
    const int32_t* block_table; int n_table;
    const uint8_t* tags;                                    /* [L][NB] */
    const uint64_t* blk_off;                                /* [L][NB] */
    uint8_t* const* layer_payload;                          /* [L] destination buffers */
    const uint64_t* layer_bytes;                            /* [L] */
} pkvo_gather_args;

/* Encode one section (K or V) of one block: values are the pool's bf16 rows read as fp32; tokens past the end of
 * the suffix encode as zeros.  Quantiser: per group of G channels of one (token, head), s = fp16(amax / qmax),
 * code = clamp(rint(x / s), -qmax, qmax) with ties to even, s == 0 -> code 0; qmax = 127 (int8) or 7 (int4). */
static void encode_section(const pkvo_gather_args* a, const uint16_t* pool, int l, int j, int valid, int fmt,
                           uint8_t* codes, uint8_t* scales) {
    const int B = a->B, H = a->H, D = a->D, G = a->G, P = a->P;
    float* x = (float*)malloc(sizeof(float) * (size_t)G);
    int8_t* q = (int8_t*)malloc((size_t)G);
    for (int t = 0; t < B; t++) {
        int64_t u = (int64_t)j * B + t + a->src_shift;
        const uint16_t* row = NULL;
        if (t < valid)
            row = pool + (int64_t)l * a->stride_layer + (int64_t)a->block_table[u / P] * a->stride_page +
                  (u % P) * a->stride_token;
        for (int h = 0; h < H; h++) {
            const uint16_t* src = row ? row + (int64_t)h * a->stride_head : NULL;
            uint64_t e0 = ((uint64_t)t * H + h) * D;
            if (fmt == PKVO_FMT_BF16) {
                for (int c = 0; c < D; c++) {
                    uint16_t b = src ? src[c] : 0;
                    memcpy(codes + 2 * (e0 + c), &b, 2);
                }
                continue;
            }
            for (int g = 0; g < D / G; g++) {
                for (int i = 0; i < G; i++) x[i] = src ? pkvo_bf16_to_f32(src[g * G + i]) : 0.0f;
                uint16_t sb;
                pkvo_quantise_group(x, G, fmt == PKVO_FMT_INT8 ? 127 : 7, q, &sb);
                memcpy(scales + 2 * (((uint64_t)t * H + h) * (D / G) + g), &sb, 2);
                for (int i = 0; i < G; i++) {
                    uint64_t e = e0 + (uint64_t)g * G + i;
                    if (fmt == PKVO_FMT_INT8) codes[e] = (uint8_t)q[i];
                    else {
                        uint8_t nib = (uint8_t)q[i] & 15u;
                        if (e & 1) codes[e >> 1] = (uint8_t)((codes[e >> 1] & 0x0f) | (nib << 4));
                        else       codes[e >> 1] = (uint8_t)((codes[e >> 1] & 0xf0) | nib);
                    }
                }
            }
        }
    }
    free(x); free(q);
}

/* Write the record of every block of every layer.  A block whose tag, record extent or source pages are out of
 * range is skipped whole (its bytes are left as they were) and the call returns PKVO_E_BOUNDS at the end. */
int pkvo_quantize_gather(const pkvo_gather_args* a) {
    if (a->L <= 0 || a->H <= 0 || a->D <= 0 || a->B <= 0 || a->P <= 0 || a->G <= 0 || a->D % a->G || a->n < 0 ||
        a->src_shift < 0 || a->src_shift >= a->P)
        return PKVO_E_INVALID;
    const int NB = (a->n + a->B - 1) / a->B;
    const uint64_t elems = (uint64_t)a->B * a->H * a->D;
    int status = PKVO_OK;
    for (int l = 0; l < a->L; l++)
        for (int j = 0; j < NB; j++) {
            int tag = a->tags[(int64_t)l * NB + j];
            uint64_t rec = pkvo_record_bytes(tag, a->B, a->H, a->D, a->G);
            uint64_t off = a->blk_off[(int64_t)l * NB + j];
            int bad = rec == 0 || off > a->layer_bytes[l] || rec > a->layer_bytes[l] - off;
            int valid = a->n - j * a->B < a->B ? a->n - j * a->B : a->B;
            for (int t = 0; t < valid && !bad; t++) {
                int64_t u = (int64_t)j * a->B + t + a->src_shift;
                if (u / a->P >= a->n_table) { bad = 1; break; }
                int32_t page = a->block_table[u / a->P];
                if (page < 0 || page >= a->n_pages) bad = 1;
            }
            if (bad) { status = PKVO_E_BOUNDS; continue; }
            const int kf = k_fmt(tag), vf = v_fmt(tag);
            uint8_t* kc = a->layer_payload[l] + off;
            uint8_t* ks = kc + codes_bytes(kf, elems);
            uint8_t* vc = ks + scales_bytes(kf, elems, a->G);
            uint8_t* vs = vc + codes_bytes(vf, elems);
            encode_section(a, a->k_pool, l, j, valid, kf, kc, ks);
            encode_section(a, a->v_pool, l, j, valid, vf, vc, vs);
        }
    return status;
}

/* ------------------------------------------------------------------ token-level selection (Eqs. 9-12 as printed) */
/* The paper's own form of the selection: the importance score is per TOKEN, H is the set of the top-kappa tokens
 * outside the dirty token set D, and only then is D u H rounded to blocks:
 *   D   = the first min(max(dirty_tokens, 0), n) suffix tokens                      (Eq. 9)
 *   H_l = the min(top_tokens, #candidates) tokens outside D with the largest score; ties: lower token index (Eq. 11)
 *   R_l = blocks holding a token of D u H_l,  F_l = the other blocks, both ascending (Eq. 12)
 * token_mass is u64 [L][n] (the exact attention mass of Eq. 10 at token granularity, B = 1 in pkvo_block_mass).
 * LAYERS_SHARED ranks on the mass summed over layers, the request-level reading of Eq. 10.
 * Outputs as pkvo_select, plus an optional token mask u8 [L][n] (1 = token in D u H_l). */
int pkvo_select_tokens(const uint64_t* token_mass, int L, int n, int B, int dirty_tokens, int top_tokens, int layer_mode,
                       uint8_t* token_mask, uint8_t* mask, int32_t* repair_idx, int32_t* repair_cnt,
                       int32_t* reuse_idx, int32_t* reuse_cnt) {
    if (L <= 0 || n < 0 || B <= 0 || top_tokens < 0) return PKVO_E_INVALID;
    if (layer_mode != PKVO_LAYERS_INDEPENDENT && layer_mode != PKVO_LAYERS_SHARED) return PKVO_E_INVALID;
    int NB = (n + B - 1) / B;
    int64_t nd64 = dirty_tokens < 0 ? 0 : dirty_tokens;
    if (nd64 > n) nd64 = n;
    int nd = (int)nd64;
    cand_t* cand = (cand_t*)malloc(sizeof(cand_t) * (size_t)(n > 0 ? n : 1));
    uint8_t* tmask = (uint8_t*)malloc((size_t)(n > 0 ? n : 1));
    uint64_t* shared = NULL;
    if (layer_mode == PKVO_LAYERS_SHARED) {
        shared = (uint64_t*)calloc((size_t)(n > 0 ? n : 1), sizeof(uint64_t));
        for (int l = 0; l < L; l++) for (int i = 0; i < n; i++) shared[i] += token_mass[(int64_t)l * n + i];
    }
    for (int l = 0; l < L; l++) {
        const uint64_t* m = shared ? shared : token_mass + (int64_t)l * n;
        int nc = 0;
        for (int i = 0; i < n; i++) {
            tmask[i] = i < nd;
            if (i >= nd) { cand[nc].mass = m[i]; cand[nc].idx = i; nc++; }
        }
        qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
        int take = top_tokens < nc ? top_tokens : nc;
        for (int i = 0; i < take; i++) tmask[cand[i].idx] = 1;
        if (token_mask) memcpy(token_mask + (int64_t)l * n, tmask, (size_t)n);
        int nr = 0, nf = 0;
        for (int j = 0; j < NB; j++) {
            int hit = 0;
            for (int i = j * B; i < (j + 1) * B && i < n; i++) hit |= tmask[i];   /* BlockRound: blocks that intersect */
            mask[(int64_t)l * NB + j] = (uint8_t)hit;
            if (hit) repair_idx[(int64_t)l * NB + nr++] = j;
            else     reuse_idx[(int64_t)l * NB + nf++] = j;
        }
        for (int i = nr; i < NB; i++) repair_idx[(int64_t)l * NB + i] = -1;
        for (int i = nf; i < NB; i++) reuse_idx[(int64_t)l * NB + i] = -1;
        repair_cnt[l] = nr; reuse_cnt[l] = nf;
    }
    free(cand); free(tmask); free(shared);
    return PKVO_OK;
}

/* ------------------------------------------------------------------ precision planner (Eqs. 13-14) */
/* Per block b of the suffix: Z_i = sqrt(A_i * e_i) for its tokens (A_i the normalised stored attention mass, e_i the
 * normalised residual of the candidate low-bit V representation), r_b = alpha * max Z + (1 - alpha) * mean Z, and
 *   tag = BF16 (the full-precision tier)  if r_b >= tau_H
 *         INT8 (K8/V8)                    if tau_L <= r_b < tau_H
 *         INT4 (K8/V4)                    if r_b < tau_L and G4(b)
 *         INT8                            if r_b < tau_L and not G4(b)
 * The paper leaves the low-bit test G4 open; the reading here is G4(b) = (max_i e_i <= eps4).  All arithmetic is
 * fp32 with every operation rounded on its own, tokens taken in ascending order, so that the decision is made in
 * one fixed precision on both sides.  attn, resid: fp32 [n]; tags u8 [NB]; risk fp32 [NB] (optional). */
int pkvo_plan_precision(const float* attn, const float* resid, int n, int B, float alpha, float tau_L, float tau_H,
                        float eps4, uint8_t* tags, float* risk) {
    if (n < 0 || B <= 0 || !(alpha >= 0.0f && alpha <= 1.0f) || !(tau_L < tau_H)) return PKVO_E_INVALID;
    int NB = (n + B - 1) / B;
    for (int j = 0; j < NB; j++) {
        float zmax = 0.0f, zsum = 0.0f, emax = 0.0f;
        int cnt = 0;
        for (int i = j * B; i < (j + 1) * B && i < n; i++) {
            volatile float prod = attn[i] * resid[i];
            float z = sqrtf(prod);
            if (z > zmax) zmax = z;
            if (resid[i] > emax) emax = resid[i];
            volatile float s = zsum + z;
            zsum = s;
            cnt++;
        }
        volatile float mean = zsum / (float)cnt;
        volatile float t1 = alpha * zmax;
        volatile float om = 1.0f - alpha;
        volatile float t2 = om * mean;
        float r = t1 + t2;
        if (risk) risk[j] = r;
        uint8_t tag;
        if (r >= tau_H) tag = PKVO_TAG_BF16;
        else if (r >= tau_L) tag = PKVO_TAG_INT8;
        else tag = emax <= eps4 ? PKVO_TAG_INT4 : PKVO_TAG_INT8;
        tags[j] = tag;
    }
    return PKVO_OK;
}
