/*
 * FFD oracle: a plain, slow, fp64 CPU statement of the sparse decode-attention path of
 * "Faster Than Flash" (FFD): 2-bit mid-rise key quantizer (App. A.1), approximate scores from the
 * 2-bit keys, pseudo-max over sink + local blocks (Sec. 3.2, Alg. 1 "Pseudo-max estimation"),
 * top-delta block selection (Eq. 1, Alg. 1 "Top-delta selection"), exact softmax attention over the
 * kept blocks (Alg. 1 "Fine-grained refinement"), and dense softmax attention.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists to define correctness for the CUDA library and to be timed as
 * a reported CPU baseline.  It shares no code with the CUDA path and the product never calls it.
 *
 * Style: every step is the definition written out, token by token and channel by channel, in double
 * precision on the exact values of the bf16 / fp16 inputs.  No blocking, no fusion, no reordering.  The
 * only parallelism is an OpenMP loop over independent units: (sequence, query head) pairs in the decode
 * functions, blocks in the quantizer.
 *
 * Readings of the paper that this file fixes (each is a reading, not something the paper prints; the
 * ones marked "parity unpinned" have no independent pin):
 *   - bit width 2, codebook {-1.5,-0.5,+0.5,+1.5}, scale = absmax/1.5            (App. A.1, printed)
 *   - the deeper thumbnails of App. "Bandwidth Proportionality of Quantization Depth" (4 and 8 bits): the paper
 *     prints no formulas for them; reading: the same symmetric mid-rise construction with 2^b levels
 *     +-(k + 1/2), k = 0 .. 2^(b-1) - 1, scale = absmax / (2^(b-1) - 1/2), nearest level with ties outward
 *     (for b = 2 this is the printed codebook and scale)                        (parity unpinned: a reading)
 *   - one scale per (64-token block, KV head, channel), absmax over the block's valid rows;
 *     stored as fp16 = RNE(fp32(absmax)/1.5f), saturated at 65504             (parity unpinned)
 *   - nearest level written as comparisons: |x| >= s -> outer level, x = 0 -> +0.5; this equals the
 *     arg-min of App. A.1 everywhere except exact ties
 *   - approximate scores and the pseudo-max carry 1/sqrt(d); delta is a natural-log logit gap (Eq. 1-2)
 *   - the pseudo-max uses the quantized scores (Alg. 1), so the kept set is never empty
 *   - sink set = first n_sink blocks, local set = last n_local blocks (incl. the partial tail)
 *                                                                              (parity unpinned)
 *   - selection is per query head; whole 64-token blocks are kept or skipped  (parity unpinned)
 *   - the partial tail block is quantized over its valid rows; rows past seq_len never contribute
 *                                                                              (parity unpinned)
 *   - refinement uses the full 16-bit K (the two-term form of Sec. 3.3 equals q.k when the residual
 *     is exact), softmax over the kept tokens only
 *   - optional 8-bit residual format (Sec. 3.1 "k -> {k^quant, k^res}", Alg. 1 Dequant, Sec. 3.3 two-term
 *     score): the paper does not print the residual quantizer.  Reading: symmetric int8 on the grid
 *     s/254 of the channel's own 2-bit scale s (the residual of a mid-rise level lies in [-s/2, s/2]),
 *     code8 = clamp(rint(r * (254/s)), -127, 127), r = x - level*s, all three operations in IEEE
 *     binary32 (the precision the code is decided in); refinement then uses
 *     K^full = level*s + code8*s/254 in place of the 16-bit K                  (parity unpinned: the
 *     grid is this file's choice; what is pinned is the error bound and the two-term identity)
 *
 * Layouts (all host pointers, row-major, innermost last):
 *   q        bf16 bits  [B, Hq, D]
 *   k_cache  bf16 bits  [num_pages, Hkv, BLK, D]      v_cache the same
 *   codes    u8 0..3    [num_pages, Hkv, BLK, D]      level = code - 1.5
 *   scales   fp16 bits  [num_pages, Hkv, D]
 *   k_res    int8       [num_pages, Hkv, BLK, D]      residual in units of scale/254
 *   block_table int32   [B, max_blocks]  logical block -> physical page; NULL = b*max_blocks + blk
 *   seq_lens int32      [B]
 *   query head h belongs to KV head h / (Hq/Hkv).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;

void ffd_oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int ffd_oracle_get_threads(void) { return g_threads; }
int ffd_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ---- number formats -------------------------------------------------------------------------- */

/* bf16 is the top half of an IEEE binary32. */
static double bf16_value(uint16_t bits) {
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double fp16_value(uint16_t bits) {
    int sign = (bits >> 15) & 1;
    int expo = (bits >> 10) & 0x1f;
    int frac = bits & 0x3ff;
    double v;
    if (expo == 0) v = ldexp((double)frac, -24);                 /* subnormal: frac * 2^-24 */
    else if (expo == 31) v = frac ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    return sign ? -v : v;
}

/* Round a finite non-negative binary32 to binary16, ties to even, by the definition: pick the fp16
 * quantum for the value's binade, round the ratio to the nearest even integer. */
static uint16_t fp16_round_nonneg(float f) {
    double v = (double)f;
    if (v == 0.0) return 0;
    int e;
    (void)frexp(v, &e);            /* v = m * 2^e, m in [0.5,1)  ->  floor(log2 v) = e-1 */
    int binade = e - 1;
    if (binade < -14) binade = -14; /* subnormal range shares the quantum 2^-24 */
    double quantum = ldexp(1.0, binade - 10);
    double n = rint(v / quantum);   /* default rounding mode: to nearest, ties to even */
    double r = n * quantum;
    if (r >= 65536.0) return 0x7c00; /* overflow to +inf (unreachable after saturation) */
    if (r == 0.0) return 0;
    (void)frexp(r, &e);
    binade = e - 1;
    if (binade < -14) return (uint16_t)ldexp(r, 24);             /* subnormal */
    double frac = r / ldexp(1.0, binade) - 1.0;                  /* in [0,1) */
    return (uint16_t)(((binade + 15) << 10) | (int)(frac * 1024.0));
}

/* exported so tests can pin the two conversions against a library's */
double ffd_oracle_fp16_value(uint16_t bits) { return fp16_value(bits); }
double ffd_oracle_bf16_value(uint16_t bits) { return bf16_value(bits); }
uint16_t ffd_oracle_fp16_round(float f) { return fp16_round_nonneg(f); }

static int64_t page_of(const int32_t* block_table, int b, int blk, int max_blocks) {
    return block_table ? (int64_t)block_table[(int64_t)b * max_blocks + blk]
                       : (int64_t)b * max_blocks + blk;
}

static int valid_rows(int seq_len, int blk, int BLK) {
    int rows = seq_len - blk * BLK;
    return rows > BLK ? BLK : rows;
}

/* ---- App. A.1: the quantizer ----------------------------------------------------------------- */

/* One (page, KV head) tile with b-bit thumbnails.  For every channel c: a = max over valid rows of |K[r,c]|;
 * s = fp16(fp32(a) / (2^(b-1) - 1/2)) saturated at 65504; the code of x is the index (0 .. 2^b - 1) of the nearest of
 * the 2^b levels +-(k + 1/2) * s, found by counting the cell boundaries k * s that |x| reaches (k * s is exact in
 * double): ties go outward, +-0 takes +1/2.  b = 2 is App. A.1 as printed. */
static void quantize_tile(const uint16_t* k_tile, int rows, int BLK, int D, int bits, uint8_t* codes, uint16_t* scales) {
    const int half_levels = 1 << (bits - 1);                 /* levels on each side of zero */
    const float top = (float)half_levels - 0.5f;             /* 1.5, 7.5, 127.5 */
    for (int c = 0; c < D; ++c) {
        float a = 0.0f;
        for (int r = 0; r < rows; ++r) {
            float x = (float)fabs(bf16_value(k_tile[(int64_t)r * D + c]));
            if (x > a) a = x;
        }
        float s32 = a / top;                      /* IEEE binary32 division, round to nearest */
        if (s32 > 65504.0f) s32 = 65504.0f;
        uint16_t sbits = fp16_round_nonneg(s32);
        scales[c] = sbits;
        double s = fp16_value(sbits);
        for (int r = 0; r < BLK; ++r) {
            uint8_t code = 0;                     /* padding rows: don't-care, written as 0 */
            if (r < rows) {
                double x = bf16_value(k_tile[(int64_t)r * D + c]);
                int neg = x < 0.0;                /* -0.0 is not negative */
                int m = 0;                        /* cell of |x|: [m s, (m + 1) s), the last one open-ended */
                for (int k = 1; k < half_levels; ++k)
                    if (fabs(x) >= (double)k * s) m = k;
                code = (uint8_t)(neg ? half_levels - 1 - m : half_levels + m);
            }
            codes[(int64_t)r * D + c] = code;
        }
    }
}

/* Quantize every logical block of every sequence that holds at least one valid token (bits = 2, 4 or 8). */
int ffd_oracle_quantize(const uint16_t* k_cache, uint8_t* codes, uint16_t* scales, const int32_t* block_table,
                        const int32_t* seq_lens, int B, int Hkv, int D, int BLK, int max_blocks, int num_pages, int bits) {
    if (bits != 2 && bits != 4 && bits != 8) return 5;
    for (int b = 0; b < B; ++b) {
        int nb = (seq_lens[b] + BLK - 1) / BLK;
        if (seq_lens[b] < 0 || nb > max_blocks) return 2;
        for (int blk = 0; blk < nb; ++blk) {
            int64_t page = page_of(block_table, b, blk, max_blocks);
            if (page < 0 || page >= num_pages) return 3;
        }
    }
    for (int b = 0; b < B; ++b) {
        int nb = (seq_lens[b] + BLK - 1) / BLK;
#pragma omp parallel for schedule(static) num_threads(g_threads)
        for (int blk = 0; blk < nb; ++blk) {
            int64_t page = page_of(block_table, b, blk, max_blocks);
            int rows = valid_rows(seq_lens[b], blk, BLK);
            for (int g = 0; g < Hkv; ++g) {
                int64_t tile = page * Hkv + g;
                quantize_tile(k_cache + tile * BLK * D, rows, BLK, D, bits, codes + tile * BLK * D, scales + tile * D);
            }
        }
    }
    return 0;
}

/* ---- Sec. 3.1: the 8-bit residual ------------------------------------------------------------- */

/* Residual code of one element: x (bf16 bits), its 2-bit code and the channel's scale (fp16 bits).
 * Every operation is a single IEEE binary32 operation (level*s is exact in binary32). */
static int8_t residual_code(uint16_t xbits, uint8_t code, uint16_t sbits) {
    float s = (float)fp16_value(sbits);
    if (s == 0.0f) return 0;                      /* all-zero channel: nothing to refine */
    float x = (float)bf16_value(xbits);
    float level_s = ((float)code - 1.5f) * s;     /* exact: 11 significant bits times 1.5 or 0.5 */
    float r = x - level_s;
    float inv = 254.0f / s;
    float t = rintf(r * inv);                     /* to nearest, ties to even */
    if (t > 127.0f) t = 127.0f;
    if (t < -127.0f) t = -127.0f;
    return (int8_t)t;
}

/* Residual codes of every valid token, given the 2-bit codes and scales; padding rows get 0. */
int ffd_oracle_quantize_residual(const uint16_t* k_cache, const uint8_t* codes, const uint16_t* scales, int8_t* k_res,
                                 const int32_t* block_table, const int32_t* seq_lens, int B, int Hkv, int D, int BLK,
                                 int max_blocks, int num_pages) {
    for (int b = 0; b < B; ++b) {
        int nb = (seq_lens[b] + BLK - 1) / BLK;
        if (seq_lens[b] < 0 || nb > max_blocks) return 2;
        for (int blk = 0; blk < nb; ++blk) {
            int64_t page = page_of(block_table, b, blk, max_blocks);
            if (page < 0 || page >= num_pages) return 3;
        }
    }
    for (int b = 0; b < B; ++b) {
        int nb = (seq_lens[b] + BLK - 1) / BLK;
#pragma omp parallel for schedule(static) num_threads(g_threads)
        for (int blk = 0; blk < nb; ++blk) {
            int64_t page = page_of(block_table, b, blk, max_blocks);
            int rows = valid_rows(seq_lens[b], blk, BLK);
            for (int g = 0; g < Hkv; ++g) {
                int64_t tile = page * Hkv + g;
                for (int r = 0; r < BLK; ++r)
                    for (int c = 0; c < D; ++c) {
                        int64_t e = (tile * BLK + r) * D + c;
                        k_res[e] = r < rows ? residual_code(k_cache[e], codes[e], scales[tile * D + c]) : 0;
                    }
            }
        }
    }
    return 0;
}

/* Alg. 1 "Dequant": the key the refinement sees in the residual format. */
static double dequant_full(uint8_t code, int8_t res, uint16_t sbits) {
    double s = fp16_value(sbits);
    return ((double)code - 1.5) * s + (double)res * s / 254.0;
}

/* ---- Alg. 1 for one (sequence, query head) ---------------------------------------------------- */

typedef struct {
    const uint16_t *q, *k_cache, *v_cache, *scales;
    const uint8_t* codes;
    const int32_t *block_table, *seq_lens;
    int B, Hq, Hkv, D, BLK, max_blocks, num_pages, n_sink, n_local;
    double sm_scale, delta;
    double level_offset;        /* level of code c = c - level_offset: (2^b - 1) / 2 = 1.5, 7.5, 127.5 */
    const uint8_t* forced_mask; /* nullable [B,Hq,max_blocks]: use these decisions instead of top-delta */
    double *out, *lse, *block_max, *mtilde;
    uint8_t* kept;
    const int8_t* k_res;        /* nullable: refine from Dequant(codes, k_res) instead of the 16-bit K */
    int rule;                   /* selection rule, see ffd_oracle_decode */
    int top_k;                  /* rule 3 only */
    double* thr;                /* nullable [B,Hq,max_blocks]: the threshold every block's maximum was compared with */
} decode_args;

static void softmax_attention_over_mask(const decode_args* a, int b, int h, const uint8_t* keep, double* out,
                                        double* lse) {
    int D = a->D, BLK = a->BLK, g = h / (a->Hq / a->Hkv);
    int N = a->seq_lens[b], nb = (N + BLK - 1) / BLK;
    const uint16_t* qv = a->q + ((int64_t)b * a->Hq + h) * D;
    /* pass 1: the exact logits of kept tokens and their maximum */
    double* s = (double*)malloc(sizeof(double) * (size_t)(nb > 0 ? nb : 1) * BLK);
    double M = -INFINITY;
    for (int blk = 0; blk < nb; ++blk) {
        if (!keep[blk]) continue;
        int64_t tile = page_of(a->block_table, b, blk, a->max_blocks) * a->Hkv + g;
        int rows = valid_rows(N, blk, BLK);
        for (int r = 0; r < rows; ++r) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c) {
                int64_t e = (tile * BLK + r) * D + c;
                double k = a->k_res ? dequant_full(a->codes[e], a->k_res[e], a->scales[tile * D + c])
                                    : bf16_value(a->k_cache[e]);
                dot += bf16_value(qv[c]) * k;
            }
            s[blk * BLK + r] = a->sm_scale * dot;
            if (s[blk * BLK + r] > M) M = s[blk * BLK + r];
        }
    }
    /* pass 2: softmax weights and the weighted sum of V */
    double L = 0.0;
    for (int c = 0; c < D; ++c) out[c] = 0.0;
    for (int blk = 0; blk < nb; ++blk) {
        if (!keep[blk]) continue;
        int64_t tile = page_of(a->block_table, b, blk, a->max_blocks) * a->Hkv + g;
        int rows = valid_rows(N, blk, BLK);
        for (int r = 0; r < rows; ++r) {
            double p = exp(s[blk * BLK + r] - M);
            L += p;
            for (int c = 0; c < D; ++c) out[c] += p * bf16_value(a->v_cache[(tile * BLK + r) * D + c]);
        }
    }
    if (L > 0.0) {
        for (int c = 0; c < D; ++c) out[c] /= L;
        *lse = M + log(L);
    } else {
        *lse = -INFINITY; /* empty sequence: zeros */
    }
    free(s);
}

static void decode_one(const decode_args* a, int b, int h) {
    int D = a->D, BLK = a->BLK, g = h / (a->Hq / a->Hkv);
    int N = a->seq_lens[b], nb = (N + BLK - 1) / BLK;
    const uint16_t* qv = a->q + ((int64_t)b * a->Hq + h) * D;
    int64_t row = ((int64_t)b * a->Hq + h);
    double* bm = a->block_max + row * a->max_blocks;
    uint8_t* keep = a->kept + row * a->max_blocks;

    /* approximate scores from the dequantized 2-bit keys; per-block maximum */
    for (int blk = 0; blk < nb; ++blk) {
        int64_t tile = page_of(a->block_table, b, blk, a->max_blocks) * a->Hkv + g;
        int rows = valid_rows(N, blk, BLK);
        double best = -INFINITY;
        for (int r = 0; r < rows; ++r) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c) {
                double khat = ((double)a->codes[(tile * BLK + r) * D + c] - a->level_offset) * fp16_value(a->scales[tile * D + c]);
                dot += bf16_value(qv[c]) * khat;
            }
            double s_approx = a->sm_scale * dot;
            if (s_approx > best) best = s_approx;
        }
        bm[blk] = best;
    }
    /* pseudo-max over the sink and local blocks */
    double mt = -INFINITY;
    for (int blk = 0; blk < nb; ++blk)
        if (blk < a->n_sink || blk >= nb - a->n_local)
            if (bm[blk] > mt) mt = bm[blk];
    a->mtilde[row] = mt;
    /* the threshold of every block under the selection rule */
    double* thr = (double*)malloc(sizeof(double) * (size_t)(nb > 0 ? nb : 1));
    if (a->rule == 0) {            /* Alg. 1 / Eq. 1: the pseudo-max of the sink and local blocks */
        for (int blk = 0; blk < nb; ++blk) thr[blk] = mt - a->delta;
    } else if (a->rule == 1) {     /* the comparison rule of Sec. 5.2: the maximum over all blocks (a first pass of its own) */
        double m = -INFINITY;
        for (int blk = 0; blk < nb; ++blk)
            if (bm[blk] > m) m = bm[blk];
        for (int blk = 0; blk < nb; ++blk) thr[blk] = m - a->delta;
    } else if (a->rule == 2) {     /* a streaming scan's own reference: the pseudo-max raised by every block maximum
                                      met so far, blocks taken in logical order, the block itself included */
        double run = mt;
        for (int blk = 0; blk < nb; ++blk) {
            if (bm[blk] > run) run = bm[blk];
            thr[blk] = run - a->delta;
        }
    } else {                       /* fixed budget (Fig. 1a): the top_k blocks by block maximum; blocks equal to the
                                      k-th largest maximum are all kept; delta plays no part */
        double tau = -INFINITY;
        if (a->top_k < nb) {
            /* the k-th largest by repeated extraction (k is small next to nb; clarity over speed) */
            uint8_t* used = (uint8_t*)calloc((size_t)(nb > 0 ? nb : 1), 1);
            for (int i = 0; i < a->top_k; ++i) {
                int arg = -1;
                for (int blk = 0; blk < nb; ++blk)
                    if (!used[blk] && (arg < 0 || bm[blk] > bm[arg])) arg = blk;
                used[arg] = 1;
                tau = bm[arg];
            }
            free(used);
        }
        for (int blk = 0; blk < nb; ++blk) thr[blk] = tau;
    }
    for (int blk = 0; blk < nb; ++blk) {
        if (a->thr) a->thr[row * a->max_blocks + blk] = thr[blk];
        if (a->forced_mask) keep[blk] = a->forced_mask[row * a->max_blocks + blk];
        else keep[blk] = (a->rule != 3 && isinf(a->delta)) ? 1 : (bm[blk] >= thr[blk]);
    }
    free(thr);
    /* exact attention over the kept blocks */
    softmax_attention_over_mask(a, b, h, keep, a->out + row * D, a->lse + row);
}

static int check_geometry(const decode_args* a) {
    if (a->Hq % a->Hkv) return 1;
    for (int b = 0; b < a->B; ++b) {
        int nb = (a->seq_lens[b] + a->BLK - 1) / a->BLK;
        if (a->seq_lens[b] < 0 || nb > a->max_blocks) return 2;
        for (int blk = 0; blk < nb; ++blk) {
            int64_t page = page_of(a->block_table, b, blk, a->max_blocks);
            if (page < 0 || page >= a->num_pages) return 3;
        }
    }
    return 0;
}

/* Sparse decode step.  Rows of kept / block_max beyond a sequence's block count are left untouched.
 * k_res: NULL = refine from the 16-bit K; else from the 2-bit + 8-bit reconstruction (k_cache is then unused).
 * units: nullable list of n_units (b, h) pairs to compute; NULL = all B*Hq pairs.
 * rule: which reference the block maxima are compared with.  0 = the paper's method (Alg. 1, Eq. 1): m_tilde - delta.
 * 1 = global approximate maximum - delta (Sec. 5.2's comparison).  2 = scan-order running maximum - delta: the pseudo-max
 * raised by the block maxima met so far in logical block order (the whole sequence is one scan; the split geometry of an
 * implementation plays no part).  3 = top-k by block maximum (Fig. 1a's fixed budget; the selection-overhead comparison
 * of Sec. 4.4), ties with the k-th value kept, 1 <= top_k.  thr_out: nullable, the per-block thresholds. */
int ffd_oracle_decode(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache, const uint8_t* codes,
                      const uint16_t* scales, const int32_t* block_table, const int32_t* seq_lens, int B, int Hq,
                      int Hkv, int D, int BLK, int max_blocks, int num_pages, int n_sink, int n_local,
                      double sm_scale, double delta, const uint8_t* forced_mask, const int32_t* units, int n_units,
                      double* out, double* lse, uint8_t* kept, double* block_max, double* mtilde, const int8_t* k_res,
                      int bits, int rule, int top_k, double* thr_out) {
    if (bits != 2 && bits != 4 && bits != 8) return 5;
    if (rule < 0 || rule > 3 || (rule == 3 && top_k < 1)) return 6;
    if (k_res && bits != 2) return 5;             /* the residual format is defined on the 2-bit thumbnails */
    decode_args a = {q, k_cache, v_cache, scales, codes, block_table, seq_lens, B, Hq, Hkv, D, BLK, max_blocks,
                     num_pages, n_sink, n_local, sm_scale, delta, (double)((1 << bits) - 1) / 2.0, forced_mask, out, lse,
                     block_max, mtilde, kept, k_res, rule, top_k, thr_out};
    int rc = check_geometry(&a);
    if (rc) return rc;
    if (isnan(delta) || delta < 0.0) return 4;
    int total = units ? n_units : B * Hq;
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
    for (int u = 0; u < total; ++u) {
        int b = units ? units[2 * u] : u / Hq;
        int h = units ? units[2 * u + 1] : u % Hq;
        decode_one(&a, b, h);
    }
    return 0;
}

/* Dense softmax attention over every valid token: softmax(q K^T / sqrt(d)) V. */
int ffd_oracle_dense(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache, const int32_t* block_table,
                     const int32_t* seq_lens, int B, int Hq, int Hkv, int D, int BLK, int max_blocks, int num_pages,
                     double sm_scale, const int32_t* units, int n_units, double* out, double* lse) {
    decode_args a = {q, k_cache, v_cache, NULL, NULL, block_table, seq_lens, B, Hq, Hkv, D, BLK, max_blocks,
                     num_pages, 0, 0, sm_scale, INFINITY, 1.5, NULL, out, lse, NULL, NULL, NULL, NULL, 0, 0, NULL};
    int rc = check_geometry(&a);
    if (rc) return rc;
    int total = units ? n_units : B * Hq;
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
    for (int u = 0; u < total; ++u) {
        int b = units ? units[2 * u] : u / Hq;
        int h = units ? units[2 * u + 1] : u % Hq;
        uint8_t* all = (uint8_t*)malloc((size_t)(max_blocks > 0 ? max_blocks : 1));
        memset(all, 1, (size_t)(max_blocks > 0 ? max_blocks : 1));
        int64_t row = (int64_t)b * Hq + h;
        softmax_attention_over_mask(&a, b, h, all, out + row * D, lse + row);
        free(all);
    }
    return 0;
}
