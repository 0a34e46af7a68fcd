/*
 * CPU checker for the progressive SQuant solver (SQuant-E -> SQuant-K -> SQuant-C).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded restatement of
 * the method, written to be checked against the paper by eye.  Nothing in the product
 * path may call it; only the test-suite, the smoke check and the benchmark's CPU-baseline
 * leg do.  It shares no code, header, table or helper with the CUDA implementation.
 *
 * Notation follows the paper (Sec. 2.1): M output channels, N kernels per output channel,
 * K = kh*kw elements per kernel; a fully connected layer is (M, N, 1).  Weights are
 * row-major [M][N][K]; the "flat index" of an element is its offset n*K + i inside its
 * output channel.
 *
 * Steps, per output channel m (the M sub-problems are independent, Sec. 3.4 "On-the-Fly
 * Framework"):
 *
 *  scale   The paper takes the scale vector s as an input of Algorithm 1 and only says
 *          that the range is set per output channel (Sec. 4).  Reading used here:
 *          symmetric absmax, s_m = max|W[m]| / qmax in IEEE fp32, qmax = 2^(bits-1) - 1.
 *          A channel whose absmax is below 2^-100 (which includes the all-zero channel)
 *          gets s_m = 1, so every code is 0.
 *          Algorithm 1 itself takes the scale vector as an INPUT, and Sec. 2.2 clips
 *          round(w / s) to the integer range; with a caller-supplied scale (scales_in, one
 *          per output channel) that clip really fires.  The paper says nothing about clipped
 *          elements in SQuant-K / SQuant-C.  Reading used here: a clipped element keeps its
 *          saturated code, its perturbation p = q - w/s (now possibly far beyond 0.5) enters
 *          every kernel and channel sum like any other, and it can never be flipped outward
 *          (the flipped code would leave the range), so it is never a candidate; when a
 *          kernel or channel has fewer candidates than round(|e|) asks for, all of them are
 *          flipped and the remaining |e| > 0.5 is what the error sums report.  A supplied
 *          scale that is not a positive finite number is replaced by 1.  Perturbations are
 *          held in 64 bits; |w / s| is assumed below 2^12.
 *
 *  E       Algorithm 1 "Scale and SQuant-E (Rounding)" / Eq. 9: x = w / s_m (IEEE fp32
 *          division), q = round-to-nearest(x) with ties to even, clipped to [qmin, qmax]
 *          (Sec. 2.2), perturbation p = q - x ("rounded up" is positive, as in App. B.1's
 *          0.7 -> 1 gives +0.3).  p is then converted ONCE to fixed point,
 *          P = nearbyint(p * 2^30); every later sum, comparison and threshold is integer
 *          arithmetic on P, so results do not depend on summation order.
 *
 *  K       Algorithm 2 (SQuantFlip) on each kernel: e = sum_i P; only elements whose
 *          perturbation has the sign of e are candidates; k = round(|e|); flip the k
 *          candidates with the largest |P| by one step against that sign.  Ties of
 *          round(|e|) at exactly one half go to the smaller k (App. B.3 gives the target
 *          interval as (-0.5, 0.5]; a flip never lowers the element term, App. B.2), ties
 *          of |P| go to the lower flat index.  An element whose flipped code would leave
 *          [qmin, qmax] is not a candidate.
 *
 *  update  Algorithm 3 (UpdatePerturbation): each kernel keeps exactly one candidate for
 *          SQuant-C.  "Over SQuant" (k > |e|): the last flipped element, with its
 *          perturbation AFTER the flip (0.5 <= |v| < 1; the example in App. B.3 uses
 *          -0.7), so that SQuant-C flips it back.  "Under SQuant" (otherwise): the first
 *          un-flipped candidate (the (k+1)-th largest), |v| <= 0.5.  e = 0: no candidate.
 *
 *  C       Algorithm 2 again on the channel, with the kernels' candidates as keys:
 *          e_c = the TRUE sum of all perturbations of the channel (Eq. 11 constrains the
 *          sum over all n, i); candidates are the kernels whose v has the sign of e_c;
 *          k_c = round(|e_c|) (same tie rule); the k_c kernels with the largest |v|
 *          (ties: lower kernel index) get their one candidate element flipped.
 *          Without SQuant-K in the mode mask every element is its own candidate.
 *
 *  emit    int8 codes, fp32 scales, and the final signed error sums per kernel and per
 *          channel as (float)(integer sum) * 2^-30.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SQO_ONE  ((int64_t)1 << 30)
#define SQO_HALF ((int64_t)1 << 29)

enum { SQO_MODE_E = 1u, SQO_MODE_K = 2u, SQO_MODE_C = 4u };
enum { SQO_FLAG_NARROW_RANGE = 1u, SQO_FLAG_PACK_INT4 = 2u };
enum { SQO_OK = 0, SQO_ERR_ARG = -1, SQO_ERR_NOMEM = -2 };

typedef struct {
    int32_t bits;    /* 2..8 */
    uint32_t mode;   /* SQO_MODE_E | SQO_MODE_K | SQO_MODE_C */
    uint32_t flags;  /* SQO_FLAG_NARROW_RANGE: codes in [-qmax, qmax];
                        SQO_FLAG_PACK_INT4 (bits <= 4): two codes per byte, low nibble = even flat
                        index, ceil(N*K/2) bytes per output channel */
} sqo_options;

typedef struct {
    int64_t mag;  /* |perturbation| in units of 2^-30 */
    int32_t idx;  /* flat index inside the output channel */
} sqo_cand;

/* Order of Algorithm 2's TopK: larger |perturbation| first, equal ones by lower index. */
static int sqo_cand_cmp(const void *a, const void *b)
{
    const sqo_cand *x = (const sqo_cand *)a, *y = (const sqo_cand *)b;
    if (x->mag != y->mag) return x->mag > y->mag ? -1 : 1;
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;
    return 0;
}

/* k = round(|e|) of Algorithm 2, |e| in units of 2^-30; exactly-half goes down. */
static int64_t sqo_flip_count(int64_t abs_e)
{
    return (abs_e + SQO_HALF - 1) >> 30;
}

static int sqo_sign64(int64_t v) { return (v > 0) - (v < 0); }

typedef struct {
    int32_t *q;      /* [N*K] integer codes */
    int64_t *P;      /* [N*K] fixed-point perturbations */
    uint8_t *flip;   /* [N*K] bit0: flipped by SQuant-K, bit1: flipped by SQuant-C */
    int64_t *cv;     /* [N*K] SQuant-C candidate value per slot (0 = none) */
    int32_t *cj;     /* [N*K] SQuant-C candidate flat index per slot */
    sqo_cand *list;  /* [N*K] scratch for sorting */
} sqo_work;

/* fp32 -> bfloat16 (the upper 16 bits of the fp32 pattern), round to nearest, ties to even. */
static uint16_t sqo_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof(u));
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static void sqo_channel(const float *w, int32_t N, int32_t K, const sqo_options *opt, const float *scale_in,
                        sqo_work *wk, int8_t *codes, float *scale_out,
                        float *kernel_err, float *channel_err, float *dequant, uint16_t *dequant_bf16)
{
    const int32_t NK = N * K;
    const int32_t qmax = (1 << (opt->bits - 1)) - 1;
    const int32_t qmin = (opt->flags & SQO_FLAG_NARROW_RANGE) ? -qmax : -qmax - 1;
    int32_t *q = wk->q;
    int64_t *P = wk->P;

    /* scale: the caller's (Algorithm 1 takes s as an input), else symmetric absmax */
    float s;
    if (scale_in) {
        s = *scale_in;
        if (!(s > 0.0f && s < INFINITY)) s = 1.0f;
    } else {
        float a = 0.0f;
        for (int32_t j = 0; j < NK; ++j) {
            float t = fabsf(w[j]);
            if (t > a) a = t;
        }
        s = (a < 0x1p-100f) ? 1.0f : a / (float)qmax;
    }
    *scale_out = s;

    /* SQuant-E (Eq. 9): round to nearest, clip, perturbation, one conversion to fixed point */
    for (int32_t j = 0; j < NK; ++j) {
        float x = w[j] / s;
        float qf = nearbyintf(x);
        if (qf > (float)qmax) qf = (float)qmax;
        if (qf < (float)qmin) qf = (float)qmin;
        float p = qf - x;
        q[j] = (int32_t)qf;
        P[j] = (int64_t)nearbyint((double)p * 0x1p30);   /* exact: p is an fp32 number */
        wk->flip[j] = 0;
    }

    /* SQuant-K (Algorithm 2 per kernel) and the candidate of Algorithm 3 */
    int32_t n_slots = 0;              /* number of SQuant-C candidate slots */
    if (opt->mode & SQO_MODE_K) {
        for (int32_t n = 0; n < N; ++n) {
            int32_t *qk = q + (size_t)n * K;
            int64_t *Pk = P + (size_t)n * K;
            int64_t e = 0;
            for (int32_t i = 0; i < K; ++i) e += Pk[i];
            wk->cv[n] = 0;
            wk->cj[n] = n * K;
            if (e == 0) continue;
            const int sgn = sqo_sign64(e);
            const int64_t abs_e = e > 0 ? e : -e;
            int32_t nc = 0;
            for (int32_t i = 0; i < K; ++i) {
                int32_t flipped = qk[i] - sgn;
                if (sqo_sign64(Pk[i]) == sgn && flipped >= qmin && flipped <= qmax) {
                    wk->list[nc].mag = Pk[i] > 0 ? Pk[i] : -Pk[i];
                    wk->list[nc].idx = n * K + i;
                    ++nc;
                }
            }
            qsort(wk->list, (size_t)nc, sizeof(sqo_cand), sqo_cand_cmp);
            int64_t k = sqo_flip_count(abs_e);
            if (k > nc) k = nc;
            for (int64_t r = 0; r < k; ++r) {
                int32_t j = wk->list[r].idx;
                q[j] -= sgn;
                P[j] -= sgn * SQO_ONE;
                wk->flip[j] |= 1;
            }
            if (k * SQO_ONE > abs_e) {              /* Over SQuant: last flipped, post-flip value */
                int32_t j = wk->list[k - 1].idx;
                wk->cv[n] = P[j];
                wk->cj[n] = j;
            } else if (k < nc) {                    /* Under SQuant: first un-flipped candidate */
                int32_t j = wk->list[k].idx;
                wk->cv[n] = P[j];
                wk->cj[n] = j;
            }
        }
        n_slots = N;
    } else {
        for (int32_t j = 0; j < NK; ++j) {          /* no SQuant-K: each element is its own slot */
            wk->cv[j] = P[j];
            wk->cj[j] = j;
        }
        n_slots = NK;
    }

    /* SQuant-C (Algorithm 2 on the channel, Eq. 11) */
    if (opt->mode & SQO_MODE_C) {
        int64_t ec = 0;
        for (int32_t j = 0; j < NK; ++j) ec += P[j];
        if (ec != 0) {
            const int sgn = sqo_sign64(ec);
            const int64_t abs_e = ec > 0 ? ec : -ec;
            int32_t nc = 0;
            for (int32_t t = 0; t < n_slots; ++t) {
                int64_t v = wk->cv[t];
                int32_t j = wk->cj[t];
                int32_t flipped = q[j] - sgn;
                if (sqo_sign64(v) == sgn && flipped >= qmin && flipped <= qmax) {
                    wk->list[nc].mag = v > 0 ? v : -v;
                    wk->list[nc].idx = j;
                    ++nc;
                }
            }
            qsort(wk->list, (size_t)nc, sizeof(sqo_cand), sqo_cand_cmp);
            int64_t k = sqo_flip_count(abs_e);
            if (k > nc) k = nc;
            for (int64_t r = 0; r < k; ++r) {
                int32_t j = wk->list[r].idx;
                q[j] -= sgn;
                P[j] -= sgn * SQO_ONE;
                wk->flip[j] |= 2;
            }
        }
    }

    /* emit */
    int64_t total = 0;
    for (int32_t n = 0; n < N; ++n) {
        int64_t e = 0;
        for (int32_t i = 0; i < K; ++i) e += P[(size_t)n * K + i];
        total += e;
        if (kernel_err) kernel_err[n] = (float)e * 0x1p-30f;
    }
    if (channel_err) *channel_err = (float)total * 0x1p-30f;
    if (dequant)   /* what Algorithm 1 returns: C * s */
        for (int32_t j = 0; j < NK; ++j) dequant[j] = (float)q[j] * s;
    if (dequant_bf16)   /* the same product (fp32), stored as bfloat16 */
        for (int32_t j = 0; j < NK; ++j) dequant_bf16[j] = sqo_bf16((float)q[j] * s);
    if (opt->flags & SQO_FLAG_PACK_INT4) {
        for (int32_t j = 0; j < NK; j += 2) {
            unsigned lo = (unsigned)q[j] & 15u;
            unsigned hi = (j + 1 < NK) ? ((unsigned)q[j + 1] & 15u) : 0u;
            codes[j / 2] = (int8_t)(lo | (hi << 4));
        }
    } else {
        for (int32_t j = 0; j < NK; ++j) codes[j] = (int8_t)q[j];
    }
}

/*
 * Quantize one layer.  All pointers are HOST pointers owned by the caller.
 *   w            [M][N][K] fp32
 *   codes        out [M][N][K] int8 (with SQO_FLAG_PACK_INT4: [M][ceil(N*K/2)] nibble pairs)
 *   scales       out [M]
 *   kernel_err   out [M][N], may be NULL
 *   channel_err  out [M], may be NULL
 *   pert         out [M][N][K] final fixed-point perturbations (2^-30 units), may be NULL
 *   flip         out [M][N][K] flip record (bit0 SQuant-K, bit1 SQuant-C), may be NULL
 *   dequant      out [M][N][K] fp32 code * scale (Algorithm 1's return value), may be NULL
 *   scales_in    in  [M] caller-supplied scales (Algorithm 1's input s), may be NULL: absmax scales
 *   dequant_bf16 out [M][N][K] bfloat16 of the fp32 product code * scale (round to nearest even), may be NULL
 * pert is the perturbation clamped to 32 bits (exact whenever no element is clipped by more than
 * one step).  Inputs must be finite.  Returns SQO_OK or a negative error.
 */
int sqo_quantize_layer_scaled(const float *w, int32_t M, int32_t N, int32_t K, const sqo_options *opt,
                              int8_t *codes, float *scales, float *kernel_err, float *channel_err,
                              int32_t *pert, uint8_t *flip, float *dequant, const float *scales_in,
                              uint16_t *dequant_bf16)
{
    if (!w || !opt || !codes || !scales || M < 0 || N <= 0 || K <= 0) return SQO_ERR_ARG;
    if (opt->bits < 2 || opt->bits > 8 || !(opt->mode & SQO_MODE_E)) return SQO_ERR_ARG;
    if ((opt->flags & SQO_FLAG_PACK_INT4) && opt->bits > 4) return SQO_ERR_ARG;
    if ((int64_t)N * K > (int64_t)1 << 30) return SQO_ERR_ARG;
    const size_t NK = (size_t)N * K;
    sqo_work wk;
    wk.q = (int32_t *)malloc(NK * sizeof(int32_t));
    wk.P = (int64_t *)malloc(NK * sizeof(int64_t));
    wk.flip = (uint8_t *)malloc(NK);
    wk.cv = (int64_t *)malloc(NK * sizeof(int64_t));
    wk.cj = (int32_t *)malloc(NK * sizeof(int32_t));
    wk.list = (sqo_cand *)malloc(NK * sizeof(sqo_cand));
    int rc = SQO_OK;
    if (!wk.q || !wk.P || !wk.flip || !wk.cv || !wk.cj || !wk.list) {
        rc = SQO_ERR_NOMEM;
    } else {
        for (int32_t m = 0; m < M; ++m) {
            sqo_channel(w + (size_t)m * NK, N, K, opt, scales_in ? scales_in + m : NULL, &wk,
                        codes + (size_t)m * ((opt->flags & SQO_FLAG_PACK_INT4) ? (NK + 1) / 2 : NK), scales + m,
                        kernel_err ? kernel_err + (size_t)m * N : NULL,
                        channel_err ? channel_err + m : NULL,
                        dequant ? dequant + (size_t)m * NK : NULL,
                        dequant_bf16 ? dequant_bf16 + (size_t)m * NK : NULL);
            if (pert)
                for (size_t j = 0; j < NK; ++j) {
                    int64_t v = wk.P[j];
                    pert[(size_t)m * NK + j] = (int32_t)(v > INT32_MAX ? INT32_MAX : (v < INT32_MIN ? INT32_MIN : v));
                }
            if (flip) memcpy(flip + (size_t)m * NK, wk.flip, NK);
        }
    }
    free(wk.q); free(wk.P); free(wk.flip); free(wk.cv); free(wk.cj); free(wk.list);
    return rc;
}

/* The same with absmax scales (no supplied scales). */
int sqo_quantize_layer(const float *w, int32_t M, int32_t N, int32_t K, const sqo_options *opt,
                       int8_t *codes, float *scales, float *kernel_err, float *channel_err,
                       int32_t *pert, uint8_t *flip, float *dequant)
{
    return sqo_quantize_layer_scaled(w, M, N, K, opt, codes, scales, kernel_err, channel_err, pert, flip, dequant, NULL, NULL);
}
