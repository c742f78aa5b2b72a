/*
 * CPU oracle for CD-Adam (communication-compressed distributed AMSGrad).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, single-threaded, slow restatement of
 * the paper's Algorithm 1 and of the compressors of its Appendix A.  It exists so that the
 * CUDA library can be checked against something that can be read against the paper by eye.
 * It shares no code with the CUDA path, is never linked into it, and must never be called
 * from it.  Only tests, the smoke check and the CPU-baseline leg of the benchmark use it.
 *
 * Arithmetic: every vector operation of Algorithm 1 is done in IEEE binary32 with one
 * rounding per printed operation and no fused multiply-add (compile with
 * -ffp-contract=off).  The one quantity whose evaluation order the paper leaves open, the
 * l1 norm inside the scaled-sign compressor, is evaluated EXACTLY (integer accumulation of
 * significands), so that its value does not depend on any summation order:
 *     scale = fl32( fl64(exact sum |x_j|) / fl64(count) ).
 *
 * Notation follows the paper: n workers, dimension d, worker Markov state ghat^(i)
 * ("\hat g^{(i)}"), server aggregate ghat ("\hat g"), shared second Markov state gtil
 * ("\tilde g"), moments m, v, vhat, model x, step size alpha, beta1, beta2, nu.
 *
 * Parity pins (tests/, CPU only): exact rational worked examples, math.fsum for the exact
 * l1 sum, brute-force sort for top-k, the closed form of Appendix A for the scaled-sign
 * error, the Markov identity ghat_t - ghat_{t-1} = c_t, and an independently written
 * vanilla AMSGrad for the identity compressor; for the naive-compression mode a second
 * hand-worked step and its statelessness; for the decoupled weight decay and the step-size
 * milestones the closed form x_t = x_1 prod (1 - alpha_t lambda) at zero gradients and an
 * independently written recursion; for the error-feedback mode a hand-worked three-iteration
 * run and the server recursion rebuilt from the messages; for the given-scales branch of the
 * sampled checks the bit-for-bit repeat of a computed run and planted hand-over mistakes.
 * No function here is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

enum { ORC_SIGN = 0, ORC_TOPK = 1, ORC_IDENTITY = 2, ORC_RANDK = 3 };
enum { ORC_MARKOV = 0, ORC_EF = 1, ORC_NAIVE = 2 };

/* ------------------------------------------------------------------------------------ */
/* Exact l1 norm of binary32 data.                                                        */
/* ------------------------------------------------------------------------------------ */

/* |x| = sig * 2^(e-150) with integer sig < 2^24 and biased exponent e in 1..254 (zeros and
 * subnormals use e = 1 without the hidden bit).  bin[e] holds the integer sum of the
 * significands seen with exponent e; 2^40 values fit before a bin could overflow. */
typedef struct {
    uint64_t bin[256];
} l1_accumulator;

static void l1_clear(l1_accumulator *a) { memset(a, 0, sizeof *a); }

static void l1_add(l1_accumulator *a, float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    b &= 0x7fffffffu;
    uint32_t e = b >> 23;
    uint32_t sig = b & 0x7fffffu;
    if (e != 0) sig |= 0x800000u; else e = 1;
    a->bin[e] += sig;
}

/* Nearest binary64 (ties to even) of the exact sum held in the accumulator. */
static double l1_round_to_double(const l1_accumulator *a)
{
    /* big = sum_e bin[e] << (e-1), an integer equal to (exact sum) * 2^149. */
    enum { LIMBS = 6 };
    uint64_t big[LIMBS];
    memset(big, 0, sizeof big);
    for (int e = 1; e <= 254; ++e) {
        uint64_t v = a->bin[e];
        if (v == 0) continue;
        int shift = e - 1, limb = shift / 64, off = shift % 64;
        uint64_t lo = v << off;
        uint64_t hi = off ? (v >> (64 - off)) : 0;
        /* add lo at limb, hi at limb+1, propagating carries */
        uint64_t carry = 0;
        for (int p = limb; p < LIMBS; ++p) {
            uint64_t add = (p == limb) ? lo : (p == limb + 1 ? hi : 0);
            uint64_t s = big[p] + add;
            uint64_t c1 = s < add;
            uint64_t s2 = s + carry;
            uint64_t c2 = s2 < carry;
            big[p] = s2;
            carry = c1 | c2;
            if (p > limb + 1 && carry == 0) break;
        }
    }
    int top = -1;
    for (int p = LIMBS - 1; p >= 0 && top < 0; --p)
        if (big[p])
            for (int b = 63; b >= 0; --b)
                if ((big[p] >> b) & 1) { top = p * 64 + b; break; }
    if (top < 0) return 0.0;
    if (top <= 52) return ldexp((double)big[0], -149);
    /* keep bits top..top-52, round on bit top-53, sticky below */
    uint64_t mant = 0;
    for (int b = top; b >= top - 52; --b)
        mant = (mant << 1) | ((big[b / 64] >> (b % 64)) & 1);
    int rb = top - 53;
    int round_bit = (int)((big[rb / 64] >> (rb % 64)) & 1);
    int sticky = 0;
    for (int b = rb - 1; b >= 0 && !sticky; --b)
        sticky = (int)((big[b / 64] >> (b % 64)) & 1);
    if (round_bit && (sticky || (mant & 1))) mant += 1;   /* may become 2^53: still exact */
    return ldexp((double)mant, top - 52 - 149);
}

/* Correctly rounded binary64 value of sum_j |x_j| (no dependence on order). */
double oracle_l1_exact(const float *x, int64_t count)
{
    l1_accumulator a;
    l1_clear(&a);
    for (int64_t j = 0; j < count; ++j) l1_add(&a, x[j]);
    return l1_round_to_double(&a);
}

/* ------------------------------------------------------------------------------------ */
/* Compressors (Appendix A).  Each writes the dense decoded vector c and its payload.     */
/* ------------------------------------------------------------------------------------ */

/* Scaled sign, applied independently to each contiguous segment [off[r], off[r+1]):
 *   C(x)_j = (||x_seg||_1 / |seg|) * sign(x_j),   sign(0) = +1  (one bit cannot say 0).
 * bits: ceil(d/32) words, bit (j mod 32) of word j/32, least significant first,
 * 1 = non-negative; unused high bits of the last word are 0.  scales: q floats. */
void oracle_compress_sign(const float *x, int64_t d, int q, const int64_t *off,
                          uint32_t *bits, float *scales, float *c)
{
    int64_t words = (d + 31) / 32;
    memset(bits, 0, (size_t)words * sizeof(uint32_t));
    for (int r = 0; r < q; ++r) {
        int64_t lo = off[r], hi = off[r + 1];
        double l1 = oracle_l1_exact(x + lo, hi - lo);
        float s = (float)(l1 / (double)(hi - lo));
        scales[r] = s;
        for (int64_t j = lo; j < hi; ++j) {
            int nonneg = x[j] >= 0.0f;
            if (nonneg) bits[j / 32] |= (uint32_t)1 << (j % 32);
            c[j] = nonneg ? s : -s;
        }
    }
}

static int cmp_u64_desc(const void *pa, const void *pb)
{
    uint64_t a = *(const uint64_t *)pa, b = *(const uint64_t *)pb;
    return (a < b) - (a > b);
}

/* Top-k: order coordinates by (|x_j| descending, j ascending) and keep the first k.
 * Payload: k (index, value) pairs listed by ascending index; c is x there and 0 elsewhere. */
void oracle_compress_topk(const float *x, int64_t d, int64_t k,
                          uint32_t *idx, float *val, float *c)
{
    /* one sortable key per coordinate: magnitude bits above, reversed index below, so a
     * single descending sort realises "larger |x| first, then lower index first". */
    uint64_t *key = (uint64_t *)malloc((size_t)d * sizeof(uint64_t));
    for (int64_t j = 0; j < d; ++j) {
        uint32_t b;
        memcpy(&b, &x[j], sizeof b);
        b &= 0x7fffffffu;   /* for finite non-negative floats integer order = value order */
        key[j] = ((uint64_t)b << 32) | (uint64_t)(0xffffffffu - (uint32_t)j);
    }
    qsort(key, (size_t)d, sizeof(uint64_t), cmp_u64_desc);
    memset(c, 0, (size_t)d * sizeof(float));
    for (int64_t t = 0; t < k; ++t) {
        uint32_t j = 0xffffffffu - (uint32_t)(key[t] & 0xffffffffu);
        c[j] = x[j];
    }
    /* list the kept coordinates by ascending index */
    uint8_t *kept = (uint8_t *)calloc((size_t)d, 1);
    for (int64_t t = 0; t < k; ++t)
        kept[0xffffffffu - (uint32_t)(key[t] & 0xffffffffu)] = 1;
    int64_t t = 0;
    for (int64_t j = 0; j < d; ++j)
        if (kept[j]) { idx[t] = (uint32_t)j; val[t] = x[j]; ++t; }
    free(kept);
    free(key);
}

/* Rand-k: C(x) = sum_{j in S} x_j e_j for a set S of k distinct coordinates drawn uniformly at
 * random.  The draw is an INPUT here (S, k increasing coordinates), so both sides of a
 * comparison use the same set.  Payload: the k (index, value) pairs; c is x on S, 0 elsewhere. */
void oracle_compress_randk(const float *x, int64_t d, int64_t k, const uint32_t *S,
                           uint32_t *idx, float *val, float *c)
{
    memset(c, 0, (size_t)d * sizeof(float));
    for (int64_t t = 0; t < k; ++t) {
        uint32_t j = S[t];
        idx[t] = j;
        val[t] = x[j];
        c[j] = x[j];
    }
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1                                                                           */
/* ------------------------------------------------------------------------------------ */

typedef struct oracle_ctx {
    int64_t d, k;
    int n, compressor, mode, q;
    int64_t *kseg;           /* top-k applied per segment: entries kept in each (NULL: whole vector) */
    float wd;                /* decoupled weight decay lambda (0 = none) */
    float base_lr, gamma;    /* step-size milestones */
    int n_milestones;
    int64_t milestones[64];
    float beta1, beta2, lr, nu;
    int64_t *off;            /* q+1 segment offsets */
    int64_t steps;
    /* state */
    float *ghat_w;           /* n*d : worker Markov state (EF mode: worker error delta^(i)) */
    float *ghat_s;           /* d   : server aggregate (unused in EF mode) */
    float *gtil;             /* d   : second Markov state (EF mode: server error delta) */
    float *m, *v, *vhat, *x; /* d each */
    /* scratch */
    float *u, *c, *acc;
    /* last payloads */
    uint32_t *w_bits;        /* n*words */
    float *w_scales;         /* n*q */
    uint32_t *w_idx;         /* n*k */
    float *w_val;            /* n*k */
    uint32_t *s_bits;        /* words */
    float *s_scales;         /* q */
    uint32_t *s_idx;         /* k */
    float *s_val;            /* k */
    /* sampled checks only: scales given from outside instead of computed (NULL = compute) */
    float *force_w_scales;   /* n*q */
    float *force_s_scales;   /* q */
    /* rand-k: the coordinate sets of the coming iteration (inputs) */
    uint32_t *rand_w;        /* n*k */
    uint32_t *rand_s;        /* k */
} oracle_ctx;

static float *zeros(int64_t count) { return (float *)calloc((size_t)(count > 0 ? count : 1), sizeof(float)); }

void oracle_destroy(oracle_ctx *o)
{
    if (!o) return;
    free(o->off); free(o->ghat_w); free(o->ghat_s); free(o->gtil);
    free(o->m); free(o->v); free(o->vhat); free(o->x);
    free(o->u); free(o->c); free(o->acc);
    free(o->w_bits); free(o->w_scales); free(o->w_idx); free(o->w_val);
    free(o->s_bits); free(o->s_scales); free(o->s_idx); free(o->s_val);
    free(o->force_w_scales); free(o->force_s_scales);
    free(o->rand_w); free(o->rand_s); free(o->kseg);
    free(o);
}

static void alloc_payloads(oracle_ctx *o)
{
    int64_t words = (o->d + 31) / 32;
    free(o->w_scales); free(o->s_scales);
    o->w_scales = zeros((int64_t)o->n * o->q);
    o->s_scales = zeros(o->q);
    if (!o->w_bits) {
        o->w_bits = (uint32_t *)calloc((size_t)(o->n * words), sizeof(uint32_t));
        o->s_bits = (uint32_t *)calloc((size_t)words, sizeof(uint32_t));
        int64_t kk = o->k > 0 ? o->k : 1;
        o->w_idx = (uint32_t *)calloc((size_t)(o->n * kk), sizeof(uint32_t));
        o->w_val = zeros(o->n * kk);
        o->s_idx = (uint32_t *)calloc((size_t)kk, sizeof(uint32_t));
        o->s_val = zeros(kk);
    }
}

/* Inputs of Algorithm 1: x_1 (set later, default 0), alpha, beta1, beta2, nu, C.
 * All state starts at zero (the initialisation of Algorithm 1: C(0) = 0). */
oracle_ctx *oracle_create(int64_t d, int n, int compressor, int64_t k,
                          float beta1, float beta2, float lr, float nu)
{
    if (d < 1 || n < 1 || compressor < 0 || compressor > 3) return NULL;
    if ((compressor == ORC_TOPK || compressor == ORC_RANDK) && (k < 1 || k > d)) return NULL;
    oracle_ctx *o = (oracle_ctx *)calloc(1, sizeof *o);
    o->d = d; o->n = n; o->compressor = compressor;
    o->k = (compressor == ORC_TOPK || compressor == ORC_RANDK) ? k : 0;
    o->mode = ORC_MARKOV;
    o->beta1 = beta1; o->beta2 = beta2; o->lr = lr; o->nu = nu;
    o->q = 1;
    o->off = (int64_t *)malloc(2 * sizeof(int64_t));
    o->off[0] = 0; o->off[1] = d;
    o->ghat_w = zeros((int64_t)n * d);
    o->ghat_s = zeros(d); o->gtil = zeros(d);
    o->m = zeros(d); o->v = zeros(d); o->vhat = zeros(d); o->x = zeros(d);
    o->u = zeros(d); o->c = zeros(d); o->acc = zeros(d);
    alloc_payloads(o);
    return o;
}

int oracle_set_segments(oracle_ctx *o, int q, const int64_t *off)
{
    if (!o || q < 1 || off[0] != 0 || off[q] != o->d) return -1;
    for (int r = 0; r < q; ++r) if (off[r + 1] <= off[r]) return -1;
    free(o->off);
    o->off = (int64_t *)malloc((size_t)(q + 1) * sizeof(int64_t));
    memcpy(o->off, off, (size_t)(q + 1) * sizeof(int64_t));
    o->q = q;
    alloc_payloads(o);
    return 0;
}

/* Top-k applied to every segment on its own (the per-tensor use of a compressor, as for the
 * scaled sign): segment r keeps its kseg[r] coordinates of largest magnitude, ties to the
 * lower index.  The message is the concatenation of the segments' (index, value) lists, so it
 * is still listed by ascending index and has k = sum_r kseg[r] entries. */
int oracle_set_topk_segments(oracle_ctx *o, int q, const int64_t *off, const int64_t *kseg)
{
    if (!o || o->compressor != ORC_TOPK || o->steps != 0) return -1;
    if (q < 1 || off[0] != 0 || off[q] != o->d) return -1;
    int64_t total = 0;
    for (int r = 0; r < q; ++r) {
        if (off[r + 1] <= off[r] || kseg[r] < 1 || kseg[r] > off[r + 1] - off[r]) return -1;
        total += kseg[r];
    }
    if (oracle_set_segments(o, q, off) != 0) return -1;
    free(o->kseg);
    o->kseg = (int64_t *)malloc((size_t)q * sizeof(int64_t));
    memcpy(o->kseg, kseg, (size_t)q * sizeof(int64_t));
    o->k = total;
    free(o->w_idx); free(o->w_val); free(o->s_idx); free(o->s_val);
    o->w_idx = (uint32_t *)calloc((size_t)(o->n * total), sizeof(uint32_t));
    o->w_val = zeros(o->n * total);
    o->s_idx = (uint32_t *)calloc((size_t)total, sizeof(uint32_t));
    o->s_val = zeros(total);
    return 0;
}

int oracle_set_mode(oracle_ctx *o, int mode)
{
    if (!o || (mode != ORC_MARKOV && mode != ORC_EF && mode != ORC_NAIVE) || o->steps != 0) return -1;
    o->mode = mode;
    return 0;
}

int oracle_set_lr(oracle_ctx *o, float lr) { if (!o) return -1; o->lr = lr; o->n_milestones = 0; return 0; }

/* Decoupled weight decay lambda (the image-classification experiments of Section 6 use a
 * weight decay; the paper does not print the formula, the decoupled form is the reading):
 *   x_{t+1} = x_t - alpha_t m_t / sqrt(vhat_t + nu) - (alpha_t lambda) x_t. */
int oracle_set_weight_decay(oracle_ctx *o, float lambda)
{
    if (!o || !(lambda >= 0.0f)) return -1;
    o->wd = lambda;
    return 0;
}

/* Step-size milestones (Section 6: the step size is multiplied by 0.1 at two points of the
 * run): the step with 1-based number t uses alpha_t = base * gamma^(number of milestones
 * < t), the product taken by repeated binary32 multiplication.  Milestones count completed
 * steps and must be increasing; gamma in (0, 1] keeps alpha_t non-increasing (Algorithm 1). */
int oracle_set_lr_milestones(oracle_ctx *o, float base, int count, const int64_t *after_steps, float gamma)
{
    if (!o || count < 0 || count > 64 || !(gamma > 0.0f && gamma <= 1.0f)) return -1;
    for (int i = 0; i < count; ++i)
        if (after_steps[i] < 0 || (i > 0 && after_steps[i] <= after_steps[i - 1])) return -1;
    o->base_lr = base; o->gamma = gamma; o->n_milestones = count;
    for (int i = 0; i < count; ++i) o->milestones[i] = after_steps[i];
    if (count == 0) o->lr = base;
    return 0;
}

/* name: 0 ghat_w (n*d), 1 ghat_s, 2 gtil, 3 m, 4 v, 5 vhat, 6 x */
float *oracle_state(oracle_ctx *o, int name)
{
    switch (name) {
    case 0: return o->ghat_w; case 1: return o->ghat_s; case 2: return o->gtil;
    case 3: return o->m; case 4: return o->v; case 5: return o->vhat; case 6: return o->x;
    }
    return NULL;
}

/* who = worker index 0..n-1, or -1 for the server */
uint32_t *oracle_payload_bits(oracle_ctx *o, int who)
{ return who < 0 ? o->s_bits : o->w_bits + (int64_t)who * ((o->d + 31) / 32); }
float *oracle_payload_scales(oracle_ctx *o, int who)
{ return who < 0 ? o->s_scales : o->w_scales + (int64_t)who * o->q; }
uint32_t *oracle_payload_idx(oracle_ctx *o, int who)
{ return who < 0 ? o->s_idx : o->w_idx + (int64_t)who * o->k; }
float *oracle_payload_val(oracle_ctx *o, int who)
{ return who < 0 ? o->s_val : o->w_val + (int64_t)who * o->k; }

/* For checks on a SAMPLE of the coordinates of a larger problem: the scaled-sign scales
 * are global reductions that a sample cannot reproduce, so they are supplied (after having
 * been verified on the full data with oracle_l1_exact) and only bits and the decoded vector
 * are computed here.  Pass NULL to return to computed scales. */
int oracle_force_scales(oracle_ctx *o, const float *worker_scales, const float *server_scales)
{
    if (!o || o->compressor != ORC_SIGN) return -1;
    free(o->force_w_scales); free(o->force_s_scales);
    o->force_w_scales = o->force_s_scales = NULL;
    if (worker_scales) {
        o->force_w_scales = (float *)malloc((size_t)o->n * o->q * sizeof(float));
        memcpy(o->force_w_scales, worker_scales, (size_t)o->n * o->q * sizeof(float));
    }
    if (server_scales) {
        o->force_s_scales = (float *)malloc((size_t)o->q * sizeof(float));
        memcpy(o->force_s_scales, server_scales, (size_t)o->q * sizeof(float));
    }
    return 0;
}

static void sign_with_given_scales(oracle_ctx *o, const float *u, const float *given,
                                   uint32_t *bits, float *scales, float *c)
{
    memset(bits, 0, (size_t)((o->d + 31) / 32) * sizeof(uint32_t));
    for (int r = 0; r < o->q; ++r) {
        const float s = given[r];
        scales[r] = s;
        for (int64_t j = o->off[r]; j < o->off[r + 1]; ++j) {
            int nonneg = u[j] >= 0.0f;
            if (nonneg) bits[j / 32] |= (uint32_t)1 << (j % 32);
            c[j] = nonneg ? s : -s;
        }
    }
}

/* Rand-k: the coordinate sets (k increasing, distinct coordinates each) the n workers and the
 * server use in the next call of oracle_step. */
int oracle_set_random_sets(oracle_ctx *o, const uint32_t *workers, const uint32_t *server)
{
    if (!o || o->compressor != ORC_RANDK || !workers || !server) return -1;
    if (!o->rand_w) {
        o->rand_w = (uint32_t *)malloc((size_t)o->n * o->k * sizeof(uint32_t));
        o->rand_s = (uint32_t *)malloc((size_t)o->k * sizeof(uint32_t));
    }
    memcpy(o->rand_w, workers, (size_t)o->n * o->k * sizeof(uint32_t));
    memcpy(o->rand_s, server, (size_t)o->k * sizeof(uint32_t));
    return 0;
}

/* c = C(u) with the context's compressor; who selects where the payload is kept. */
static void compress(oracle_ctx *o, const float *u, float *c, int who)
{
    const float *given = who < 0 ? o->force_s_scales
                                 : (o->force_w_scales ? o->force_w_scales + (int64_t)who * o->q : NULL);
    if (o->compressor == ORC_SIGN && given)
        sign_with_given_scales(o, u, given, oracle_payload_bits(o, who),
                               oracle_payload_scales(o, who), c);
    else if (o->compressor == ORC_SIGN)
        oracle_compress_sign(u, o->d, o->q, o->off, oracle_payload_bits(o, who),
                             oracle_payload_scales(o, who), c);
    else if (o->compressor == ORC_TOPK && o->kseg) {
        uint32_t *idx = oracle_payload_idx(o, who);
        float *val = oracle_payload_val(o, who);
        for (int r = 0; r < o->q; ++r) {             /* C on every segment on its own */
            const int64_t lo = o->off[r], len = o->off[r + 1] - lo;
            oracle_compress_topk(u + lo, len, o->kseg[r], idx, val, c + lo);
            for (int64_t t = 0; t < o->kseg[r]; ++t) idx[t] += (uint32_t)lo;   /* positions in the whole vector */
            idx += o->kseg[r];
            val += o->kseg[r];
        }
    } else if (o->compressor == ORC_TOPK)
        oracle_compress_topk(u, o->d, o->k, oracle_payload_idx(o, who),
                             oracle_payload_val(o, who), c);
    else if (o->compressor == ORC_RANDK)
        oracle_compress_randk(u, o->d, o->k, who < 0 ? o->rand_s : o->rand_w + (int64_t)who * o->k,
                              oracle_payload_idx(o, who), oracle_payload_val(o, who), c);
    else
        memcpy(c, u, (size_t)o->d * sizeof(float));
}

/* AMSGrad update of Algorithm 1 (its last four assignments) with gradient estimate ge:
 *   m = beta1 m + (1-beta1) ge;  v = beta2 v + (1-beta2) ge^2;  vhat = max(vhat, v);
 *   x = x - alpha * m / sqrt(vhat + nu)          (nu inside the root, no bias correction) */
static void amsgrad(oracle_ctx *o, const float *ge)
{
    const float b1 = o->beta1, b2 = o->beta2;
    const float omb1 = 1.0f - b1, omb2 = 1.0f - b2;
    const float lrwd = o->lr * o->wd;
    for (int64_t j = 0; j < o->d; ++j) {
        float g = ge[j];
        float m1 = b1 * o->m[j];
        float m2 = omb1 * g;
        o->m[j] = m1 + m2;
        float v1 = b2 * o->v[j];
        float gg = g * g;
        float v2 = omb2 * gg;
        o->v[j] = v1 + v2;
        o->vhat[j] = o->vhat[j] >= o->v[j] ? o->vhat[j] : o->v[j];
        float den = sqrtf(o->vhat[j] + o->nu);
        float num = o->lr * o->m[j];
        float xold = o->x[j];
        float xnew = xold - num / den;
        if (o->wd != 0.0f) {                         /* decoupled weight decay */
            float decay = lrwd * xold;
            xnew = xnew - decay;
        }
        o->x[j] = xnew;
    }
}

/* One iteration of Algorithm 1 on the n stochastic gradients g (n*d, row i = worker i). */
static void step_markov(oracle_ctx *o, const float *g)
{
    const int64_t d = o->d;
    memset(o->acc, 0, (size_t)d * sizeof(float));
    for (int i = 0; i < o->n; ++i) {                 /* on worker i */
        const float *gi = g + (int64_t)i * d;
        float *gh = o->ghat_w + (int64_t)i * d;
        for (int64_t j = 0; j < d; ++j) o->u[j] = gi[j] - gh[j];
        compress(o, o->u, o->c, i);                  /* c^(i) = C(g^(i) - ghat^(i)) */
        for (int64_t j = 0; j < d; ++j) gh[j] = gh[j] + o->c[j];
        for (int64_t j = 0; j < d; ++j) o->acc[j] = o->acc[j] + o->c[j];  /* i ascending */
    }
    const float fn = (float)o->n;                    /* on the server */
    for (int64_t j = 0; j < d; ++j) o->ghat_s[j] = o->ghat_s[j] + o->acc[j] / fn;
    for (int64_t j = 0; j < d; ++j) o->u[j] = o->ghat_s[j] - o->gtil[j];
    compress(o, o->u, o->c, -1);                     /* c = C(ghat - gtil) */
    for (int64_t j = 0; j < d; ++j) o->gtil[j] = o->gtil[j] + o->c[j];
    amsgrad(o, o->gtil);                             /* on every worker, identically */
}

/* Classical error feedback (the comparison scheme of the paper's Section 4), both ways:
 *   worker: p = g + delta^(i); c^(i) = C(p); delta^(i) = p - c^(i)
 *   server: p = mean_i c^(i) + delta; c = C(p); delta = p - c;  AMSGrad on c.
 * delta^(i) is kept in ghat_w, the server delta in gtil. */
static void step_ef(oracle_ctx *o, const float *g)
{
    const int64_t d = o->d;
    memset(o->acc, 0, (size_t)d * sizeof(float));
    for (int i = 0; i < o->n; ++i) {
        const float *gi = g + (int64_t)i * d;
        float *del = o->ghat_w + (int64_t)i * d;
        for (int64_t j = 0; j < d; ++j) o->u[j] = gi[j] + del[j];
        compress(o, o->u, o->c, i);
        for (int64_t j = 0; j < d; ++j) del[j] = o->u[j] - o->c[j];
        for (int64_t j = 0; j < d; ++j) o->acc[j] = o->acc[j] + o->c[j];
    }
    const float fn = (float)o->n;
    for (int64_t j = 0; j < d; ++j) o->u[j] = o->acc[j] / fn + o->gtil[j];
    compress(o, o->u, o->c, -1);
    for (int64_t j = 0; j < d; ++j) o->gtil[j] = o->u[j] - o->c[j];
    amsgrad(o, o->c);
}

/* Naive compression (Section 4, first paragraph) carried over to AMSGrad, the third
 * comparison scheme of the experiments of Section 6: no state on either side,
 *   worker: c^(i) = C(g^(i));   server: c = C(mean_i c^(i));   AMSGrad on c.
 * (The section prints the SGD form with the uplink compressed; compressing the downlink with
 * the same C is the reading that puts it under the same communication budget as the other
 * schemes.)  ghat_w, ghat_s and gtil stay zero. */
static void step_naive(oracle_ctx *o, const float *g)
{
    const int64_t d = o->d;
    memset(o->acc, 0, (size_t)d * sizeof(float));
    for (int i = 0; i < o->n; ++i) {
        compress(o, g + (int64_t)i * d, o->c, i);
        for (int64_t j = 0; j < d; ++j) o->acc[j] = o->acc[j] + o->c[j];
    }
    const float fn = (float)o->n;
    for (int64_t j = 0; j < d; ++j) o->u[j] = o->acc[j] / fn;
    compress(o, o->u, o->c, -1);
    amsgrad(o, o->c);
}

int oracle_step(oracle_ctx *o, const float *g)
{
    if (!o || !g) return -1;
    if (o->compressor == ORC_RANDK && !o->rand_w) return -1;
    if (o->n_milestones > 0) {
        float lr = o->base_lr;
        for (int i = 0; i < o->n_milestones; ++i)
            if (o->milestones[i] <= o->steps) lr = lr * o->gamma;
        o->lr = lr;
    }
    if (o->mode == ORC_MARKOV) step_markov(o, g);
    else if (o->mode == ORC_EF) step_ef(o, g);
    else step_naive(o, g);
    o->steps += 1;
    return 0;
}
