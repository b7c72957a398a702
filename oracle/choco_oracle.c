/*
 * CPU oracle for the CHOCO-Gossip / CHOCO-SGD step -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the method computes, written
 * from the paper.  It shares no code with the CUDA library and must never be
 * reached from a product code path: only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * What follows the paper:
 *   - the compression operators of Appendix C ("Compression Schemes"): top_a,
 *     random_a (biased form), gsgd_b (biased and unbiased forms), scaled sign;
 *   - the per-worker updates of Algorithm 1 (gossip, compression, public copies,
 *     gradient step) in the form that
 *     keeps three vectors per worker (x_i, x^_i and s_i = sum_j w_ij x^_j), the
 *     storage the end of Section 3 describes;
 *   - the consensus distance of Section 6, (1/n) sum_i ||x_i - xbar||^2.
 *
 * Precision: the paper's experiments hold float32 values, so all state arithmetic is
 * float32 (round to nearest even, no fused multiply-add: build with
 * -ffp-contract=off); metrics are float64.  Where the paper leaves the arithmetic open
 * (order of operations, tie-breaks, how a norm is summed, bit layout) the choice made
 * is stated next to the code.
 *
 * Parity pins live in tests/ (brute force, closed forms, known-answer vectors of the
 * published Philox4x32-10 generator, invariants of Assumption 4).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy */
/* as 1, 2, 3", SC'11).  The paper only says that sender and receiver share a  */
/* seed (Appendix C, random_a); the generator is this build's choice.          */
/* ------------------------------------------------------------------------- */

void oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * One 32-bit word per coordinate, keyed on (seed, step, worker, coordinate) and a
 * stream number (0: random_a selection keys, 1: gsgd_b dither).  Counter =
 * (coord / 4, worker, low 32 bits of step, (high bits of step << 8) | stream), key =
 * (low, high) half of the seed; coordinate c takes output word c mod 4.
 */
void oracle_random_words(uint64_t seed, uint64_t step, uint32_t worker, uint32_t stream,
                         int64_t d, uint32_t* words)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (int64_t c4 = 0; c4 * 4 < d; ++c4) {
        uint32_t ctr[4] = { (uint32_t)c4, worker, (uint32_t)step,
                            ((uint32_t)(step >> 32) << 8) | stream };
        uint32_t o[4];
        oracle_philox4x32_10(ctr, key, o);
        for (int e = 0; e < 4 && c4 * 4 + e < d; ++e) words[c4 * 4 + e] = o[e];
    }
}

/* u in [0,1): the top 24 bits of the word, exactly representable in float32. */
void oracle_words_to_unit(const uint32_t* words, int64_t d, float* u)
{
    for (int64_t c = 0; c < d; ++c) u[c] = (float)(words[c] >> 8) * 0x1p-24f;
}

/* ------------------------------------------------------------------------- */
/* Summation order for norms.  The paper does not say how ||.||_1 and ||.||_2  */
/* are accumulated; float32 addition is not associative, so the order is fixed  */
/* here: a pairwise tree over the coordinate index.  Level 0 holds the terms;   */
/* each level adds neighbours (2j, 2j+1); an odd element out is carried up      */
/* unchanged (the same as padding with +0 to a power of two).                   */
/* ------------------------------------------------------------------------- */

float oracle_tree_sum(float* a, int64_t m)
{
    if (m <= 0) return 0.0f;
    while (m > 1) {
        int64_t half = m / 2;
        for (int64_t j = 0; j < half; ++j) a[j] = a[2 * j] + a[2 * j + 1];
        if (m & 1) a[half] = a[m - 1];
        m = half + (m & 1);
    }
    return a[0];
}

/* ------------------------------------------------------------------------- */
/* Selection shared by top_a and random_a: keep the k entries with the largest  */
/* 32-bit key; equal keys are ordered by ascending coordinate (the paper allows  */
/* any permutation pi that sorts the magnitudes, Appendix C; this picks one).    */
/* Indices come back in ascending order.                                         */
/* ------------------------------------------------------------------------- */

static int cmp_u64(const void* a, const void* b)
{
    uint64_t x = *(const uint64_t*)a, y = *(const uint64_t*)b;
    return (x > y) - (x < y);
}
static int cmp_u32(const void* a, const void* b)
{
    uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
    return (x > y) - (x < y);
}

int oracle_select_largest(const uint32_t* key, int64_t d, int64_t k, uint32_t* idx_out)
{
    if (k < 0 || k > d) return -1;
    uint64_t* order = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(d > 0 ? d : 1));
    if (!order) return -2;
    /* ascending sort of (~key, index) == descending key, then ascending index */
    for (int64_t c = 0; c < d; ++c) order[c] = ((uint64_t)(~key[c]) << 32) | (uint64_t)(uint32_t)c;
    qsort(order, (size_t)d, sizeof(uint64_t), cmp_u64);
    for (int64_t e = 0; e < k; ++e) idx_out[e] = (uint32_t)order[e];
    qsort(idx_out, (size_t)k, sizeof(uint32_t), cmp_u32);
    free(order);
    return 0;
}

static uint32_t f32_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return u;
}

/* v = x - x^ (Algorithm 1, the argument of Q in the compression step) */
void oracle_difference(const float* x, const float* xhat, int64_t d, float* v)
{
    for (int64_t c = 0; c < d; ++c) v[c] = x[c] - xhat[c];
}

/*
 * top_a (Appendix C): keep the k = floor(a d) coordinates of largest magnitude, zero
 * the rest.  Magnitudes are compared through the bit pattern of |v| (monotone for
 * finite floats; +0 and -0 compare equal).  q and mask are dense [d]; idx/val are the
 * message (positions and float32 values: 2 * 32 * k bits).
 */
int oracle_compress_topk(const float* v, int64_t d, int64_t k, uint32_t* idx, float* val,
                         float* q, uint8_t* mask)
{
    uint32_t* key = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(d > 0 ? d : 1));
    if (!key) return -2;
    for (int64_t c = 0; c < d; ++c) key[c] = f32_bits(v[c]) & 0x7FFFFFFFu;
    int rc = oracle_select_largest(key, d, k, idx);
    free(key);
    if (rc) return rc;
    memset(q, 0, sizeof(float) * (size_t)d);
    memset(mask, 0, (size_t)d);
    for (int64_t e = 0; e < k; ++e) {
        val[e] = v[idx[e]];
        q[idx[e]] = val[e];
        mask[idx[e]] = 1;
    }
    return 0;
}

/*
 * random_a, biased form q = v (.) u with ||u||_1 = k (Appendix C).  The mask is the
 * set of the k coordinates with the smallest random word (ties by coordinate), which
 * is uniform over k-subsets; `words` are the d random words of this (step, worker),
 * passed in so that a test can supply its own.  Only the k values are the message
 * (32 * k bits): a receiver regenerates idx from the shared seed.
 */
int oracle_compress_randk(const float* v, const uint32_t* words, int64_t d, int64_t k,
                          uint32_t* idx, float* val, float* q, uint8_t* mask)
{
    uint32_t* key = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(d > 0 ? d : 1));
    if (!key) return -2;
    for (int64_t c = 0; c < d; ++c) key[c] = ~words[c];
    int rc = oracle_select_largest(key, d, k, idx);
    free(key);
    if (rc) return rc;
    memset(q, 0, sizeof(float) * (size_t)d);
    memset(mask, 0, (size_t)d);
    for (int64_t e = 0; e < k; ++e) {
        val[e] = v[idx[e]];
        q[idx[e]] = val[e];
        mask[idx[e]] = 1;
    }
    return 0;
}

/*
 * scaled sign (Appendix C): q = (||v||_1 / d) * sgn(v).  sgn(0) is not defined by the
 * paper; here a coordinate is negative iff v < 0 (so +0 and -0 map to +scale), which
 * makes ||q - v||^2 = ||v||^2 - ||v||_1^2 / d hold exactly.  Message: d sign bits,
 * bit (c mod 32) of word c / 32, set iff v_c < 0, unused tail bits zero; plus the
 * float32 scale: d + 32 bits.
 */
int oracle_compress_sign(const float* v, int64_t d, uint32_t* bits, float* scale_out, float* q)
{
    float* a = (float*)malloc(sizeof(float) * (size_t)(d > 0 ? d : 1));
    if (!a) return -2;
    for (int64_t c = 0; c < d; ++c) a[c] = fabsf(v[c]);
    float l1 = oracle_tree_sum(a, d);
    free(a);
    float scale = l1 / (float)d;
    int64_t nwords = (d + 31) / 32;
    memset(bits, 0, sizeof(uint32_t) * (size_t)nwords);
    for (int64_t c = 0; c < d; ++c) {
        int neg = v[c] < 0.0f;
        if (neg) bits[c / 32] |= 1u << (c % 32);
        q[c] = neg ? -scale : scale;
    }
    *scale_out = scale;
    return 0;
}

/* tau of the biased gsgd_b (Appendix C) for a block of `len` coordinates and
 * s = 2^(b-1) levels: 1 + min(len / s^2, sqrt(len) / s); float64 then rounded once. */
float oracle_qsgd_tau(int64_t len, int32_t s)
{
    double a = (double)len / ((double)s * (double)s);
    double b = sqrt((double)len) / (double)s;
    return (float)(1.0 + (a < b ? a : b));
}

/* width of the stored level field: smallest of 1, 2, 4, 8, 16 bits holding 0..s-1 (b = 16 bits
 * per coordinate, the first QSGD row of Table 1, is s = 2^15 with 16-bit fields) */
int32_t oracle_qsgd_level_bits(int32_t s)
{
    int32_t w = 1;
    while ((1 << w) < s) w *= 2;
    return w;
}

/*
 * gsgd_b (Appendix C) with s = 2^(b-1):
 *     q = (nu / tau) * sig(v) * (1/s) * floor(s |v| / nu + u),   nu = ||v||_2,
 * applied per block of `bucket` consecutive coordinates (bucket = 0: the whole row is
 * one block; the last block may be shorter and uses its own length in tau).
 * biased = 0 drops the 1/tau factor.  Readings the paper leaves open:
 *   - nu^2 is the pairwise-tree sum of the rounded squares, nu = sqrtf of it;
 *   - r = (s * |v|) / nu, level = floor(r + u) in float32;
 *   - the paper states levels lie in {0..s-1}, yet the formula reaches s when
 *     |v_c| / nu is within 1/s of one; the level is saturated to s - 1 so that it fits;
 *   - nu = 0 gives level 0 and q = +0;
 *   - q = (nu / (tau * s)) * level, negated where v < 0 (sig(0) = +1).
 * Message per row: float32 nu per block, one sign bit per coordinate (as for sign),
 * and the levels in fields of oracle_qsgd_level_bits(s) bits, coordinate c at bit
 * offset c * width, least significant first (s <= 32768: fields of at most 16 bits).
 */
int oracle_compress_qsgd(const float* v, const float* u, int64_t d, int32_t s, int64_t bucket,
                         int32_t biased, float* norms, uint32_t* signbits, uint8_t* levels,
                         float* q)
{
    if (bucket <= 0) bucket = d;
    if (s < 2 || s > 32768) return -1;
    int32_t wbits = oracle_qsgd_level_bits(s);
    int64_t nwords = (d + 31) / 32;
    int64_t nbytes = (d * wbits + 7) / 8;
    memset(signbits, 0, sizeof(uint32_t) * (size_t)nwords);
    memset(levels, 0, (size_t)nbytes);
    float* sq = (float*)malloc(sizeof(float) * (size_t)bucket);
    if (!sq) return -2;
    int64_t b = 0;
    for (int64_t c0 = 0; c0 < d; c0 += bucket, ++b) {
        int64_t len = (d - c0 < bucket) ? d - c0 : bucket;
        for (int64_t c = 0; c < len; ++c) sq[c] = v[c0 + c] * v[c0 + c];
        float nu = sqrtf(oracle_tree_sum(sq, len));
        float tau = biased ? oracle_qsgd_tau(len, s) : 1.0f;
        float scale = nu / (tau * (float)s);
        norms[b] = nu;
        for (int64_t c = c0; c < c0 + len; ++c) {
            int32_t level = 0;
            if (nu != 0.0f) {
                float r = ((float)s * fabsf(v[c])) / nu;
                level = (int32_t)floorf(r + u[c]);
                if (level > s - 1) level = s - 1;
            }
            int neg = v[c] < 0.0f;
            if (neg) signbits[c / 32] |= 1u << (c % 32);
            int64_t bit = c * wbits;
            levels[bit / 8] |= (uint8_t)(level << (bit % 8));
            if (wbits == 16) levels[bit / 8 + 1] = (uint8_t)(level >> 8); /* little-endian field */
            float mag = scale * (float)level;
            q[c] = neg ? -mag : mag;
        }
    }
    free(sq);
    return 0;
}

/*
 * One worker's update in three-vector form.  With q_j = Q(x_j - x^_j) already formed
 * for this worker and its neighbours (Algorithm 1, compression step):
 *     x^_i  <- x^_i + q_i                              (public copy, j = i)
 *     s_i   <- s_i + sum_j w_ij q_j                    (the same for all j, folded into
 *                                                       s_i = sum_j w_ij x^_j)
 *     x_i   <- (x_i - eta g_i) + gamma (s_i - x^_i)    (the gradient step, then the gossip
 *                                                       step of the next iteration, which is
 *                                                       gamma sum_j w_ij (x^_j - x^_i)
 *                                                       because rows of W sum to one)
 * Operation order, fixed here because the paper does not give one: neighbours are
 * added in the order given (CSR column order), acc = +0; acc = acc + w_ij * q_j; then
 * s' = s + acc; c = s' - x^'; x' = (x - eta * g) + gamma * c, i.e. the gradient step and then
 * the gossip step (x' = x + gamma * c when g is NULL).  For sparse q (mask given) coordinates that no neighbour touches
 * leave s and x^ as they are.
 */
void oracle_apply_row(int64_t d, float* x, float* xhat, float* s, const float* g,
                      int32_t nnb, const float* const* q_nb, const uint8_t* const* mask_nb,
                      const float* w_nb, int32_t self_pos, float eta, float gamma)
{
    for (int64_t c = 0; c < d; ++c) {
        float xh = xhat[c];
        if (!mask_nb || mask_nb[self_pos][c]) xh = xh + q_nb[self_pos][c];
        float acc = 0.0f;
        int any = 0;
        for (int32_t e = 0; e < nnb; ++e) {
            if (mask_nb && !mask_nb[e][c]) continue;
            acc = acc + w_nb[e] * q_nb[e][c];
            any = 1;
        }
        float sn = s[c];
        if (any) sn = sn + acc;
        float cons = sn - xh;
        float xn = x[c];
        if (g) xn = xn - eta * g[c];
        xn = xn + gamma * cons;
        xhat[c] = xh;
        s[c] = sn;
        x[c] = xn;
    }
}

/*
 * Momentum variant (Algorithm 2): the gradient step becomes
 *     v <- (g + lambda x) + beta v ;  x <- x - eta v
 * with x the iterate the gradient was taken at, followed by the gossip correction of
 * the next iteration as in oracle_apply_row:
 *     m' = (g + lambda * x) + beta * m ;  x' = (x - eta * m') + gamma * c.
 * Appendix D says only that Nesterov momentum can be adapted in the same way and gives no
 * formula.  The reading taken here (nesterov != 0) is the look-ahead form common in
 * deep-learning optimisers: the memory is updated as above and the step is taken along
 *     (g + lambda * x) + beta * m'
 * instead of m'.
 */
void oracle_apply_row_momentum(int64_t d, float* x, float* xhat, float* s, const float* g,
                               float* mom, int32_t nnb, const float* const* q_nb,
                               const uint8_t* const* mask_nb, const float* w_nb,
                               int32_t self_pos, float eta, float gamma, float lambda,
                               float beta, int32_t nesterov)
{
    for (int64_t c = 0; c < d; ++c) {
        float xh = xhat[c];
        if (!mask_nb || mask_nb[self_pos][c]) xh = xh + q_nb[self_pos][c];
        float acc = 0.0f;
        int any = 0;
        for (int32_t e = 0; e < nnb; ++e) {
            if (mask_nb && !mask_nb[e][c]) continue;
            acc = acc + w_nb[e] * q_nb[e][c];
            any = 1;
        }
        float sn = s[c];
        if (any) sn = sn + acc;
        float cons = sn - xh;
        float gl = g[c] + lambda * x[c];
        float mn = gl + beta * mom[c];
        float dir = mn;
        if (nesterov) dir = gl + beta * mn;
        float xn = (x[c] - eta * dir) + gamma * cons;
        xhat[c] = xh;
        s[c] = sn;
        mom[c] = mn;
        x[c] = xn;
    }
}

/* consensus distance of Section 6 without the 1/n: sum_i ||x_i - xbar||^2, float64 */
double oracle_consensus_error(const float* x, int64_t n, int64_t d, int64_t ld)
{
    double total = 0.0;
    for (int64_t c = 0; c < d; ++c) {
        double mean = 0.0;
        for (int64_t i = 0; i < n; ++i) mean += (double)x[i * ld + c];
        mean /= (double)n;
        for (int64_t i = 0; i < n; ++i) {
            double t = (double)x[i * ld + c] - mean;
            total += t * t;
        }
    }
    return total;
}
