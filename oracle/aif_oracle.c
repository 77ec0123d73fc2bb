/*
 * AIF pre-ranking scoring pass -- CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 definition of what the scoring pass
 * computes.  It is used by the tests, by the smoke check and by the bench's cpu_baseline / reference
 * legs.  The product (the CUDA library) never calls, links or includes it, and this file includes
 * nothing of the product: every constant, hash, table and layout below is written out here a second
 * time on purpose.
 *
 * Every candidate is evaluated on its own, from the full concatenated input vector, with no tiling,
 * no decomposition of the first layer and no cached partial results, in double precision over the
 * exact input values (fp32, or bf16 bit patterns widened exactly).
 *
 * Where the paper fixes the computation the function cites the passage.  Where the paper is silent
 * the choice is named "reading" in the comment; those readings have no pin in the paper itself
 * ("parity unpinned by the paper"): FFN form and mean pooling in eq. 2, the sum that combines the
 * two user vectors, SimTier tier edges and tier count, the order of the concatenated input, the
 * normalisation options of LSH-DIN / SimTier, and the bucket hash of the cross features.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC (see build.py beside this file).  OpenMP only spreads
 * independent candidates (or independent sequence rows) over host cores; it changes no arithmetic.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_BUCKET_MOD = 0, ORC_BUCKET_HASH = 1 };
enum { ORC_BLK_ATT = 1, ORC_BLK_CROSS = 2, ORC_BLK_BEA = 4, ORC_BLK_LSH_DIN = 8, ORC_BLK_SIMTIER = 16 };
enum { ORC_NORM_NONE = 0, ORC_NORM_MEAN = 1 };

typedef struct {
    int32_t dtype;        /* storage type of E, T, V, bea_w, weights, and of u / S when given projected */
    int64_t M;            /* rows of the item table */
    int32_t d;            /* width of item / user vectors */
    int32_t F, B, dc;     /* cross fields, buckets per field, width of a cross embedding */
    int32_t n_hidden;     /* hidden layers of the scoring MLP */
    int32_t hidden[4];
    int32_t bucket_mode;
    int32_t blocks;       /* ORC_BLK_* mask */
    int32_t n_bridge;     /* n of Algorithm 1 */
    int32_t lsh_bits;     /* d' of eq. 5 */
    int32_t n_tiers;      /* N of eq. 9 */
    int32_t lsh_din_norm; /* ORC_NORM_NONE: eq. 8 as printed (a sum); ORC_NORM_MEAN: divided by l */
    int32_t simtier_norm; /* ORC_NORM_NONE: raw counts (eq. 9); ORC_NORM_MEAN: counts divided by l */
    int32_t emit_sigmoid;
    int32_t n_categories; /* 0: the interaction blocks see the whole sequence; > 0: only the sub-sequence of the
                             candidate's category (Section 3.3, SIM-hard) */
} orc_cfg;

typedef struct {
    const void *W[4];     /* W[k]: [hidden[k] x in_k] row-major; in_0 = orc_input_width(cfg) */
    const float *b[4];    /* [hidden[k]] */
    const void *w_out;    /* [hidden[n_hidden-1]] */
    const float *b_out;   /* [1] */
} orc_mlp_weights;

typedef struct {
    const void *W_profile; /* [d x dU] */
    const void *W_seq;     /* [d x dU] */
    const void *W_a;       /* [d x d] */
    const float *b_a;      /* [d] */
    const void *W_b;       /* [d x d] */
    const float *b_b;      /* [d] */
} orc_user_weights;

/* One stored element, widened exactly to double. */
static double ld(const void *p, int64_t i, int dtype)
{
    if (dtype == ORC_F32) return (double)((const float *)p)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------------------------
 * Cross-feature bucket of a candidate (Section 3.3: the real-time half of a cross feature indexes
 * the user's pre-cached part by an attribute of the candidate).  Reading: the attribute is a bucket
 * derived from the id -- id mod B, or a 64-bit mix of (id, field) mod B.  The mix is the published
 * splitmix64 output function applied to id * 0x9E3779B97F4A7C15 + field.
 * ------------------------------------------------------------------------------------------- */
uint64_t orc_mix64(uint64_t id, uint64_t field)
{
    uint64_t z = id * 0x9E3779B97F4A7C15ULL + field;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

int64_t orc_bucket(int64_t id, int field, int B, int mode)
{
    if (mode == ORC_BUCKET_MOD) return id % B;
    return (int64_t)(orc_mix64((uint64_t)id, (uint64_t)field) % (uint64_t)B);
}

/* Category of an item (Section 3.3: SIM-hard selects sub-sequences "based on the candidate items' category").
 * Reading: like the cross-feature attribute, the category is derived from the id, with the bucket function applied
 * to a field number of its own. */
enum { ORC_CATEGORY_FIELD = 3239 };
int64_t orc_category(int64_t id, int n_categories, int mode) { return orc_bucket(id, ORC_CATEGORY_FIELD, n_categories, mode); }

/* ---------------------------------------------------------------------------------------------
 * LSH signatures (Section 4.2).
 * ------------------------------------------------------------------------------------------- */

/* eq. 5: bit k = ReLU(Sign(m . W_hash[k])): 1 iff the projection is strictly positive. */
void orc_lsh_hash_bits(const double *m, const double *W_hash, int d, int dbits, uint8_t *bits)
{
    for (int k = 0; k < dbits; ++k) {
        double p = 0.0;
        for (int c = 0; c < d; ++c) p += m[c] * W_hash[(int64_t)k * d + c];
        bits[k] = p > 0.0 ? 1 : 0;
    }
}

/* Eight bits -> one uint8, first bit most significant (the worked example 00110101b = 53). */
void orc_pack_bits(const uint8_t *bits, int nbits, uint8_t *out)
{
    for (int byte = 0; byte < nbits / 8; ++byte) {
        unsigned v = 0;
        for (int k = 0; k < 8; ++k) v = (v << 1) | (bits[byte * 8 + k] & 1u);
        out[byte] = (uint8_t)v;
    }
}

/* The 1 x 256 lookup table that replaces PopulationCount for uint8 signatures. */
static int popcount_lut[256];
static int popcount_lut_ready = 0;
static void build_lut(void)
{
    for (int v = 0; v < 256; ++v) {
        int c = 0;
        for (int k = 0; k < 8; ++k) c += (v >> k) & 1;
        popcount_lut[v] = c;
    }
    popcount_lut_ready = 1;
}

int orc_popcount_lut(int v)
{
    if (!popcount_lut_ready) build_lut();
    return popcount_lut[v & 255];
}

/* eq. 6 numerator: number of bit positions where the two signatures agree (XNOR, then count).
 * via_lut = 1 takes the table-lookup route, 0 counts bit by bit. */
int orc_lsh_matches(const uint8_t *a, const uint8_t *b, int nbytes, int via_lut)
{
    int k = 0;
    for (int i = 0; i < nbytes; ++i) {
        unsigned x = (unsigned)(uint8_t) ~(a[i] ^ b[i]);
        if (via_lut) {
            k += orc_popcount_lut((int)x);
        } else {
            for (int t = 0; t < 8; ++t) k += (x >> t) & 1u;
        }
    }
    return k;
}

/* eq. 7: M_sim[i][j] = matches / d'. */
void orc_lsh_similarity(const uint8_t *sig_items, int b, const uint8_t *sig_seq, int l, int dbits, double *sim)
{
    int nbytes = dbits / 8;
    for (int i = 0; i < b; ++i)
        for (int j = 0; j < l; ++j)
            sim[(int64_t)i * l + j] =
                (double)orc_lsh_matches(sig_items + (int64_t)i * nbytes, sig_seq + (int64_t)j * nbytes, nbytes, 1) /
                (double)dbits;
}

/* eq. 8 (read as M_sim times the projected sequence): din = sum_j sim_j * S_j, optionally / l. */
void orc_lsh_din(const double *sim, const double *S, int l, int d, int norm, double *out)
{
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j < l; ++j)
        for (int c = 0; c < d; ++c) out[c] += sim[j] * S[(int64_t)j * d + c];
    if (norm == ORC_NORM_MEAN)
        for (int c = 0; c < d; ++c) out[c] /= (double)l;
}

/* eq. 9: histogram of the similarities over N tiers.  Reading: N equal-width intervals over [0,1],
 * the last one closed; decided on the integer match count so that no float compare is involved:
 * tier = min(N-1, floor(matches * N / d')). */
int orc_tier_of(int matches, int dbits, int n_tiers)
{
    int t = (matches * n_tiers) / dbits;
    return t < n_tiers - 1 ? t : n_tiers - 1;
}

void orc_simtier(const int *matches, int l, int dbits, int n_tiers, int norm, double *out)
{
    for (int t = 0; t < n_tiers; ++t) out[t] = 0.0;
    for (int j = 0; j < l; ++j) out[orc_tier_of(matches[j], dbits, n_tiers)] += 1.0;
    if (norm == ORC_NORM_MEAN)
        for (int t = 0; t < n_tiers; ++t) out[t] /= (double)l;
}

/* ---------------------------------------------------------------------------------------------
 * Attention of one query row over a sequence: softmax(q S^T / sqrt(d)) S.
 * Used for the dense target attention (candidate vector as the query; Section 4.2 describes it as
 * similarity with every historical item followed by pooling) and for eqs. 2 and 3.
 * ------------------------------------------------------------------------------------------- */
void orc_attention(const double *q, const double *S, int l, int d, double *out)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)l);
    double m = -INFINITY;
    for (int j = 0; j < l; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += q[c] * S[(int64_t)j * d + c];
        s[j] = dot / sqrt((double)d);
        if (s[j] > m) m = s[j];
    }
    double z = 0.0;
    for (int j = 0; j < l; ++j) {
        s[j] = exp(s[j] - m);
        z += s[j];
    }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j < l; ++j) {
        double a = s[j] / z;
        for (int c = 0; c < d; ++c) out[c] += a * S[(int64_t)j * d + c];
    }
    free(s);
}

/* Algorithm 1 line 4: v = w_hat V, one candidate row. */
void orc_bea(const double *w_hat, const double *V, int n, int dp, double *out)
{
    for (int c = 0; c < dp; ++c) out[c] = 0.0;
    for (int k = 0; k < n; ++k)
        for (int c = 0; c < dp; ++c) out[c] += w_hat[k] * V[(int64_t)k * dp + c];
}

/* y = W x + b, W [rows x cols] row-major in storage type. */
static void linear(const void *W, int dtype, const float *b, int rows, int cols, const double *x, double *y)
{
    for (int r = 0; r < rows; ++r) {
        double acc = b ? (double)b[r] : 0.0;
        for (int c = 0; c < cols; ++c) acc += ld(W, (int64_t)r * cols + c, dtype) * x[c];
        y[r] = acc;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Item side, nearline (Section 3.2 eq. 4; Algorithm 1 step 3; Section 4.2 eq. 5).  One call computes,
 * for n items, what the nearline pipeline stores in the index table.
 *   eq. 4   I^ = MLP(I).  Reading (the paper names no widths or activation): one hidden layer,
 *           I^ = W_1 ReLU(W_0 I + b_0) + b_1, widths dI -> hI -> d, linear output.
 *   Alg. 1  step 3: w^ = Softmax(I_id B^T / sqrt(d)), one row of n_bridge weights per item; I_id is the
 *           item's d-wide id embedding (an input of its own; the algorithm's I is d-wide).
 *   eq. 5   signature bits of the item's multi-modal embedding M (see orc_lsh_hash_bits), packed
 *           first-bit-most-significant.
 * Inputs in storage type `dtype`; outputs in double (vectors, weights) and bytes (signatures).  A NULL
 * output (with its inputs) skips that part.
 * ------------------------------------------------------------------------------------------- */
void orc_item_nearline(int dtype, int64_t n, int dI, int hI, int d, const void *I_raw, const void *W0, const float *b0,
                       const void *W1, const float *b1, double *I_hat, int n_bridge, const void *I_id, const void *bridges,
                       double *w_hat, int d_mm, int dbits, const void *M_mm, const void *W_hash, uint8_t *sig)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        if (I_hat) {
            double *x = (double *)malloc(sizeof(double) * (size_t)(dI + hI));
            double *h = x + dI;
            for (int c = 0; c < dI; ++c) x[c] = ld(I_raw, i * dI + c, dtype);
            linear(W0, dtype, b0, hI, dI, x, h);
            for (int j = 0; j < hI; ++j) h[j] = h[j] > 0.0 ? h[j] : 0.0;
            linear(W1, dtype, b1, d, hI, h, I_hat + i * d);
            free(x);
        }
        if (w_hat) {
            double s[64], mx = -INFINITY, den = 0.0;
            for (int k = 0; k < n_bridge; ++k) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += ld(I_id, i * d + c, dtype) * ld(bridges, (int64_t)k * d + c, dtype);
                s[k] = acc / sqrt((double)d);
                if (s[k] > mx) mx = s[k];
            }
            for (int k = 0; k < n_bridge; ++k) den += exp(s[k] - mx);
            for (int k = 0; k < n_bridge; ++k) w_hat[i * n_bridge + k] = exp(s[k] - mx) / den;
        }
        if (sig) {
            double *m = (double *)malloc(sizeof(double) * (size_t)d_mm * (size_t)(1 + dbits));
            double *Wd = m + d_mm;
            uint8_t bits[1024];
            for (int c = 0; c < d_mm; ++c) m[c] = ld(M_mm, i * d_mm + c, dtype);
            for (int64_t c = 0; c < (int64_t)d_mm * dbits; ++c) Wd[c] = ld(W_hash, c, dtype);
            orc_lsh_hash_bits(m, Wd, d_mm, dbits, bits);
            orc_pack_bits(bits, dbits, sig + i * (dbits / 8));
            free(m);
        }
    }
}

/* Algorithm 1 steps 1-2, user side: W = Softmax(B U^T / sqrt(d)) [n x m] (one softmax per bridge over the m user-side
 * feature embeddings), then V = f(U, W | Theta_u) [n x d].  Reading of f (the paper leaves the network open): one linear
 * layer on the attention-weighted features, V_k = W_f (sum_j W_kj U_j).  bridges [n x d], U [m x d], W_f [d x d] in
 * storage type; V_out [n x d], W_out [n x m] (may be NULL) in double. */
void orc_bea_user(int dtype, int n, int m, int d, const void *bridges, const void *U, const void *W_f, double *V_out, double *W_out)
{
    double *w = (double *)malloc(sizeof(double) * (size_t)(m + d));
    double *a = w + m;
    for (int k = 0; k < n; ++k) {
        double mx = -INFINITY, den = 0.0;
        for (int j = 0; j < m; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += ld(bridges, (int64_t)k * d + c, dtype) * ld(U, (int64_t)j * d + c, dtype);
            w[j] = acc / sqrt((double)d);
            if (w[j] > mx) mx = w[j];
        }
        for (int j = 0; j < m; ++j) den += exp(w[j] - mx);
        for (int j = 0; j < m; ++j) w[j] = exp(w[j] - mx) / den;
        if (W_out)
            for (int j = 0; j < m; ++j) W_out[(int64_t)k * m + j] = w[j];
        for (int c = 0; c < d; ++c) {
            a[c] = 0.0;
            for (int j = 0; j < m; ++j) a[c] += w[j] * ld(U, (int64_t)j * d + c, dtype);
        }
        linear(W_f, dtype, NULL, d, d, a, V_out + (int64_t)k * d);
    }
    free(w);
}

/* The projections behind eq. 5's bits, for tests that need to know how close to zero a bit was decided. */
void orc_lsh_projections(int dtype, int64_t n, int d_mm, int dbits, const void *M_mm, const void *W_hash, double *proj)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int k = 0; k < dbits; ++k) {
            double p = 0.0;
            for (int c = 0; c < d_mm; ++c) p += ld(M_mm, i * d_mm + c, dtype) * ld(W_hash, (int64_t)k * d_mm + c, dtype);
            proj[i * dbits + k] = p;
        }
}

/* ---------------------------------------------------------------------------------------------
 * User side, eqs. 1-3 (Section 3.1).  Readings: FFN(x) = ReLU(x W_a^T + b_a) W_b^T + b_b, Pooling =
 * mean over the sequence, combined vector = U_self_attention + U_profile_attention.
 * profile [dU], seq [l x dU] in storage type; u_out [d], S_out [l x d] (= U^_seq) in double.
 * ------------------------------------------------------------------------------------------- */
void orc_user_state(const orc_cfg *cfg, const orc_user_weights *w, int dU, const void *profile, const void *seq,
                    int l, double *u_out, double *S_out)
{
    const int d = cfg->d, dt = cfg->dtype;
    double *prof_hat = (double *)calloc((size_t)d, sizeof(double));
    /* eq. 1 */
    for (int j = 0; j < d; ++j) {
        double acc = 0.0;
        for (int k = 0; k < dU; ++k) acc += ld(profile, k, dt) * ld(w->W_profile, (int64_t)j * dU + k, dt);
        prof_hat[j] = acc;
    }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < l; ++i)
        for (int j = 0; j < d; ++j) {
            double acc = 0.0;
            for (int k = 0; k < dU; ++k)
                acc += ld(seq, (int64_t)i * dU + k, dt) * ld(w->W_seq, (int64_t)j * dU + k, dt);
            S_out[(int64_t)i * d + j] = acc;
        }
    /* eq. 2: every sequence row attends over the whole sequence, then FFN, then mean pooling */
    double *Z = (double *)calloc((size_t)l * d, sizeof(double));
#pragma omp parallel for schedule(dynamic, 8)
    for (int i = 0; i < l; ++i) {
        double *ctx = (double *)malloc(sizeof(double) * d * 2);
        double *hid = ctx + d;
        orc_attention(S_out + (int64_t)i * d, S_out, l, d, ctx);
        linear(w->W_a, dt, w->b_a, d, d, ctx, hid);
        for (int j = 0; j < d; ++j) hid[j] = hid[j] > 0.0 ? hid[j] : 0.0;
        linear(w->W_b, dt, w->b_b, d, d, hid, Z + (int64_t)i * d);
        free(ctx);
    }
    double *u_prof = (double *)calloc((size_t)d, sizeof(double));
    /* eq. 3 */
    orc_attention(prof_hat, S_out, l, d, u_prof);
    for (int j = 0; j < d; ++j) {
        double pooled = 0.0;
        for (int i = 0; i < l; ++i) pooled += Z[(int64_t)i * d + j];
        u_out[j] = pooled / (double)l + u_prof[j];
    }
    free(prof_hat);
    free(Z);
    free(u_prof);
}

/* ---------------------------------------------------------------------------------------------
 * The real-time model input of one candidate (hybrid inputs, Sections 2 and 3): reading of the order
 *   [ u | e | att | cross f=0..F-1 | v_bea | lsh_din | simtier ]   (disabled blocks leave no columns).
 * ------------------------------------------------------------------------------------------- */
int orc_input_width(const orc_cfg *cfg)
{
    int w = cfg->d + cfg->d;
    if (cfg->blocks & ORC_BLK_ATT) w += cfg->d;
    if (cfg->blocks & ORC_BLK_CROSS) w += cfg->F * cfg->dc;
    if (cfg->blocks & ORC_BLK_BEA) w += cfg->d;
    if (cfg->blocks & ORC_BLK_LSH_DIN) w += cfg->d;
    if (cfg->blocks & ORC_BLK_SIMTIER) w += cfg->n_tiers;
    return w;
}

typedef struct {
    const void *E;          /* [M x d] item vectors (the nearline table, Section 3.2) */
    const void *bea_w;      /* [M x n] item-side BEA weights (Algorithm 1 line 3), or NULL */
    const uint8_t *sig;     /* [M x d'/8] item signatures, or NULL */
    const double *u;        /* [d] combined user vector */
    const double *S;        /* [l x d] projected behaviour sequence */
    int32_t l;
    const void *T;          /* [F x B x dc] user-side part of the cross features, or NULL */
    const void *V;          /* [n x d] user-side BEA vectors (Algorithm 1 line 2), or NULL */
    const uint8_t *sig_seq; /* [l x d'/8] signatures of the sequence items, or NULL */
    const int32_t *seq_cat; /* [l] category of every sequence item (the parsed <user, category, sub_sequence> form of
                               Section 3.3), or NULL when n_categories = 0 */
} orc_request;

void orc_build_input(const orc_cfg *cfg, const orc_request *rq, int64_t id, double *x)
{
    const int d = cfg->d, dt = cfg->dtype;
    int o = 0;
    for (int c = 0; c < d; ++c) x[o++] = rq->u[c];
    double *e = x + o;
    for (int c = 0; c < d; ++c) x[o++] = ld(rq->E, id * d + c, dt);
    /* Section 3.3 (SIM-hard): with categories on, the sequence the interaction blocks see is the sub-sequence of the
     * user's behaviours whose category is the candidate's, in their original order.  Reading for an empty sub-sequence
     * (the paper is silent): attention output, LSH-DIN output and tier counts are all zero. */
    const double *S = rq->S;
    const uint8_t *sig_seq = rq->sig_seq;
    int l = rq->l;
    double *S_sub = NULL;
    uint8_t *sig_sub = NULL;
    if (cfg->n_categories > 0) {
        const int64_t cat = orc_category(id, cfg->n_categories, cfg->bucket_mode);
        const int nbytes = cfg->lsh_bits / 8;
        S_sub = (double *)malloc(sizeof(double) * (size_t)(rq->l > 0 ? rq->l : 1) * (size_t)d);
        if (rq->sig_seq) sig_sub = (uint8_t *)malloc((size_t)(rq->l > 0 ? rq->l : 1) * (size_t)(nbytes > 0 ? nbytes : 1));
        l = 0;
        for (int j = 0; j < rq->l; ++j)
            if (rq->seq_cat[j] == cat) {
                memcpy(S_sub + (int64_t)l * d, rq->S + (int64_t)j * d, sizeof(double) * (size_t)d);
                if (sig_sub) memcpy(sig_sub + (int64_t)l * nbytes, rq->sig_seq + (int64_t)j * nbytes, (size_t)nbytes);
                l += 1;
            }
        S = S_sub, sig_seq = sig_sub;
    }
    if (cfg->blocks & ORC_BLK_ATT) {
        if (l > 0) orc_attention(e, S, l, d, x + o);
        else
            for (int c = 0; c < d; ++c) x[o + c] = 0.0;
        o += d;
    }
    if (cfg->blocks & ORC_BLK_CROSS) {
        for (int f = 0; f < cfg->F; ++f) {
            int64_t bkt = orc_bucket(id, f, cfg->B, cfg->bucket_mode);
            for (int c = 0; c < cfg->dc; ++c) x[o++] = ld(rq->T, ((int64_t)f * cfg->B + bkt) * cfg->dc + c, dt);
        }
    }
    if (cfg->blocks & ORC_BLK_BEA) {
        int n = cfg->n_bridge;
        double *wh = (double *)malloc(sizeof(double) * ((size_t)n + (size_t)n * d));
        double *V = wh + n;
        for (int k = 0; k < n; ++k) wh[k] = ld(rq->bea_w, id * n + k, dt);
        for (int k = 0; k < n * d; ++k) V[k] = ld(rq->V, k, dt);
        orc_bea(wh, V, n, d, x + o);
        o += d;
        free(wh);
    }
    if (cfg->blocks & (ORC_BLK_LSH_DIN | ORC_BLK_SIMTIER)) {
        int nbytes = cfg->lsh_bits / 8;
        int *matches = (int *)malloc(sizeof(int) * (size_t)(l > 0 ? l : 1));
        double *sim = (double *)malloc(sizeof(double) * (size_t)(l > 0 ? l : 1));
        for (int j = 0; j < l; ++j) {
            matches[j] = orc_lsh_matches(rq->sig + id * nbytes, sig_seq + (int64_t)j * nbytes, nbytes, 1);
            sim[j] = (double)matches[j] / (double)cfg->lsh_bits;
        }
        if (cfg->blocks & ORC_BLK_LSH_DIN) {
            if (l > 0) orc_lsh_din(sim, S, l, d, cfg->lsh_din_norm, x + o);
            else
                for (int c = 0; c < d; ++c) x[o + c] = 0.0;
            o += d;
        }
        if (cfg->blocks & ORC_BLK_SIMTIER) {
            if (l > 0) orc_simtier(matches, l, cfg->lsh_bits, cfg->n_tiers, cfg->simtier_norm, x + o);
            else
                for (int t = 0; t < cfg->n_tiers; ++t) x[o + t] = 0.0;
            o += cfg->n_tiers;
        }
        free(matches);
        free(sim);
    }
    free(S_sub);
    free(sig_sub);
}

/* The shallow scoring MLP on the full concatenated input (Section 1): ReLU hidden layers, linear
 * output; optional sigmoid. */
double orc_mlp(const orc_cfg *cfg, const orc_mlp_weights *w, const double *x)
{
    int in = orc_input_width(cfg);
    int maxw = in;
    for (int k = 0; k < cfg->n_hidden; ++k)
        if (cfg->hidden[k] > maxw) maxw = cfg->hidden[k];
    double *a = (double *)malloc(sizeof(double) * (size_t)maxw * 2);
    double *bq = a + maxw;
    memcpy(a, x, sizeof(double) * (size_t)in);
    for (int k = 0; k < cfg->n_hidden; ++k) {
        linear(w->W[k], cfg->dtype, w->b[k], cfg->hidden[k], in, a, bq);
        for (int j = 0; j < cfg->hidden[k]; ++j) a[j] = bq[j] > 0.0 ? bq[j] : 0.0;
        in = cfg->hidden[k];
    }
    double logit = (double)w->b_out[0];
    for (int j = 0; j < in; ++j) logit += ld(w->w_out, j, cfg->dtype) * a[j];
    free(a);
    if (cfg->emit_sigmoid) return 1.0 / (1.0 + exp(-logit));
    return logit;
}

/* Scores n candidates of one request.  An id outside [0, M) yields NaN.  Returns the number of bad ids.
 * x_out (optional) receives the n concatenated input vectors. */
int orc_score(const orc_cfg *cfg, const orc_mlp_weights *w, const orc_request *rq, const int32_t *ids, int n,
              double *out, double *x_out)
{
    const int width = orc_input_width(cfg);
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4) reduction(+ : bad)
    for (int i = 0; i < n; ++i) {
        int64_t id = ids[i];
        if (id < 0 || id >= cfg->M) {
            out[i] = NAN;
            bad += 1;
            continue;
        }
        double *x = (double *)malloc(sizeof(double) * (size_t)width);
        orc_build_input(cfg, rq, id, x);
        out[i] = orc_mlp(cfg, w, x);
        if (x_out) memcpy(x_out + (int64_t)i * width, x, sizeof(double) * (size_t)width);
        free(x);
    }
    return bad;
}

/* Item side: the table write of the nearline pipeline (Section 3.2, 3.4): full (ids NULL: rows 0..n-1)
 * or incremental (row i of `rows` replaces table row ids[i]).  Byte copy, row_bytes per row.
 * Out-of-range ids are skipped and counted. */
int orc_table_refresh(uint8_t *table, int64_t M, int64_t row_bytes, const int32_t *ids, int64_t n,
                      const uint8_t *rows)
{
    int bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t r = ids ? (int64_t)ids[i] : i;
        if (r < 0 || r >= M) {
            bad += 1;
            continue;
        }
        memcpy(table + r * row_bytes, rows + i * row_bytes, (size_t)row_bytes);
    }
    return bad;
}
