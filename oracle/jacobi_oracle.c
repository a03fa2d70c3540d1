/*
 * CPU oracle for parallel autoregressive sampling by fixed-point iteration.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, single-threaded
 * restatement of the method in "Accelerating Feedforward Computation via
 * Parallel Nonlinear Equation Solving" (arXiv 2002.03629).  It exists so that
 * the CUDA library can be checked against it; it shares no code, table or
 * constant with that library and must never be called from the product path.
 *
 * What is written out here, with the passage each part follows:
 *   - the recurrence x_t = h_t(u, x_{1:t-1}) for ancestral sampling with the
 *     random numbers u fixed in advance            (Eq. 1; Appendix A.3)
 *   - nonlinear Jacobi iteration                    (Eq. 3; Algorithm 1)
 *   - nonlinear Gauss-Seidel = one feedforward pass (Eq. 4; Section 3.2)
 *   - Jacobi-GS and GS-Jacobi block hybrids         (Algorithms 2 and 3)
 *
 * h_t is one conditional of a masked autoregressive network: either a masked
 * MLP (MADE) or a stack of masked 3x3 convolutions with a 1x1 head.  All sums
 * are accumulated in double precision in index order over every term, masked
 * (zero) terms included.  Where the network is declared bf16, weights and
 * hidden activations are rounded to bf16 (round-to-nearest-even) at the same
 * points the method's description fixes: weights after masking, activations
 * after bias and nonlinearity.  Logits are rounded once to float; the integer
 * decision (threshold or argmax) is then taken in float arithmetic.
 *
 * Pins (tests/test_oracle_*.py): brute-force enumeration of all outcomes on a
 * 16-position binary model, the convergence propositions of Section 3, the
 * worked Examples 1-3 of Section 4.1 realised as hand-built networks, the
 * autoregressive property by bit flips, a hand-computed 3-position network,
 * numpy re-computation of the forward pass (default and caller-given degrees),
 * the decision margins recomputed from the logits and checked by moving the
 * noise just short of and just past them, and, for the categorical inverse
 * CDF, enumeration of all outcomes of a 3-way model, its law by chi-square and
 * exact boundary cases.  Iteration counts on the
 * random-weight workloads have no value in the paper to compare with:
 * "parity unpinned" for those counts (they are bounded by the propositions
 * and checked on Examples 1-3 only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_NOISE_UNIFORM_ICDF = 0, ORC_NOISE_LOGISTIC = 1, ORC_NOISE_GUMBEL = 2, ORC_NOISE_UNIFORM_CAT = 3 };
enum { ORC_ACT_RELU = 0, ORC_ACT_GELU_TANH = 1 };
enum { ORC_PREC_F32 = 0, ORC_PREC_BF16 = 1 };
enum { ORC_KIND_MADE = 0, ORC_KIND_CONV = 1 };

#define ORC_MAX_LAYERS 16

/* ---------------------------------------------------------------- rounding */

/* float -> nearest bf16 (ties to even), returned as a float. */
static float round_bf16(float v)
{
    uint32_t bits;
    memcpy(&bits, &v, 4);
    if ((bits & 0x7f800000u) == 0x7f800000u) return v;      /* inf / nan unchanged */
    uint32_t lsb = (bits >> 16) & 1u;
    bits += 0x7fffu + lsb;
    bits &= 0xffff0000u;
    memcpy(&v, &bits, 4);
    return v;
}

static double act_fn(int act, double v)
{
    if (act == ORC_ACT_RELU) return v > 0.0 ? v : 0.0;
    /* tanh form of GELU */
    double y = 0.7978845608028654 * (v + 0.044715 * v * v * v);
    return 0.5 * v * (1.0 + tanh(y));
}

/* pre-activation (double) -> stored hidden activation */
static float hidden_value(int act, int prec, double pre)
{
    float pre_f = (float)pre;
    float a = (float)act_fn(act, (double)pre_f);
    return prec == ORC_PREC_BF16 ? round_bf16(a) : a;
}

/* ------------------------------------------------------------------- model */

typedef struct orc_model {
    int kind;
    int T;              /* number of positions (states s_1..s_T) */
    int C;              /* logits per position: 1 binary, else classes */
    int act, prec;
    int n_lut;
    float *lut;         /* input encoding: network input for symbol v */

    /* MADE */
    int L;                              /* hidden layers */
    int n[ORC_MAX_LAYERS + 2];          /* widths: n[0]=T, n[1..L], n[L+1]=T*C */
    int *deg[ORC_MAX_LAYERS + 2];       /* degree of every unit of every layer */
    float *Wm[ORC_MAX_LAYERS + 1];      /* masked (and rounded) weights [n[l+1]][n[l]] */
    float *b[ORC_MAX_LAYERS + 1];

    /* conv */
    int height, width, in_ch, ch, n_conv;
    float *Wc[ORC_MAX_LAYERS + 1];      /* masked conv weights [cout][3][3][cin]; head [in_ch*C][ch] */
    float *bc[ORC_MAX_LAYERS + 1];
} orc_model;

void orc_model_destroy(orc_model *m)
{
    if (!m) return;
    free(m->lut);
    for (int l = 0; l < ORC_MAX_LAYERS + 2; ++l) free(m->deg[l]);
    for (int l = 0; l < ORC_MAX_LAYERS + 1; ++l) {
        free(m->Wm[l]); free(m->b[l]); free(m->Wc[l]); free(m->bc[l]);
    }
    free(m);
}

/*
 * Masked MLP.  Degrees: input position d (0-based) has degree d+1; hidden unit
 * j of a layer of width H has degree 1 + floor(j*(T-1)/H) unless the caller
 * gives degrees; output unit (d, c) has degree d+1.  A hidden unit may read a
 * unit of the layer below whose degree is <= its own; an output may only read
 * hidden units of strictly smaller degree, so logits of position d depend on
 * positions < d alone, which is what makes Eq. 5 a triangular system.
 *
 * W[l]: unmasked float [n[l+1]][n[l]], b[l]: float [n[l+1]], l = 0..L.
 * hidden_deg: NULL or L arrays of n[l+1] ints.
 */
orc_model *orc_made_create(int T, int C, int L, const int *H, int act, int prec,
                           const float *const *W, const float *const *b,
                           const float *lut, int n_lut, const int *const *hidden_deg)
{
    if (L < 1 || L > ORC_MAX_LAYERS || T < 1 || C < 1 || C > 256) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->kind = ORC_KIND_MADE; m->T = T; m->C = C; m->L = L; m->act = act; m->prec = prec;
    m->n_lut = n_lut;
    m->lut = (float *)malloc(sizeof(float) * (size_t)n_lut);
    for (int i = 0; i < n_lut; ++i)
        m->lut[i] = prec == ORC_PREC_BF16 ? round_bf16(lut[i]) : lut[i];
    m->n[0] = T;
    for (int l = 0; l < L; ++l) m->n[l + 1] = H[l];
    m->n[L + 1] = T * C;
    for (int l = 0; l <= L + 1; ++l) m->deg[l] = (int *)malloc(sizeof(int) * (size_t)m->n[l]);
    for (int d = 0; d < T; ++d) m->deg[0][d] = d + 1;
    for (int l = 1; l <= L; ++l)
        for (int j = 0; j < m->n[l]; ++j)
            m->deg[l][j] = hidden_deg && hidden_deg[l - 1]
                               ? hidden_deg[l - 1][j]
                               : 1 + (int)(((long long)j * (T - 1)) / m->n[l]);
    for (int d = 0; d < T; ++d)
        for (int c = 0; c < C; ++c) m->deg[L + 1][d * C + c] = d + 1;
    for (int l = 0; l <= L; ++l) {
        int nin = m->n[l], nout = m->n[l + 1];
        m->Wm[l] = (float *)malloc(sizeof(float) * (size_t)nin * (size_t)nout);
        m->b[l] = (float *)malloc(sizeof(float) * (size_t)nout);
        for (int i = 0; i < nout; ++i) {
            for (int j = 0; j < nin; ++j) {
                int keep = (l == L) ? (m->deg[l + 1][i] > m->deg[l][j])
                                    : (m->deg[l + 1][i] >= m->deg[l][j]);
                float w = keep ? W[l][(size_t)i * nin + j] : 0.0f;
                m->Wm[l][(size_t)i * nin + j] = prec == ORC_PREC_BF16 ? round_bf16(w) : w;
            }
            m->b[l][i] = b[l][i];
        }
    }
    return m;
}

int orc_T(const orc_model *m) { return m->T; }
int orc_C(const orc_model *m) { return m->C; }
/* masked weights as the oracle holds them (for tests that recompute with numpy) */
const float *orc_masked_weight(const orc_model *m, int l)
{
    return m->kind == ORC_KIND_MADE ? m->Wm[l] : m->Wc[l];
}
const int *orc_degrees(const orc_model *m, int l) { return m->deg[l]; }

/* pre-activation of unit i of layer l+1 given the whole layer below */
static double made_unit(const orc_model *m, int l, int i, const float *below)
{
    const float *w = m->Wm[l] + (size_t)i * m->n[l];
    double acc = 0.0;
    for (int j = 0; j < m->n[l]; ++j) acc += (double)w[j] * (double)below[j];
    return acc + (double)m->b[l][i];
}

typedef struct {
    float *a[ORC_MAX_LAYERS + 1];   /* a[0] encoded input, a[1..L] hidden */
} made_ws;

static void made_ws_alloc(const orc_model *m, made_ws *ws)
{
    for (int l = 0; l <= m->L; ++l) ws->a[l] = (float *)calloc((size_t)m->n[l], sizeof(float));
}
static void made_ws_free(const orc_model *m, made_ws *ws)
{
    for (int l = 0; l <= m->L; ++l) free(ws->a[l]);
}

/* all logits of the network on input x: z[T*C] */
static void made_forward(const orc_model *m, const uint8_t *x, float *z)
{
    made_ws ws; made_ws_alloc(m, &ws);
    for (int d = 0; d < m->T; ++d) ws.a[0][d] = m->lut[x[d]];
    for (int l = 0; l < m->L; ++l)
        for (int i = 0; i < m->n[l + 1]; ++i)
            ws.a[l + 1][i] = hidden_value(m->act, m->prec, made_unit(m, l, i, ws.a[l]));
    for (int i = 0; i < m->n[m->L + 1]; ++i) z[i] = (float)made_unit(m, m->L, i, ws.a[m->L]);
    made_ws_free(m, &ws);
}

/* ---------------------------------------------------------------- sampling */

/*
 * h_t's last step (Appendix A.3): turn the conditional's logits into the value
 * of x_t using the random numbers reserved for position t.
 *   UNIFORM_ICDF  x = [u < sigmoid(z)]             (inverse-CDF for a Bernoulli)
 *   LOGISTIC      x = [z + eps > 0]                (eps logistic: same law)
 *   GUMBEL        x = argmax_c (z_c + g_c), lowest index among equal maxima
 *   UNIFORM_CAT   x = the first class c with u < F_c, F_c = sum_{i<=c} softmax(z)_i
 *                 (inverse-CDF for a categorical: one uniform number per position)
 * nz: C logits of this position; noise: 1 value, or C values for GUMBEL.
 */

/* unnormalised cumulative distribution of softmax(nz): cum[c] = sum_{i<=c} exp(nz[i] - max);
 * returns the total cum[C-1] */
static double softmax_cumulative(int C, const float *nz, double *cum)
{
    double mx = (double)nz[0];
    for (int c = 1; c < C; ++c) if ((double)nz[c] > mx) mx = (double)nz[c];
    double run = 0.0;
    for (int c = 0; c < C; ++c) { run += exp((double)nz[c] - mx); cum[c] = run; }
    return run;
}

static int sample_position(int C, const float *nz, const float *noise, int nk)
{
    if (nk == ORC_NOISE_UNIFORM_CAT) {
        double cum[256];
        double tot = softmax_cumulative(C, nz, cum);
        double target = (double)noise[0] * tot;
        for (int c = 0; c < C; ++c)
            if (target < cum[c]) return c;
        return C - 1;       /* u so close to 1 that rounding left it at the total */
    }
    if (nk == ORC_NOISE_UNIFORM_ICDF) {
        float p = (float)(1.0 / (1.0 + exp(-(double)nz[0])));
        return noise[0] < p ? 1 : 0;
    }
    if (nk == ORC_NOISE_LOGISTIC) {
        float s = nz[0] + noise[0];
        return s > 0.0f ? 1 : 0;
    }
    int best = 0;
    float best_v = nz[0] + noise[0];
    for (int c = 1; c < C; ++c) {
        float v = nz[c] + noise[c];
        if (v > best_v) { best_v = v; best = c; }
    }
    return best;
}

/* distance of the decision from a tie, in logit units */
static float decision_margin(int C, const float *nz, const float *noise, int nk)
{
    if (nk == ORC_NOISE_UNIFORM_CAT) {
        /* u lies between the cumulative probabilities F_{x-1} and F_x.  Moving every logit by at
         * most d moves a cumulative probability by at most d/2, so twice the distance of u from
         * the nearer boundary is the tie distance in logit units (the outermost boundaries 0
         * and 1 do not move). */
        double cum[256];
        double tot = softmax_cumulative(C, nz, cum);
        double u = (double)noise[0];
        int x = sample_position(C, nz, noise, nk);
        double gap = INFINITY;
        if (x > 0) gap = u - cum[x - 1] / tot;
        if (x < C - 1 && cum[x] / tot - u < gap) gap = cum[x] / tot - u;
        return (float)(2.0 * gap);
    }
    if (nk == ORC_NOISE_UNIFORM_ICDF) {
        double u = (double)noise[0];
        return (float)fabs((double)nz[0] - (log(u) - log1p(-u)));
    }
    if (nk == ORC_NOISE_LOGISTIC) return fabsf(nz[0] + noise[0]);
    float top = -INFINITY, second = -INFINITY;
    for (int c = 0; c < C; ++c) {
        float v = nz[c] + noise[c];
        if (v > top) { second = top; top = v; }
        else if (v > second) second = v;
    }
    return top - second;
}

static size_t noise_stride(const orc_model *m, int nk)
{
    return nk == ORC_NOISE_GUMBEL ? (size_t)m->C : 1;
}

/* ------------------------------------------------- MADE: sequential sweep */

/*
 * Positions a..b-1 computed in order, each from the positions before it
 * (Eq. 1), updating y in place; positions < a of y are taken as given.
 * Hidden units are evaluated once each, as soon as every position they may
 * read is known (a unit of degree g reads positions < g), with the same
 * full-row dot product the complete forward pass uses, so the logits are the
 * ones made_forward would give on the finished prefix.
 */
static void made_sweep(const orc_model *m, uint8_t *y, int a, int b, const float *noise, int nk)
{
    made_ws ws; made_ws_alloc(m, &ws);
    size_t ns = noise_stride(m, nk);
    float *zt = (float *)malloc(sizeof(float) * (size_t)m->C);
    for (int d = 0; d < m->T; ++d) ws.a[0][d] = m->lut[y[d]];
    for (int l = 0; l < m->L; ++l)
        for (int i = 0; i < m->n[l + 1]; ++i)
            if (m->deg[l + 1][i] <= a)
                ws.a[l + 1][i] = hidden_value(m->act, m->prec, made_unit(m, l, i, ws.a[l]));
    for (int t = a; t < b; ++t) {
        if (t > a)
            for (int l = 0; l < m->L; ++l)
                for (int i = 0; i < m->n[l + 1]; ++i)
                    if (m->deg[l + 1][i] == t)
                        ws.a[l + 1][i] = hidden_value(m->act, m->prec, made_unit(m, l, i, ws.a[l]));
        for (int c = 0; c < m->C; ++c) zt[c] = (float)made_unit(m, m->L, t * m->C + c, ws.a[m->L]);
        y[t] = (uint8_t)sample_position(m->C, zt, noise + (size_t)t * ns, nk);
        ws.a[0][t] = m->lut[y[t]];
    }
    free(zt);
    made_ws_free(m, &ws);
}

/* ------------------------------------------------------ masked conv model */

/*
 * Stack of n_conv masked 3x3 convolutions (zero padding, ReLU) and a 1x1 head.
 * Image [height][width][in_ch], position t = (y*width + x)*in_ch + c (raster
 * order, channels innermost).  Hidden channel k belongs to colour group
 * floor(in_ch*k/ch).  A 3x3 kernel keeps the row above and the pixel to the
 * left entirely; at the centre tap the first layer (type A) keeps input groups
 * strictly below the output's group and the later layers (type B) keep groups
 * <= it.  The head gives sub-pixel c its C logits from hidden groups <= c.
 * So a hidden unit of group g at pixel p reads positions < p*in_ch + g only.
 *
 * W[0]: [ch][3][3][in_ch]; W[1..n_conv-1]: [ch][3][3][ch]; W[n_conv]: [in_ch*C][ch].
 */
static int conv_group(const orc_model *m, int k) { return (int)(((long long)m->in_ch * k) / m->ch); }

orc_model *orc_conv_create(int height, int width, int in_ch, int ch, int n_conv, int C, int prec,
                           const float *const *W, const float *const *b,
                           const float *lut, int n_lut)
{
    if (n_conv < 1 || n_conv > ORC_MAX_LAYERS || C < 1 || C > 256) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->kind = ORC_KIND_CONV; m->height = height; m->width = width; m->in_ch = in_ch; m->ch = ch;
    m->n_conv = n_conv; m->C = C; m->T = height * width * in_ch; m->act = ORC_ACT_RELU; m->prec = prec;
    m->n_lut = n_lut;
    m->lut = (float *)malloc(sizeof(float) * (size_t)n_lut);
    for (int i = 0; i < n_lut; ++i)
        m->lut[i] = prec == ORC_PREC_BF16 ? round_bf16(lut[i]) : lut[i];
    for (int l = 0; l < n_conv; ++l) {
        int cin = l == 0 ? in_ch : ch;
        size_t nw = (size_t)ch * 9 * cin;
        m->Wc[l] = (float *)malloc(sizeof(float) * nw);
        m->bc[l] = (float *)malloc(sizeof(float) * (size_t)ch);
        for (int co = 0; co < ch; ++co) {
            int go = conv_group(m, co);
            for (int ky = 0; ky < 3; ++ky)
                for (int kx = 0; kx < 3; ++kx)
                    for (int ci = 0; ci < cin; ++ci) {
                        int gi = l == 0 ? ci : conv_group(m, ci);
                        int keep;
                        if (ky == 0) keep = 1;
                        else if (ky == 1 && kx == 0) keep = 1;
                        else if (ky == 1 && kx == 1) keep = l == 0 ? (gi < go) : (gi <= go);
                        else keep = 0;
                        size_t idx = (((size_t)co * 3 + ky) * 3 + kx) * cin + ci;
                        float w = keep ? W[l][idx] : 0.0f;
                        m->Wc[l][idx] = prec == ORC_PREC_BF16 ? round_bf16(w) : w;
                    }
            m->bc[l][co] = b[l][co];
        }
    }
    int nout = in_ch * C;
    m->Wc[n_conv] = (float *)malloc(sizeof(float) * (size_t)nout * ch);
    m->bc[n_conv] = (float *)malloc(sizeof(float) * (size_t)nout);
    for (int o = 0; o < nout; ++o) {
        int go = o / C;
        for (int ci = 0; ci < ch; ++ci) {
            float w = conv_group(m, ci) <= go ? W[n_conv][(size_t)o * ch + ci] : 0.0f;
            m->Wc[n_conv][(size_t)o * ch + ci] = prec == ORC_PREC_BF16 ? round_bf16(w) : w;
        }
        m->bc[n_conv][o] = b[n_conv][o];
    }
    return m;
}

/* pre-activation of channel co of conv layer l at pixel (py, px); below: [height][width][cin] */
static double conv_unit(const orc_model *m, int l, int py, int px, int co, const float *below)
{
    int cin = l == 0 ? m->in_ch : m->ch;
    double acc = 0.0;
    for (int ky = 0; ky < 3; ++ky)
        for (int kx = 0; kx < 3; ++kx) {
            int yy = py + ky - 1, xx = px + kx - 1;
            if (yy < 0 || yy >= m->height || xx < 0 || xx >= m->width) continue;  /* zero padding */
            const float *w = m->Wc[l] + (((size_t)co * 3 + ky) * 3 + kx) * cin;
            const float *in = below + ((size_t)yy * m->width + xx) * cin;
            for (int ci = 0; ci < cin; ++ci) acc += (double)w[ci] * (double)in[ci];
        }
    return acc + (double)m->bc[l][co];
}

static double head_unit(const orc_model *m, int pix, int o, const float *top)
{
    const float *w = m->Wc[m->n_conv] + (size_t)o * m->ch;
    const float *in = top + (size_t)pix * m->ch;
    double acc = 0.0;
    for (int ci = 0; ci < m->ch; ++ci) acc += (double)w[ci] * (double)in[ci];
    return acc + (double)m->bc[m->n_conv][o];
}

typedef struct { float *a[ORC_MAX_LAYERS + 1]; } conv_ws;

static void conv_ws_alloc(const orc_model *m, conv_ws *ws)
{
    size_t npix = (size_t)m->height * m->width;
    ws->a[0] = (float *)calloc(npix * m->in_ch, sizeof(float));
    for (int l = 1; l <= m->n_conv; ++l) ws->a[l] = (float *)calloc(npix * m->ch, sizeof(float));
}
static void conv_ws_free(const orc_model *m, conv_ws *ws)
{
    for (int l = 0; l <= m->n_conv; ++l) free(ws->a[l]);
}

static void conv_forward(const orc_model *m, const uint8_t *x, float *z)
{
    conv_ws ws; conv_ws_alloc(m, &ws);
    int npix = m->height * m->width;
    for (int t = 0; t < m->T; ++t) ws.a[0][t] = m->lut[x[t]];
    for (int l = 0; l < m->n_conv; ++l)
        for (int p = 0; p < npix; ++p)
            for (int co = 0; co < m->ch; ++co)
                ws.a[l + 1][(size_t)p * m->ch + co] =
                    hidden_value(m->act, m->prec, conv_unit(m, l, p / m->width, p % m->width, co, ws.a[l]));
    for (int p = 0; p < npix; ++p)
        for (int o = 0; o < m->in_ch * m->C; ++o)
            z[(size_t)p * m->in_ch * m->C + o] = (float)head_unit(m, p, o, ws.a[m->n_conv]);
    conv_ws_free(m, &ws);
}

/* Sequential sweep over positions a..b-1; see made_sweep.  A hidden unit of
 * group g at pixel p becomes computable once positions < p*in_ch + g are known. */
static void conv_sweep(const orc_model *m, uint8_t *y, int a, int b, const float *noise, int nk)
{
    conv_ws ws; conv_ws_alloc(m, &ws);
    size_t ns = noise_stride(m, nk);
    int npix = m->height * m->width;
    float *zt = (float *)malloc(sizeof(float) * (size_t)m->C);
    for (int t = 0; t < m->T; ++t) ws.a[0][t] = m->lut[y[t]];
    for (int l = 0; l < m->n_conv; ++l)
        for (int p = 0; p < npix; ++p)
            for (int co = 0; co < m->ch; ++co)
                if (p * m->in_ch + conv_group(m, co) <= a)
                    ws.a[l + 1][(size_t)p * m->ch + co] =
                        hidden_value(m->act, m->prec, conv_unit(m, l, p / m->width, p % m->width, co, ws.a[l]));
    for (int t = a; t < b; ++t) {
        int p = t / m->in_ch, c = t % m->in_ch;
        if (t > a)
            for (int l = 0; l < m->n_conv; ++l)
                for (int co = 0; co < m->ch; ++co)
                    if (conv_group(m, co) == c)
                        ws.a[l + 1][(size_t)p * m->ch + co] =
                            hidden_value(m->act, m->prec, conv_unit(m, l, p / m->width, p % m->width, co, ws.a[l]));
        for (int k = 0; k < m->C; ++k) zt[k] = (float)head_unit(m, p, c * m->C + k, ws.a[m->n_conv]);
        y[t] = (uint8_t)sample_position(m->C, zt, noise + (size_t)t * ns, nk);
        ws.a[0][t] = m->lut[y[t]];
    }
    free(zt);
    conv_ws_free(m, &ws);
}

/* ------------------------------------------------------ model dispatchers */

/* logits of every position for the iterate x: z[T*C] */
void orc_forward_logits(const orc_model *m, const uint8_t *x, float *z)
{
    if (m->kind == ORC_KIND_MADE) made_forward(m, x, z); else conv_forward(m, x, z);
}

static void sweep(const orc_model *m, uint8_t *y, int a, int b, const float *noise, int nk)
{
    if (m->kind == ORC_KIND_MADE) made_sweep(m, y, a, b, noise, nk); else conv_sweep(m, y, a, b, noise, nk);
}

/* one parallel update of all positions: x_out[t] = h_t(u, x_in[0..t-1]) for every t
 * (the inner parallel loop of Algorithm 1) */
void orc_jacobi_step(const orc_model *m, const uint8_t *x_in, const float *noise, int nk, uint8_t *x_out)
{
    size_t ns = noise_stride(m, nk);
    float *z = (float *)malloc(sizeof(float) * (size_t)m->T * m->C);
    orc_forward_logits(m, x_in, z);
    for (int t = 0; t < m->T; ++t)
        x_out[t] = (uint8_t)sample_position(m->C, z + (size_t)t * m->C, noise + (size_t)t * ns, nk);
    free(z);
}

/* tie distance of every position's decision, teacher-forced on x */
void orc_margins(const orc_model *m, const uint8_t *x, const float *noise, int nk, float *margin)
{
    size_t ns = noise_stride(m, nk);
    float *z = (float *)malloc(sizeof(float) * (size_t)m->T * m->C);
    orc_forward_logits(m, x, z);
    for (int t = 0; t < m->T; ++t)
        margin[t] = decision_margin(m->C, z + (size_t)t * m->C, noise + (size_t)t * ns, nk);
    free(z);
}

/* ----------------------------------------------------------------- solvers
 * All solvers work on ONE sample: noise is [T] (or [T][C] for GUMBEL), x is
 * uint8 [T].  States are integers, so the stopping tolerance epsilon is 0 and
 * the forward difference test is exact equality.
 */

/* Feedforward computation in the plainest form (Eq. 1): for each t a complete
 * forward pass on the current x, of which only position t is kept. */
void orc_sequential_literal(const orc_model *m, const float *noise, int nk, uint8_t *x)
{
    size_t ns = noise_stride(m, nk);
    float *z = (float *)malloc(sizeof(float) * (size_t)m->T * m->C);
    memset(x, 0, (size_t)m->T);
    for (int t = 0; t < m->T; ++t) {
        orc_forward_logits(m, x, z);
        x[t] = (uint8_t)sample_position(m->C, z + (size_t)t * m->C, noise + (size_t)t * ns, nk);
    }
    free(z);
}

/* The same feedforward pass with every hidden unit evaluated once. */
void orc_sequential(const orc_model *m, const float *noise, int nk, uint8_t *x)
{
    memset(x, 0, (size_t)m->T);
    sweep(m, x, 0, m->T, noise, nk);
}

/* One Gauss-Seidel iteration on the triangular system (Eq. 4 applied to Eq. 5):
 * position t is solved with the new values of positions < t, which for a
 * triangular system is the feedforward pass whatever the starting point. */
void orc_gauss_seidel(const orc_model *m, const float *noise, int nk, const uint8_t *init, uint8_t *x)
{
    if (init) memcpy(x, init, (size_t)m->T); else memset(x, 0, (size_t)m->T);
    sweep(m, x, 0, m->T, noise, nk);
}

/*
 * Algorithm 1.  x^0 = init (zeros if NULL); repeat k <- k+1, x^k = G(x^{k-1})
 * until k == cap or x^k == x^{k-1}, where cap = T, lowered to max_iters when
 * 0 < max_iters < T.  Returns the final k in *iters.  *converged is 1 when the
 * forward difference vanished or k reached T (Proposition 1 then guarantees
 * the exact result).  If x_star is given, *k_correct is the first k with
 * x^k == x_star (0 if the start already equals it, -1 if never reached).
 */
void orc_jacobi(const orc_model *m, const float *noise, int nk, const uint8_t *init, int max_iters,
                uint8_t *x, int *iters, int *converged, const uint8_t *x_star, int *k_correct)
{
    int T = m->T;
    int cap = (max_iters > 0 && max_iters < T) ? max_iters : T;
    uint8_t *prev = (uint8_t *)malloc((size_t)T);
    if (init) memcpy(x, init, (size_t)T); else memset(x, 0, (size_t)T);
    int kc = -1;
    if (x_star && memcmp(x, x_star, (size_t)T) == 0) kc = 0;
    int k = 0, same = 0;
    do {
        k += 1;
        memcpy(prev, x, (size_t)T);
        orc_jacobi_step(m, prev, noise, nk, x);
        same = memcmp(prev, x, (size_t)T) == 0;
        if (x_star && kc < 0 && memcmp(x, x_star, (size_t)T) == 0) kc = k;
    } while (k < cap && !same);
    if (iters) *iters = k;
    if (converged) *converged = (same || k == T) ? 1 : 0;
    if (k_correct) *k_correct = kc;
    free(prev);
}

/*
 * Algorithm 3 (GS-Jacobi).  Blocks of `block` consecutive positions (the last
 * one shorter if block does not divide T) are taken in order; inside block
 * [a, b) Jacobi iterations update only the block's positions, reading the
 * finished positions < a and the block's previous iterate, until k == |B_i|
 * (lowered to max_iters if 0 < max_iters < |B_i|) or the block stops changing.
 * The block's start values come from init.  *iters = sum of inner iterations.
 */
void orc_gs_jacobi(const orc_model *m, const float *noise, int nk, const uint8_t *init, int block,
                   int max_iters, uint8_t *x, int *iters, int *converged)
{
    int T = m->T;
    uint8_t *next = (uint8_t *)malloc((size_t)T);
    if (init) memcpy(x, init, (size_t)T); else memset(x, 0, (size_t)T);
    int total = 0, conv_all = 1;
    for (int a = 0; a < T; a += block) {
        int b = a + block < T ? a + block : T;
        int len = b - a;
        int cap = (max_iters > 0 && max_iters < len) ? max_iters : len;
        int k = 0, same = 0;
        do {
            k += 1;
            orc_jacobi_step(m, x, noise, nk, next);
            same = memcmp(next + a, x + a, (size_t)len) == 0;
            memcpy(x + a, next + a, (size_t)len);       /* only the block is updated */
        } while (k < cap && !same);
        total += k;
        if (!(same || k == len)) conv_all = 0;
    }
    if (iters) *iters = total;
    if (converged) *converged = conv_all;
    free(next);
}

/*
 * Algorithm 2 (Jacobi-GS).  Every outer iteration updates all blocks from the
 * previous outer iterate: block [a, b) is swept sequentially, position j
 * reading x^{k-1} for positions < a and the freshly computed x^k for a..j-1.
 * Stops at k == M (number of blocks; lowered to max_iters if 0 < max_iters < M)
 * or when the whole iterate is unchanged.  *iters = outer iterations.
 */
void orc_jacobi_gs(const orc_model *m, const float *noise, int nk, const uint8_t *init, int block,
                   int max_iters, uint8_t *x, int *iters, int *converged)
{
    int T = m->T;
    int M = (T + block - 1) / block;
    int cap = (max_iters > 0 && max_iters < M) ? max_iters : M;
    uint8_t *prev = (uint8_t *)malloc((size_t)T);
    uint8_t *y = (uint8_t *)malloc((size_t)T);
    if (init) memcpy(x, init, (size_t)T); else memset(x, 0, (size_t)T);
    int k = 0, same = 0;
    do {
        k += 1;
        memcpy(prev, x, (size_t)T);
        for (int a = 0; a < T; a += block) {
            int b = a + block < T ? a + block : T;
            memcpy(y, prev, (size_t)T);
            sweep(m, y, a, b, noise, nk);
            memcpy(x + a, y + a, (size_t)(b - a));
        }
        same = memcmp(prev, x, (size_t)T) == 0;
    } while (k < cap && !same);
    if (iters) *iters = k;
    if (converged) *converged = (same || k == M) ? 1 : 0;
    free(prev); free(y);
}

/* Algorithm 2 with each position obtained from a complete forward pass on the
 * mixed iterate (x^{k-1} before the block, x^k inside it): small cases only. */
void orc_jacobi_gs_literal(const orc_model *m, const float *noise, int nk, const uint8_t *init, int block,
                           int max_iters, uint8_t *x, int *iters, int *converged)
{
    int T = m->T;
    int M = (T + block - 1) / block;
    int cap = (max_iters > 0 && max_iters < M) ? max_iters : M;
    size_t ns = noise_stride(m, nk);
    uint8_t *prev = (uint8_t *)malloc((size_t)T);
    uint8_t *y = (uint8_t *)malloc((size_t)T);
    float *z = (float *)malloc(sizeof(float) * (size_t)T * m->C);
    if (init) memcpy(x, init, (size_t)T); else memset(x, 0, (size_t)T);
    int k = 0, same = 0;
    do {
        k += 1;
        memcpy(prev, x, (size_t)T);
        for (int a = 0; a < T; a += block) {
            int b = a + block < T ? a + block : T;
            memcpy(y, prev, (size_t)T);
            for (int j = a; j < b; ++j) {
                orc_forward_logits(m, y, z);
                y[j] = (uint8_t)sample_position(m->C, z + (size_t)j * m->C, noise + (size_t)j * ns, nk);
            }
            memcpy(x + a, y + a, (size_t)(b - a));
        }
        same = memcmp(prev, x, (size_t)T) == 0;
    } while (k < cap && !same);
    if (iters) *iters = k;
    if (converged) *converged = (same || k == M) ? 1 : 0;
    free(prev); free(y); free(z);
}

/* ------------------------------------------------- continuous states (masked MLP)
 * The paper's MADE has logistic conditionals (Section 5.3.1, Appendix C.3): every state x_t is a real
 * number, the network reads the states themselves and gives position t two numbers, a location m_t
 * and a log-scale l_t, from x_{<t}; with the uniform number u_t reserved for the position (Appendix
 * A.3) the inverse CDF of the logistic law gives  x_t = m_t + exp(l_t) * logit(u_t).  The noise
 * passed in is logit(u_t) already (the same array as for binary positions with logistic noise).
 * C must be 2: logit 2t is m_t, logit 2t+1 is l_t.  In a bf16 model the inputs are rounded to bf16
 * like any activation.  States are floats; the update is evaluated in double and rounded once.
 */
static void made_forward_real(const orc_model *m, const float *x, float *z)
{
    made_ws ws; made_ws_alloc(m, &ws);
    for (int d = 0; d < m->T; ++d) ws.a[0][d] = m->prec == ORC_PREC_BF16 ? round_bf16(x[d]) : x[d];
    for (int l = 0; l < m->L; ++l)
        for (int i = 0; i < m->n[l + 1]; ++i)
            ws.a[l + 1][i] = hidden_value(m->act, m->prec, made_unit(m, l, i, ws.a[l]));
    for (int i = 0; i < m->n[m->L + 1]; ++i) z[i] = (float)made_unit(m, m->L, i, ws.a[m->L]);
    made_ws_free(m, &ws);
}

void orc_forward_logits_real(const orc_model *m, const float *x, float *z) { made_forward_real(m, x, z); }

static float real_state(const float *zt, float eps_t)
{
    return (float)((double)zt[0] + exp((double)zt[1]) * (double)eps_t);
}

/* one parallel update of all positions (inner loop of Algorithm 1) */
void orc_jacobi_step_real(const orc_model *m, const float *x_in, const float *noise, float *x_out)
{
    float *z = (float *)malloc(sizeof(float) * (size_t)m->T * 2);
    made_forward_real(m, x_in, z);
    for (int t = 0; t < m->T; ++t) x_out[t] = real_state(z + 2 * t, noise[t]);
    free(z);
}

/* Eq. 1 in the plainest form: for each t a complete forward pass on the current x, of which position t is kept */
void orc_sequential_real(const orc_model *m, const float *noise, float *x)
{
    float *z = (float *)malloc(sizeof(float) * (size_t)m->T * 2);
    for (int t = 0; t < m->T; ++t) x[t] = 0.0f;
    for (int t = 0; t < m->T; ++t) {
        made_forward_real(m, x, z);
        x[t] = real_state(z + 2 * t, noise[t]);
    }
    free(z);
}

/*
 * Algorithm 1 with the stopping rule of Section 2.2.1: x^0 = init (zeros if NULL); repeat k <- k+1,
 * x^k = G(x^{k-1}) until k == cap or max_t |x^k_t - x^{k-1}_t| <= eps (the paper leaves the norm open
 * and stops its image samplers on the largest deviation, Section 5.3.2: the maximum norm here).
 * cap = T, lowered to max_iters when 0 < max_iters < T.  *converged is 1 when the forward difference
 * test fired or k reached T (Proposition 1: exact then).
 */
void orc_jacobi_real(const orc_model *m, const float *noise, const float *init, float eps, int max_iters,
                     float *x, int *iters, int *converged)
{
    int T = m->T;
    int cap = (max_iters > 0 && max_iters < T) ? max_iters : T;
    float *prev = (float *)malloc(sizeof(float) * (size_t)T);
    for (int t = 0; t < T; ++t) x[t] = init ? init[t] : 0.0f;
    int k = 0, stop = 0;
    do {
        k += 1;
        memcpy(prev, x, sizeof(float) * (size_t)T);
        orc_jacobi_step_real(m, prev, noise, x);
        float dmax = 0.0f;
        for (int t = 0; t < T; ++t) {
            float d = fabsf(x[t] - prev[t]);
            if (!(d <= dmax)) dmax = d;                 /* a NaN difference counts as a change */
        }
        stop = dmax <= eps;
    } while (k < cap && !stop);
    if (iters) *iters = k;
    if (converged) *converged = (stop || k == T) ? 1 : 0;
    free(prev);
}

/* Algorithm 3 on continuous states: blocks in order, Jacobi inside block [a, b) until k == |B_i| or the
 * block's largest change is <= eps; the block starts from init.  *iters = sum of inner iterations. */
void orc_gs_jacobi_real(const orc_model *m, const float *noise, const float *init, int block, float eps,
                        int max_iters, float *x, int *iters, int *converged)
{
    int T = m->T;
    float *next = (float *)malloc(sizeof(float) * (size_t)T);
    for (int t = 0; t < T; ++t) x[t] = init ? init[t] : 0.0f;
    int total = 0, conv_all = 1;
    for (int a = 0; a < T; a += block) {
        int b = a + block < T ? a + block : T;
        int len = b - a;
        int cap = (max_iters > 0 && max_iters < len) ? max_iters : len;
        int k = 0, stop = 0;
        do {
            k += 1;
            orc_jacobi_step_real(m, x, noise, next);
            float dmax = 0.0f;
            for (int t = a; t < b; ++t) {
                float d = fabsf(next[t] - x[t]);
                if (!(d <= dmax)) dmax = d;
            }
            stop = dmax <= eps;
            memcpy(x + a, next + a, sizeof(float) * (size_t)len);
        } while (k < cap && !stop);
        total += k;
        if (!(stop || k == len)) conv_all = 0;
    }
    if (iters) *iters = total;
    if (converged) *converged = conv_all;
    free(next);
}
