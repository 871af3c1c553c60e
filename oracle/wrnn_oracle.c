/*
 * WaveRNN sampling-step ORACLE  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, CPU-only restatement of the WaveRNN sampling step of
 * "Efficient Neural Audio Synthesis" (Eq. 2, the masked-input paragraph
 * after it, and the evaluation order given in the caption of Fig. 1).
 * Scalar loops, dense matrices (a sparse model is a dense one whose pruned
 * 4x4 blocks are zero, Section 3.2), every sum accumulated in double in
 * index order, no blocking and no reordering.  It shares no code with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.
 *
 * Conventions the paper leaves open (each is a stated reading, not a fact
 * of the paper, so parity for it is "unpinned" outside this file):
 *   - biases exist ("omitted for brevity", Section 2): one per gate row,
 *     added outside the r o (R_e h) product, one per output-layer row;
 *   - the conditioning vector enters additively on all 3H gate
 *     pre-activations (the paper only says generation "is conditioned");
 *   - scaling of an 8-bit value v to [-1,1] is v/127.5 - 1 (0 -> -1, 255 -> +1);
 *   - initial state h = 0 and previous sample (c,f) = (128,0);
 *   - 16-bit sample = 256*c + f (coarse = high 8 bits, fine = low 8 bits,
 *     Fig. 1 caption), emitted as int16 by subtracting 32768;
 *   - sampling is temperature 1 inverse-CDF with strict '>' and the
 *     smallest qualifying index.
 *
 * Row order of every 3H-row object: u rows [0,H), r rows [H,2H), e rows
 * [2H,3H) (the order of Eq. 2); inside each gate the first H/2 rows are the
 * coarse half, the last H/2 the fine half ("split", Eq. 2).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 * as easy as 1, 2, 3", SC'11): counter-based generator, 10 rounds.     */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {            /* key schedule: bumped between rounds */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The uniform of (seed, stream, step, head): counter = (step low word, head,
 * stream, step high word), key = (seed low word, seed high word); the top
 * 24 bits of output word 0 scaled by 2^-24, so u is in [0,1).           */
double orc_uniform(uint64_t seed, uint32_t stream, uint64_t step, uint32_t head)
{
    uint32_t ctr[4] = { (uint32_t)(step & 0xFFFFFFFFu), head, stream, (uint32_t)(step >> 32) };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return (double)(out[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------ */
/* bf16 storage: keep the top 16 bits of the fp32 pattern, rounding to
 * nearest, ties to even.  Returned as the fp32 value of that bf16.     */

float orc_bf16_round_scalar(float v)
{
    uint32_t bits;
    memcpy(&bits, &v, 4);
    if ((bits & 0x7F800000u) == 0x7F800000u) {      /* Inf / NaN: truncate, keep NaN a NaN */
        if (bits & 0x007FFFFFu) bits |= 0x00400000u;
        bits &= 0xFFFF0000u;
    } else {
        uint32_t dropped = bits & 0xFFFFu;
        uint32_t kept_lsb = (bits >> 16) & 1u;
        bits &= 0xFFFF0000u;
        if (dropped > 0x8000u || (dropped == 0x8000u && kept_lsb)) bits += 0x10000u;
    }
    float r;
    memcpy(&r, &bits, 4);
    return r;
}

void orc_bf16_round(const float *in, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_bf16_round_scalar(in[i]);
}

/* Zero every br x bc block of W[rows][cols] whose mask entry is 0 (mask is [rows/br][cols/bc]; Section 3.2:
 * non-overlapping blocks pruned or kept together, 4 x 4 or m x 1 -- m rows, one column -- with m = 16;
 * 1 x 1 is the unstructured case). */
void orc_apply_block_mask_shape(float *W, int rows, int cols, const uint8_t *mask, int br, int bc)
{
    int nbc = cols / bc;
    for (int r = 0; r < rows; ++r)
        for (int c = 0; c < cols; ++c)
            if (!mask[(r / br) * nbc + (c / bc)]) W[(int64_t)r * cols + c] = 0.0f;
}

/* The 4 x 4 case. */
void orc_apply_block_mask(float *W, int rows, int cols, const uint8_t *mask)
{
    orc_apply_block_mask_shape(W, rows, cols, mask, 4, 4);
}

/* ------------------------------------------------------------------ */
/* Coarse / fine split of a 16-bit sample (Fig. 1 caption) and the int16 map. */

void orc_split16(uint16_t x, uint8_t *c, uint8_t *f) { *c = (uint8_t)(x >> 8); *f = (uint8_t)(x & 255u); }
uint16_t orc_join16(uint8_t c, uint8_t f) { return (uint16_t)(256u * c + f); }
int16_t orc_to_int16(uint8_t c, uint8_t f) { return (int16_t)((int32_t)(256 * c + f) - 32768); }

/* 8-bit value scaled to [-1,1] (paragraph after Eq. 2). */
double orc_scale8(int v) { return (double)v / 127.5 - 1.0; }

/* ------------------------------------------------------------------ */
/* Subscale fold / unfold (Section 4, Eq. 4): sub-tensor s holds u_{B i + s}. */

void orc_fold(const int16_t *x, int64_t n_total, int B, int16_t *sub)
{
    int64_t len = n_total / B;
    for (int s = 0; s < B; ++s)
        for (int64_t i = 0; i < len; ++i) sub[(int64_t)s * len + i] = x[(int64_t)B * i + s];
}

void orc_unfold(const int16_t *sub, int64_t n_total, int B, int16_t *x)
{
    int64_t len = n_total / B;
    for (int s = 0; s < B; ++s)
        for (int64_t i = 0; i < len; ++i) x[(int64_t)B * i + s] = sub[(int64_t)s * len + i];
}

/* ------------------------------------------------------------------ */
/* softmax + inverse-CDF draw over 256 logits (Eq. 2 softmax; "c_t is
 * sampled from P(c_t)", Fig. 1 caption).  probs (may be NULL) receives the
 * softmax; *margin (may be NULL) the distance from u to the nearest
 * normalised CDF boundary.                                             */

int orc_softmax_sample(const float *logits, int n, double u, double *probs, double *margin)
{
    double m = logits[0];
    for (int k = 1; k < n; ++k) if (logits[k] > m) m = logits[k];
    double *w = (double *)malloc(sizeof(double) * (size_t)n);
    double S = 0.0;
    for (int k = 0; k < n; ++k) { w[k] = exp((double)logits[k] - m); S += w[k]; }
    int pick = -1;
    double A = 0.0, best = 1e300;
    for (int k = 0; k < n; ++k) {
        A += w[k];
        if (pick < 0 && A > u * S) pick = k;
        double d = fabs(u - A / S);
        if (k < n - 1 && d < best) best = d;    /* the last boundary (=1) is never crossed */
        if (probs) probs[k] = w[k] / S;
    }
    if (pick < 0) pick = n - 1;
    if (margin) *margin = best;
    free(w);
    return pick;
}

/* ------------------------------------------------------------------ */

typedef struct {
    int32_t H;            /* state size, even                                     */
    int32_t cond_dim;     /* 0 = no conditioning                                  */
    const float *R;       /* [3H][H]                                              */
    const float *I;       /* [3H][3]  columns (c_{t-1}, f_{t-1}, c_t)             */
    const float *b_gate;  /* [3H] or NULL                                         */
    const float *W_cond;  /* [3H][cond_dim] or NULL                               */
    const float *O1, *b1; /* [H/2][H/2], [H/2]                                    */
    const float *O2, *b2; /* [256][H/2], [256]                                    */
    const float *O3, *b3, *O4, *b4;
} orc_params;

static double sigmoid_d(double x) { return 1.0 / (1.0 + exp(-x)); }

/* One stream row, n_steps steps.  Everything indexed relative to this row. */
static void run_row(const orc_params *p, const float *cond_row, int n_frames, int hop,
                    int row_stride, int row_offset, int64_t n_steps, int64_t step0,
                    uint64_t seed, uint32_t stream, float *h /*[H] in/out*/,
                    uint8_t *c_prev, uint8_t *f_prev,
                    const uint8_t *c_forced, const uint8_t *f_forced,
                    int16_t *out, uint8_t *c_out, uint8_t *f_out, double *margins /*[n_steps][2]*/,
                    float *dbg_gates, int64_t gates_stride, float *dbg_h, int64_t h_stride,
                    float *dbg_logits, int64_t logits_stride, int *err)
{
    const int H = p->H, Hh = H / 2, G = 3 * H, D = p->cond_dim;
    double *a = (double *)malloc(sizeof(double) * (size_t)G);
    double *g = (double *)malloc(sizeof(double) * (size_t)G);
    double *gate = (double *)malloc(sizeof(double) * (size_t)G);
    float *hn = (float *)malloc(sizeof(float) * (size_t)H);
    double *q = (double *)malloc(sizeof(double) * (size_t)Hh);
    float logit[256];
    int64_t g_frame = -1;
    int cp = *c_prev, fp = *f_prev;

    for (int64_t s = 0; s < n_steps; ++s) {
        const int64_t t = step0 + s;
        /* conditioning: held frame, projected, plus the gate bias */
        int64_t k = (D > 0) ? (t * row_stride + row_offset) / hop : 0;
        if (D > 0 && (k < 0 || k >= n_frames)) { *err = 1; break; }
        if (k != g_frame) {
            for (int row = 0; row < G; ++row) {
                double acc = p->b_gate ? (double)p->b_gate[row] : 0.0;
                for (int d = 0; d < D; ++d)
                    acc += (double)p->W_cond[(int64_t)row * D + d] * (double)cond_row[k * D + d];
                g[row] = acc;
            }
            g_frame = k;
        }
        const double x0 = orc_scale8(cp), x1 = orc_scale8(fp);

        /* a = R h_{t-1}: the single matrix-vector product for all three gates */
        for (int row = 0; row < G; ++row) {
            double acc = 0.0;
            const float *Rr = p->R + (int64_t)row * H;
            for (int j = 0; j < H; ++j) acc += (double)Rr[j] * (double)h[j];
            a[row] = acc;
        }

        int c_t = 0, f_t = 0;
        for (int half = 0; half < 2; ++half) {
            const int j0 = half ? Hh : 0, j1 = half ? H : Hh;
            /* c_t reaches only the fine half of u, r, e (masked matrix I*) */
            const double x2 = half ? orc_scale8(c_t) : 0.0;
            for (int j = j0; j < j1; ++j) {
                const float *Iu = p->I + (int64_t)j * 3;
                const float *Ir = p->I + (int64_t)(H + j) * 3;
                const float *Ie = p->I + (int64_t)(2 * H + j) * 3;
                double pu = a[j] + Iu[0] * x0 + Iu[1] * x1 + g[j];
                double pr = a[H + j] + Ir[0] * x0 + Ir[1] * x1 + g[H + j];
                double pe_in = Ie[0] * x0 + Ie[1] * x1 + g[2 * H + j];
                if (half) { pu += Iu[2] * x2; pr += Ir[2] * x2; pe_in += Ie[2] * x2; }
                double u = sigmoid_d(pu);
                double r = sigmoid_d(pr);
                double e = tanh(r * a[2 * H + j] + pe_in);
                gate[j] = u; gate[H + j] = r; gate[2 * H + j] = e;
                hn[j] = (float)(u * (double)h[j] + (1.0 - u) * e);   /* fp32 state */
            }
            /* output head on this half of the new state */
            const float *Oa = half ? p->O3 : p->O1, *ba = half ? p->b3 : p->b1;
            const float *Ob = half ? p->O4 : p->O2, *bb = half ? p->b4 : p->b2;
            for (int i = 0; i < Hh; ++i) {
                double acc = ba ? (double)ba[i] : 0.0;
                for (int j = 0; j < Hh; ++j) acc += (double)Oa[(int64_t)i * Hh + j] * (double)hn[j0 + j];
                q[i] = acc > 0.0 ? acc : 0.0;
            }
            for (int i = 0; i < 256; ++i) {
                double acc = bb ? (double)bb[i] : 0.0;
                for (int j = 0; j < Hh; ++j) acc += (double)Ob[(int64_t)i * Hh + j] * q[j];
                logit[i] = (float)acc;
            }
            double uu = orc_uniform(seed, stream, (uint64_t)t, (uint32_t)half);
            double margin;
            int idx = orc_softmax_sample(logit, 256, uu, NULL, &margin);
            if (margins) margins[2 * s + half] = margin;
            if (dbg_logits) memcpy(dbg_logits + s * logits_stride + half * 256, logit, sizeof(logit));
            if (half == 0) {
                if (c_out) c_out[s] = (uint8_t)idx;
                c_t = c_forced ? c_forced[s] : idx;
            } else {
                if (f_out) f_out[s] = (uint8_t)idx;
                f_t = f_forced ? f_forced[s] : idx;
            }
        }
        if (dbg_gates) for (int row = 0; row < G; ++row) dbg_gates[s * gates_stride + row] = (float)gate[row];
        if (dbg_h) memcpy(dbg_h + s * h_stride, hn, sizeof(float) * (size_t)H);
        memcpy(h, hn, sizeof(float) * (size_t)H);
        if (out) out[s] = orc_to_int16((uint8_t)c_t, (uint8_t)f_t);
        cp = c_t; fp = f_t;
    }
    *c_prev = (uint8_t)cp; *f_prev = (uint8_t)fp;
    free(a); free(g); free(gate); free(hn); free(q);
}

/*
 * Advance `batch` independent stream rows by n_steps.  Row b has the global
 * row id gb = stream0 + b: it uses Philox stream id gb, conditioning frames
 * cond[b][n_frames][cond_dim] and frame index
 * ((step0+s)*row_stride + gb*row_offset_mul) div hop.  With
 * c_forced/f_forced non-NULL ([batch][n_steps]) the drawn indices are only
 * recorded (c_out/f_out) and the forced values are fed back instead.
 * Optional dumps: dbg_gates [n_steps][batch][3H] (post-activation u|r|e),
 * dbg_h [n_steps][batch][H], dbg_logits [n_steps][batch][2][256],
 * margins [batch][n_steps][2].  Rows are independent (Section 4: shared
 * weights, separate streams), so they may be spread over `threads` threads;
 * the arithmetic of a row does not depend on that.  Returns 0, or 1 when a
 * frame index fell outside [0,n_frames).
 */
int orc_run(const orc_params *p, const float *cond, int n_frames, int hop,
            int row_stride, int row_offset_mul, int64_t n_steps, int batch, int64_t step0,
            uint64_t seed, uint32_t stream0, float *h /*[batch][H]*/, uint8_t *c_prev, uint8_t *f_prev,
            const uint8_t *c_forced, const uint8_t *f_forced,
            int16_t *out /*[batch][n_steps]*/, uint8_t *c_out, uint8_t *f_out, double *margins,
            float *dbg_gates, float *dbg_h, float *dbg_logits, int threads)
{
    const int H = p->H, G = 3 * H, D = p->cond_dim;
    int err_any = 0;
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        int err = 0;
        run_row(p, cond ? cond + (int64_t)b * n_frames * D : NULL, n_frames, hop,
                row_stride, (int)(stream0 + (uint32_t)b) * row_offset_mul, n_steps, step0, seed,
                stream0 + (uint32_t)b,
                h + (int64_t)b * H, c_prev + b, f_prev + b,
                c_forced ? c_forced + (int64_t)b * n_steps : NULL,
                f_forced ? f_forced + (int64_t)b * n_steps : NULL,
                out ? out + (int64_t)b * n_steps : NULL,
                c_out ? c_out + (int64_t)b * n_steps : NULL,
                f_out ? f_out + (int64_t)b * n_steps : NULL,
                margins ? margins + (int64_t)b * n_steps * 2 : NULL,
                dbg_gates ? dbg_gates + (int64_t)b * G : NULL, (int64_t)batch * G,
                dbg_h ? dbg_h + (int64_t)b * H : NULL, (int64_t)batch * H,
                dbg_logits ? dbg_logits + (int64_t)b * 512 : NULL, (int64_t)batch * 512, &err);
        if (err) {
#pragma omp atomic write
            err_any = 1;
        }
    }
    return err_any;
}

/* ====================================================================== */
/* Fused Subscale WaveRNN 2x (the paper's subsection of that name; batched
 * sampling and the lag between sub-tensors are in the subsection before it).
 *
 * What the paper fixes: a Subscale WaveRNN 2x whose two sub-tensors are not
 * batched but given one part each of the hidden state of a single WaveRNN;
 * 8 softmaxes of 4 bits; future horizon F = 2; the sub-tensors' samples are
 * the network's direct inputs, no conditioning network; 32 bits per step.
 * Everything else below is a stated reading (parity for it is unpinned
 * outside this file):
 *   - sub-tensor 0 holds a_i = u_{2i}, sub-tensor 1 holds b_i = u_{2i+1};
 *     step t emits a_t from part A of the state (units [0,H/2), the "coarse"
 *     half of Eq. 2) and then b_{t-2} from part B (units [H/2,H)): part B sees
 *     a_t inside the step exactly as the fine half sees c_t in Eq. 2, so b_j is
 *     conditioned on a_{<= j+2}: F = 2;
 *   - x_t = [nibbles of a_{t-1}, nibbles of the previous step's b, nibbles of
 *     a_t], most significant nibble first, a nibble v scaled to v/7.5 - 1;
 *     I* is [3H][12] and its last four columns reach only the rows of part B;
 *   - each part keeps the head of Eq. 2, softmax(O2 relu(O1 y)), with
 *     O2 of 64 rows: rows [16k, 16k+16) are the softmax of nibble k, and the four
 *     nibbles of a sample are drawn independently given the state;
 *   - sample = sum_k nibble_k << (12 - 4k), emitted as int16 minus 32768;
 *   - uniforms: the same counter generator with head = 4 * part + k;
 *   - before the first step a_{-1} = b = 0x8000 and h = 0.
 * Gate rows, biases, conditioning and the draw are as for the base model.    */

double orc_scale4(int v) { return (double)v / 7.5 - 1.0; }
void orc_split_nibbles(uint16_t x, uint8_t n[4]) { for (int k = 0; k < 4; ++k) n[k] = (uint8_t)((x >> (12 - 4 * k)) & 15u); }
uint16_t orc_join_nibbles(const uint8_t n[4]) { return (uint16_t)((n[0] << 12) | (n[1] << 8) | (n[2] << 4) | n[3]); }

/*
 * One stream, n_steps steps from step0.  p->I is [3H][12], p->O2 / p->O4 are
 * [64][H/2], p->b2 / p->b4 [64]; the other fields as for orc_run.  a_prev /
 * b_prev: the two samples emitted by the previous step (in / out).  With
 * a_forced / b_forced the drawn samples are only recorded and the forced
 * ones fed back.  out is [2][n_steps] (row 0: a_t, row 1: the b of step t);
 * margins [n_steps][8]; dbg_gates [n_steps][3H]; dbg_h [n_steps][H];
 * dbg_logits [n_steps][2][64].  Returns 0, or 1 when a frame index fell
 * outside [0, n_frames).
 */
int orc_fs2_run(const orc_params *p, const float *cond, int n_frames, int hop, int64_t n_steps, int64_t step0,
                uint64_t seed, uint32_t stream, float *h, uint16_t *a_prev, uint16_t *b_prev,
                const uint16_t *a_forced, const uint16_t *b_forced, uint16_t *a_out, uint16_t *b_out,
                int16_t *out, double *margins, float *dbg_gates, float *dbg_h, float *dbg_logits)
{
    const int H = p->H, Hh = H / 2, G = 3 * H, D = p->cond_dim;
    double *a = (double *)malloc(sizeof(double) * (size_t)G);
    double *g = (double *)malloc(sizeof(double) * (size_t)G);
    double *gate = (double *)malloc(sizeof(double) * (size_t)G);
    float *hn = (float *)malloc(sizeof(float) * (size_t)H);
    double *q = (double *)malloc(sizeof(double) * (size_t)Hh);
    float logit[64];
    int64_t g_frame = -1;
    int err = 0;
    uint16_t ap = *a_prev, bp = *b_prev;

    for (int64_t s = 0; s < n_steps && !err; ++s) {
        const int64_t t = step0 + s;
        int64_t k = (D > 0) ? t / hop : 0;
        if (D > 0 && (k < 0 || k >= n_frames)) { err = 1; break; }
        if (k != g_frame) {
            for (int row = 0; row < G; ++row) {
                double acc = p->b_gate ? (double)p->b_gate[row] : 0.0;
                for (int d = 0; d < D; ++d) acc += (double)p->W_cond[(int64_t)row * D + d] * (double)cond[k * D + d];
                g[row] = acc;
            }
            g_frame = k;
        }
        double x[12];
        uint8_t nb[4];
        orc_split_nibbles(ap, nb); for (int c = 0; c < 4; ++c) x[c] = orc_scale4(nb[c]);
        orc_split_nibbles(bp, nb); for (int c = 0; c < 4; ++c) x[4 + c] = orc_scale4(nb[c]);
        for (int c = 8; c < 12; ++c) x[c] = 0.0;

        for (int row = 0; row < G; ++row) {
            double acc = 0.0;
            const float *Rr = p->R + (int64_t)row * H;
            for (int j = 0; j < H; ++j) acc += (double)Rr[j] * (double)h[j];
            a[row] = acc;
        }

        uint16_t smp[2] = {0, 0};
        for (int part = 0; part < 2; ++part) {
            const int j0 = part ? Hh : 0, j1 = part ? H : Hh;
            const int ncol = part ? 12 : 8;             /* a_t reaches only part B (masked I*) */
            for (int j = j0; j < j1; ++j) {
                const float *Iu = p->I + (int64_t)j * 12;
                const float *Ir = p->I + (int64_t)(H + j) * 12;
                const float *Ie = p->I + (int64_t)(2 * H + j) * 12;
                double pu = a[j] + g[j], pr = a[H + j] + g[H + j], pe_in = g[2 * H + j];
                for (int c = 0; c < ncol; ++c) { pu += Iu[c] * x[c]; pr += Ir[c] * x[c]; pe_in += Ie[c] * x[c]; }
                double u = sigmoid_d(pu);
                double r = sigmoid_d(pr);
                double e = tanh(r * a[2 * H + j] + pe_in);
                gate[j] = u; gate[H + j] = r; gate[2 * H + j] = e;
                hn[j] = (float)(u * (double)h[j] + (1.0 - u) * e);
            }
            const float *Oa = part ? p->O3 : p->O1, *ba = part ? p->b3 : p->b1;
            const float *Ob = part ? p->O4 : p->O2, *bb = part ? p->b4 : p->b2;
            for (int i = 0; i < Hh; ++i) {
                double acc = ba ? (double)ba[i] : 0.0;
                for (int j = 0; j < Hh; ++j) acc += (double)Oa[(int64_t)i * Hh + j] * (double)hn[j0 + j];
                q[i] = acc > 0.0 ? acc : 0.0;
            }
            for (int i = 0; i < 64; ++i) {
                double acc = bb ? (double)bb[i] : 0.0;
                for (int j = 0; j < Hh; ++j) acc += (double)Ob[(int64_t)i * Hh + j] * q[j];
                logit[i] = (float)acc;
            }
            uint8_t drawn[4];
            for (int kk = 0; kk < 4; ++kk) {
                double uu = orc_uniform(seed, stream, (uint64_t)t, (uint32_t)(4 * part + kk));
                double margin;
                drawn[kk] = (uint8_t)orc_softmax_sample(logit + 16 * kk, 16, uu, NULL, &margin);
                if (margins) margins[8 * s + 4 * part + kk] = margin;
            }
            if (dbg_logits) memcpy(dbg_logits + s * 128 + part * 64, logit, sizeof(logit));
            const uint16_t v = orc_join_nibbles(drawn);
            if (part == 0) {
                if (a_out) a_out[s] = v;
                smp[0] = a_forced ? a_forced[s] : v;
                orc_split_nibbles(smp[0], nb);
                for (int c = 0; c < 4; ++c) x[8 + c] = orc_scale4(nb[c]);
            } else {
                if (b_out) b_out[s] = v;
                smp[1] = b_forced ? b_forced[s] : v;
            }
        }
        if (dbg_gates) for (int row = 0; row < G; ++row) dbg_gates[s * G + row] = (float)gate[row];
        if (dbg_h) memcpy(dbg_h + s * H, hn, sizeof(float) * (size_t)H);
        memcpy(h, hn, sizeof(float) * (size_t)H);
        if (out) { out[s] = (int16_t)((int32_t)smp[0] - 32768); out[n_steps + s] = (int16_t)((int32_t)smp[1] - 32768); }
        ap = smp[0]; bp = smp[1];
    }
    *a_prev = ap; *b_prev = bp;
    free(a); free(g); free(gate); free(hn); free(q);
    return err;
}

/* Interleave the two streams of orc_fs2_run into the original order: u_{2i} = a_i, u_{2i+1} = b_i, where b_i is the b
 * of step i + 2 (the first two b of a run are the lag's pre-roll and are dropped).  n = number of steps; u gets
 * 2 (n - 2) samples. */
void orc_fs2_unfold(const int16_t *ab /* [2][n] */, int64_t n, int16_t *u)
{
    for (int64_t i = 0; i + 2 < n; ++i) { u[2 * i] = ab[i]; u[2 * i + 1] = ab[n + i + 2]; }
}
