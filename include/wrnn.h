/*
 * wrnn.h -- C ABI of the B200 WaveRNN sampling library (libwrnn.so).
 *
 * One thing is computed here: the per-sample autoregressive sampling step of
 * the WaveRNN ("Efficient Neural Audio Synthesis", Section 2, Eq. 2):
 *
 *     x_t = [c_{t-1}, f_{t-1}, c_t]                      8-bit values scaled to [-1,1]
 *     u_t = sigmoid(R_u h_{t-1} + I*_u x_t + g_u)
 *     r_t = sigmoid(R_r h_{t-1} + I*_r x_t + g_r)
 *     e_t = tanh(r_t o (R_e h_{t-1}) + I*_e x_t + g_e)
 *     h_t = u_t o h_{t-1} + (1 - u_t) o e_t
 *     y_c, y_f = split(h_t)
 *     P(c_t) = softmax(O2 relu(O1 y_c + b1) + b2),  P(f_t) = softmax(O4 relu(O3 y_f + b3) + b4)
 *
 * evaluated in the order of Fig. 1: R h for both halves, coarse gates, draw c_t,
 * fine gates (I* lets c_t reach only the fine half), draw f_t; the 16-bit sample is
 * 256 c_t + f_t.  g = W_cond frame + b_gate is the per-step conditioning vector
 * (held for `hop` samples).  Dense (Section 2.1), 4x4 block-sparse (Section 3.2)
 * and batched / subscale-folded (Section 4) forms share these entry points; the Fused Subscale
 * WaveRNN 2x (Section 4.4, wrnn_fs2_*) and subscale generation with dependent rows on the staggered
 * schedule (Sections 4.1, 4.2, wrnn_sample_subscale_dependent) are built on the same step.
 *
 * Conventions: C linkage; every function returns a wrnn_status (0 = ok) unless
 * noted; pointers are marked HOST or DEVICE; the caller owns every buffer it
 * passes; nothing here takes or returns a C++ or torch type.  Argument errors are
 * reported synchronously and nothing is launched.  Work is enqueued on the given
 * CUDA stream (a cudaStream_t passed as void*, NULL = default stream) and is
 * asynchronous unless noted.  One call in flight per model.  There is no CPU path:
 * without a usable CUDA device every compute entry point returns WRNN_ERR_CUDA.
 *
 * Row order of every 3H-row object: u rows [0,H), r rows [H,2H), e rows [2H,3H);
 * inside each gate rows [0,H/2) belong to the coarse half, [H/2,H) to the fine half.
 */
#ifndef WRNN_H
#define WRNN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wrnn_model wrnn_model;   /* opaque; owns the device memory it allocates */

typedef enum {
    WRNN_OK = 0,
    WRNN_ERR_INVALID_ARG = 1,
    WRNN_ERR_UNSUPPORTED = 2,   /* shape / dtype / batch has no kernel, or it does not fit the device */
    WRNN_ERR_NOMEM = 3,
    WRNN_ERR_CUDA = 4,
    WRNN_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out; the kernel returned cleanly */
    WRNN_ERR_CHECK = 6          /* checked build (models created under WRNN_DEBUG=1): an index left its array or a guard  */
                                /* word behind a shared-memory region was overwritten; the access was skipped, the kernel */
                                /* returned cleanly; wrnn_last_error names the CTA and the region                         */
} wrnn_status;

typedef enum { WRNN_F32 = 0, WRNN_BF16 = 1 } wrnn_dtype;

/* Which kernel family wrnn_sample / wrnn_step_teacher_forced use. */
typedef enum {
    WRNN_KERNEL_AUTO = 0,       /* the fastest one that supports the model and batch          */
    WRNN_KERNEL_GENERIC = 1,    /* weights streamed from L2 every step; any shape; bring-up path */
    WRNN_KERNEL_RESIDENT = 2,   /* persistent kernel, weights resident in shared memory (one row; 2 to 16 rows of a dense bf16 H = 896 model) */
    WRNN_KERNEL_BATCHED = 3,    /* tensor-pipe contractions over all rows (dense bf16, >= 2 rows)  */
    WRNN_KERNEL_SPARSE = 4,     /* block-sparse model resident in 16-CTA clusters (one row)        */
    WRNN_KERNEL_BCLUSTER = 5    /* rows dealt to 16-CTA clusters, tcgen05 contractions (dense bf16, >= 2 rows) */
} wrnn_kernel;

/*
 * Model description for wrnn_create.  All pointers HOST, fp32, row-major, read
 * during the call only (the library keeps packed copies on the device).
 */
typedef struct {
    int32_t H;                  /* state size, a multiple of 8                                        */
    int32_t cond_dim;           /* length of a conditioning frame; 0 = unconditioned                  */
    const float *R;             /* [3H][H]   recurrent matrix, gates stacked u|r|e (Eq. 2)            */
    const float *I;             /* [3H][3]   input matrix, columns (c_{t-1}, f_{t-1}, c_t); column 2  */
                                /*           is ignored on coarse rows (the mask of I*, Section 2)    */
    const float *b_gate;        /* [3H] or NULL (= 0)                                                 */
    const float *W_cond;        /* [3H][cond_dim], NULL iff cond_dim == 0                             */
    const float *O1, *b1;       /* [H/2][H/2], [H/2]   coarse hidden layer (b* may be NULL = 0)       */
    const float *O2, *b2;       /* [256][H/2], [256]   coarse logits                                  */
    const float *O3, *b3;       /* fine hidden layer, same shapes                                     */
    const float *O4, *b4;       /* fine logits                                                        */
    const uint8_t *mask_R;      /* [3H/br][H/bc] 1 = block kept (Section 3.2), NULL = dense; br x bc  */
                                /* is the block shape given below (4 x 4 unless stated otherwise)     */
    const uint8_t *mask_O1;     /* [H/2/br][H/2/bc] or NULL                                           */
    const uint8_t *mask_O3;     /* [H/2/br][H/2/bc] or NULL                                           */
    int32_t dtype;              /* wrnn_dtype: storage type of R, I, W_cond, O1..O4 (bf16 = round to  */
                                /* nearest even at create); biases, state and all arithmetic are fp32 */
    int32_t kernel;             /* wrnn_kernel                                                        */
    int32_t mask_block_rows;    /* rows and columns of one block of the three masks (Section 3.2:     */
    int32_t mask_block_cols;    /* 4 x 4, or m x 1 = 16 rows of one column, or 1 x 1 = unstructured); */
                                /* 0, 0 means 4 x 4.  Both must divide H/2.  Every shape runs on the  */
                                /* generic kernel; 4 x 4 and 16 x 1 also on the sparse cluster kernel  */
    int32_t variant;            /* 0: WaveRNN (Eq. 2, shapes as above).  1: Fused Subscale WaveRNN 2x */
                                /* (Section 4.4): I is [3H][12] (nibbles of a_{t-1}, of the previous  */
                                /* b, of a_t; the last four columns are ignored on part-A rows),      */
                                /* O2 / O4 are [64][H/2] and b2 / b4 [64]: rows 16 k .. 16 k + 15 are  */
                                /* the softmax of nibble k.  Dense bf16, one stream, the resident     */
                                /* kernel only; stepped with the wrnn_fs2_* calls below               */
} wrnn_params;

/*
 * wrnn_create: validate, apply the block masks, round to the storage type, pack and
 * upload.  max_batch (>= 1) sizes the per-row exchange and state buffers.  Synchronous;
 * allocates device memory on the current device.  On failure *out is NULL.
 */
int wrnn_create(const wrnn_params *params, int32_t max_batch, wrnn_model **out);
void wrnn_destroy(wrnn_model *m);   /* NULL is allowed; synchronises the device */

/*
 * Carry state of `batch` stream rows.  DEVICE pointers, caller-owned, read at the
 * start and written at the end of a call; a NULL pointer means the default initial
 * value (h = 0; previous sample 0, i.e. c_prev = 128, f_prev = 0) and no write-back.
 * Row b has the global row id stream0 + b, which selects its Philox stream and its
 * conditioning offset; step0 is the absolute index of the first step of the call.
 * Generating T steps in one call equals generating T1 then T - T1 with the state
 * carried over and step0 advanced.
 */
typedef struct {
    float *h;            /* [batch][H] */
    uint8_t *c_prev;     /* [batch]    */
    uint8_t *f_prev;     /* [batch]    */
    int64_t step0;
    uint32_t stream0;
    uint32_t reserved;
} wrnn_state;

/*
 * Conditioning and step geometry shared by the two stepping calls.
 * Frame index of row b at step s of the call:
 *     ((step0 + s) * row_stride + (stream0 + b) * row_offset_mul) / hop      (integer division)
 * which must stay below n_frames.  (1, 0) is an ordinary stream; (B, 1) is row b of a
 * B-way subscale fold (Section 4.1: row b holds samples B i + b).
 */
typedef struct {
    const float *cond;   /* DEVICE [batch][n_frames][cond_dim] fp32; NULL iff cond_dim == 0 */
    int32_t n_frames;
    int32_t hop;         /* samples per frame, > 0 */
    int32_t row_stride;
    int32_t row_offset_mul;
} wrnn_cond;

/*
 * wrnn_sample: free-running generation (Fig. 1).  For every row and step draws
 * c_t then f_t with uniforms Philox4x32-10(key = seed; counter = (step lo, head,
 * global row id, step hi)), word 0 >> 8 scaled by 2^-24, head 0 = coarse, 1 = fine;
 * inverse CDF: smallest k whose running sum of exp(l - max l) exceeds u times the total.
 * out: DEVICE int16 [batch][n_steps], value 256 c + f - 32768.
 * st may be NULL (default state, step0 = 0, stream0 = 0).
 * May grow an internal scratch buffer (synchronously) when batch * n_frames exceeds
 * what earlier calls needed.
 */
int wrnn_sample(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch,
                uint64_t seed, const wrnn_state *st, int16_t *out, void *cuda_stream);

/*
 * wrnn_sample_noalloc: wrnn_sample for callers that must not allocate.  (The paper has no counterpart;
 * this exists for the way the library gets embedded.)  A real-time audio thread, a caller that is inside a
 * region where device allocation is forbidden or would synchronise the whole device, or one running under a
 * fixed memory budget creates its model ahead of time and then needs a sampling call that never reaches
 * cudaMalloc / cudaFree -- wrnn_sample may grow its conditioning scratch on a larger request.  This entry
 * point takes the same arguments and always runs the any-shape step kernel, so it produces exactly the samples of
 * wrnn_sample on a model created with WRNN_KERNEL_GENERIC (on other models wrnn_sample runs a specialised kernel
 * whose summation order may turn a draw that sits on a CDF boundary the other way), but every byte of per-call scratch -- projected conditioning, state and head exchange buffers, the barrier
 * counter -- lives in one fixed 8 MiB array inside the library's device image.  Each GPU that loads the
 * library carries that array until the process exits.
 *   - Sizes whose scratch does not fit (roughly batch * n_frames * 3H * 4 bytes plus batch * 5H * 4) are
 *     refused with WRNN_ERR_UNSUPPORTED and a message that states both numbers; nothing is launched.
 *   - The array's device address is looked up once per device, with that device current: by wrnn_create for the
 *     device the model lives on, otherwise by the first call of this entry point on a device; such a first call
 *     should come before any stream capture.
 *   - All calls, on all models and streams, share the one array and it keeps what the previous call left
 *     behind; the entry point re-zeroes what must start at zero, but two calls that overlap on the GPU race on
 *     it.  Serialise them (one stream, or events).
 * No cudaMalloc, cudaFree or allocating library routine is called.  Asynchronous on cuda_stream.
 */
int wrnn_sample_noalloc(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch,
                        uint64_t seed, const wrnn_state *st, int16_t *out, void *cuda_stream);

/*
 * wrnn_step_teacher_forced: the same steps, but the samples fed back are given.
 * Step s uses (c_forced, f_forced)[b][s-1] as the previous sample (the state's
 * c_prev / f_prev at s = 0) and c_forced[b][s] in the fine gates.  The indices the
 * device itself draws are written to c_out / f_out.  All DEVICE; forced arrays and
 * c_out / f_out are uint8 [batch][n_steps].  Optional dumps (NULL = off):
 *   dbg_gates  [n_steps][batch][3H]     post-activation u | r | e
 *   dbg_h      [n_steps][batch][H]      h_t
 *   dbg_logits [n_steps][batch][2][256] pre-softmax logits, coarse then fine
 */
int wrnn_step_teacher_forced(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch,
                             uint64_t seed, const wrnn_state *st,
                             const uint8_t *c_forced, const uint8_t *f_forced,
                             uint8_t *c_out, uint8_t *f_out,
                             float *dbg_gates, float *dbg_h, float *dbg_logits, void *cuda_stream);

/*
 * Subscale fold / unfold (Section 4.1, Eq. 4): sub-tensor s holds x[B i + s].
 * x: DEVICE int16 [n_total]; sub: DEVICE int16 [B][n_total / B]; B must divide n_total.
 */
int wrnn_fold(const int16_t *x, int64_t n_total, int32_t B, int16_t *sub, void *cuda_stream);
int wrnn_unfold(const int16_t *sub, int64_t n_total, int32_t B, int16_t *x, void *cuda_stream);

/*
 * wrnn_sample_subscale: generate one sequence of n_total samples as B interleaved
 * sub-sequences advanced in lock-step as a batch of B (Section 4.2), then unfold.
 * cond: [B][n_frames][cond_dim] (row s conditions sub-sequence s), geometry forced to
 * (row_stride, row_offset_mul) = (B, 1).  out: DEVICE int16 [n_total] in original order.
 */
int wrnn_sample_subscale(wrnn_model *m, const float *cond, int32_t n_frames, int32_t hop,
                         int64_t n_total, int32_t B, uint64_t seed, int16_t *out, void *cuda_stream);

/*
 * Subscale generation with dependent rows and the staggered schedule of batched sampling (Sections 4.1, 4.2): sub-tensor r
 * (samples u_{B i + r}) is conditioned on the sub-tensors z < r, on their positions up to F ahead of its own, and starts
 * `lag` steps after sub-tensor r - 1, so that after (B - 1) lag steps all B rows advance together through the shared
 * WaveRNN.  The conditioning network is computed `chunk` positions ahead at a time (the paper's L), hence lag >= F + chunk
 * (and a multiple of chunk, so that the rows' chunks line up).  The network here is one masked convolution (a stated
 * reading; the paper's has ten layers):
 *     v_r[i] = frames[r][(B i + r) div hop] + relu(bias + sum_{delta=1..r} sum_{d=0..F} V[delta-1][d] x(u_{r-delta}[i + d]))
 * with x(u) = u / 32768 and positions beyond the row length contributing nothing; row r is a WaveRNN stream with Philox
 * stream id r, step = position, conditioning vector v_r[i] at step i.  The result does not depend on chunk or lag.
 * frames: DEVICE [B][n_frames][cond_dim]; V: DEVICE [B-1][F+1][cond_dim]; bias: DEVICE [cond_dim]; out: DEVICE int16
 * [n_total] in the original order.  B <= max_batch given at create.  Asynchronous on cuda_stream.  Dense bf16 H = 896
 * models of up to 16 rows advance all active rows in one launch of the multi-stream resident kernel (a lone row on the
 * single-stream resident kernel); other dense bf16 models use the cluster-partitioned kernel for two or more active rows;
 * everything else runs on the any-shape kernel.
 * wrnn_subscale_conditioning computes v_row[0..L) alone from a given history (DEVICE int16 [B][L]) into
 * v (DEVICE [L][cond_dim]).
 */
int wrnn_sample_subscale_dependent(wrnn_model *m, const float *frames, int32_t n_frames, int32_t hop, const float *V,
                                   const float *bias, int32_t F, int32_t chunk, int32_t lag, int64_t n_total, int32_t B,
                                   uint64_t seed, int16_t *out, void *cuda_stream);
int wrnn_subscale_conditioning(const int16_t *hist, const float *frames, const float *V, const float *bias, int32_t B,
                               int64_t L, int32_t F, int32_t cond_dim, int32_t n_frames, int32_t hop, int32_t row, float *v,
                               void *cuda_stream);
/* The stepping launches of that schedule, in order, without running anything (host only, no device needed): call i is
 * calls[4 i .. 4 i + 3] = (first row, number of rows, position of the first row, steps); row b of a call is at the
 * first row's position minus b * lag.  HOST calls[max_calls][4].  Returns the number of launches of the schedule (which
 * may exceed max_calls: only the first max_calls are written), or minus a wrnn_status for bad arguments. */
int wrnn_subscale_schedule(int32_t B, int64_t L, int32_t chunk, int32_t lag, int64_t *calls, int32_t max_calls);

/*
 * The conditioning network of the Subscale WaveRNN with the shape the paper states (Section 5.3: a masked dilated 1-D CNN,
 * ten layers, kernels of size 3, 384 convolution channels, 768 residual channels, five stages of increasing dilation, a
 * future horizon of F = 128 positions; Section 4.1: relus, the mask over the past connections).  The paper prints no
 * equations for it; the reading built here (sub-tensor s, position i, x(u) = u / 32768):
 *     X[i][z]    = x(u_{B i + z}) for z < s, 0 otherwise            block input, masked to the earlier sub-tensors
 *     x_0[i]     = W_in X[i] + b_in
 *     a_l[i]     = relu(b_conv[l] + sum_{t < taps} W_conv[l][t] x_l[i + t dilation[l]])      forward connections only
 *     x_{l+1}[i] = x_l[i] + W_res[l] a_l[i] + b_res[l]
 *     v_s[i]     = frames[s][(B i + s) div hop] + W_out relu(x_last[i]) + b_out
 * positions at or beyond the row length hold the zero vector in every layer; the reach of the network is
 * (taps - 1) * sum of the dilations (124 for 1,1,2,2,4,4,8,8,16,16).  All pointers HOST fp32 row-major, read during the
 * call; the matrices are rounded to bf16 (nearest even), biases stay fp32:
 *     W_in [res_ch][B], b_in [res_ch]; W_conv [n_layers][taps][conv_ch][res_ch], b_conv [n_layers][conv_ch];
 *     W_res [n_layers][res_ch][conv_ch], b_res [n_layers][res_ch]; W_out [cond_dim][res_ch], b_out [cond_dim].
 * The products run on the tensor cores (tiles of 128 positions): conv_ch must be a multiple of 192, res_ch of 128,
 * B <= 64, cond_dim <= 64, every dilation <= 64; other shapes return WRNN_ERR_UNSUPPORTED.
 */
typedef struct wrnn_subscale_net wrnn_subscale_net;     /* opaque; owns its device memory */
typedef struct {
    int32_t B, n_layers, taps, conv_ch, res_ch, cond_dim;
    const int32_t *dilation;                            /* HOST [n_layers] */
    const float *W_in, *b_in, *W_conv, *b_conv, *W_res, *b_res, *W_out, *b_out;
} wrnn_subscale_net_params;
int wrnn_subscale_net_create(const wrnn_subscale_net_params *params, wrnn_subscale_net **out);    /* synchronous; current device */
void wrnn_subscale_net_destroy(wrnn_subscale_net *net);                                            /* NULL allowed */
/* v (DEVICE [L][cond_dim]) = conditioning vectors of sub-tensor `row` at all L positions from the history hist (DEVICE int16
 * [B][L]); frames DEVICE [B][n_frames][cond_dim].  Asynchronous on cuda_stream; may grow the network's activation buffers
 * (synchronously).  wrnn_subscale_net_status, after synchronising: WRNN_OK, or WRNN_ERR_TIMEOUT when a bounded wait of the
 * tensor pipeline ran out. */
int wrnn_subscale_net_conditioning(wrnn_subscale_net *net, const int16_t *hist, const float *frames, int32_t n_frames, int32_t hop,
                                   int32_t row, int64_t L, float *v, void *cuda_stream);
int wrnn_subscale_net_status(wrnn_subscale_net *net);
/* wrnn_sample_subscale_dependent with this network in place of the one-layer convolution: B = the network's B; F >= the
 * network's reach; lag a multiple of chunk and >= F + chunk.  Per chunk the network is evaluated for chunk + reach positions
 * of every active row (the positions ahead are recomputed by the next chunk).  Asynchronous on cuda_stream. */
int wrnn_sample_subscale_net(wrnn_model *m, wrnn_subscale_net *net, const float *frames, int32_t n_frames, int32_t hop, int32_t F,
                             int32_t chunk, int32_t lag, int64_t n_total, uint64_t seed, int16_t *out, void *cuda_stream);

/* One stepping call of the staggered schedule on caller-owned buffers: rows r_lo .. r_lo + n_rows - 1 of the B sub-tensors
 * advance n_steps positions, row b of the call from position p_lo - b * lag on (the unit wrnn_sample_subscale_net is made of,
 * exposed so that the sub-tensors can be spread over several devices, each generating some rows and passing the samples on one
 * way, online: Section 5.3's closing paragraph).  hist: DEVICE int16 [B][L], read for the rows below r_lo + n_rows (positions up
 * to F ahead must be there) and written in place for the rows of the call; h [B][H], c_prev / f_prev [B]: DEVICE carry state
 * of all rows, read and written for the rows of the call (start from h = 0, c_prev = 128, f_prev = 0).  n_rows <= max_batch.
 * Asynchronous on cuda_stream. */
int wrnn_subscale_net_rows(wrnn_model *m, wrnn_subscale_net *net, const float *frames, int32_t n_frames, int32_t hop, int32_t lag, int16_t *hist,
                           int64_t L, float *h, uint8_t *c_prev, uint8_t *f_prev, int32_t r_lo, int32_t n_rows, int64_t p_lo, int32_t n_steps,
                           uint64_t seed, void *cuda_stream);

/*
 * Host-buffer convenience for callers without device pointers: copies cond
 * (HOST [batch][n_frames][cond_dim]) to the device, runs wrnn_sample from the
 * default state and copies the samples back to out (HOST int16 [batch][n_steps]).
 * Synchronous.
 */
int wrnn_sample_host(wrnn_model *m, const float *cond_host, int32_t n_frames, int32_t hop,
                     int32_t row_stride, int32_t row_offset_mul, int64_t n_steps, int32_t batch,
                     uint64_t seed, int16_t *out_host);

/* After the stream has been synchronised: WRNN_OK, or what the last kernel reported. */
int wrnn_poll_status(wrnn_model *m);
/* Diagnostic text of the last error on this model (or of the last failed create when
 * m == NULL).  Not thread-safe; valid until the next call. */
const char *wrnn_last_error(wrnn_model *m);

/* Introspection used by the benchmark and the tests (HOST out-pointers, any may be NULL):
 * kernel family in use, CTAs and threads per CTA of the persistent kernel for `batch`
 * rows, bytes of packed weights read per step, dynamic shared memory per CTA. */
int wrnn_launch_info(wrnn_model *m, int32_t batch, int32_t *kernel, int32_t *n_ctas,
                     int32_t *n_threads, int64_t *weight_bytes_per_step, int32_t *smem_bytes);

/*
 * Fused Subscale WaveRNN 2x (Section 4.4: a Subscale WaveRNN 2x whose two sub-tensors each get one part of the hidden
 * state of a single WaveRNN; 8 softmaxes of 4 bits, future horizon F = 2, the generated samples are the direct inputs;
 * 32 bits per step).  Reading used here: sub-tensor 0 holds a_i = u_{2i}, sub-tensor 1 holds b_i = u_{2i+1}; step t
 * emits a_t from part A (units [0, H/2)) and then b_{t-2} from part B (units [H/2, H)), which sees a_t inside the step
 * as the fine half sees c_t in Eq. 2; a 16-bit sample is four nibbles, most significant first, each drawn from its own
 * 16-way softmax over 16 consecutive logits of the part's head, and fed back scaled to v / 7.5 - 1.  Uniforms: the
 * same Philox keying with head = 4 * part + nibble.  Models are created by wrnn_create with variant = 1; batch is 1.
 *
 * State: DEVICE pointers as for wrnn_state; a_prev / b_prev hold the two samples of the previous step as unsigned
 * 16-bit values (NULL = 0x8000).  cond: as for wrnn_sample with batch 1 (frame index (step0 + s) * row_stride / hop).
 * wrnn_fs2_sample writes DEVICE out[2][n_steps] int16 (value - 32768): row 0 = a_t, row 1 = the sample part B emitted in
 * step t (= b_{t-2}).  wrnn_fs2_step_teacher_forced records the drawn samples in a_out / b_out (DEVICE [n_steps] or
 * NULL) and feeds a_forced / b_forced back instead; dumps as for wrnn_step_teacher_forced with logits [n_steps][2][64].
 * wrnn_fs2_unfold interleaves the two rows into the original order, dropping the two pre-roll samples of row 1:
 * u[2 i] = ab[0][i], u[2 i + 1] = ab[1][i + 2] for i < n_steps - 2 (DEVICE u of 2 (n_steps - 2) samples).
 * All asynchronous on cuda_stream; errors as for the calls above; WRNN_ERR_UNSUPPORTED for a model of the other variant.
 */
typedef struct {
    float *h;            /* [H] */
    uint16_t *a_prev;    /* [1] */
    uint16_t *b_prev;    /* [1] */
    int64_t step0;
    uint32_t stream0;
    uint32_t reserved;
} wrnn_fs2_state;

int wrnn_fs2_sample(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, uint64_t seed, const wrnn_fs2_state *st,
                    int16_t *out, void *cuda_stream);
int wrnn_fs2_step_teacher_forced(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, uint64_t seed,
                                 const wrnn_fs2_state *st, const uint16_t *a_forced, const uint16_t *b_forced,
                                 uint16_t *a_out, uint16_t *b_out, float *dbg_gates, float *dbg_h, float *dbg_logits,
                                 void *cuda_stream);
int wrnn_fs2_unfold(const int16_t *ab, int64_t n_steps, int16_t *u, void *cuda_stream);
/* Host-buffer convenience, synchronous: cond_host HOST [n_frames][cond_dim] -> device, wrnn_fs2_sample from the default
 * state, wrnn_fs2_unfold, and the 2 (n_steps - 2) interleaved samples back to u_host (HOST int16). */
int wrnn_fs2_sample_host(wrnn_model *m, const float *cond_host, int32_t n_frames, int32_t hop, int64_t n_steps,
                         uint64_t seed, int16_t *u_host);

/* Diagnostic of the resident single-stream kernel (Section 2.1: after the persistent kernel the
 * remaining overhead is the synchronisation between multiprocessors): SM-clock cycles that warp 0 of
 * CTA 0 spent in each phase of a step, summed over the last finished call on this model (HOST
 * out16[16]).  A step has a fine half (entries 0..5, 12, 14) and a coarse half (6..11, 13, 15):
 *   0 / 6   wait for the input half of the state from the whole chip (L2 exchange)
 *   12 / 13 hidden-layer and recurrent partial products + CTA barrier
 *   1 / 7   hidden-layer finish and send to the cluster
 *   2 / 8   wait for the cluster's hidden layer + CTA barrier
 *   14 / 15 logits partial products + CTA barrier
 *   3 / 9   logits finish and send to the cluster
 *   4 / 10  wait for the cluster's logits
 *   5 / 11  softmax draw, gates of the other half, publish
 * A dense fp32 model runs the fp32 variant of the kernel: the same slots, with "partial products" read as its
 * plain fp32 row products, and 2 / 8 a second chip-wide wait (the hidden layer crosses L2 there).
 * The lean single-stream kernel (the default for a dense bf16 H = 896 model) has eight phases per half, fine half in
 * entries 0..7 and coarse half in 8..15: wait for the state half; hidden-layer products; hidden-layer sums and send;
 * recurrent products; recurrent sums and gate preparation (while other warps wait for the cluster's hidden layer and
 * multiply the output-layer rows); CTA barrier behind those rows and send; wait for the cluster's logits; draw, gates,
 * publish.  wrnn_phase_names writes the sixteen names that belong to
 * the last profiled call, comma-separated, into buf (HOST, cap bytes).
 * The stamps cost the stamped warp, which is on the critical path of the whole chip, some tens of cycles each, so they
 * are taken only while wrnn_phase_profile(m, 1) is in effect (default off); wrnn_phase_cycles then reports the last
 * finished call.  Synchronous. */
int wrnn_phase_profile(wrnn_model *m, int32_t enable);
int wrnn_phase_names(wrnn_model *m, char *buf, int32_t cap);
int wrnn_phase_cycles(wrnn_model *m, int64_t *out16);

/* Floor of a chip-wide exchange on this device: nanoseconds per all-gather of K tagged fp32 values through
 * L2 among n_ctas co-resident CTAs of n_threads threads in an otherwise empty persistent kernel (Section 2.1:
 * once the weights are resident, what remains per step is the synchronisation between multiprocessors; the
 * sampling step needs two such exchanges).  Measured twice -- pollers starting at once, and pollers held back 150 cycles
 * after their CTA's own publication, as the sampling kernels do -- and the smaller figure is reported.  K must be a
 * multiple of n_ctas.  HOST out-pointer.  Synchronous; allocates and frees a small device buffer. */
int wrnn_measure_exchange_floor(int32_t n_ctas, int32_t n_threads, int32_t K, int32_t iters, float *ns_per_exchange);

/* Measured counterpart of the nominal shared-memory bandwidth that bounds "every resident weight read once per step"
 * (Section 2.1: the model stays on chip across the whole utterance): n_ctas CTAs (one per SM when n_ctas <= the SM
 * count) of n_threads threads each read a resident buffer of bytes_per_cta bytes `iters` times with 16-byte loads;
 * *gb_per_s receives the aggregate rate (HOST out-pointer).  bytes_per_cta: a multiple of 16 up to 227 KiB.
 * Synchronous; allocates and frees a small device buffer. */
int wrnn_measure_smem_stream(int32_t n_ctas, int32_t n_threads, int32_t bytes_per_cta, int32_t iters, float *gb_per_s);

/* Self-test of the bounded device-side waits (the error path of every persistent kernel here): a two-CTA kernel whose
 * first CTA waits at the grid barrier for an arrival that never comes, gives up after limit_ns (1 us .. 1 s of the
 * global timer) and returns.  *code receives the device status word (WRNN_ERR_TIMEOUT when the wait ran out as it
 * should), the optional HOST out-pointers the (cta, step, phase) it recorded (0, 7, 3) and the kernel's duration.
 * Nothing faults and the context stays usable.  Synchronous; allocates and frees two small device buffers. */
int wrnn_selftest_bounded_wait(int64_t limit_ns, int32_t *code, int32_t *cta, int32_t *step, int32_t *phase, float *waited_ms);

/* Self-test of the give-up paths of the sampling kernels themselves (the failure is made on the host side of the
 * protocol: a message is withheld; nothing faults, traps or spins without bound).  From the next launch on this model,
 * CTA `cta` withholds at step `step` (relative to the call) what it would hand to the other CTAs: the state values it
 * publishes (shared-memory-resident and sparse kernels), one operand load of its own tensor pipeline (cluster-partitioned
 * kernel), or its arrivals at the grid barrier (any-shape and grid-phased kernels); limit_ns (0 = the default of two
 * seconds, at most two seconds) bounds every device-side wait of the launch.  The waits that depend on the missing piece
 * run out, the first CTA to give up records WRNN_ERR_TIMEOUT with (cta, step, phase), every CTA leaves through its normal
 * exit and wrnn_poll_status reports it.  cta = -1 restores normal operation (limit_ns still applies).  Host only. */
int wrnn_selftest_lost_word(wrnn_model *m, int64_t limit_ns, int32_t cta, int64_t step);

/* Kernels launched by this library in this process since load (all models). */
int64_t wrnn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* WRNN_H */
