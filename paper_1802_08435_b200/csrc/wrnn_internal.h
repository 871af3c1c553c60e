// Host-side structures shared by the translation units of libwrnn.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdlib>
#include <string>
#include <vector>

#include "../../include/wrnn.h"
#include "wrnn_device.cuh"

namespace wrnn {

// A matrix stored as compressed block rows of 4x4 blocks (Section 3.2).  A dense matrix is
// the same structure with every block present.  vals holds nnz blocks of 16 weights each,
// block-row-major inside a block (vals[i][4 r + c] = W[4 br + r][4 bc + c]), in the model's
// storage type (fp32 or bf16).
struct BsrDev {
    int rows4 = 0, cols4 = 0, nnz = 0;
    int *row_ptr = nullptr;        // [rows4 + 1]
    uint16_t *col = nullptr;       // [nnz] block column
    void *vals = nullptr;          // [nnz][16]
};

// Host image of the same thing (after masking and rounding), kept for the packers of the
// specialised kernels.
struct BsrHost {
    int rows4 = 0, cols4 = 0;
    std::vector<int> row_ptr;
    std::vector<uint16_t> col;
    std::vector<float> vals;       // fp32 values (already rounded to the storage type)
};

// Everything one stepping call needs besides the model (device pointers).
struct StepArgs {
    const float *cond;       // [batch][n_frames][cond_dim] (unused by the step kernels: g is projected)
    int n_frames, hop, row_stride, row_offset_mul;
    long long n_steps;
    int batch;
    unsigned long long seed;
    long long step0;
    unsigned stream0;
    const float *h_in;  float *h_out;            // may be null
    const uint8_t *c_in, *f_in; uint8_t *c_st_out, *f_st_out;
    const uint8_t *c_forced, *f_forced;          // [batch][n_steps] or null
    uint8_t *c_out, *f_out;                      // [batch][n_steps] or null
    int16_t *out;                                // [batch][n_steps] or null
    float *dbg_gates, *dbg_h, *dbg_logits;       // or null
    // staggered subscale rows: row b of the call is row_lag steps behind row b - 1 and takes one conditioning frame per
    // step of the call (0 = rows in lock step); out_pitch = samples between the rows of `out` (0 = n_steps)
    int row_lag;
    long long out_pitch;
    // fused subscale variant: 16-bit samples of parts A and B in place of the bytes above (batch 1)
    const uint16_t *a_in, *b_in; uint16_t *a_st_out, *b_st_out;
    const uint16_t *a_forced, *b_forced;         // [n_steps] or null
    uint16_t *a_out, *b_out;                     // [n_steps] or null
};

struct ResidentPack;   // packed weights of the shared-memory-resident kernels (opaque here)
struct BatchedPack;    // fragment-packed weights and activation images of the batched kernel (opaque here)
struct SparsePack;     // compressed block rows of the single-cluster block-sparse kernel (opaque here)
struct ResF32Pack;     // per-CTA fp32 weight shards of the single-stream fp32 resident kernel (opaque here)
struct ResLeanPack;      // per-CTA weights of the lean single-stream resident kernel (opaque here)
struct ResMultiPack;  // per-CTA weights of the multi-stream resident kernel (opaque here)
struct BcPack;         // per-CTA weight slices and stacked activation images of the cluster-partitioned multi-row kernel

}  // namespace wrnn

struct wrnn_subscale_net;   // the conditioning network of the Subscale WaveRNN (wrnn_subnet.cu)

struct wrnn_model {
    int H = 0, cond_dim = 0, dtype = 0, kernel = 0, max_batch = 0;
    int variant = 0;                // 0: WaveRNN (Eq. 2); 1: Fused Subscale WaveRNN 2x (I has 12 columns, O2 / O4 64 rows)
    int device = 0, n_sms = 0;
    bool sparse = false;
    int mask_br = 4, mask_bc = 4;   // shape of one block of the sparsity masks (Section 3.2)

    // generic format
    wrnn::BsrDev R, O1, O2, O3, O4;
    float *I = nullptr;            // [3H][3] fp32 (values rounded to storage type; masked column zeroed)
    float *b_gate = nullptr, *b1 = nullptr, *b2 = nullptr, *b3 = nullptr, *b4 = nullptr;
    float *W_condT = nullptr;      // [cond_dim][3H] fp32 (rounded values), transposed for coalescing
    int64_t weight_bytes = 0;      // packed bytes read per step (values + indices + row pointers)

    // per-call scratch owned by the model
    float *g = nullptr;            // projected conditioning [batch][n_frames][3H]
    size_t g_cap = 0;              // floats
    float *hbuf[2] = {nullptr, nullptr};   // [max_batch][H]
    float *a_fine = nullptr;       // [max_batch][3][H/2]  R h of the fine rows, kept across the coarse head
    float *q = nullptr;            // [max_batch][H/2]
    float *logits = nullptr;       // [max_batch][256]
    uint8_t *c_cur = nullptr, *c_prev = nullptr, *f_prev = nullptr;   // [max_batch]
    unsigned long long *bar = nullptr;     // grid barrier counter
    wrnn::DevStatus *status = nullptr;     // device status word
    // host staging for wrnn_sample_host
    float *stage_cond = nullptr; size_t stage_cond_cap = 0;
    int16_t *stage_out = nullptr; size_t stage_out_cap = 0;
    uint8_t *sub_scratch = nullptr; size_t sub_cap = 0;   // history, conditioning and carry state of wrnn_sample_subscale_dependent

    wrnn::ResidentPack *resident = nullptr;
    wrnn::ResLeanPack *reslean = nullptr;
    bool prof_lean = false;           // the last call with phase timing ran on the lean single-stream resident kernel
    wrnn::ResF32Pack *resf32 = nullptr;
    wrnn::ResMultiPack *resmulti = nullptr;
    // wrnn_selftest_lost_word: bound of every device-side wait (0 = the default of two seconds) and the CTA / step whose
    // publication (or operand load) is withheld (-1 = none)
    unsigned long long dbg_limit_ns = 0;
    int dbg_skip_cta = -1;
    long long dbg_skip_step = -1;
    unsigned long long wait_limit_ns() const { return dbg_limit_ns ? dbg_limit_ns : 2000000000ull; }
    bool prof_enabled = false;      // wrnn_phase_profile: the resident kernels stamp their phases
    bool prof_multi = false;        // the last call with phase timing ran on the multi-stream resident kernel
    wrnn::BatchedPack *batched = nullptr;
    wrnn::SparsePack *sparse_pack = nullptr;
    wrnn::BcPack *bcluster = nullptr;

    // host images for packers
    wrnn::BsrHost hR, hO1, hO2, hO3, hO4;
    std::vector<float> hI, hb_gate, hb1, hb2, hb3, hb4;

    std::string err;
};

namespace wrnn {

extern std::atomic<long long> g_launches;

// Whether the persistent cluster kernels are launched with the cooperative attribute (the driver then refuses the launch
// unless all clusters can be co-resident).  Co-residency is checked against the occupancy API when a model is created, so
// the attribute is a second line of defence; it is dropped under WRNN_NO_COOP=1 and when a CUDA injection library is
// loaded into the process (a profiler: kernel replay does not accept cooperative cluster launches).
inline bool coop_launch_allowed()
{
    const char *no_coop = getenv("WRNN_NO_COOP");
    if (no_coop && no_coop[0] == '1') return false;
    const char *inj = getenv("CUDA_INJECTION64_PATH");
    return !(inj && inj[0]);
}

// wrnn_api.cu: argument checks shared by the stepping entry points (fills the cond / state part of StepArgs)
int check_step(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, const wrnn_state *st, StepArgs *a);

// wrnn_generic.cu
int generic_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem);
int generic_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);   // returns wrnn_status
int cond_project(wrnn_model *m, const float *cond, int batch, int n_frames, cudaStream_t s);
void noalloc_warm(int device);   // resolves the device address of the fixed scratch array of wrnn_sample_noalloc (once per device)
int fold_launch(const int16_t *x, long long n_total, int B, int16_t *sub, bool unfold, cudaStream_t s);
int fs2_unfold_launch(const int16_t *ab, long long n, int16_t *u, cudaStream_t s);
int subscale_cond_launch(const int16_t *hist, const float *frames, const float *V, const float *bias, float *v, int B, long long L, int F,
                         int D, int n_frames, int hop, int r_lo, int n_rows, long long p_lo, int lag, int n_steps, cudaStream_t s);

// wrnn_subnet.cu: the masked dilated conditioning network on the tensor cores, for the segments of one stepping call
int subnet_run(wrnn_subscale_net *n, const int16_t *hist, const float *frames, int n_frames, int hop, long long L, int r_lo, int n_rows,
               long long p_lo, int lag, int n_steps, float *v, unsigned long long limit_ns, cudaStream_t s);
int subnet_reach(const wrnn_subscale_net *n);
int subnet_B(const wrnn_subscale_net *n);
int subnet_cond_dim(const wrnn_subscale_net *n);

// wrnn_resident.cu
int resident_supported(const wrnn_model *m, int batch, std::string *why);
int resident_prepare(wrnn_model *m);                                  // pack + upload at create
void resident_destroy(wrnn_model *m);
int resident_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem,
                         int64_t *weight_bytes);
int resident_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);
int resident_phase_cycles(const wrnn_model *m, long long *out16);
int resident_pair_supported(const wrnn_model *m, int batch);          // two streams per launch on the same weights (batch 2 or 4)
int resident_pair_run(wrnn_model *m, const StepArgs &a, int pair, cudaStream_t s);

// host packers shared by the resident kernels (wrnn_resident.cu)
void dense_row_bf16(const BsrHost &M, int row, int c0, int n, uint16_t *dst);       // dense row of a block-row matrix -> bf16 bits of columns [c0, c0 + n)
void pack_tile(const std::vector<std::vector<uint16_t>> &rows, int K, uint16_t *dst);   // rows[16][K] -> m16n8k16 A fragments [K/16][32 lanes][8]

// wrnn_reslean.cu: one stream of a dense bf16 H = 896 model, the row-split resident kernel with a shorter chain per half-step
int reslean_supported(const wrnn_model *m, int batch);
int reslean_prepare(wrnn_model *m);
void reslean_destroy(wrnn_model *m);
int reslean_launch_info(const wrnn_model *m, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int reslean_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);
int reslean_phase_cycles(const wrnn_model *m, long long *out16);

// wrnn_resmulti.cu: 2 to 16 lock-step streams of a dense bf16 H = 896 model on resident weights
int resmulti_supported(const wrnn_model *m, int batch);
int resmulti_prepare(wrnn_model *m);
void resmulti_destroy(wrnn_model *m);
int resmulti_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int resmulti_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);
int resmulti_phase_cycles(const wrnn_model *m, long long *out16);

// wrnn_resf32.cu: the same role for dense fp32 models (every matrix sharded chip-wide, nothing replicated)
int resf32_supported(const wrnn_model *m, int batch, std::string *why);
int resf32_prepare(wrnn_model *m);
void resf32_destroy(wrnn_model *m);
int resf32_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int resf32_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);
int resf32_phase_cycles(const wrnn_model *m, long long *out16);

// wrnn_sparse.cu
int sparse_supported(const wrnn_model *m, int batch, std::string *why);
int sparse_prepare(wrnn_model *m);
void sparse_destroy(wrnn_model *m);
int sparse_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int sparse_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);

// wrnn_batched.cu
int batched_supported(const wrnn_model *m, int batch, std::string *why);
int batched_prepare(wrnn_model *m);
void batched_destroy(wrnn_model *m);
int batched_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int batched_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);
std::vector<uint16_t> dense_bf16_bits(const BsrHost &M);   // host block rows -> dense row-major bf16 bits

// wrnn_bcluster.cu
int bcluster_supported(const wrnn_model *m, int batch, std::string *why);
int bcluster_prepare(wrnn_model *m);
void bcluster_destroy(wrnn_model *m);
int bcluster_launch_info(const wrnn_model *m, int batch, int *n_ctas, int *n_threads, int *smem, int64_t *weight_bytes);
int bcluster_run(wrnn_model *m, const StepArgs &a, cudaStream_t s);

}  // namespace wrnn
