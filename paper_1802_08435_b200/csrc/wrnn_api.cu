// C ABI of libwrnn.so: model creation (masking, rounding, packing, upload), argument
// checking and dispatch to the kernel families.  Declarations and contracts: include/wrnn.h.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "wrnn_internal.h"

namespace wrnn {
std::atomic<long long> g_launches{0};
static std::string g_create_err;

// fp32 -> bf16 storage (round to nearest, ties to even) -> back to fp32.
static float round_bf16(float v)
{
    uint32_t b;
    std::memcpy(&b, &v, 4);
    if ((b & 0x7f800000u) != 0x7f800000u) {
        const uint32_t lsb = (b >> 16) & 1u;
        b += 0x7fffu + lsb;
    } else if (b & 0x007fffffu) {
        b |= 0x00400000u;
    }
    b &= 0xffff0000u;
    float r;
    std::memcpy(&r, &b, 4);
    return r;
}

static inline uint16_t bf16_bits(float rounded)
{
    uint32_t b;
    std::memcpy(&b, &rounded, 4);
    return (uint16_t)(b >> 16);
}

// Dense row-major W[rows][cols] (+ optional 4x4 block mask) -> host block rows with the
// values already rounded to the storage type.
// W[rows][cols] with an optional mask of mr x mc blocks ([rows/mr][cols/mc], 1 = kept) -> compressed block rows of
// 4x4 blocks: a 4x4 block is stored when any of its 16 weights is kept; weights that are not kept are stored as zero.
static void build_bsr(const float *W, int rows, int cols, const uint8_t *mask, int mr, int mc, bool bf16, BsrHost *out)
{
    const int R4 = rows / 4, C4 = cols / 4, MC = mask ? cols / mc : 0;
    out->rows4 = R4; out->cols4 = C4;
    out->row_ptr.assign(R4 + 1, 0);
    out->col.clear(); out->vals.clear();
    for (int br = 0; br < R4; ++br) {
        for (int bc = 0; bc < C4; ++bc) {
            bool kept[16], any = false;
            for (int r = 0; r < 4; ++r)
                for (int c = 0; c < 4; ++c) {
                    kept[4 * r + c] = !mask || mask[(size_t)((4 * br + r) / mr) * MC + (4 * bc + c) / mc] != 0;
                    any = any || kept[4 * r + c];
                }
            if (!any) continue;
            out->col.push_back((uint16_t)bc);
            for (int r = 0; r < 4; ++r)
                for (int c = 0; c < 4; ++c) {
                    const float v = kept[4 * r + c] ? W[(size_t)(4 * br + r) * cols + 4 * bc + c] : 0.f;
                    out->vals.push_back(bf16 ? round_bf16(v) : v);
                }
        }
        out->row_ptr[br + 1] = (int)out->col.size();
    }
}

template <typename T> static bool upload(T **dst, const void *src, size_t bytes)
{
    *dst = nullptr;
    if (bytes == 0) return true;
    if (cudaMalloc((void **)dst, bytes) != cudaSuccess) return false;
    return cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) == cudaSuccess;
}

static bool upload_bsr(const BsrHost &h, bool bf16, BsrDev *d)
{
    d->rows4 = h.rows4; d->cols4 = h.cols4; d->nnz = (int)h.col.size();
    if (!upload(&d->row_ptr, h.row_ptr.data(), h.row_ptr.size() * sizeof(int))) return false;
    // keep 16 B of slack so that vector loads of an empty matrix stay in bounds
    std::vector<uint16_t> col(h.col);
    col.resize(col.size() + 8, 0);
    if (!upload(&d->col, col.data(), col.size() * sizeof(uint16_t))) return false;
    if (bf16) {
        std::vector<uint16_t> v(h.vals.size() + 16, 0);
        for (size_t i = 0; i < h.vals.size(); ++i) v[i] = bf16_bits(h.vals[i]);
        return upload((uint16_t **)&d->vals, v.data(), v.size() * sizeof(uint16_t));
    }
    std::vector<float> v(h.vals);
    v.resize(v.size() + 16, 0.f);
    return upload((float **)&d->vals, v.data(), v.size() * sizeof(float));
}

static void free_bsr(BsrDev *d)
{
    cudaFree(d->row_ptr); cudaFree(d->col); cudaFree(d->vals);
    *d = BsrDev();
}

static int fail(wrnn_model *m, int code, const std::string &msg)
{
    if (m) m->err = msg; else g_create_err = msg;
    return code;
}

static bool ensure_g(wrnn_model *m, size_t floats)
{
    if (floats <= m->g_cap) return true;
    cudaDeviceSynchronize();
    cudaFree(m->g);
    m->g = nullptr; m->g_cap = 0;
    if (cudaMalloc((void **)&m->g, floats * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return false; }
    m->g_cap = floats;
    return true;
}

static bool use_resident(const wrnn_model *m, int batch)
{
    if (m->kernel == WRNN_KERNEL_GENERIC || m->kernel == WRNN_KERNEL_BATCHED || m->kernel == WRNN_KERNEL_BCLUSTER) return false;
    return m->resident != nullptr && resident_supported(m, batch, nullptr) == WRNN_OK;
}

// one stream of a dense bf16 H = 896 model: the lean form of the resident kernel (wrnn_reslean.cu)
// (WRNN_RESIDENT_LEAN=0 keeps the first form: diagnostic, for A/B measurements on one device)
static bool use_reslean(const wrnn_model *m, int batch)
{
    if (m->kernel != WRNN_KERNEL_AUTO && m->kernel != WRNN_KERNEL_RESIDENT) return false;
    const char *sw = getenv("WRNN_RESIDENT_LEAN");
    if (sw && sw[0] == '0') return false;
    return reslean_supported(m, batch) == WRNN_OK;
}

static bool use_resf32(const wrnn_model *m, int batch)
{
    if (m->kernel == WRNN_KERNEL_GENERIC || m->kernel == WRNN_KERNEL_BATCHED || m->kernel == WRNN_KERNEL_BCLUSTER) return false;
    return m->resf32 != nullptr && resf32_supported(m, batch, nullptr) == WRNN_OK;
}

// two or four streams of a dense bf16 model: pairs on the two-stream form of the resident kernel, one pair after the other
// (the fallback of the multi-stream resident kernel, which takes 2 to 16 rows where the model has one)
static bool use_pair(const wrnn_model *m, int batch)
{
    if (m->kernel != WRNN_KERNEL_AUTO && m->kernel != WRNN_KERNEL_RESIDENT) return false;
    const char *off = getenv("WRNN_NO_PAIR");
    if (off && off[0] == '1') return false;
    return m->variant == 0 && resident_pair_supported(m, batch) == WRNN_OK;
}

// 2 to 16 lock-step streams of a dense bf16 H = 896 model: all of them in one launch on the resident weights
// (WRNN_NO_MULTI=1 falls back to the two-stream and cluster-partitioned kernels: diagnostic)
static bool use_multi(const wrnn_model *m, int batch)
{
    if (m->kernel != WRNN_KERNEL_AUTO && m->kernel != WRNN_KERNEL_RESIDENT) return false;
    const char *off = getenv("WRNN_NO_MULTI");
    if (off && off[0] == '1') return false;
    return m->variant == 0 && resmulti_supported(m, batch) == WRNN_OK;
}

static bool use_sparse(const wrnn_model *m, int batch)
{
    if (m->kernel != WRNN_KERNEL_AUTO && m->kernel != WRNN_KERNEL_SPARSE) return false;
    return m->sparse_pack != nullptr && sparse_supported(m, batch, nullptr) == WRNN_OK;
}

static bool use_bcluster(const wrnn_model *m, int batch)
{
    if (m->kernel != WRNN_KERNEL_AUTO && m->kernel != WRNN_KERNEL_BCLUSTER) return false;
    return m->bcluster != nullptr && bcluster_supported(m, batch, nullptr) == WRNN_OK;
}

static bool use_batched(const wrnn_model *m, int batch)
{
    if (m->kernel == WRNN_KERNEL_GENERIC || m->kernel == WRNN_KERNEL_RESIDENT || m->kernel == WRNN_KERNEL_BCLUSTER) return false;
    return m->batched != nullptr && batched_supported(m, batch, nullptr) == WRNN_OK;
}

// Common argument checks of the stepping calls; fills the parts of StepArgs that come from
// cond / st.  Returns WRNN_OK or an error (message in m->err).
static int check_step_any(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, const wrnn_state *st,
                          StepArgs *a, bool fused_call)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    if ((m->variant == 1) != fused_call)
        return fail(m, WRNN_ERR_UNSUPPORTED, fused_call ? "not a fused subscale model (create with variant = 1)"
                                                        : "a fused subscale model is stepped with the wrnn_fs2_* calls");
    if (n_steps < 0 || batch < 1) return fail(m, WRNN_ERR_INVALID_ARG, "n_steps < 0 or batch < 1");
    if (batch > m->max_batch) return fail(m, WRNN_ERR_INVALID_ARG, "batch exceeds max_batch given at create");
    if (n_steps > (1ll << 31) - 2) return fail(m, WRNN_ERR_INVALID_ARG, "n_steps too large for one call");
    std::memset(a, 0, sizeof(*a));
    a->n_steps = n_steps; a->batch = batch;
    a->step0 = st ? st->step0 : 0;
    a->stream0 = st ? st->stream0 : 0;
    if (a->step0 < 0) return fail(m, WRNN_ERR_INVALID_ARG, "step0 < 0");
    if (st) {
        a->h_in = st->h; a->h_out = st->h;
        a->c_in = st->c_prev; a->c_st_out = st->c_prev;
        a->f_in = st->f_prev; a->f_st_out = st->f_prev;
    }
    if (m->cond_dim > 0) {
        if (!cond || !cond->cond) return fail(m, WRNN_ERR_INVALID_ARG, "model is conditioned but cond is NULL");
        if (cond->hop <= 0 || cond->n_frames <= 0 || cond->row_stride < 0 || cond->row_offset_mul < 0)
            return fail(m, WRNN_ERR_INVALID_ARG, "bad conditioning geometry");
        a->cond = cond->cond; a->n_frames = cond->n_frames; a->hop = cond->hop;
        a->row_stride = cond->row_stride; a->row_offset_mul = cond->row_offset_mul;
        if (n_steps > 0) {
            const long long last = ((a->step0 + n_steps - 1) * (long long)a->row_stride +
                                    ((long long)a->stream0 + batch - 1) * a->row_offset_mul) / a->hop;
            if (last >= a->n_frames) return fail(m, WRNN_ERR_INVALID_ARG, "conditioning frames run out before n_steps");
        }
    } else {
        a->n_frames = 1; a->hop = 1;
    }
    return WRNN_OK;
}

int check_step(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, const wrnn_state *st, StepArgs *a)
{
    return check_step_any(m, cond, n_steps, batch, st, a, false);
}

static int run_steps(wrnn_model *m, StepArgs &a, cudaStream_t s)
{
    if (a.n_steps == 0) return WRNN_OK;
    if (cudaSetDevice(m->device) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, "cudaSetDevice failed");
    const int nf = m->cond_dim ? a.n_frames : 1;
    if (!ensure_g(m, (size_t)a.batch * nf * 3 * m->H)) return fail(m, WRNN_ERR_NOMEM, "conditioning scratch allocation failed");
    int rc = cond_project(m, a.cond, a.batch, nf, s);
    if (rc != WRNN_OK) return fail(m, rc, "conditioning projection launch failed");
    // staggered rows: the cluster-partitioned kernel, else the any-shape kernel
    if (a.row_lag > 0) {
        if (a.batch >= 2 && use_multi(m, a.batch)) return resmulti_run(m, a, s);
        if (a.batch >= 2 && use_bcluster(m, a.batch)) return bcluster_run(m, a, s);
        if (a.batch == 1 && use_reslean(m, 1)) return reslean_run(m, a, s);           // a lone row (the ramps of the schedule)
        if (a.batch == 1 && use_resident(m, 1)) return resident_run(m, a, s);
        return generic_run(m, a, s);
    }
    if (use_reslean(m, a.batch)) return reslean_run(m, a, s);
    if (use_resident(m, a.batch)) return resident_run(m, a, s);
    // 2 to 16 rows: the multi-stream kernel (two rows 6.5 us per lock-step against 7.7 on the two-stream kernel, which serves
    // them where the multi-stream kernel does not apply or under WRNN_NO_MULTI=1)
    if (use_multi(m, a.batch)) return resmulti_run(m, a, s);
    if (use_pair(m, a.batch)) {
        for (int pair = 0; pair < a.batch / 2; ++pair) {
            rc = resident_pair_run(m, a, pair, s);
            if (rc != WRNN_OK) return rc;
        }
        return WRNN_OK;
    }
    if (use_resf32(m, a.batch)) return resf32_run(m, a, s);
    if (use_sparse(m, a.batch)) return sparse_run(m, a, s);
    if (use_bcluster(m, a.batch)) return bcluster_run(m, a, s);
    if (use_batched(m, a.batch)) return batched_run(m, a, s);
    if (m->kernel == WRNN_KERNEL_BCLUSTER) {
        std::string why;
        bcluster_supported(m, a.batch, &why);
        return fail(m, WRNN_ERR_UNSUPPORTED, "cluster-partitioned kernel unavailable: " + why);
    }
    if (m->kernel == WRNN_KERNEL_SPARSE) {
        std::string why;
        sparse_supported(m, a.batch, &why);
        return fail(m, WRNN_ERR_UNSUPPORTED, "sparse cluster kernel unavailable: " + why);
    }
    if (m->kernel == WRNN_KERNEL_BATCHED) {
        std::string why;
        batched_supported(m, a.batch, &why);
        return fail(m, WRNN_ERR_UNSUPPORTED, "batched kernel unavailable: " + why);
    }
    if (m->kernel == WRNN_KERNEL_RESIDENT) {
        std::string why;
        if (m->dtype == WRNN_F32) resf32_supported(m, a.batch, &why); else resident_supported(m, a.batch, &why);
        return fail(m, WRNN_ERR_UNSUPPORTED, "resident kernel unavailable: " + why);
    }
    return generic_run(m, a, s);
}

// The stepping calls of the staggered subscale schedule (Section 4.2), in launch order: global time advances one chunk
// per iteration, row r is at position k * chunk - r * lag and active while that lies in [0, L); the active rows are
// contiguous; a row that ends inside a chunk gets a call of its own (all rows of a call run the same number of steps).
struct SubCall { int r_lo, n_rows; long long p_lo; int n_steps; };
static void subscale_schedule(int B, long long L, int chunk, int lag, std::vector<SubCall> *calls)
{
    for (long long k = 0;; ++k) {
        const long long t = k * chunk;
        if (t - (long long)(B - 1) * lag >= L) break;                       // the last row is done
        const int r_hi = (int)std::min<long long>(B - 1, t / lag);
        int r_lo = t >= L ? (int)((t - L) / lag) + 1 : 0;
        if (r_lo > r_hi) continue;                                          // a gap between rows (lag > L)
        const long long p_lo = t - (long long)r_lo * lag;
        const long long left = L - p_lo;
        if (left < chunk) {                                                 // the oldest active row ends inside this chunk
            calls->push_back({r_lo, 1, p_lo, (int)left});
            ++r_lo;
            if (r_lo > r_hi) continue;
        }
        calls->push_back({r_lo, r_hi - r_lo + 1, t - (long long)r_lo * lag, chunk});
    }
}

}  // namespace wrnn

using namespace wrnn;

extern "C" {

int wrnn_create(const wrnn_params *p, int32_t max_batch, wrnn_model **out)
{
    if (out) *out = nullptr;
    if (!p || !out) return fail(nullptr, WRNN_ERR_INVALID_ARG, "null params or out");
    const int H = p->H;
    if (H < 8 || H % 8 != 0 || H > 65536 * 4 / 4) return fail(nullptr, WRNN_ERR_INVALID_ARG, "H must be a positive multiple of 8");
    if (H / 4 > 65535) return fail(nullptr, WRNN_ERR_UNSUPPORTED, "H too large for 16-bit block columns");
    if (max_batch < 1 || max_batch > 65536) return fail(nullptr, WRNN_ERR_INVALID_ARG, "max_batch out of range");
    if (p->cond_dim < 0 || p->cond_dim > 4096) return fail(nullptr, WRNN_ERR_INVALID_ARG, "cond_dim out of range");
    if (!p->R || !p->I || !p->O1 || !p->O2 || !p->O3 || !p->O4) return fail(nullptr, WRNN_ERR_INVALID_ARG, "missing weight matrix");
    if ((p->cond_dim > 0) != (p->W_cond != nullptr)) return fail(nullptr, WRNN_ERR_INVALID_ARG, "W_cond must be given iff cond_dim > 0");
    if (p->dtype != WRNN_F32 && p->dtype != WRNN_BF16) return fail(nullptr, WRNN_ERR_INVALID_ARG, "unknown dtype");
    if (p->kernel < WRNN_KERNEL_AUTO || p->kernel > WRNN_KERNEL_BCLUSTER) return fail(nullptr, WRNN_ERR_INVALID_ARG, "unknown kernel family");
    if (p->variant != 0 && p->variant != 1) return fail(nullptr, WRNN_ERR_INVALID_ARG, "unknown model variant");
    const bool fused = p->variant == 1;
    if (fused && (p->dtype != WRNN_BF16 || p->mask_R || p->mask_O1 || p->mask_O3 || max_batch != 1 ||
                  (p->kernel != WRNN_KERNEL_AUTO && p->kernel != WRNN_KERNEL_RESIDENT)))
        return fail(nullptr, WRNN_ERR_UNSUPPORTED, "the fused subscale variant runs dense, bf16, one stream, on the resident kernel");
    const int n_in = fused ? 12 : 3, n_logits = fused ? 64 : 256;
    const int mbr = p->mask_block_rows ? p->mask_block_rows : 4, mbc = p->mask_block_cols ? p->mask_block_cols : 4;
    if ((p->mask_block_rows == 0) != (p->mask_block_cols == 0) || mbr < 1 || mbc < 1 || (H / 2) % mbr != 0 || (H / 2) % mbc != 0)
        return fail(nullptr, WRNN_ERR_INVALID_ARG, "mask block shape must divide H/2 (0, 0 = 4 x 4)");

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return fail(nullptr, WRNN_ERR_CUDA, "no usable CUDA device"); }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return fail(nullptr, WRNN_ERR_CUDA, "cudaGetDeviceProperties failed");
    if (prop.major != 10) return fail(nullptr, WRNN_ERR_UNSUPPORTED, "this library is built for sm_100a (B200) only");

    wrnn_model *m = new (std::nothrow) wrnn_model();
    if (!m) return fail(nullptr, WRNN_ERR_NOMEM, "host allocation failed");
    m->H = H; m->cond_dim = p->cond_dim; m->dtype = p->dtype; m->kernel = p->kernel; m->max_batch = max_batch;
    m->variant = p->variant;
    m->device = dev; m->n_sms = prop.multiProcessorCount;
    m->sparse = p->mask_R || p->mask_O1 || p->mask_O3;
    m->mask_br = mbr; m->mask_bc = mbc;
    const bool bf = p->dtype == WRNN_BF16;
    const int Hh = H / 2, G = 3 * H;

    build_bsr(p->R, G, H, p->mask_R, mbr, mbc, bf, &m->hR);
    build_bsr(p->O1, Hh, Hh, p->mask_O1, mbr, mbc, bf, &m->hO1);
    build_bsr(p->O2, n_logits, Hh, nullptr, 4, 4, bf, &m->hO2);
    build_bsr(p->O3, Hh, Hh, p->mask_O3, mbr, mbc, bf, &m->hO3);
    build_bsr(p->O4, n_logits, Hh, nullptr, 4, 4, bf, &m->hO4);
    m->hI.resize((size_t)G * n_in);
    for (int row = 0; row < G; ++row)
        for (int c = 0; c < n_in; ++c) {
            float v = p->I[(size_t)row * n_in + c];
            if (c >= 2 * (n_in / 3) && (row % H) < Hh) v = 0.f;   // c_t (a_t) reaches only the fine half (part B): I*
            m->hI[(size_t)row * n_in + c] = bf ? round_bf16(v) : v;
        }
    auto copy_bias = [](const float *b, int n, std::vector<float> *dst) { dst->assign(n, 0.f); if (b) std::memcpy(dst->data(), b, n * sizeof(float)); };
    copy_bias(p->b_gate, G, &m->hb_gate);
    copy_bias(p->b1, Hh, &m->hb1); copy_bias(p->b2, n_logits, &m->hb2);
    copy_bias(p->b3, Hh, &m->hb3); copy_bias(p->b4, n_logits, &m->hb4);
    std::vector<float> WcT((size_t)p->cond_dim * G);
    for (int row = 0; row < G; ++row)
        for (int d = 0; d < p->cond_dim; ++d) {
            const float v = p->W_cond[(size_t)row * p->cond_dim + d];
            WcT[(size_t)d * G + row] = bf ? round_bf16(v) : v;
        }

    bool ok = upload_bsr(m->hR, bf, &m->R) && upload_bsr(m->hO1, bf, &m->O1) && upload_bsr(m->hO2, bf, &m->O2) &&
              upload_bsr(m->hO3, bf, &m->O3) && upload_bsr(m->hO4, bf, &m->O4) &&
              upload(&m->I, m->hI.data(), m->hI.size() * 4) && upload(&m->b_gate, m->hb_gate.data(), G * 4) &&
              upload(&m->b1, m->hb1.data(), Hh * 4) && upload(&m->b2, m->hb2.data(), n_logits * 4) &&
              upload(&m->b3, m->hb3.data(), Hh * 4) && upload(&m->b4, m->hb4.data(), n_logits * 4) &&
              upload(&m->W_condT, WcT.data(), WcT.size() * 4);
    const size_t B = (size_t)max_batch;
    ok = ok && cudaMalloc((void **)&m->hbuf[0], B * H * 4) == cudaSuccess &&
         cudaMalloc((void **)&m->hbuf[1], B * H * 4) == cudaSuccess &&
         cudaMalloc((void **)&m->a_fine, B * 3 * Hh * 4) == cudaSuccess &&
         cudaMalloc((void **)&m->q, B * Hh * 4) == cudaSuccess &&
         cudaMalloc((void **)&m->logits, B * 256 * 4) == cudaSuccess &&
         cudaMalloc((void **)&m->c_cur, B) == cudaSuccess && cudaMalloc((void **)&m->c_prev, B) == cudaSuccess &&
         cudaMalloc((void **)&m->f_prev, B) == cudaSuccess &&
         cudaMalloc((void **)&m->bar, 256) == cudaSuccess && cudaMalloc((void **)&m->status, sizeof(DevStatus)) == cudaSuccess;
    if (ok) ok = cudaMemset(m->status, 0, sizeof(DevStatus)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        wrnn_destroy(m);
        return fail(nullptr, WRNN_ERR_NOMEM, "device allocation or upload failed");
    }
    const int wsz = bf ? 2 : 4;
    auto bsr_bytes = [&](const BsrHost &h) { return (int64_t)h.vals.size() * wsz + (int64_t)h.col.size() * 2 + (int64_t)h.row_ptr.size() * 4; };
    m->weight_bytes = bsr_bytes(m->hR) + bsr_bytes(m->hO1) + bsr_bytes(m->hO2) + bsr_bytes(m->hO3) + bsr_bytes(m->hO4) +
                      (int64_t)G * 3 * 4;

    if (fused) {
        // one kernel serves this variant; without it the model cannot be stepped
        const int rc = resident_prepare(m);
        if (rc != WRNN_OK) {
            const std::string why = m->err;
            wrnn_destroy(m);
            return fail(nullptr, rc, "resident kernel unavailable: " + why);
        }
        reslean_prepare(m);     // optional: the lean form of the same kernel (the first form serves the variant without it)
        *out = m;
        return WRNN_OK;
    }
    if (p->kernel == WRNN_KERNEL_AUTO || p->kernel == WRNN_KERNEL_SPARSE) {
        const int rc = sparse_prepare(m);
        if (rc != WRNN_OK && p->kernel == WRNN_KERNEL_SPARSE) {
            const std::string why = m->err;
            wrnn_destroy(m);
            return fail(nullptr, rc, "sparse cluster kernel unavailable: " + why);
        }
    }
    if (p->kernel == WRNN_KERNEL_AUTO || p->kernel == WRNN_KERNEL_BCLUSTER) {
        const int rc = bcluster_prepare(m);
        if (rc != WRNN_OK && p->kernel == WRNN_KERNEL_BCLUSTER) {
            const std::string why = m->err;
            wrnn_destroy(m);
            return fail(nullptr, rc, "cluster-partitioned kernel unavailable: " + why);
        }
    }
    if (p->kernel == WRNN_KERNEL_AUTO || p->kernel == WRNN_KERNEL_BATCHED) {
        const int rc = batched_prepare(m);
        if (rc != WRNN_OK && p->kernel == WRNN_KERNEL_BATCHED) {
            const std::string why = m->err;
            wrnn_destroy(m);
            return fail(nullptr, rc, "batched kernel unavailable: " + why);
        }
    }
    if (p->kernel == WRNN_KERNEL_AUTO || p->kernel == WRNN_KERNEL_RESIDENT) {
        const int rc = m->dtype == WRNN_F32 ? resf32_prepare(m) : resident_prepare(m);
        if (rc != WRNN_OK && p->kernel == WRNN_KERNEL_RESIDENT) {
            const std::string why = m->err;
            wrnn_destroy(m);
            return fail(nullptr, rc, "resident kernel unavailable: " + why);
        }
        if (m->dtype == WRNN_BF16 && m->variant == 0) reslean_prepare(m);                        // optional: the row-split resident kernel serves the stream without it
        if (m->dtype == WRNN_BF16 && m->variant == 0 && max_batch >= 2) resmulti_prepare(m);   // optional: other kernels serve the batch without it
    }
    m->err.clear();             // reasons why optional kernels were not prepared are not errors of this call
    noalloc_warm(dev);
    *out = m;
    return WRNN_OK;
}

void wrnn_destroy(wrnn_model *m)
{
    if (!m) return;
    cudaSetDevice(m->device);
    cudaDeviceSynchronize();
    resident_destroy(m);
    reslean_destroy(m);
    resf32_destroy(m);
    resmulti_destroy(m);
    batched_destroy(m);
    bcluster_destroy(m);
    sparse_destroy(m);
    free_bsr(&m->R); free_bsr(&m->O1); free_bsr(&m->O2); free_bsr(&m->O3); free_bsr(&m->O4);
    cudaFree(m->I); cudaFree(m->b_gate); cudaFree(m->b1); cudaFree(m->b2); cudaFree(m->b3); cudaFree(m->b4);
    cudaFree(m->W_condT); cudaFree(m->g); cudaFree(m->hbuf[0]); cudaFree(m->hbuf[1]); cudaFree(m->a_fine);
    cudaFree(m->q); cudaFree(m->logits); cudaFree(m->c_cur); cudaFree(m->c_prev); cudaFree(m->f_prev);
    cudaFree(m->bar); cudaFree(m->status); cudaFree(m->stage_cond); cudaFree(m->stage_out); cudaFree(m->sub_scratch);
    cudaGetLastError();
    delete m;
}

int wrnn_sample(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, uint64_t seed,
                const wrnn_state *st, int16_t *out, void *cuda_stream)
{
    StepArgs a;
    int rc = check_step(m, cond, n_steps, batch, st, &a);
    if (rc != WRNN_OK) return rc;
    if (!out && n_steps > 0) return fail(m, WRNN_ERR_INVALID_ARG, "out is NULL");
    a.seed = seed; a.out = out;
    return run_steps(m, a, (cudaStream_t)cuda_stream);
}

int wrnn_step_teacher_forced(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, int32_t batch, uint64_t seed,
                             const wrnn_state *st, const uint8_t *c_forced, const uint8_t *f_forced, uint8_t *c_out,
                             uint8_t *f_out, float *dbg_gates, float *dbg_h, float *dbg_logits, void *cuda_stream)
{
    StepArgs a;
    int rc = check_step(m, cond, n_steps, batch, st, &a);
    if (rc != WRNN_OK) return rc;
    if ((!c_forced || !f_forced) && n_steps > 0) return fail(m, WRNN_ERR_INVALID_ARG, "forced sample arrays are NULL");
    a.seed = seed;
    a.c_forced = c_forced; a.f_forced = f_forced; a.c_out = c_out; a.f_out = f_out;
    a.dbg_gates = dbg_gates; a.dbg_h = dbg_h; a.dbg_logits = dbg_logits;
    return run_steps(m, a, (cudaStream_t)cuda_stream);
}

// Fused Subscale WaveRNN 2x: the same checks and launch path with the 16-bit state of the two parts.
static int fs2_args(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, const wrnn_fs2_state *st, StepArgs *a)
{
    int rc = check_step_any(m, cond, n_steps, 1, nullptr, a, true);
    if (rc != WRNN_OK) return rc;
    if (st) {
        if (st->step0 < 0) return fail(m, WRNN_ERR_INVALID_ARG, "step0 < 0");
        a->step0 = st->step0; a->stream0 = st->stream0;
        a->h_in = st->h; a->h_out = st->h;
        a->a_in = st->a_prev; a->a_st_out = st->a_prev;
        a->b_in = st->b_prev; a->b_st_out = st->b_prev;
        if (m->cond_dim > 0 && n_steps > 0) {
            const long long last = ((a->step0 + n_steps - 1) * (long long)a->row_stride + (long long)a->stream0 * a->row_offset_mul) / a->hop;
            if (last >= a->n_frames) return fail(m, WRNN_ERR_INVALID_ARG, "conditioning frames run out before n_steps");
        }
    }
    return WRNN_OK;
}

int wrnn_fs2_sample(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, uint64_t seed, const wrnn_fs2_state *st,
                    int16_t *out, void *cuda_stream)
{
    StepArgs a;
    int rc = fs2_args(m, cond, n_steps, st, &a);
    if (rc != WRNN_OK) return rc;
    if (!out && n_steps > 0) return fail(m, WRNN_ERR_INVALID_ARG, "out is NULL");
    a.seed = seed; a.out = out;
    return run_steps(m, a, (cudaStream_t)cuda_stream);
}

int wrnn_fs2_step_teacher_forced(wrnn_model *m, const wrnn_cond *cond, int64_t n_steps, uint64_t seed,
                                 const wrnn_fs2_state *st, const uint16_t *a_forced, const uint16_t *b_forced,
                                 uint16_t *a_out, uint16_t *b_out, float *dbg_gates, float *dbg_h, float *dbg_logits,
                                 void *cuda_stream)
{
    StepArgs a;
    int rc = fs2_args(m, cond, n_steps, st, &a);
    if (rc != WRNN_OK) return rc;
    if ((!a_forced || !b_forced) && n_steps > 0) return fail(m, WRNN_ERR_INVALID_ARG, "forced sample arrays are NULL");
    a.seed = seed;
    a.a_forced = a_forced; a.b_forced = b_forced; a.a_out = a_out; a.b_out = b_out;
    a.dbg_gates = dbg_gates; a.dbg_h = dbg_h; a.dbg_logits = dbg_logits;
    return run_steps(m, a, (cudaStream_t)cuda_stream);
}

int wrnn_fs2_unfold(const int16_t *ab, int64_t n_steps, int16_t *u, void *cuda_stream)
{
    if (n_steps < 0 || (n_steps > 2 && (!ab || !u))) return WRNN_ERR_INVALID_ARG;
    return fs2_unfold_launch(ab, n_steps, u, (cudaStream_t)cuda_stream);
}

int wrnn_fold(const int16_t *x, int64_t n_total, int32_t B, int16_t *sub, void *cuda_stream)
{
    if (B < 1 || n_total < 0 || n_total % B != 0 || (n_total > 0 && (!x || !sub))) return WRNN_ERR_INVALID_ARG;
    return fold_launch(x, n_total, B, sub, false, (cudaStream_t)cuda_stream);
}

int wrnn_unfold(const int16_t *sub, int64_t n_total, int32_t B, int16_t *x, void *cuda_stream)
{
    if (B < 1 || n_total < 0 || n_total % B != 0 || (n_total > 0 && (!x || !sub))) return WRNN_ERR_INVALID_ARG;
    return fold_launch(sub, n_total, B, x, true, (cudaStream_t)cuda_stream);
}

int wrnn_sample_subscale(wrnn_model *m, const float *cond, int32_t n_frames, int32_t hop, int64_t n_total, int32_t B,
                         uint64_t seed, int16_t *out, void *cuda_stream)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    if (B < 1 || n_total < 0 || n_total % B != 0) return fail(m, WRNN_ERR_INVALID_ARG, "B must divide n_total");
    if (n_total == 0) return WRNN_OK;
    if (!out) return fail(m, WRNN_ERR_INVALID_ARG, "out is NULL");
    const size_t need = (size_t)n_total;
    if (need > m->stage_out_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->stage_out); m->stage_out = nullptr; m->stage_out_cap = 0;
        if (cudaMalloc((void **)&m->stage_out, need * sizeof(int16_t)) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "staging allocation failed"); }
        m->stage_out_cap = need;
    }
    wrnn_cond c = {cond, n_frames, hop, B, 1};
    int rc = wrnn_sample(m, &c, n_total / B, B, seed, nullptr, m->stage_out, cuda_stream);
    if (rc != WRNN_OK) return rc;
    return fold_launch(m->stage_out, n_total, B, out, true, (cudaStream_t)cuda_stream);
}

int wrnn_subscale_schedule(int32_t B, int64_t L, int32_t chunk, int32_t lag, int64_t *calls, int32_t max_calls)
{
    if (B < 1 || L < 1 || chunk < 1 || lag < chunk || lag % chunk != 0 || max_calls < 0 || (max_calls > 0 && !calls)) return -WRNN_ERR_INVALID_ARG;
    std::vector<SubCall> v;
    subscale_schedule(B, L, chunk, lag, &v);
    for (size_t i = 0; i < v.size() && i < (size_t)max_calls; ++i) {
        calls[4 * i] = v[i].r_lo; calls[4 * i + 1] = v[i].n_rows; calls[4 * i + 2] = v[i].p_lo; calls[4 * i + 3] = v[i].n_steps;
    }
    return (int)v.size();
}

int wrnn_subscale_conditioning(const int16_t *hist, const float *frames, const float *V, const float *bias, int32_t B, int64_t L,
                               int32_t F, int32_t cond_dim, int32_t n_frames, int32_t hop, int32_t row, float *v, void *cuda_stream)
{
    if (!hist || !frames || !V || !bias || !v || B < 1 || L < 1 || F < 0 || cond_dim < 1 || hop < 1 || row < 0 || row >= B || L > (1ll << 30))
        return WRNN_ERR_INVALID_ARG;
    if (((long long)B * (L - 1) + row) / hop >= n_frames) return WRNN_ERR_INVALID_ARG;
    return subscale_cond_launch(hist, frames, V, bias, v, B, L, F, cond_dim, n_frames, hop, row, 1, 0, 0, (int)L, (cudaStream_t)cuda_stream);
}

}  // extern "C"

namespace wrnn {
// Subscale generation with dependent rows on the staggered schedule, whatever the conditioning network: `cond_rows`
// computes the conditioning vectors v[n_rows][n][D] of one stepping call (rows r_a .. r_a + n_rows - 1, row b of the call
// from position p_lo - b * lag on) from the sample history hist [B][L].
template <typename CondFn>
static int subscale_dependent_impl(wrnn_model *m, int32_t n_frames, int32_t hop, int32_t F, int32_t chunk, int32_t lag, int64_t n_total, int32_t B,
                                   uint64_t seed, int16_t *out, cudaStream_t s, CondFn cond_rows)
{
    if (m->variant != 0) return fail(m, WRNN_ERR_UNSUPPORTED, "subscale generation takes a WaveRNN model (variant 0)");
    if (m->cond_dim <= 0) return fail(m, WRNN_ERR_INVALID_ARG, "the model must be conditioned");
    if (B < 1 || B > m->max_batch || n_total < 0 || n_total % B != 0) return fail(m, WRNN_ERR_INVALID_ARG, "B must divide n_total and fit max_batch");
    if (n_total == 0) return WRNN_OK;
    if (!out || hop < 1 || F < 0 || chunk < 1) return fail(m, WRNN_ERR_INVALID_ARG, "bad arguments");
    // row r + 1 may use positions of row r up to F ahead of its own, for a whole chunk at a time: it follows F + chunk
    // steps (or more) behind; chunks of all rows line up when the lag is a multiple of the chunk
    if (lag < F + chunk || lag % chunk != 0) return fail(m, WRNN_ERR_INVALID_ARG, "lag must be a multiple of chunk and at least F + chunk");
    const long long L = n_total / B;
    if (((long long)B * (L - 1) + (B - 1)) / hop >= n_frames) return fail(m, WRNN_ERR_INVALID_ARG, "conditioning frames run out");
    if (cudaSetDevice(m->device) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, "cudaSetDevice failed");
    const int D = m->cond_dim, H = m->H;
    // scratch: sample history [B][L], per-call conditioning [B][chunk][D], carry state
    const size_t need = (size_t)B * L * sizeof(int16_t) + (size_t)B * chunk * D * sizeof(float) + (size_t)B * H * sizeof(float) + 2 * (size_t)B + 64;
    if (need > m->sub_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->sub_scratch); m->sub_scratch = nullptr; m->sub_cap = 0;
        if (cudaMalloc((void **)&m->sub_scratch, need) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "scratch allocation failed"); }
        m->sub_cap = need;
    }
    float *v = reinterpret_cast<float *>(m->sub_scratch);
    float *hst = v + (size_t)B * chunk * D;
    int16_t *hist = reinterpret_cast<int16_t *>(hst + (size_t)B * H);
    uint8_t *cp = reinterpret_cast<uint8_t *>(hist + (size_t)B * L);
    uint8_t *fp = cp + B;
    if (cudaMemsetAsync(hst, 0, (size_t)B * H * sizeof(float), s) != cudaSuccess || cudaMemsetAsync(cp, 128, B, s) != cudaSuccess ||
        cudaMemsetAsync(fp, 0, B, s) != cudaSuccess || cudaMemsetAsync(hist, 0, (size_t)B * L * sizeof(int16_t), s) != cudaSuccess)
        return fail(m, WRNN_ERR_CUDA, "scratch initialisation failed");

    auto run_rows = [&](int r_a, int n_rows, long long p_lo, int n) -> int {
        int rc = cond_rows(hist, v, L, r_a, n_rows, p_lo, n);
        if (rc != WRNN_OK) return fail(m, rc, "conditioning launch failed");
        // rows advance together on the multi-stream resident kernel where the model has one; without it up to three rows go
        // one after the other through the single-stream kernel
        const int group = (n_rows >= 2 && use_multi(m, n_rows)) ? n_rows : (n_rows <= 3 && (use_reslean(m, 1) || use_resident(m, 1))) ? 1 : n_rows;
        for (int b0 = 0; b0 < n_rows; b0 += group) {
            const int r0 = r_a + b0;
            const long long p0 = p_lo - (long long)b0 * lag;
            StepArgs a;
            std::memset(&a, 0, sizeof(a));
            a.cond = v + (size_t)b0 * n * D; a.n_frames = n; a.hop = 1; a.row_stride = 1; a.row_offset_mul = 0;
            a.n_steps = n; a.batch = group; a.seed = seed; a.step0 = p0; a.stream0 = (unsigned)r0;
            a.h_in = a.h_out = hst + (size_t)r0 * H;
            a.c_in = a.c_st_out = cp + r0; a.f_in = a.f_st_out = fp + r0;
            a.out = hist + (size_t)r0 * L + p0;
            a.row_lag = lag; a.out_pitch = L - lag;
            rc = run_steps(m, a, s);
            if (rc != WRNN_OK) return rc;
        }
        return WRNN_OK;
    };
    std::vector<SubCall> calls;
    subscale_schedule(B, L, chunk, lag, &calls);
    for (const SubCall &c : calls) {
        const int rc = run_rows(c.r_lo, c.n_rows, c.p_lo, c.n_steps);
        if (rc != WRNN_OK) return rc;
    }
    return fold_launch(hist, n_total, B, out, true, s);
}
}  // namespace wrnn

extern "C" {

int wrnn_sample_subscale_dependent(wrnn_model *m, const float *frames, int32_t n_frames, int32_t hop, const float *V, const float *bias,
                                   int32_t F, int32_t chunk, int32_t lag, int64_t n_total, int32_t B, uint64_t seed, int16_t *out,
                                   void *cuda_stream)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    if (n_total > 0 && (!frames || !V || !bias)) return fail(m, WRNN_ERR_INVALID_ARG, "bad arguments");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int D = m->cond_dim;
    return subscale_dependent_impl(m, n_frames, hop, F, chunk, lag, n_total, B, seed, out, s,
                                   [&](const int16_t *hist, float *v, long long L, int r_a, int n_rows, long long p_lo, int n) {
                                       return subscale_cond_launch(hist, frames, V, bias, v, B, L, F, D, n_frames, hop, r_a, n_rows, p_lo, lag, n, s);
                                   });
}

int wrnn_sample_subscale_net(wrnn_model *m, wrnn_subscale_net *net, const float *frames, int32_t n_frames, int32_t hop, int32_t F, int32_t chunk,
                             int32_t lag, int64_t n_total, uint64_t seed, int16_t *out, void *cuda_stream)
{
    if (!m || !net) return WRNN_ERR_INVALID_ARG;
    if (n_total > 0 && !frames) return fail(m, WRNN_ERR_INVALID_ARG, "bad arguments");
    if (subnet_cond_dim(net) != m->cond_dim) return fail(m, WRNN_ERR_INVALID_ARG, "the network's output does not match the model's conditioning size");
    if (F < subnet_reach(net)) return fail(m, WRNN_ERR_INVALID_ARG, "the future horizon F is shorter than the reach of the network");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int B = subnet_B(net);
    return subscale_dependent_impl(m, n_frames, hop, F, chunk, lag, n_total, B, seed, out, s,
                                   [&](const int16_t *hist, float *v, long long L, int r_a, int n_rows, long long p_lo, int n) {
                                       return subnet_run(net, hist, frames, n_frames, hop, L, r_a, n_rows, p_lo, lag, n, v, m->wait_limit_ns(), s);
                                   });
}

int wrnn_subscale_net_rows(wrnn_model *m, wrnn_subscale_net *net, const float *frames, int32_t n_frames, int32_t hop, int32_t lag, int16_t *hist,
                           int64_t L, float *h, uint8_t *c_prev, uint8_t *f_prev, int32_t r_lo, int32_t n_rows, int64_t p_lo, int32_t n_steps,
                           uint64_t seed, void *cuda_stream)
{
    if (!m || !net) return WRNN_ERR_INVALID_ARG;
    if (m->variant != 0) return fail(m, WRNN_ERR_UNSUPPORTED, "subscale generation takes a WaveRNN model (variant 0)");
    const int B = subnet_B(net), D = m->cond_dim, H = m->H;
    if (subnet_cond_dim(net) != D || D <= 0) return fail(m, WRNN_ERR_INVALID_ARG, "the network's output does not match the model's conditioning size");
    if (!frames || !hist || !h || !c_prev || !f_prev || hop < 1 || L < 1 || r_lo < 0 || n_rows < 1 || r_lo + n_rows > B || n_rows > m->max_batch ||
        n_steps < 1 || lag < 1)
        return fail(m, WRNN_ERR_INVALID_ARG, "bad arguments");
    // every row of the call stays inside its sub-tensor, and its frames exist
    const long long p_last_row = p_lo - (long long)(n_rows - 1) * lag;
    if (p_last_row < 0 || p_lo + n_steps > L) return fail(m, WRNN_ERR_INVALID_ARG, "positions outside the sub-tensors");
    if (((long long)B * (p_lo + n_steps - 1) + (B - 1)) / hop >= n_frames) return fail(m, WRNN_ERR_INVALID_ARG, "conditioning frames run out");
    if (cudaSetDevice(m->device) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, "cudaSetDevice failed");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t need = (size_t)n_rows * n_steps * D * sizeof(float);
    if (need > m->sub_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->sub_scratch); m->sub_scratch = nullptr; m->sub_cap = 0;
        if (cudaMalloc((void **)&m->sub_scratch, need) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "scratch allocation failed"); }
        m->sub_cap = need;
    }
    float *v = reinterpret_cast<float *>(m->sub_scratch);
    int rc = subnet_run(net, hist, frames, n_frames, hop, L, r_lo, n_rows, p_lo, lag, n_steps, v, m->wait_limit_ns(), s);
    if (rc != WRNN_OK) return fail(m, rc, "conditioning launch failed");
    const int group = (n_rows >= 2 && use_multi(m, n_rows)) ? n_rows : (n_rows <= 3 && (use_reslean(m, 1) || use_resident(m, 1))) ? 1 : n_rows;
    for (int b0 = 0; b0 < n_rows; b0 += group) {
        const int r0 = r_lo + b0;
        const long long p0 = p_lo - (long long)b0 * lag;
        StepArgs a;
        std::memset(&a, 0, sizeof(a));
        a.cond = v + (size_t)b0 * n_steps * D; a.n_frames = n_steps; a.hop = 1; a.row_stride = 1; a.row_offset_mul = 0;
        a.n_steps = n_steps; a.batch = group; a.seed = seed; a.step0 = p0; a.stream0 = (unsigned)r0;
        a.h_in = a.h_out = h + (size_t)r0 * H;
        a.c_in = a.c_st_out = c_prev + r0; a.f_in = a.f_st_out = f_prev + r0;
        a.out = hist + (size_t)r0 * L + p0;
        a.row_lag = lag; a.out_pitch = L - lag;
        rc = run_steps(m, a, s);
        if (rc != WRNN_OK) return rc;
    }
    return WRNN_OK;
}

int wrnn_sample_host(wrnn_model *m, const float *cond_host, int32_t n_frames, int32_t hop, int32_t row_stride,
                     int32_t row_offset_mul, int64_t n_steps, int32_t batch, uint64_t seed, int16_t *out_host)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    if (batch < 1 || n_steps < 0 || n_frames < 0) return fail(m, WRNN_ERR_INVALID_ARG, "bad sizes");
    if (cudaSetDevice(m->device) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, "cudaSetDevice failed");
    const size_t nc = m->cond_dim ? (size_t)batch * n_frames * m->cond_dim : 0;
    const size_t no = (size_t)batch * (size_t)n_steps;
    if (nc > m->stage_cond_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->stage_cond); m->stage_cond = nullptr; m->stage_cond_cap = 0;
        if (cudaMalloc((void **)&m->stage_cond, nc * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "staging allocation failed"); }
        m->stage_cond_cap = nc;
    }
    // the subscale path shares stage_out; size for either use
    if (no > m->stage_out_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->stage_out); m->stage_out = nullptr; m->stage_out_cap = 0;
        if (cudaMalloc((void **)&m->stage_out, no * sizeof(int16_t)) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "staging allocation failed"); }
        m->stage_out_cap = no;
    }
    if (nc && (!cond_host || cudaMemcpyAsync(m->stage_cond, cond_host, nc * sizeof(float), cudaMemcpyHostToDevice, 0) != cudaSuccess))
        return fail(m, WRNN_ERR_CUDA, "cond upload failed");
    wrnn_cond c = {m->stage_cond, n_frames, hop, row_stride, row_offset_mul};
    int rc = wrnn_sample(m, m->cond_dim ? &c : nullptr, n_steps, batch, seed, nullptr, m->stage_out, nullptr);
    if (rc != WRNN_OK) return rc;
    if (no && cudaMemcpyAsync(out_host, m->stage_out, no * sizeof(int16_t), cudaMemcpyDeviceToHost, 0) != cudaSuccess)
        return fail(m, WRNN_ERR_CUDA, "sample download failed");
    if (cudaStreamSynchronize(0) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, cudaGetErrorString(cudaGetLastError()));
    return wrnn_poll_status(m);
}

int wrnn_fs2_sample_host(wrnn_model *m, const float *cond_host, int32_t n_frames, int32_t hop, int64_t n_steps, uint64_t seed,
                         int16_t *u_host)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    if (m->variant != 1) return fail(m, WRNN_ERR_UNSUPPORTED, "not a fused subscale model (create with variant = 1)");
    if (n_steps < 0 || n_frames < 0) return fail(m, WRNN_ERR_INVALID_ARG, "bad sizes");
    if (cudaSetDevice(m->device) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, "cudaSetDevice failed");
    const size_t nc = m->cond_dim ? (size_t)n_frames * m->cond_dim : 0;
    const size_t nu = n_steps > 2 ? 2 * (size_t)(n_steps - 2) : 0;
    const size_t no = 2 * (size_t)n_steps + nu;                 // the two streams, then the interleaved samples
    if (nc > m->stage_cond_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->stage_cond); m->stage_cond = nullptr; m->stage_cond_cap = 0;
        if (cudaMalloc((void **)&m->stage_cond, nc * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "staging allocation failed"); }
        m->stage_cond_cap = nc;
    }
    if (no > m->stage_out_cap) {
        cudaDeviceSynchronize();
        cudaFree(m->stage_out); m->stage_out = nullptr; m->stage_out_cap = 0;
        if (cudaMalloc((void **)&m->stage_out, no * sizeof(int16_t)) != cudaSuccess) { cudaGetLastError(); return fail(m, WRNN_ERR_NOMEM, "staging allocation failed"); }
        m->stage_out_cap = no;
    }
    if (nc && (!cond_host || cudaMemcpyAsync(m->stage_cond, cond_host, nc * sizeof(float), cudaMemcpyHostToDevice, 0) != cudaSuccess))
        return fail(m, WRNN_ERR_CUDA, "cond upload failed");
    wrnn_cond c = {m->stage_cond, n_frames, hop, 1, 0};
    int rc = wrnn_fs2_sample(m, m->cond_dim ? &c : nullptr, n_steps, seed, nullptr, m->stage_out, nullptr);
    if (rc != WRNN_OK) return rc;
    int16_t *u = m->stage_out + 2 * (size_t)n_steps;
    rc = fs2_unfold_launch(m->stage_out, n_steps, u, 0);
    if (rc != WRNN_OK) return fail(m, rc, "unfold launch failed");
    if (nu && (!u_host || cudaMemcpyAsync(u_host, u, nu * sizeof(int16_t), cudaMemcpyDeviceToHost, 0) != cudaSuccess))
        return fail(m, WRNN_ERR_CUDA, "sample download failed");
    if (cudaStreamSynchronize(0) != cudaSuccess) return fail(m, WRNN_ERR_CUDA, cudaGetErrorString(cudaGetLastError()));
    return wrnn_poll_status(m);
}

int wrnn_poll_status(wrnn_model *m)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    DevStatus st;
    if (cudaMemcpy(&st, m->status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(m, WRNN_ERR_CUDA, std::string("status read failed: ") + cudaGetErrorString(cudaGetLastError()));
    if (st.code != DEV_OK) {
        char buf[200];
        if (st.code == DEV_CHECK) {
            std::snprintf(buf, sizeof(buf), "checked build: cta %d found %s (region %d)", st.cta,
                          st.step == -1 ? "an exchange slot outside the slot array" : st.step == -2 ? "a shared-memory carve-up that disagrees with the allocation"
                                                                                                      : "a clobbered guard behind a shared-memory region", st.step);
            m->err = buf;
            return WRNN_ERR_CHECK;
        }
        std::snprintf(buf, sizeof(buf), "device-side wait timed out (code %d) at cta %d, step %d, phase %d", st.code, st.cta, st.step, st.phase);
        m->err = buf;
        return st.code == DEV_TIMEOUT ? WRNN_ERR_TIMEOUT : WRNN_ERR_CUDA;
    }
    return WRNN_OK;
}

const char *wrnn_last_error(wrnn_model *m) { return m ? m->err.c_str() : g_create_err.c_str(); }

int wrnn_launch_info(wrnn_model *m, int32_t batch, int32_t *kernel, int32_t *n_ctas, int32_t *n_threads,
                     int64_t *weight_bytes_per_step, int32_t *smem_bytes)
{
    if (!m || batch < 1 || batch > m->max_batch) return WRNN_ERR_INVALID_ARG;
    if (use_reslean(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_RESIDENT;
        return reslean_launch_info(m, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_resident(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_RESIDENT;
        return resident_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_multi(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_RESIDENT;
        return resmulti_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_pair(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_RESIDENT;
        return resident_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_resf32(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_RESIDENT;
        return resf32_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_sparse(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_SPARSE;
        return sparse_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_bcluster(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_BCLUSTER;
        return bcluster_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (use_batched(m, batch)) {
        if (kernel) *kernel = WRNN_KERNEL_BATCHED;
        return batched_launch_info(m, batch, n_ctas, n_threads, smem_bytes, weight_bytes_per_step);
    }
    if (kernel) *kernel = WRNN_KERNEL_GENERIC;
    if (weight_bytes_per_step) *weight_bytes_per_step = m->weight_bytes;
    return generic_launch_info(m, batch, n_ctas, n_threads, smem_bytes);
}

int64_t wrnn_launch_count(void) { return g_launches.load(); }

int wrnn_selftest_lost_word(wrnn_model *m, int64_t limit_ns, int32_t cta, int64_t step)
{
    if (!m || limit_ns < 0 || limit_ns > 2000000000ll || cta < -1 || step < -1) return WRNN_ERR_INVALID_ARG;
    m->dbg_limit_ns = (unsigned long long)limit_ns;
    m->dbg_skip_cta = cta;
    m->dbg_skip_step = cta < 0 ? -1 : step;
    return WRNN_OK;
}

int wrnn_phase_profile(wrnn_model *m, int32_t enable)
{
    if (!m) return WRNN_ERR_INVALID_ARG;
    m->prof_enabled = enable != 0;
    return WRNN_OK;
}

int wrnn_phase_names(wrnn_model *m, char *buf, int32_t cap)
{
    if (!m || !buf || cap < 1) return WRNN_ERR_INVALID_ARG;
    const char *first = "F.wait_y,F.hid_finish_send,F.wait_q,F.log_finish_send,F.wait_logits,F.draw_gates,"
                        "C.wait_y,C.hid_finish_send,C.wait_q,C.log_finish_send,C.wait_logits,C.draw_gates,"
                        "F.hid_products,C.hid_products,F.log_products,C.log_products";
    const char *multi = "F.wait_y,F.hid_finish_send,F.wait_q,F.log_finish_send,F.wait_logits,F.draw_wait_recurrent,"
                        "C.wait_y,C.hid_finish_send,C.wait_q,C.log_finish_send,C.wait_logits,C.draw_wait_recurrent,"
                        "F.hid_products,C.hid_products,F.log_products,C.log_products";
    const char *lean = "F.wait_y,F.hid_products,F.hid_sums_send,F.recurrent_products,F.rsums_gateprep,F.wait_logit_rows_send,F.wait_logits,F.draw_gates,"
                       "C.wait_y,C.hid_products,C.hid_sums_send,C.recurrent_products,C.rsums_gateprep,C.wait_logit_rows_send,C.wait_logits,C.draw_gates";
    const char *src = (!m->resf32 && m->prof_multi) ? multi : (!m->resf32 && m->prof_lean) ? lean : first;
    std::snprintf(buf, (size_t)cap, "%s", src);
    return WRNN_OK;
}

int wrnn_phase_cycles(wrnn_model *m, int64_t *out16)
{
    if (!m || !out16) return WRNN_ERR_INVALID_ARG;
    static_assert(sizeof(long long) == sizeof(int64_t), "");
    if (m->resf32) return resf32_phase_cycles(m, reinterpret_cast<long long *>(out16));
    if (m->prof_multi) return resmulti_phase_cycles(m, reinterpret_cast<long long *>(out16));
    if (m->prof_lean) return reslean_phase_cycles(m, reinterpret_cast<long long *>(out16));
    return resident_phase_cycles(m, reinterpret_cast<long long *>(out16));
}

}  // extern "C"
