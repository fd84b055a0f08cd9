// C ABI of libmmasim: argument validation, model objects, dispatch to the kernels.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include "mmasim_internal.h"

namespace mmasim {

static thread_local char g_error[512] = "";
static thread_local char g_kernel[64] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
}
void set_kernel_name(const char* name) { snprintf(g_kernel, sizeof(g_kernel), "%s", name); }

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// MMASIM_OK if p is device-accessible memory; ERR_INVALID_ARG for plain host memory; ERR_CUDA otherwise.
int check_device_ptr(const void* p, const char* name) {
    cudaPointerAttributes attr;
    const cudaError_t err = cudaPointerGetAttributes(&attr, p);
    if (err != cudaSuccess) {
        cudaGetLastError();
        set_error("cudaPointerGetAttributes(%s) failed: %s", name, cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    if (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) return MMASIM_OK;
    set_error("%s is not a device pointer", name);
    return MMASIM_ERR_INVALID_ARG;
}

// Shape rules shared by gemm and dot_batch.  Returns MMASIM_OK or an error status.
int check_k(const DevModel& m, int64_t K) {
    if (K < 1) { set_error("K must be >= 1"); return MMASIM_ERR_SHAPE; }
    if (m.family == FAM_FMA) return MMASIM_OK;
    if (m.family == FAM_FTZ) {
        if (K % m.P) { set_error("K = %lld is not a multiple of P = %d", (long long)K, m.P); return MMASIM_ERR_SHAPE; }
        return MMASIM_OK;
    }
    const int64_t L = K < m.L ? K : m.L;
    if (K % L) {
        set_error("K = %lld is not a multiple of L = min(K, L_max) = %lld", (long long)K, (long long)L);
        return MMASIM_ERR_SHAPE;
    }
    if (m.family == FAM_GST && (L % 32)) { set_error("GST-FDPA models need K to be a multiple of 32"); return MMASIM_ERR_SHAPE; }
    if (m.family == FAM_GTR && (L % 2)) { set_error("GTR-FDPA models need an even K"); return MMASIM_ERR_SHAPE; }
    if (m.family == FAM_ST && K > 32 && (K % 32)) { set_error("ST-FDPA models need K to be a multiple of 32"); return MMASIM_ERR_SHAPE; }
    return MMASIM_OK;
}

int run_gemm(const mmasim_model* model, const GemmArgs& g, int flags, cudaStream_t stream) {
    const DevModel& m = model->dev;
    if (!(flags & MMASIM_GEMM_FORCE_GENERIC) && !m.literal_emax) {
        if (fast_tfdpa_supported(m, g)) return launch_fast_tfdpa(m, g, stream);
        if (fast_fp_supported(m, g)) return launch_fast_fp(m, g, stream);
        if (fast_gst_supported(m, g)) return launch_fast_gst(m, g, stream);
    }
    set_kernel_name("generic");
    return launch_generic(m, g, stream);
}

int build_args(const mmasim_model* model, int64_t M, int64_t N, int64_t K, const void* A, const void* B,
               const void* C, void* D, const mmasim_gemm_opts* opts, GemmArgs* out) {
    if (!model) { set_error("model is NULL"); return MMASIM_ERR_INVALID_ARG; }
    if (!A || !B || !D) { set_error("A, B and D must not be NULL"); return MMASIM_ERR_INVALID_ARG; }
    if (M < 1 || N < 1) { set_error("M and N must be >= 1"); return MMASIM_ERR_SHAPE; }
    const DevModel& m = model->dev;
    int st = check_k(m, K);
    if (st != MMASIM_OK) return st;
    GemmArgs g;
    std::memset(&g, 0, sizeof(g));
    g.M = M; g.N = N; g.K = K;
    g.A = A; g.B = B; g.C = C; g.D = D;
    g.lda = g.ldb = K;
    g.ldc = g.ldd = N;
    g.copy_timeouts = copy_timeout_counter();
    if (m.k_block) g.ld_sfa = g.ld_sfb = (K + m.k_block - 1) / m.k_block;
    if (opts) {
        if (opts->lda) g.lda = opts->lda;
        if (opts->ldb) g.ldb = opts->ldb;
        if (opts->ldc) g.ldc = opts->ldc;
        if (opts->ldd) g.ldd = opts->ldd;
        g.sfa = static_cast<const uint8_t*>(opts->sfa);
        g.sfb = static_cast<const uint8_t*>(opts->sfb);
        g.k_chunk = opts->k_chunk;
        g.row_scale = opts->row_scale;
        g.col_scale = opts->col_scale;
    }
    if (g.lda < K || g.ldb < K || g.ldc < N || g.ldd < N) { set_error("leading dimension smaller than the row length"); return MMASIM_ERR_SHAPE; }
    if (m.packed4 && ((g.lda | g.ldb | K) & 1)) { set_error("packed FP4 operands need even K and leading dimensions"); return MMASIM_ERR_SHAPE; }
    if (m.k_block && (!g.sfa || !g.sfb)) { set_error("this model needs scale factors (opts->sfa, opts->sfb)"); return MMASIM_ERR_INVALID_ARG; }
    if (!m.k_block && (g.sfa || g.sfb)) { set_error("this model takes no scale factors"); return MMASIM_ERR_INVALID_ARG; }
    const bool fdpa32 = m.family != FAM_FMA && m.family != FAM_FTZ && m.acc == ACC_F32;
    if (g.k_chunk) {
        if (!fdpa32) { set_error("k_chunk needs an FDPA model with an FP32 accumulator"); return MMASIM_ERR_UNSUPPORTED; }
        const int64_t L = K < m.L ? K : m.L;
        if (g.k_chunk < 0 || g.k_chunk % L || K % g.k_chunk) { set_error("k_chunk must be a multiple of L that divides K"); return MMASIM_ERR_SHAPE; }
    }
    if ((g.row_scale != nullptr) != (g.col_scale != nullptr)) { set_error("row_scale and col_scale must be given together"); return MMASIM_ERR_INVALID_ARG; }
    if (g.row_scale && !fdpa32) { set_error("dequantisation scales need an FDPA model with an FP32 accumulator"); return MMASIM_ERR_UNSUPPORTED; }
    *out = g;
    return MMASIM_OK;
}

}  // namespace

namespace {
// Device memory the library takes for itself (the staging buffers of mmasim_gemm_host, the decoded operand blocks of
// the tuned kernels): one memory pool per device, the library's own (the device's default pool and its attributes are
// the caller's and stay untouched), created on first use, keeping up to 1 GiB between calls.
constexpr int MAX_DEVICES = 64;
std::mutex g_pool_mutex;
cudaMemPool_t g_pools[MAX_DEVICES] = {};

}  // namespace

cudaError_t scratch_pool(cudaMemPool_t* out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    if (!g_pools[dev]) {
        cudaMemPoolProps props;
        std::memset(&props, 0, sizeof(props));
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t pool = nullptr;
        err = cudaMemPoolCreate(&pool, &props);
        if (err != cudaSuccess) return err;
        unsigned long long keep = 1ull << 30;
        err = cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        if (err != cudaSuccess) { cudaMemPoolDestroy(pool); return err; }
        g_pools[dev] = pool;
    }
    *out = g_pools[dev];
    return cudaSuccess;
}


}  // namespace mmasim

using namespace mmasim;

extern "C" {

mmasim_model* mmasim_create_model_ex(int arch, int a_fmt, int b_fmt, int acc_fmt, const mmasim_overrides* ov) {
    mmasim_model tmp;
    const char* why = "";
    if (!registry_lookup(arch, a_fmt, b_fmt, acc_fmt, &tmp, &why)) {
        set_error("mmasim_create_model: %s (arch %d, input %d x %d, accumulator %d)", why, arch, a_fmt, b_fmt, acc_fmt);
        return nullptr;
    }
    if (ov) {
        DevModel& d = tmp.dev;
        const bool fdpa = d.family == FAM_T || d.family == FAM_ST || d.family == FAM_TR || d.family == FAM_GTR;
        if ((ov->l_max >= 0 || ov->F >= 0 || ov->F2 >= 0 || ov->rho >= 0 || ov->inner_round >= 0) && !fdpa) {
            set_error("overrides apply to T-, ST-, TR- and GTR-FDPA models only");
            return nullptr;
        }
        if (ov->l_max >= 0) {
            if (ov->l_max < 1 || ov->l_max > 64 || (d.family == FAM_GTR && (ov->l_max & 1)) || (d.family == FAM_ST && ov->l_max != 32)) {
                set_error("l_max override out of range"); return nullptr;
            }
            d.L = ov->l_max;
        }
        if (ov->F >= 0) { if (ov->F > 30 || ov->F < 1) { set_error("F override must be in 1..30"); return nullptr; } d.F = ov->F; }
        if (ov->F2 >= 0) { if (d.F2 == 0 || ov->F2 > 36) { set_error("F2 override not applicable"); return nullptr; } d.F2 = ov->F2; }
        if (d.F2 && d.F2 < d.F) { set_error("F2 must be >= F"); return nullptr; }
        if (ov->rho >= 0) {
            const bool fp16 = d.acc == ACC_F16;
            const bool ok = fp16 ? ov->rho == MMASIM_RNE_FP16 : (ov->rho >= MMASIM_RZ_FP32 && ov->rho <= MMASIM_RNE_FP32);
            if (!ok) { set_error("rho override does not match the accumulator type"); return nullptr; }
            d.rho = ov->rho;
        }
        if (ov->inner_round >= 0) {
            if (ov->inner_round > 1 || d.family != FAM_TR) { set_error("inner_round applies to TR-FDPA models only"); return nullptr; }
            d.inner_round = ov->inner_round;
        }
        if (ov->literal_emax > 0) {
            if (!fdpa && d.family != FAM_GST) { set_error("literal_emax applies to T-, ST-, GST-, TR- and GTR-FDPA models only"); return nullptr; }
            d.literal_emax = 1;
        }
        tmp.info.l_max = d.L; tmp.info.F = d.F; tmp.info.F2 = d.F2; tmp.info.rho = d.rho; tmp.info.inner_round = d.inner_round;
    }
    mmasim_model* m = new (std::nothrow) mmasim_model(tmp);
    if (!m) set_error("out of host memory");
    return m;
}

mmasim_model* mmasim_create_model(int arch, int in_fmt, int acc_fmt) {
    return mmasim_create_model_ex(arch, in_fmt, in_fmt, acc_fmt, nullptr);
}

void mmasim_destroy_model(mmasim_model* model) { delete model; }

int mmasim_model_info(const mmasim_model* model, mmasim_info* out) {
    if (!model || !out) { set_error("mmasim_model_info: NULL argument"); return MMASIM_ERR_INVALID_ARG; }
    *out = model->info;
    return MMASIM_OK;
}

int mmasim_gemm_ex(const mmasim_model* model, int64_t M, int64_t N, int64_t K, const void* A, const void* B,
                   const void* C, void* D, const mmasim_gemm_opts* opts, void* stream) {
    GemmArgs g;
    int st = build_args(model, M, N, K, A, B, C, D, opts, &g);
    if (st != MMASIM_OK) return st;
    if (!aligned16(A) || !aligned16(B) || !aligned16(D) || (C && !aligned16(C))) {
        set_error("A, B, C and D must be 16-byte aligned");
        return MMASIM_ERR_ALIGN;
    }
    if ((st = check_device_ptr(A, "A")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(B, "B")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if (C && (st = check_device_ptr(C, "C")) != MMASIM_OK) return st;
    if (g.sfa && (st = check_device_ptr(g.sfa, "opts->sfa")) != MMASIM_OK) return st;
    if (g.sfb && (st = check_device_ptr(g.sfb, "opts->sfb")) != MMASIM_OK) return st;
    if (g.row_scale && (st = check_device_ptr(g.row_scale, "opts->row_scale")) != MMASIM_OK) return st;
    if (g.col_scale && (st = check_device_ptr(g.col_scale, "opts->col_scale")) != MMASIM_OK) return st;
    return run_gemm(model, g, opts ? opts->flags : 0, static_cast<cudaStream_t>(stream));
}

int mmasim_gemm_noalloc(const mmasim_model* model, int64_t M, int64_t N, int64_t K, const void* A, const void* B,
                        const void* C, void* D, const mmasim_gemm_opts* opts, void* stream) {
    GemmArgs g;
    int st = build_args(model, M, N, K, A, B, C, D, opts, &g);
    if (st != MMASIM_OK) return st;
    if (!aligned16(A) || !aligned16(B) || !aligned16(D) || (C && !aligned16(C))) {
        set_error("A, B, C and D must be 16-byte aligned");
        return MMASIM_ERR_ALIGN;
    }
    if ((st = check_device_ptr(A, "A")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(B, "B")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if (C && (st = check_device_ptr(C, "C")) != MMASIM_OK) return st;
    if (g.row_scale && (st = check_device_ptr(g.row_scale, "opts->row_scale")) != MMASIM_OK) return st;
    if (g.col_scale && (st = check_device_ptr(g.col_scale, "opts->col_scale")) != MMASIM_OK) return st;
    return launch_gemm_noalloc(model->dev, g, static_cast<cudaStream_t>(stream));
}

int mmasim_gemm(const mmasim_model* model, int64_t M, int64_t N, int64_t K, const void* A, const void* B,
                const void* C, void* D, void* stream) {
    return mmasim_gemm_ex(model, M, N, K, A, B, C, D, nullptr, stream);
}

int mmasim_dot_batch(const mmasim_model* model, int64_t n, int64_t K, const void* A, const void* B,
                     const void* C, void* D, void* stream) {
    if (!model) { set_error("model is NULL"); return MMASIM_ERR_INVALID_ARG; }
    if (!A || !B || !D) { set_error("A, B and D must not be NULL"); return MMASIM_ERR_INVALID_ARG; }
    if (n < 1) { set_error("n must be >= 1"); return MMASIM_ERR_SHAPE; }
    const DevModel& m = model->dev;
    if (m.k_block) { set_error("mmasim_dot_batch supports unscaled models only"); return MMASIM_ERR_UNSUPPORTED; }
    int st = check_k(m, K);
    if (st != MMASIM_OK) return st;
    if (!aligned16(A) || !aligned16(B) || !aligned16(D) || (C && !aligned16(C))) {
        set_error("A, B, C and D must be 16-byte aligned");
        return MMASIM_ERR_ALIGN;
    }
    if ((st = check_device_ptr(A, "A")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(B, "B")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if (C && (st = check_device_ptr(C, "C")) != MMASIM_OK) return st;
    GemmArgs g;
    std::memset(&g, 0, sizeof(g));
    g.M = n; g.N = 1; g.K = K;
    g.A = A; g.B = B; g.C = C; g.D = D;
    g.lda = g.ldb = K;
    g.ldc = g.ldd = 1;
    g.dot_mode = 1;
    if (!m.literal_emax && dot_stream_supported(m, g)) return launch_dot_stream(m, g, static_cast<cudaStream_t>(stream));
    set_kernel_name("generic_dot");
    return launch_generic(m, g, static_cast<cudaStream_t>(stream));
}

int mmasim_gemm_host(const mmasim_model* model, int64_t M, int64_t N, int64_t K, const void* A, const void* B,
                     const void* C, void* D, const mmasim_gemm_opts* opts) {
    GemmArgs g;
    int st = build_args(model, M, N, K, A, B, C, D, opts, &g);
    if (st != MMASIM_OK) return st;
    const mmasim_info& info = model->info;
    const size_t a_bytes = size_t((M - 1) * g.lda + K) * info.a_bits / 8;
    const size_t b_bytes = size_t((N - 1) * g.ldb + K) * info.b_bits / 8;
    const size_t c_bytes = size_t((M - 1) * g.ldc + N) * info.acc_bytes;
    const size_t d_bytes = size_t((M - 1) * g.ldd + N) * info.acc_bytes;
    const size_t sfa_bytes = g.sfa ? size_t(M * g.ld_sfa) : 0, sfb_bytes = g.sfb ? size_t(N * g.ld_sfb) : 0;
    void *dA = nullptr, *dB = nullptr, *dC = nullptr, *dD = nullptr, *dSA = nullptr, *dSB = nullptr, *dRS = nullptr, *dCS = nullptr;
    cudaError_t err = cudaSuccess;
    // Stream-ordered allocations on a stream of this call's own: after the first call the buffers come out of the
    // library's own memory pool (which keeps up to 1 GiB between calls) and the call synchronises once, at the end.
    // Large problems are cut into a few row panels of D (outputs are independent, Section 3.1 Step 1): B once, then per
    // panel its rows of A and C in, the kernel, its rows of D out, on three streams chained by events, so that the
    // copies of one panel run beside the arithmetic of another (two compute streams, so that a panel's last CTAs
    // share the SMs with the next panel's first).
    // the counter of bulk-copy timeouts before the call: a kernel of this call that gives up makes it grow
    unsigned int timeouts_before = 0u;
    if (g.copy_timeouts) cudaMemcpy(&timeouts_before, g.copy_timeouts, sizeof(unsigned int), cudaMemcpyDeviceToHost);
    constexpr int MAX_PANELS = 16;
    int panels = 1;
    int64_t panel_rows = M;
    if (M >= 1024 && a_bytes + b_bytes + c_bytes + d_bytes >= (size_t(32) << 20)) {
        // whole CTA tiles, at most about eight panels, and at least 256 tiles of 128 x 128 per panel: with fewer a
        // panel's kernel leaves most of the 296 CTA slots of the GPU empty
        panel_rows = ((M + 7) / 8 + 127) / 128 * 128;
        const int64_t fill_rows = 128 * ((256 + (N + 127) / 128 - 1) / ((N + 127) / 128));
        if (panel_rows < fill_rows) panel_rows = fill_rows;
        if (panel_rows < 512) panel_rows = 512;
        panels = int((M + panel_rows - 1) / panel_rows);
        if (panels > MAX_PANELS) { panels = 1; panel_rows = M; }
    }
    cudaStream_t s_in = nullptr, s_k[2] = {nullptr, nullptr}, s_out = nullptr;
    cudaEvent_t ev_in[MAX_PANELS] = {}, ev_k[MAX_PANELS] = {};
    err = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking);
    if (err == cudaSuccess && panels > 1) {
        err = cudaStreamCreateWithFlags(&s_k[0], cudaStreamNonBlocking);
        if (err == cudaSuccess) err = cudaStreamCreateWithFlags(&s_k[1], cudaStreamNonBlocking);
        if (err == cudaSuccess) err = cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking);
        for (int p = 0; p < panels && err == cudaSuccess; ++p) {
            err = cudaEventCreateWithFlags(&ev_in[p], cudaEventDisableTiming);
            if (err == cudaSuccess) err = cudaEventCreateWithFlags(&ev_k[p], cudaEventDisableTiming);
        }
    }
    cudaMemPool_t pool = nullptr;
    if (err == cudaSuccess) err = scratch_pool(&pool);
    auto alloc = [&](void** dst, const void* src, size_t bytes) {
        if (err != cudaSuccess || !src || !bytes) return;
        err = cudaMallocFromPoolAsync(dst, bytes, pool, s_in);
    };
    auto h2d = [&](void* dst, const void* src, size_t off, size_t bytes) {
        if (err != cudaSuccess || !src || !bytes) return;
        err = cudaMemcpyAsync(static_cast<unsigned char*>(dst) + off, static_cast<const unsigned char*>(src) + off, bytes,
                              cudaMemcpyHostToDevice, s_in);
    };
    alloc(&dA, A, a_bytes);
    alloc(&dB, B, b_bytes);
    alloc(&dC, C, c_bytes);
    alloc(&dSA, g.sfa, sfa_bytes);
    alloc(&dSB, g.sfb, sfb_bytes);
    alloc(&dRS, g.row_scale, size_t(M) * 4);
    alloc(&dCS, g.col_scale, size_t(N) * 4);
    alloc(&dD, D, d_bytes);
    h2d(dB, B, 0, b_bytes);
    h2d(dSB, g.sfb, 0, sfb_bytes);
    h2d(dRS, g.row_scale, 0, size_t(M) * 4);
    h2d(dCS, g.col_scale, 0, size_t(N) * 4);
    const GemmArgs host = g;
    for (int p = 0; p < panels && err == cudaSuccess && st == MMASIM_OK; ++p) {
        const int64_t r0 = p * panel_rows, rows = (r0 + panel_rows <= M ? panel_rows : M - r0);
        // byte ranges of the panel's rows (a row of packed 4-bit elements starts on a byte: leading dimensions are even)
        const size_t a_off = size_t(r0 * host.lda) * info.a_bits / 8, a_len = size_t((rows - 1) * host.lda + K) * info.a_bits / 8;
        const size_t c_off = size_t(r0 * host.ldc) * info.acc_bytes, c_len = size_t((rows - 1) * host.ldc + N) * info.acc_bytes;
        const size_t d_off = size_t(r0 * host.ldd) * info.acc_bytes, d_len = size_t((rows - 1) * host.ldd + N) * info.acc_bytes;
        h2d(dA, A, a_off, a_len);
        h2d(dC, C, c_off, c_len);
        h2d(dSA, host.sfa, size_t(r0 * host.ld_sfa), host.sfa ? size_t(rows * host.ld_sfa) : 0);
        if (err != cudaSuccess) break;
        cudaStream_t sk = panels > 1 ? s_k[p & 1] : s_in;
        if (panels > 1) {
            err = cudaEventRecord(ev_in[p], s_in);
            if (err == cudaSuccess) err = cudaStreamWaitEvent(sk, ev_in[p], 0);
            if (err != cudaSuccess) break;
        }
        GemmArgs q = host;
        q.M = rows;
        q.A = static_cast<const unsigned char*>(dA) + a_off;
        q.B = dB;
        q.C = dC ? static_cast<const unsigned char*>(dC) + c_off : nullptr;
        q.D = static_cast<unsigned char*>(dD) + d_off;
        q.sfa = dSA ? static_cast<const uint8_t*>(dSA) + r0 * host.ld_sfa : nullptr;
        q.sfb = static_cast<const uint8_t*>(dSB);
        q.row_scale = dRS ? static_cast<const float*>(dRS) + r0 : nullptr;
        q.col_scale = static_cast<const float*>(dCS);
        st = run_gemm(model, q, opts ? opts->flags : 0, sk);
        if (st != MMASIM_OK) break;
        cudaStream_t so = panels > 1 ? s_out : s_in;
        if (panels > 1) {
            err = cudaEventRecord(ev_k[p], sk);
            if (err == cudaSuccess) err = cudaStreamWaitEvent(so, ev_k[p], 0);
            if (err != cudaSuccess) break;
        }
        // only the N words of every row go back: with ldd > N the words between the rows of the caller's D are not the library's
        if (host.ldd == N)
            err = cudaMemcpyAsync(static_cast<unsigned char*>(D) + d_off, static_cast<unsigned char*>(dD) + d_off, d_len,
                                  cudaMemcpyDeviceToHost, so);
        else
            err = cudaMemcpy2DAsync(static_cast<unsigned char*>(D) + d_off, size_t(host.ldd) * info.acc_bytes,
                                    static_cast<unsigned char*>(dD) + d_off, size_t(host.ldd) * info.acc_bytes,
                                    size_t(N) * info.acc_bytes, size_t(rows), cudaMemcpyDeviceToHost, so);
    }
    // everything drains, then the buffers go back to the pool in the order of the stream they came from
    cudaStream_t all[] = {s_k[0], s_k[1], s_out};
    for (cudaStream_t s : all)
        if (s) { const cudaError_t e2 = cudaStreamSynchronize(s); if (err == cudaSuccess) err = e2; }
    if (s_in) {
        void* bufs[] = {dA, dB, dC, dD, dSA, dSB, dRS, dCS};
        for (void* b : bufs) if (b) cudaFreeAsync(b, s_in);
        const cudaError_t e2 = cudaStreamSynchronize(s_in);
        if (err == cudaSuccess) err = e2;
    }
    for (int p = 0; p < MAX_PANELS; ++p) { if (ev_in[p]) cudaEventDestroy(ev_in[p]); if (ev_k[p]) cudaEventDestroy(ev_k[p]); }
    cudaStream_t streams[] = {s_in, s_k[0], s_k[1], s_out};
    for (cudaStream_t s : streams) if (s) cudaStreamDestroy(s);
    if (err != cudaSuccess) {
        cudaGetLastError();
        set_error("mmasim_gemm_host: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    if (st == MMASIM_OK && g.copy_timeouts) {
        unsigned int timeouts_after = timeouts_before;
        cudaMemcpy(&timeouts_after, g.copy_timeouts, sizeof(unsigned int), cudaMemcpyDeviceToHost);
        if (timeouts_after != timeouts_before) {
            set_error("mmasim_gemm_host: %u CTAs gave up waiting for a bulk copy and stored nothing", timeouts_after - timeouts_before);
            return MMASIM_ERR_TIMEOUT;
        }
    }
    return st;
}

int mmasim_int_peak(int kind, int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, void* stream) {
    if (!sink || !ops_per_round || blocks < 1 || iters < 1 || kind < 0) { set_error("mmasim_int_peak: bad argument"); return MMASIM_ERR_INVALID_ARG; }
    const int st = check_device_ptr(sink, "sink");
    if (st != MMASIM_OK) return st;
    return launch_int_peak(kind, blocks, iters, sink, ops_per_round, static_cast<cudaStream_t>(stream));
}

int mmasim_hw_mma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, void* stream) {
    if (!A || !B || !D) { set_error("mmasim_hw_mma: A, B and D must not be NULL"); return MMASIM_ERR_INVALID_ARG; }
    int st;
    if ((st = check_device_ptr(A, "A")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(B, "B")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if (C && (st = check_device_ptr(C, "C")) != MMASIM_OK) return st;
    return launch_hw_mma(kind, M, K, A, B, C, D, static_cast<cudaStream_t>(stream));
}

int mmasim_hw_umma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, const void* sfa,
                   const void* sfb, int32_t* status, void* stream) {
    if (!A || !B || !D || !status) { set_error("mmasim_hw_umma: A, B, D and status must not be NULL"); return MMASIM_ERR_INVALID_ARG; }
    int st;
    if ((st = check_device_ptr(A, "A")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(B, "B")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(status, "status")) != MMASIM_OK) return st;
    if (C && (st = check_device_ptr(C, "C")) != MMASIM_OK) return st;
    if (sfa && (st = check_device_ptr(sfa, "sfa")) != MMASIM_OK) return st;
    if (sfb && (st = check_device_ptr(sfb, "sfb")) != MMASIM_OK) return st;
    if (!aligned16(A) || !aligned16(B)) { set_error("mmasim_hw_umma: A and B must be 16-byte aligned"); return MMASIM_ERR_ALIGN; }
    return launch_hw_umma(kind, M, K, A, B, C, D, sfa, sfb, status, static_cast<cudaStream_t>(stream));
}

int mmasim_error_stats(int acc_fmt, int64_t n, const void* D, const double* ref, double* stats, void* stream) {
    if (!D || !ref || !stats || n < 1) { set_error("mmasim_error_stats: bad argument"); return MMASIM_ERR_INVALID_ARG; }
    int st;
    if ((st = check_device_ptr(D, "D")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(ref, "ref")) != MMASIM_OK) return st;
    if ((st = check_device_ptr(stats, "stats")) != MMASIM_OK) return st;
    return launch_error_stats(acc_fmt == MMASIM_ACC_F16 ? ACC_F16 : (acc_fmt == MMASIM_ACC_F32 ? ACC_F32 : -1), n, D, ref, stats,
                              static_cast<cudaStream_t>(stream));
}

int mmasim_host_release(void) {
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    cudaError_t err = cudaSuccess;
    for (int d = 0; d < MAX_DEVICES; ++d)
        if (g_pools[d]) {
            const cudaError_t e = cudaMemPoolDestroy(g_pools[d]);
            if (err == cudaSuccess) err = e;
            g_pools[d] = nullptr;
        }
    if (err != cudaSuccess) {
        cudaGetLastError();
        set_error("mmasim_host_release: %s", cudaGetErrorString(err));
        return MMASIM_ERR_CUDA;
    }
    return MMASIM_OK;
}

const char* mmasim_last_kernel(void) { return g_kernel; }

int mmasim_copy_timeouts(uint64_t* count) {
    if (!count) { set_error("count is NULL"); return MMASIM_ERR_INVALID_ARG; }
    unsigned int* p = copy_timeout_counter();
    unsigned int v = 0u;
    cudaError_t err = p ? cudaMemcpy(&v, p, sizeof(v), cudaMemcpyDeviceToHost) : cudaErrorUnknown;
    if (err != cudaSuccess) { set_error("mmasim_copy_timeouts: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    *count = v;
    return MMASIM_OK;
}
const char* mmasim_last_error(void) { return g_error; }

}  // extern "C"
