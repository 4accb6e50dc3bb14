// Host side of the C ABI declared in include/ttc_lqr.h: argument validation, kernel
// selection, workspace ownership, launches on the caller's stream, and the host-buffer
// convenience entry point.  No torch types, no CPU fallback: without a CUDA device of
// compute capability 10.x every call fails with TTC_STATUS_CUDA_ERROR.
#include <cstdarg>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "common.cuh"
#include "riccati_cta.cuh"
#include "riccati_umma64.cuh"
#include "riccati_warp.cuh"
#include "ttc_layer.cuh"
#include "sigma_product.cuh"
#include "layer_grad.cuh"
#include "lqr_grad.cuh"
#include "scan_pair.cuh"
#include "scan_warp.cuh"
#include "peak_probe.cuh"

using namespace ttc;

namespace {

thread_local char g_err[512] = "";

int fail(int status, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return status;
}

#define TTC_CUDA(call)                                                                   \
    do {                                                                                 \
        cudaError_t e_ = (call);                                                         \
        if (e_ != cudaSuccess)                                                           \
            return fail(TTC_STATUS_CUDA_ERROR, "%s: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

constexpr int kMaxSlices = 32;   // token slices of the pipelined host-buffer entry point

struct DevBuf {
    void* ptr = nullptr;
    size_t bytes = 0;
};

} // namespace

struct ttc_lqr_handle {
    ttc_lqr_config cfg;
    long long N;
    int sm_count;
    size_t max_pitch;              // largest pitch a 2D copy accepts on this device
    DevBuf ws_K, ws_P, ws_E;       // scratch used by kernels
    DevBuf ws_info;                // status words of the layer-gradient backward pass when the caller takes none
    DevBuf ws_G;                   // per-instance gradients of Bbar, Qbar, Q_T before the reduction onto the bases
    DevBuf ws_Q;                   // dense Q expanded from a low-rank-plus-diagonal operand
    DevBuf ws_elem;                // scan elements (A_e, C_e, G_e, J_e per instance)
    DevBuf ws_k;                   // feed-forward terms k_t when the caller does not take them
    DevBuf ws_vec;                 // state, control and co-state sequences of the gradient entry point
    DevBuf st_in[5], st_out[5];    // device staging of ttc_lqr_solve_host
    DevBuf st_layer;               // device staging of ttc_lqr_solve_layer_host
    cudaStream_t host_stream;      // compute stream of ttc_lqr_solve_host
    cudaStream_t in_stream, out_stream;   // its copy streams (host -> device, device -> host)
    cudaEvent_t ev_in[kMaxSlices], ev_done[kMaxSlices];
    bool host_pipeline_ready;
    long long last_launches, total_launches;
    int last_kernel;
};

namespace {

int ensure(DevBuf& b, size_t bytes)
{
    if (bytes <= b.bytes)
        return TTC_OK;
    if (b.ptr) {
        cudaDeviceSynchronize();
        cudaFree(b.ptr);
        b.ptr = nullptr;
        b.bytes = 0;
    }
    cudaError_t e = cudaMalloc(&b.ptr, bytes);
    if (e != cudaSuccess) {
        b.ptr = nullptr;
        cudaGetLastError();
        return fail(TTC_STATUS_ALLOC_FAILED, "cudaMalloc(%zu bytes): %s", bytes, cudaGetErrorString(e));
    }
    b.bytes = bytes;
    return TTC_OK;
}

void release(DevBuf& b)
{
    if (b.ptr)
        cudaFree(b.ptr);
    b.ptr = nullptr;
    b.bytes = 0;
}

size_t workspace_bytes(const ttc_lqr_handle* h)
{
    size_t s = h->ws_K.bytes + h->ws_P.bytes + h->ws_E.bytes + h->ws_elem.bytes + h->ws_Q.bytes + h->ws_info.bytes + h->ws_G.bytes + h->ws_k.bytes + h->ws_vec.bytes + h->st_layer.bytes;
    for (int i = 0; i < 5; ++i)
        s += h->st_in[i].bytes + h->st_out[i].bytes;
    return s;
}

int check_operand(const char* name, const ttc_operand* o, bool allow_bf16, bool allow_null)
{
    if (!o || !o->ptr) {
        if (allow_null)
            return TTC_OK;
        return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s is null", name);
    }
    if (o->dtype != TTC_F32 && !(allow_bf16 && o->dtype == TTC_BF16))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s: dtype %d not supported", name, o->dtype);
    if (reinterpret_cast<uintptr_t>(o->ptr) & 15u)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s is not 16-byte aligned", name);
    for (int d = 0; d < 3; ++d)
        if (o->bstride[d] < 0)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s: negative stride", name);
    return TTC_OK;
}

OperandDev to_dev(const ttc_operand* o)
{
    OperandDev d;
    if (!o || !o->ptr) {
        d.ptr = nullptr;
        d.dtype = TTC_F32;
        d.s0 = d.s1 = d.s2 = 0;
        d.st = 0;
        return d;
    }
    d.ptr = o->ptr;
    d.dtype = o->dtype;
    d.s0 = o->bstride[0];
    d.s1 = o->bstride[1];
    d.s2 = o->bstride[2];
    d.st = 0;
    return d;
}

int validate_common(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                    const ttc_operand* R, const ttc_operand* x0, int H, const float* K, const float* P,
                    const float* x, const float* u, const int32_t* info, uint32_t flags)
{
    if (!h)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null handle");
    if (H < 1 || H > h->cfg.max_horizon)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "H=%d outside [1, max_horizon=%d]", H, h->cfg.max_horizon);
    if (flags & ~(TTC_OUT_FIRST_ONLY | TTC_OUT_BF16))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "unknown flag bits 0x%x", flags);
    int s;
    if ((s = check_operand("A", A, false, false))) return s;
    if ((s = check_operand("B", B, false, false))) return s;
    if ((s = check_operand("Q", Q, true, false))) return s;
    if ((s = check_operand("R", R, false, false))) return s;
    const bool need_x0 = (x != nullptr) || (u != nullptr);
    if ((s = check_operand("x0", x0, true, !need_x0))) return s;
    const void* outs[5] = {K, P, x, u, info};
    const char* names[5] = {"K", "P", "x", "u", "info"};
    for (int i = 0; i < 5; ++i)
        if (outs[i] && (reinterpret_cast<uintptr_t>(outs[i]) & 15u))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "output %s is not 16-byte aligned", names[i]);
    return TTC_OK;
}

// true when every batch and time stride of the operand is a multiple of 16 bytes, so that a row of the matrix
// (whose length is a multiple of 16 bytes for the kernels that ask) always starts on a 16-byte boundary
bool vector_rows_ok(const OperandDev& o)
{
    const long long q = o.dtype == TTC_BF16 ? 8 : 4;
    return ((o.s0 | o.s1 | o.s2 | o.st) % q) == 0;
}

// Start of an API call: make sure the small workspace exists and clear the device error word (word 1) on `st`.
int clear_device_error(ttc_lqr_handle* h, cudaStream_t st)
{
    int s = ensure(h->ws_E, sizeof(int) * 4);
    if (s)
        return s;
    TTC_CUDA(cudaMemsetAsync(static_cast<int*>(h->ws_E.ptr) + 1, 0, sizeof(int), st));
    return TTC_OK;
}

// Method of one call.  TTC_AUTO means the sequential recursion except where the scan is measured to be faster:
// time-invariant problems with n = m = 16 / 32 over long horizons with few instances.  The recursion then leaves most
// of the GPU idle while it walks H dependent steps (4.4 us per step at n = 16, 12 us at n = 32), whereas the scan's
// 2 log2(H) + 3 launches spread all N x H applications and gains over the machine (12 ns resp. 59 ns per instance
// and step): the scan wins below about 300 (n = 16) and 180 (n = 32) instances.
int pick_method(const ttc_lqr_handle* h, int H, bool time_varying, long long nwin)
{
    if (h->cfg.method == TTC_SCAN)
        return TTC_SCAN;
    const int n = h->cfg.n;
    if (h->cfg.method == TTC_AUTO && !time_varying && n == h->cfg.m && (n == 16 || n == 32) && H >= 256) {
        const long long in_flight = (long long)h->sm_count * (n == 32 ? 12 : 32);   // instances the recursion keeps resident
        if (nwin * (n == 32 ? 10 : 16) <= in_flight)
            return TTC_SCAN;
    }
    return TTC_RICCATI;
}

} // namespace

extern "C" {

const char* ttc_lqr_status_string(int status)
{
    switch (status) {
    case TTC_OK: return "TTC_OK";
    case TTC_STATUS_INVALID_ARGUMENT: return "TTC_STATUS_INVALID_ARGUMENT";
    case TTC_STATUS_CUDA_ERROR: return "TTC_STATUS_CUDA_ERROR";
    case TTC_STATUS_ALLOC_FAILED: return "TTC_STATUS_ALLOC_FAILED";
    case TTC_STATUS_UNSUPPORTED: return "TTC_STATUS_UNSUPPORTED";
    default: return "TTC_STATUS_UNKNOWN";
    }
}

const char* ttc_lqr_last_error(void) { return g_err; }

int ttc_lqr_create(const ttc_lqr_config* cfg, ttc_lqr_handle** out)
{
    if (!cfg || !out)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null cfg/out");
    *out = nullptr;
    if (cfg->n < 1 || cfg->n > 64 || cfg->m < 1 || cfg->m > 64)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "n=%d, m=%d outside [1, 64]", cfg->n, cfg->m);
    if (cfg->max_horizon < 1 || cfg->max_horizon > 65536)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "max_horizon=%d outside [1, 65536]", cfg->max_horizon);
    long long N = 1;
    for (int d = 0; d < 3; ++d) {
        if (cfg->batch[d] < 1 || cfg->batch[d] > (1ll << 31))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "batch[%d]=%lld out of range", d, (long long)cfg->batch[d]);
        N *= cfg->batch[d];
        if (N > (1ll << 31))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "more than 2^31 instances");
    }
    if (cfg->method < TTC_AUTO || cfg->method > TTC_SCAN)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "unknown method %d", cfg->method);
    if (cfg->math < TTC_MATH_AUTO || cfg->math > TTC_MATH_TF32)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "unknown math mode %d", cfg->math);
    if (cfg->math == TTC_MATH_TF32 && !(cfg->n == 64 && cfg->m == 64))
        return fail(TTC_STATUS_UNSUPPORTED, "TTC_MATH_TF32 needs n = m = 64");
    int ndev = 0;
    TTC_CUDA(cudaGetDeviceCount(&ndev));
    if (cfg->device < 0 || cfg->device >= ndev)
        return fail(TTC_STATUS_CUDA_ERROR, "device %d not present (%d devices)", cfg->device, ndev);
    cudaDeviceProp prop;
    TTC_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
    if (prop.major != 10)
        return fail(TTC_STATUS_CUDA_ERROR, "device %d is sm_%d%d; this library is built for sm_100a only",
                    cfg->device, prop.major, prop.minor);
    TTC_CUDA(cudaSetDevice(cfg->device));
    ttc_lqr_handle* h = new (std::nothrow) ttc_lqr_handle();
    if (!h)
        return fail(TTC_STATUS_ALLOC_FAILED, "host allocation failed");
    h->cfg = *cfg;
    h->N = N;
    h->sm_count = prop.multiProcessorCount;
    h->max_pitch = prop.memPitch;
    h->host_stream = nullptr;
    h->in_stream = h->out_stream = nullptr;
    h->host_pipeline_ready = false;
    h->last_launches = h->total_launches = 0;
    h->last_kernel = TTC_KERNEL_NONE;
    *out = h;
    g_err[0] = 0;
    return TTC_OK;
}

int ttc_lqr_destroy(ttc_lqr_handle* h)
{
    if (!h)
        return TTC_OK;
    cudaSetDevice(h->cfg.device);
    cudaDeviceSynchronize();
    release(h->ws_K);
    release(h->ws_P);
    release(h->ws_E);
    release(h->ws_elem);
    release(h->ws_Q);
    release(h->ws_info);
    release(h->ws_G);
    release(h->ws_k);
    release(h->ws_vec);
    for (int i = 0; i < 5; ++i) {
        release(h->st_in[i]);
        release(h->st_out[i]);
    }
    release(h->st_layer);
    if (h->host_pipeline_ready) {
        for (int i = 0; i < kMaxSlices; ++i) {
            cudaEventDestroy(h->ev_in[i]);
            cudaEventDestroy(h->ev_done[i]);
        }
        cudaStreamDestroy(h->in_stream);
        cudaStreamDestroy(h->out_stream);
    }
    if (h->host_stream)
        cudaStreamDestroy(h->host_stream);
    delete h;
    return TTC_OK;
}

int ttc_lqr_query(const ttc_lqr_handle* h, int32_t key, int64_t* value)
{
    if (!h || !value)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null handle/value");
    switch (key) {
    case TTC_QUERY_LAST_LAUNCHES: *value = h->last_launches; return TTC_OK;
    case TTC_QUERY_WORKSPACE_BYTES: *value = (int64_t)workspace_bytes(h); return TTC_OK;
    case TTC_QUERY_LAST_KERNEL: *value = h->last_kernel; return TTC_OK;
    case TTC_QUERY_TOTAL_LAUNCHES: *value = h->total_launches; return TTC_OK;
    case TTC_QUERY_DEVICE_ERROR: {
        // word 1 of the small workspace: set by a kernel whose bounded wait ran out
        *value = 0;
        if (h->ws_E.ptr && h->ws_E.bytes >= 2 * sizeof(int) && h->last_kernel == TTC_KERNEL_RICCATI_UMMA) {
            int flag = 0;
            if (cudaSetDevice(h->cfg.device) != cudaSuccess ||
                cudaMemcpy(&flag, static_cast<int*>(h->ws_E.ptr) + 1, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
                return fail(TTC_STATUS_CUDA_ERROR, "reading the device error word failed");
            *value = flag;
        }
        return TTC_OK;
    }
    default: return fail(TTC_STATUS_INVALID_ARGUMENT, "unknown query key %d", key);
    }
}

} // extern "C"

namespace {

// Enqueue the solve of the token window [t0, t0 + tcount) of the last batch dimension (all of it for
// ttc_lqr_solve; one slice at a time for the pipelined host-buffer entry point).  Arguments validated.
int solve_window(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                 const ttc_operand* R, const ttc_operand* x0, int32_t H, float* K, float* P, float* x,
                 float* u, int32_t* info, uint32_t flags, cudaStream_t st, long long t0, long long tcount,
                 const int64_t* tstride = nullptr, const ttc_operand* Qf = nullptr,
                 const ttc_operand* r = nullptr, int64_t r_tstride = 0, float* kff = nullptr, float* pvec = nullptr,
                 int r_count = -1)
{
    int s;
    const int n = h->cfg.n, m = h->cfg.m;

    SolveParams p;
    p.n = n; p.m = m; p.H = H;
    p.b0 = h->cfg.batch[0]; p.b1 = h->cfg.batch[1]; p.b2 = h->cfg.batch[2]; p.N = h->N;
    p.t0 = t0; p.tcount = tcount;
    const long long nwin = p.b0 * p.b1 * tcount;          // instances of this launch
    p.A = to_dev(A); p.B = to_dev(B); p.Q = to_dev(Q); p.R = to_dev(R); p.x0 = to_dev(x0);
    p.Qf = to_dev(Qf);
    if (tstride) {
        p.A.st = tstride[0]; p.B.st = tstride[1]; p.Q.st = tstride[2]; p.R.st = tstride[3];
    }
    p.r = to_dev(r);
    p.r.st = r_tstride;
    p.r_count = r_count < 0 ? H : r_count;
    const bool affine = p.r.ptr != nullptr;
    const bool time_varying = affine || p.Qf.ptr != nullptr || (p.A.st | p.B.st | p.Q.st | p.R.st) != 0;
    p.K = K; p.P = P; p.x = x; p.u = u; p.info = info;
    p.Kws = nullptr;
    p.kff = kff; p.pvec = pvec;
    p.first_only = (flags & TTC_OUT_FIRST_ONLY) ? 1 : 0;
    p.out_bf16 = (flags & TTC_OUT_BF16) ? 1 : 0;
    const bool obf = p.out_bf16 != 0;

    const int method = pick_method(h, H, time_varying, nwin);
    if (method == TTC_SCAN && time_varying)
        return fail(TTC_STATUS_UNSUPPORTED, "the scan method handles time-invariant problems without a linear cost only");
    // The rollout reads every K_t in forward order after the backward pass produced them in
    // reverse order; when the caller does not want K they live in the workspace.
    const bool rollout_needs_all_K = (x != nullptr) || (u != nullptr && !p.first_only);

    if (obf && (method == TTC_SCAN || time_varying))
        return fail(TTC_STATUS_UNSUPPORTED, "bfloat16 outputs are served by the sequential recursion of ttc_lqr_solve only");
    if (method == TTC_SCAN) {
        // n = m = 16 / 32: the scan that is parallel in time; it keeps every P_t (in the caller's P or in the
        // workspace).  Other shapes: the generic scan, which keeps every P_t, or a single value matrix (P_1) per
        // instance when only P_0 / u_0 are wanted.
        const bool warp_scan = n == m && (n == 16 || n == 32);
        const int pfull = warp_scan || !(p.first_only && !K && !x);
        float* Pbuf;
        if (pfull && P && !p.first_only) {
            Pbuf = P;
        } else {
            const size_t per = pfull ? (size_t)(H + 1) * n * n : (size_t)n * n;
            if ((s = ensure(h->ws_P, sizeof(float) * (size_t)h->N * per))) return s;
            Pbuf = static_cast<float*>(h->ws_P.ptr);
        }
        if ((s = ensure(h->ws_E, sizeof(int) * (size_t)h->N))) return s;
        int launches = 0;
        cudaError_t e;
        if (warp_scan) {
            // parallel in time: per doubling round one launch over every (instance, application) and one over the
            // squarings, then one over every (instance, t) for the gains, then the rollout
            if ((s = ensure(h->ws_elem, sizeof(float) * (size_t)h->N * scanw::ELEM_MATS * n * n))) return s;
            if (!K && (x || u)) {
                if ((s = ensure(h->ws_K, sizeof(float) * (size_t)h->N * H * m * n))) return s;
                p.Kws = static_cast<float*>(h->ws_K.ptr);
            }
            float* elem = static_cast<float*>(h->ws_elem.ptr);
            int* flags = static_cast<int*>(h->ws_E.ptr);
            e = n == 16 ? scanw::launch_scan_warp<16>(p, Pbuf, elem, flags, h->sm_count, st, &launches)
                        : scanw::launch_scan_warp<32>(p, Pbuf, elem, flags, h->sm_count, st, &launches);
        } else {
            e = launch_scan_path(p, Pbuf, static_cast<int*>(h->ws_E.ptr), pfull, h->sm_count, st, &launches);
        }
        if (e != cudaSuccess)
            return fail(TTC_STATUS_CUDA_ERROR, "scan path launch: %s", cudaGetErrorString(e));
        h->last_launches += launches;
        h->total_launches += launches;
        h->last_kernel = TTC_KERNEL_SCAN;
        return TTC_OK;
    } else {
        // the rollout reads float32 gains: from K itself, or from the workspace when K is not wanted or is bfloat16
        if ((!K && rollout_needs_all_K) || (obf && (K || rollout_needs_all_K))) {
            if ((s = ensure(h->ws_K, sizeof(float) * (size_t)h->N * H * m * n))) return s;
            p.Kws = static_cast<float*>(h->ws_K.ptr);
        }
        if (affine && !kff && rollout_needs_all_K) {          // the rollout adds k_t at every step
            if ((s = ensure(h->ws_k, sizeof(float) * (size_t)h->N * H * m))) return s;
            p.kff = static_cast<float*>(h->ws_k.ptr);
        }
        const bool bf16_in = (Q->dtype == TTC_BF16) || (x0 && x0->ptr && x0->dtype == TTC_BF16);
        const bool want_tf32 = h->cfg.math == TTC_MATH_TF32 || (h->cfg.math == TTC_MATH_AUTO && bf16_in);
        const bool head_shared = A->bstride[2] == 0 && B->bstride[2] == 0 && R->bstride[2] == 0;
        // The tcgen05 and the warp kernels read the rows of Q and Qf with 16-byte loads: every batch and time stride
        // of those operands must keep a row start on a 16-byte boundary (4 fp32 or 8 bf16 elements).  Other strides
        // are served by the generic kernel, which loads element by element.
        const bool q_rows_aligned = vector_rows_ok(p.Q) && (!p.Qf.ptr || vector_rows_ok(p.Qf));
        if (want_tf32 && n == 64 && m == 64 && head_shared && !time_varying && q_rows_aligned) {
            // tcgen05 kernel: persistent CTAs, four independent warpgroups each
            if ((s = ensure(h->ws_E, sizeof(int) * 4))) return s;
            int* counter = static_cast<int*>(h->ws_E.ptr);
            // word 0 = work counter of this launch; word 1 = device error word, cleared once per API call
            // (clear_device_error) so that a later window of the same call cannot erase an earlier report
            TTC_CUDA(cudaMemsetAsync(counter, 0, sizeof(int), st));
            const size_t smem = umma64::smem_bytes();
            auto kern = rollout_needs_all_K || K ? umma64::riccati_umma64_kernel<true> : umma64::riccati_umma64_kernel<false>;
            TTC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            const long long chunks = p.b0 * p.b1 * ((tcount + umma64::CHUNK - 1) / umma64::CHUNK);
            long long grid = h->sm_count;
            if (grid > chunks) grid = chunks;
            kern<<<(unsigned)grid, umma64::THREADS, smem, st>>>(p, counter, counter + 1);
            TTC_CUDA(cudaGetLastError());
            h->last_launches += 1;
            h->total_launches += 1;
            if (rollout_needs_all_K) {
                // forward loop of Alg. 1 as a second, bandwidth-bound kernel: it streams every K_t once
                const size_t rsmem = umma64::rollout_smem_bytes();
                TTC_CUDA(cudaFuncSetAttribute(umma64::rollout64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rsmem));
                const long long rchunks = p.b0 * p.b1 * ((tcount + umma64::ROLL_WARPS - 1) / umma64::ROLL_WARPS);
                long long rgrid = (long long)h->sm_count * 5;
                if (rgrid > rchunks) rgrid = rchunks;
                umma64::rollout64_kernel<<<(unsigned)rgrid, 32 * umma64::ROLL_WARPS, rsmem, st>>>(p, (K && !obf) ? K : p.Kws);
                TTC_CUDA(cudaGetLastError());
                h->last_launches += 1;
                h->total_launches += 1;
            }
            h->last_kernel = TTC_KERNEL_RICCATI_UMMA;
            return TTC_OK;
        }
        // A, B, R either all per head or all per token (a mix goes to the generic kernel)
        const bool per_token = A->bstride[2] != 0 && B->bstride[2] != 0 && R->bstride[2] != 0;
        if ((head_shared || per_token) && n == m && (n == 16 || n == 32) && q_rows_aligned) {
            // fp32 warp kernel: one instance per 16 / 32 lanes, chunks of tokens handed out by an atomic counter
            if ((s = ensure(h->ws_E, sizeof(int) * 4))) return s;
            int* counter = static_cast<int*>(h->ws_E.ptr);
            TTC_CUDA(cudaMemsetAsync(counter, 0, sizeof(int), st));
            void (*kern)(SolveParams, int*);
            size_t smem;
            long long chunks, grid;
            if (n == 32) {
                kern = per_token ? (affine ? rwarp::riccati_warp_kernel<32, true, true, true> : rwarp::riccati_warp_kernel<32, true, false, true>)
                     : affine ? rwarp::riccati_warp_kernel<32, true, true>
                     : time_varying ? rwarp::riccati_warp_kernel<32, true> : rwarp::riccati_warp_kernel<32, false>;
                smem = rwarp::smem_bytes<32>(per_token);
                chunks = p.b0 * p.b1 * ((tcount + rwarp::Shape<32>::SLOTS - 1) / rwarp::Shape<32>::SLOTS);
                grid = (long long)h->sm_count * 3;
            } else {
                kern = per_token ? (affine ? rwarp::riccati_warp_kernel<16, true, true, true> : rwarp::riccati_warp_kernel<16, true, false, true>)
                     : affine ? rwarp::riccati_warp_kernel<16, true, true>
                     : time_varying ? rwarp::riccati_warp_kernel<16, true> : rwarp::riccati_warp_kernel<16, false>;
                smem = rwarp::smem_bytes<16>(per_token);
                chunks = p.b0 * p.b1 * ((tcount + rwarp::Shape<16>::SLOTS - 1) / rwarp::Shape<16>::SLOTS);
                grid = (long long)h->sm_count * 4;
            }
            TTC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            if (grid > chunks) grid = chunks;
            kern<<<(unsigned)grid, rwarp::THREADS, smem, st>>>(p, counter);
            TTC_CUDA(cudaGetLastError());
            h->last_launches += 1;
            h->total_launches += 1;
            h->last_kernel = TTC_KERNEL_RICCATI_WARP;
            return TTC_OK;
        }
        if (obf)
            return fail(TTC_STATUS_UNSUPPORTED, "bfloat16 outputs need n = m in {16, 32} or the tensor-core path at n = m = 64 "
                                                "(per-head or per-token A, B, R; Q strides that keep 16-byte rows)");
        const size_t smem = riccati_cta_smem_bytes(n, m);
        TTC_CUDA(cudaFuncSetAttribute(riccati_cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int per_sm = 1;
        TTC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, riccati_cta_kernel, 256, smem));
        if (per_sm < 1) per_sm = 1;
        long long grid = (long long)h->sm_count * per_sm;
        if (grid > nwin) grid = nwin;
        riccati_cta_kernel<<<(unsigned)grid, 256, smem, st>>>(p);
        TTC_CUDA(cudaGetLastError());
        h->last_launches += 1;
        h->total_launches += 1;
        h->last_kernel = TTC_KERNEL_RICCATI_CTA;
    }
    return TTC_OK;
}


} // namespace

extern "C" {

int ttc_lqr_solve(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                  const ttc_operand* R, const ttc_operand* x0, int32_t H, float* K, float* P, float* x,
                  float* u, int32_t* info, uint32_t flags, void* cuda_stream)
{
    int s = validate_common(h, A, B, Q, R, x0, H, K, P, x, u, info, flags);
    if (s)
        return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    h->last_launches = 0;
    if ((s = clear_device_error(h, static_cast<cudaStream_t>(cuda_stream))))
        return s;
    return solve_window(h, A, B, Q, R, x0, H, K, P, x, u, info, flags, static_cast<cudaStream_t>(cuda_stream), 0,
                        h->cfg.batch[2]);
}

int ttc_lqr_solve_lowrank_q(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* U,
                            const ttc_operand* d, int32_t rank, float scale, const ttc_operand* R, const ttc_operand* x0,
                            int32_t H, float* K, float* P, float* x, float* u, int32_t* info, uint32_t flags,
                            void* cuda_stream)
{
    if (!h)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null handle");
    const int n = h->cfg.n;
    if (rank < 1 || rank > n)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "rank=%d outside [1, n=%d]", rank, n);
    if (!(scale >= 0.f))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "scale must be non-negative");
    int s;
    if ((s = check_operand("U", U, true, false))) return s;
    if ((s = check_operand("d", d, true, false))) return s;
    // the dense operand the solve will read: float32, one matrix per instance
    ttc_operand Qd;
    Qd.ptr = reinterpret_cast<const void*>(16);       // placeholder so that validation sees a non-null, aligned pointer
    Qd.dtype = TTC_F32; Qd.reserved = 0;
    Qd.bstride[2] = (int64_t)n * n;
    Qd.bstride[1] = Qd.bstride[2] * h->cfg.batch[2];
    Qd.bstride[0] = Qd.bstride[1] * h->cfg.batch[1];
    if ((s = validate_common(h, A, B, &Qd, R, x0, H, K, P, x, u, info, flags))) return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if ((s = ensure(h->ws_Q, sizeof(float) * (size_t)h->N * n * n))) return s;
    Qd.ptr = h->ws_Q.ptr;
    h->last_launches = 0;
    if ((s = clear_device_error(h, st))) return s;
    {
        SolveParams p;
        p.n = n; p.m = h->cfg.m; p.H = H;
        p.b0 = h->cfg.batch[0]; p.b1 = h->cfg.batch[1]; p.b2 = h->cfg.batch[2]; p.N = h->N;
        p.t0 = 0; p.tcount = p.b2;
        long long grid = h->N < (long long)h->sm_count * 8 ? h->N : (long long)h->sm_count * 8;
        expand_lowrank_q_kernel<<<(unsigned)grid, 256, sizeof(float) * (size_t)(rank + 1) * n, st>>>(
            p, to_dev(U), to_dev(d), rank, scale, static_cast<float*>(h->ws_Q.ptr));
        TTC_CUDA(cudaGetLastError());
        h->last_launches += 1;
        h->total_launches += 1;
    }
    // AUTO math: tensor-core path when the factors were handed over in bfloat16, as for a bfloat16 dense Q
    const bool bf16_factors = U->dtype == TTC_BF16;
    const int math_saved = h->cfg.math;
    if (math_saved == TTC_MATH_AUTO && bf16_factors && n == 64 && h->cfg.m == 64)
        h->cfg.math = TTC_MATH_TF32;
    s = solve_window(h, A, B, &Qd, R, x0, H, K, P, x, u, info, flags, st, 0, h->cfg.batch[2]);
    h->cfg.math = math_saved;
    return s;
}

int ttc_lqr_solve_affine(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                         const ttc_operand* R, const int64_t tstride[4], const ttc_operand* Qf,
                         const ttc_operand* r, int64_t r_tstride, const ttc_operand* x0, int32_t H,
                         float* K, float* kff, float* P, float* pvec, float* x, float* u, int32_t* info,
                         uint32_t flags, void* cuda_stream)
{
    int s = validate_common(h, A, B, Q, R, x0, H, K, P, x, u, info, flags);
    if (s)
        return s;
    if (!tstride)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null tstride");
    for (int i = 0; i < 4; ++i)
        if (tstride[i] < 0)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "negative time stride");
    if (r_tstride < 0)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "negative time stride of r");
    if ((s = check_operand("Qf", Qf, true, tstride[2] == 0)))
        return s;
    if ((s = check_operand("r", r, false, false)))
        return s;
    if ((reinterpret_cast<uintptr_t>(kff) | reinterpret_cast<uintptr_t>(pvec)) & 15u)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "outputs must be 16-byte aligned");
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    h->last_launches = 0;
    return solve_window(h, A, B, Q, R, x0, H, K, P, x, u, info, flags, static_cast<cudaStream_t>(cuda_stream), 0,
                        h->cfg.batch[2], tstride, (Qf && Qf->ptr) ? Qf : nullptr, r, r_tstride, kff, pvec);
}

int ttc_lqr_grad(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                 const ttc_operand* R, const int64_t tstride[4], const ttc_operand* Qf, const ttc_operand* x0,
                 const float* g, int32_t H, float* dA, float* dB, float* dQ, float* dQf, float* dR, float* dx0,
                 float* u0, int32_t* info, void* cuda_stream)
{
    int s = validate_common(h, A, B, Q, R, x0, H, nullptr, nullptr, nullptr, u0, info, 0);
    if (s)
        return s;
    if (!x0 || !x0->ptr)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "operand x0 is null");
    if (!tstride)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null tstride");
    for (int i = 0; i < 4; ++i)
        if (tstride[i] < 0)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "negative time stride");
    if ((s = check_operand("Qf", Qf, true, tstride[2] == 0)))
        return s;
    if (!g)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null output gradient g");
    const void* ptrs[8] = {g, dA, dB, dQ, dQf, dR, dx0, u0};
    for (int i = 0; i < 8; ++i)
        if (reinterpret_cast<uintptr_t>(ptrs[i]) & 15u)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "g and the gradient outputs must be 16-byte aligned");
    if (h->cfg.method == TTC_SCAN)
        return fail(TTC_STATUS_UNSUPPORTED, "the scan method has no gradient path");
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int n = h->cfg.n, m = h->cfg.m;
    const int D = ((n > m ? n : m) + 3) & ~3;
    if ((s = ensure(h->ws_K, sizeof(float) * (size_t)h->N * H * m * n))) return s;
    if ((s = ensure(h->ws_k, sizeof(float) * (size_t)h->N * H * m))) return s;
    if ((s = ensure(h->ws_vec, sizeof(float) * (size_t)h->N * 6 * (H + 1) * D))) return s;
    float* Kws = static_cast<float*>(h->ws_K.ptr);
    float* kws = static_cast<float*>(h->ws_k.ptr);
    h->last_launches = 0;

    // Backward pass of the primal problem (K_t) with the dual problem's linear cost riding along: r_0 = g, r_t = 0
    // afterwards, so k_0 = -S_0^{-1} g is the dual's first control and every later k_t vanishes.
    ttc_operand r;
    r.ptr = g; r.dtype = TTC_F32; r.reserved = 0;
    r.bstride[2] = m; r.bstride[1] = (int64_t)m * h->cfg.batch[2]; r.bstride[0] = r.bstride[1] * h->cfg.batch[1];
    if ((s = solve_window(h, A, B, Q, R, x0, H, Kws, nullptr, nullptr, nullptr, info, 0, st, 0, h->cfg.batch[2], tstride,
                          (Qf && Qf->ptr) ? Qf : nullptr, &r, 0, kws, nullptr, 1)))
        return s;

    grad::GradParams gp;
    SolveParams& p = gp.sp;
    p.n = n; p.m = m; p.H = H;
    p.b0 = h->cfg.batch[0]; p.b1 = h->cfg.batch[1]; p.b2 = h->cfg.batch[2]; p.N = h->N;
    p.t0 = 0; p.tcount = p.b2;
    p.A = to_dev(A); p.B = to_dev(B); p.Q = to_dev(Q); p.R = to_dev(R); p.x0 = to_dev(x0);
    p.Qf = to_dev((Qf && Qf->ptr) ? Qf : nullptr);
    p.A.st = tstride[0]; p.B.st = tstride[1]; p.Q.st = tstride[2]; p.R.st = tstride[3];
    p.r = to_dev(nullptr); p.r_count = 0;
    p.K = nullptr; p.P = nullptr; p.x = nullptr; p.u = nullptr; p.info = info; p.Kws = nullptr;
    p.kff = nullptr; p.pvec = nullptr; p.first_only = 0; p.out_bf16 = 0;
    gp.K = Kws; gp.kff = kws; gp.vec = static_cast<float*>(h->ws_vec.ptr); gp.D = D;
    {
        auto pow2 = [](int v) { return v > 0 && (v & (v - 1)) == 0; };
        long long strides = p.A.st | p.B.st;
        for (const OperandDev* o : {&p.A, &p.B})
            strides |= o->s0 | o->s1 | o->s2;
        gp.vec4 = (n % 4 == 0 && m % 4 == 0 && pow2(n / 4) && pow2(m / 4) && n <= 64 && m <= 64 && (strides & 3) == 0) ? 1 : 0;
    }
    gp.dA = dA; gp.dB = dB; gp.dQ = dQ; gp.dQf = dQf; gp.dR = dR; gp.dx0 = dx0; gp.u0 = u0;

    long long grid = (h->N + grad::WARPS - 1) / grad::WARPS;
    const long long cap = (long long)h->sm_count * 8;
    if (grid > cap) grid = cap;
    {
        long long qs = p.Q.st | p.Q.s0 | p.Q.s1 | p.Q.s2 | p.Qf.s0 | p.Qf.s1 | p.Qf.s2;
        const bool small = gp.vec4 && n <= 16 && m <= 16 && p.Q.dtype == TTC_F32 && p.Qf.dtype == TTC_F32 && (qs & 3) == 0;
        if (small) {
            const size_t smem = grad::small_smem_bytes();
            TTC_CUDA(cudaFuncSetAttribute(grad::grad_vectors_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            long long sgrid = (h->N + grad::WARPS - 1) / grad::WARPS;
            if (sgrid > (long long)h->sm_count * 2) sgrid = (long long)h->sm_count * 2;      // two CTAs fit an SM
            grad::grad_vectors_small_kernel<<<(unsigned)sgrid, 32 * grad::WARPS, smem, st>>>(gp);
        }
        else
            grad::grad_vectors_kernel<<<(unsigned)grid, 32 * grad::WARPS, 0, st>>>(gp);
    }
    TTC_CUDA(cudaGetLastError());
    h->last_launches += 1;
    h->total_launches += 1;
    if (dA || dB || dQ || dQf || dR) {
        grid = (h->N * (long long)(H + 1) + grad::WARPS - 1) / grad::WARPS;
        if (grid > cap) grid = cap;
        grad::grad_outer_kernel<<<(unsigned)grid, 32 * grad::WARPS, 0, st>>>(gp);
        TTC_CUDA(cudaGetLastError());
        h->last_launches += 1;
        h->total_launches += 1;
    }
    return TTC_OK;
}

// streams and events of the host-buffer entry points (created on first use)
static int ensure_host_pipeline(ttc_lqr_handle* h)
{
    if (h->host_pipeline_ready)
        return TTC_OK;
    TTC_CUDA(cudaStreamCreateWithFlags(&h->host_stream, cudaStreamNonBlocking));
    TTC_CUDA(cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking));
    TTC_CUDA(cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking));
    for (int i = 0; i < kMaxSlices; ++i) {
        TTC_CUDA(cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming));
        TTC_CUDA(cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
    }
    h->host_pipeline_ready = true;
    return TTC_OK;
}

int ttc_lqr_solve_tv(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                     const ttc_operand* R, const int64_t tstride[4], const ttc_operand* Qf, const ttc_operand* x0,
                     int32_t H, float* K, float* P, float* x, float* u, int32_t* info, uint32_t flags,
                     void* cuda_stream)
{
    int s = validate_common(h, A, B, Q, R, x0, H, K, P, x, u, info, flags);
    if (s)
        return s;
    if (!tstride)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null tstride");
    for (int i = 0; i < 4; ++i)
        if (tstride[i] < 0)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "negative time stride");
    if ((s = check_operand("Qf", Qf, true, tstride[2] == 0)))
        return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    h->last_launches = 0;
    return solve_window(h, A, B, Q, R, x0, H, K, P, x, u, info, flags, static_cast<cudaStream_t>(cuda_stream), 0,
                        h->cfg.batch[2], tstride, (Qf && Qf->ptr) ? Qf : nullptr);
}

static int check_layer_call(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, bool device_pointers,
                            const float* u1, const float* P0)
{
    if (!h || !in)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null handle or inputs");
    const int n = h->cfg.n;
    if (n != h->cfg.m || (n != 16 && n != 32))
        return fail(TTC_STATUS_UNSUPPORTED, "layer solve needs n == m in {16, 32} (got n=%d, m=%d)", n, h->cfg.m);
    if (T < 1 || T > h->cfg.max_horizon)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "T=%d outside [1, max_horizon=%d]", T, h->cfg.max_horizon);
    if (in->r < 1 || in->r > 64)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "r=%d outside [1, 64]", in->r);
    const void* ptrs[11] = {in->s_a, in->s_gamma_a, in->s_gamma_b, in->s_gamma_q, in->s_b, in->s_q, in->s_qf,
                            in->r_inv, in->h0, in->B_basis, in->Q_basis};
    for (int i = 0; i < 11; ++i) {
        if (!ptrs[i])
            return fail(TTC_STATUS_INVALID_ARGUMENT, "layer input %d is null", i);
        if (device_pointers && (reinterpret_cast<uintptr_t>(ptrs[i]) & 15u))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "layer input %d is not 16-byte aligned", i);
    }
    if (device_pointers && ((reinterpret_cast<uintptr_t>(u1) | reinterpret_cast<uintptr_t>(P0)) & 15u))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "outputs must be 16-byte aligned");
    return TTC_OK;
}

// all pointers are device memory here
// Instances [i0, i0 + cnt) of the handle's batch (the arrays are instance-major, the bases shared).
static int launch_layer(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, float* u1, float* P0, int32_t* info,
                        cudaStream_t st, long long i0 = 0, long long cnt = -1)
{
    const int n = h->cfg.n;
    int s;
    if ((s = ensure(h->ws_E, sizeof(int) * 4))) return s;
    int* counter = static_cast<int*>(h->ws_E.ptr);
    TTC_CUDA(cudaMemsetAsync(counter, 0, sizeof(int), st));
    layer::LayerParams p;
    p.N = cnt < 0 ? h->N : cnt;
    p.T = T;
    p.r = in->r;
    const long long on = i0 * n, orr = i0 * in->r;
    p.s_a = in->s_a + on; p.s_ga = in->s_gamma_a + on; p.s_gb = in->s_gamma_b + on; p.s_gq = in->s_gamma_q + on;
    p.s_b = in->s_b + orr; p.s_q = in->s_q + orr; p.s_qf = in->s_qf + orr;
    p.r_inv = in->r_inv + on; p.h0 = in->h0 + on;
    p.B_basis = in->B_basis; p.Q_basis = in->Q_basis;
    p.u1 = u1 ? u1 + on : nullptr; p.P0 = P0 ? P0 + on * n : nullptr; p.info = info ? info + i0 : nullptr;
    p.Kws = nullptr; p.Pws = nullptr; p.g = nullptr; p.k0 = nullptr;
    void (*kern)(layer::LayerParams, int*);
    size_t smem;
    long long chunks, grid;
    if (n == 32) {
        kern = layer::ttc_layer_kernel<32>;
        smem = layer::smem_bytes<32>();
        chunks = (p.N + rwarp::Shape<32>::SLOTS - 1) / rwarp::Shape<32>::SLOTS;
        grid = (long long)h->sm_count * 3;
    } else if (p.N <= (long long)h->sm_count * 2 * rwarp::Shape<16>::SLOTS) {
        // the machine is less than half full: 16 lanes per instance walk the chain faster than 8 lanes with two columns each
        kern = layer::ttc_layer_kernel<16>;
        smem = layer::smem_bytes<16>();
        chunks = (p.N + rwarp::Shape<16>::SLOTS - 1) / rwarp::Shape<16>::SLOTS;
        grid = (long long)h->sm_count * 4;
    } else {
        kern = layer::ttc_layer_kernel_c2<16>;
        smem = layer::smem_bytes_c2<16>();
        chunks = (p.N + layer::Shape2<16>::SLOTS - 1) / layer::Shape2<16>::SLOTS;
        grid = (long long)h->sm_count * 2;
    }
    TTC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (grid > chunks) grid = chunks;
    kern<<<(unsigned)grid, rwarp::THREADS, smem, st>>>(p, counter);
    TTC_CUDA(cudaGetLastError());
    h->last_launches += 1;
    h->total_launches += 1;
    h->last_kernel = TTC_KERNEL_LAYER;
    return TTC_OK;
}

int ttc_lqr_solve_layer(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, float* u1, float* P0,
                        int32_t* info, void* cuda_stream)
{
    int s = check_layer_call(h, in, T, true, u1, P0);
    if (s)
        return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    h->last_launches = 0;
    return launch_layer(h, in, T, u1, P0, info, static_cast<cudaStream_t>(cuda_stream));
}

int ttc_lqr_solve_layer_sigma_baseline(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, float* u1, float* P0,
                                       int32_t* info, void* cuda_stream)
{
    int s = check_layer_call(h, in, T, true, u1, P0);
    if (s)
        return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    h->last_launches = 0;
    const int n = h->cfg.n;
    layer::LayerParams p;
    p.N = h->N;
    p.T = T;
    p.r = in->r;
    p.s_a = in->s_a; p.s_ga = in->s_gamma_a; p.s_gb = in->s_gamma_b; p.s_gq = in->s_gamma_q;
    p.s_b = in->s_b; p.s_q = in->s_q; p.s_qf = in->s_qf;
    p.r_inv = in->r_inv; p.h0 = in->h0;
    p.B_basis = in->B_basis; p.Q_basis = in->Q_basis;
    p.u1 = u1; p.P0 = P0; p.info = info;
    p.Kws = nullptr; p.Pws = nullptr; p.g = nullptr; p.k0 = nullptr;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int slots = n == 32 ? rwarp::Shape<32>::SLOTS : rwarp::Shape<16>::SLOTS;
    long long grid = (p.N + slots - 1) / slots;
    const long long cap = (long long)h->sm_count * 8;
    if (grid > cap) grid = cap;
    if (n == 32) {
        const size_t smem = sigma::smem_bytes<32>();
        TTC_CUDA(cudaFuncSetAttribute(sigma::sigma_product_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sigma::sigma_product_kernel<32><<<(unsigned)grid, rwarp::THREADS, smem, st>>>(p);
    } else {
        const size_t smem = sigma::smem_bytes<16>();
        TTC_CUDA(cudaFuncSetAttribute(sigma::sigma_product_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sigma::sigma_product_kernel<16><<<(unsigned)grid, rwarp::THREADS, smem, st>>>(p);
    }
    TTC_CUDA(cudaGetLastError());
    h->last_launches += 1;
    h->total_launches += 1;
    h->last_kernel = TTC_KERNEL_SIGMA_BASELINE;
    return TTC_OK;
}

int ttc_lqr_layer_grad(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, const float* g,
                       const ttc_layer_grads* out, float* u1, int32_t* info, void* cuda_stream)
{
    int s = check_layer_call(h, in, T, true, u1, nullptr);
    if (s)
        return s;
    if (!g || !out)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null output gradient g or null result struct");
    const void* ptrs[13] = {g, out->s_a, out->s_gamma_a, out->s_gamma_b, out->s_gamma_q, out->s_b, out->s_q, out->s_qf,
                            out->r_inv, out->h0, out->B_basis, out->Q_basis, info};
    for (int i = 0; i < 13; ++i)
        if (reinterpret_cast<uintptr_t>(ptrs[i]) & 15u)
            return fail(TTC_STATUS_INVALID_ARGUMENT, "g and the gradient outputs must be 16-byte aligned");
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int n = h->cfg.n, r = in->r;
    const size_t N = (size_t)h->N, nn = (size_t)n * n;
    if ((s = ensure(h->ws_K, sizeof(float) * 2 * N * T * nn))) return s;           // every K_s, then every P_s
    if ((s = ensure(h->ws_k, sizeof(float) * N * n))) return s;
    if ((s = ensure(h->ws_vec, sizeof(float) * N * 4 * (T + 1) * n))) return s;
    if ((s = ensure(h->ws_E, sizeof(int) * 4))) return s;
    int* info_dev = info;
    if (!info_dev) {
        if ((s = ensure(h->ws_info, sizeof(int) * N))) return s;
        info_dev = static_cast<int*>(h->ws_info.ptr);
    }
    const bool bases = out->B_basis || out->Q_basis;
    if (bases && (s = ensure(h->ws_G, sizeof(float) * 3 * N * nn))) return s;
    h->last_launches = 0;

    // (1) backward Riccati pass on the synthesised parameters; every gain and k_0 = -S_0^{-1} g are kept
    layer::LayerParams p;
    p.N = h->N; p.T = T; p.r = r;
    p.s_a = in->s_a; p.s_ga = in->s_gamma_a; p.s_gb = in->s_gamma_b; p.s_gq = in->s_gamma_q;
    p.s_b = in->s_b; p.s_q = in->s_q; p.s_qf = in->s_qf;
    p.r_inv = in->r_inv; p.h0 = in->h0;
    p.B_basis = in->B_basis; p.Q_basis = in->Q_basis;
    p.u1 = u1; p.P0 = nullptr; p.info = info_dev;
    p.Kws = static_cast<float*>(h->ws_K.ptr); p.g = g; p.k0 = static_cast<float*>(h->ws_k.ptr);
    p.Pws = p.Kws + N * T * nn;
    int* counter = static_cast<int*>(h->ws_E.ptr);
    TTC_CUDA(cudaMemsetAsync(counter, 0, sizeof(int), st));
    {
        // n = 16 with the machine at least half full: two columns per lane, as in the forward call
        const bool c2 = n == 16 && p.N > (long long)h->sm_count * 2 * rwarp::Shape<16>::SLOTS;
        void (*kern)(layer::LayerParams, int*) = n == 32 ? layer::ttc_layer_kernel<32, true>
                                               : c2 ? layer::ttc_layer_kernel_c2<16, true> : layer::ttc_layer_kernel<16, true>;
        const size_t smem = n == 32 ? layer::smem_bytes<32>() : c2 ? layer::smem_bytes_c2<16>() : layer::smem_bytes<16>();
        const int slots = n == 32 ? rwarp::Shape<32>::SLOTS : c2 ? layer::Shape2<16>::SLOTS : rwarp::Shape<16>::SLOTS;
        long long chunks = (p.N + slots - 1) / slots, grid = (long long)h->sm_count * (n == 32 ? 3 : c2 ? 2 : 4);
        if (grid > chunks) grid = chunks;
        TTC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kern<<<(unsigned)grid, rwarp::THREADS, smem, st>>>(p, counter);
        TTC_CUDA(cudaGetLastError());
    }
    // (2) rollouts, co-states and the reductions of Thm 3.2's outer products onto the coefficients
    lgrad::LayerGradParams q;
    q.lp = p;
    q.vec = static_cast<float*>(h->ws_vec.ptr);
    q.info = info_dev;
    q.d_sa = out->s_a; q.d_ga = out->s_gamma_a; q.d_gb = out->s_gamma_b; q.d_gq = out->s_gamma_q;
    q.d_ri = out->r_inv; q.d_h0 = out->h0;
    q.d_sb = out->s_b; q.d_sq = out->s_q; q.d_sqf = out->s_qf;
    float* G = bases ? static_cast<float*>(h->ws_G.ptr) : nullptr;
    q.GB = G; q.GQ = G ? G + N * nn : nullptr; q.GF = G ? G + 2 * N * nn : nullptr;
    {
        const int slots = n == 32 ? rwarp::Shape<32>::SLOTS : rwarp::Shape<16>::SLOTS;
        long long grid = (p.N + slots - 1) / slots;
        const long long cap = (long long)h->sm_count * 8;
        if (grid > cap) grid = cap;
        if (n == 32) {
            const size_t smem = sizeof(lgrad::Slot<32>) * slots;
            TTC_CUDA(cudaFuncSetAttribute(lgrad::layer_grad_vectors_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            lgrad::layer_grad_vectors_kernel<32><<<(unsigned)grid, rwarp::THREADS, smem, st>>>(q);
        } else {
            const size_t smem = sizeof(lgrad::Slot<16>) * slots;
            TTC_CUDA(cudaFuncSetAttribute(lgrad::layer_grad_vectors_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            lgrad::layer_grad_vectors_kernel<16><<<(unsigned)grid, rwarp::THREADS, smem, st>>>(q);
        }
        TTC_CUDA(cudaGetLastError());
    }
    h->last_launches += 2;
    h->total_launches += 2;
    // (3) the bases are shared by every instance: their gradients are sums over the instances
    if (bases) {
        long long grid = (long long)h->sm_count * 4;
        if (grid > (long long)N) grid = (long long)N;
        if (out->B_basis) {
            TTC_CUDA(cudaMemsetAsync(out->B_basis, 0, sizeof(float) * (size_t)r * nn, st));
            lgrad::basis_reduce_kernel<<<(unsigned)grid, 256, 0, st>>>(h->N, r, (int)nn, info_dev, in->s_b, q.GB, nullptr, nullptr, out->B_basis);
            TTC_CUDA(cudaGetLastError());
            h->last_launches += 1; h->total_launches += 1;
        }
        if (out->Q_basis) {
            TTC_CUDA(cudaMemsetAsync(out->Q_basis, 0, sizeof(float) * (size_t)r * nn, st));
            lgrad::basis_reduce_kernel<<<(unsigned)grid, 256, 0, st>>>(h->N, r, (int)nn, info_dev, in->s_q, q.GQ, in->s_qf, q.GF, out->Q_basis);
            TTC_CUDA(cudaGetLastError());
            h->last_launches += 1; h->total_launches += 1;
        }
    }
    h->last_kernel = TTC_KERNEL_LAYER;
    return TTC_OK;
}

int ttc_lqr_solve_layer_host(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, float* u1, float* P0,
                             int32_t* info)
{
    int s = check_layer_call(h, in, T, false, nullptr, nullptr);
    if (s)
        return s;
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    if ((s = ensure_host_pipeline(h)))
        return s;
    h->last_launches = 0;
    const size_t N = (size_t)h->N, n = (size_t)h->cfg.n, r = (size_t)in->r;
    const void* src[11] = {in->s_a, in->s_gamma_a, in->s_gamma_b, in->s_gamma_q, in->s_b, in->s_q, in->s_qf,
                           in->r_inv, in->h0, in->B_basis, in->Q_basis};
    const size_t in_bytes[11] = {4 * N * n, 4 * N * n, 4 * N * n, 4 * N * n, 4 * N * r, 4 * N * r, 4 * N * r,
                                 4 * N * n, 4 * N * n, 4 * r * n * n, 4 * r * n * n};
    void* host_out[3] = {u1, P0, info};
    const size_t out_bytes[3] = {4 * N * n, 4 * N * n * n, 4 * N};
    auto pad = [](size_t b) { return (b + 255) & ~(size_t)255; };
    size_t total = 0;
    for (int i = 0; i < 11; ++i) total += pad(in_bytes[i]);
    for (int i = 0; i < 3; ++i) total += host_out[i] ? pad(out_bytes[i]) : 0;
    if ((s = ensure(h->st_layer, total)))
        return s;
    cudaStream_t st = h->host_stream;
    unsigned char* base = static_cast<unsigned char*>(h->st_layer.ptr);
    unsigned char* dptr[11];
    size_t off = 0;
    for (int i = 0; i < 11; ++i) {
        dptr[i] = base + off;
        off += pad(in_bytes[i]);
    }
    unsigned char* dev_out[3] = {nullptr, nullptr, nullptr};
    for (int i = 0; i < 3; ++i)
        if (host_out[i]) {
            dev_out[i] = base + off;
            off += pad(out_bytes[i]);
        }
    ttc_layer_inputs din = *in;
    din.s_a = reinterpret_cast<const float*>(dptr[0]); din.s_gamma_a = reinterpret_cast<const float*>(dptr[1]);
    din.s_gamma_b = reinterpret_cast<const float*>(dptr[2]); din.s_gamma_q = reinterpret_cast<const float*>(dptr[3]);
    din.s_b = reinterpret_cast<const float*>(dptr[4]); din.s_q = reinterpret_cast<const float*>(dptr[5]);
    din.s_qf = reinterpret_cast<const float*>(dptr[6]); din.r_inv = reinterpret_cast<const float*>(dptr[7]);
    din.h0 = reinterpret_cast<const float*>(dptr[8]);
    din.B_basis = reinterpret_cast<const float*>(dptr[9]); din.Q_basis = reinterpret_cast<const float*>(dptr[10]);

    // Slices of the instance dimension: copy in, solve and copy out overlap across slices (as in ttc_lqr_solve_host).
    // The bases are shared and go first.
    int nslice = 1;
    if (total >= ((size_t)16 << 20) && N >= 8192)
        nslice = (int)(N / 4096 < (size_t)kMaxSlices ? N / 4096 : (size_t)kMaxSlices);
    size_t per = (N + nslice - 1) / nslice;
    per = (per + 63) / 64 * 64;
    nslice = (int)((N + per - 1) / per);
    const size_t per_inst_in[9] = {4 * n, 4 * n, 4 * n, 4 * n, 4 * r, 4 * r, 4 * r, 4 * n, 4 * n};
    const size_t per_inst_out[3] = {4 * n, 4 * n * n, 4};
    for (int i = 9; i < 11; ++i)
        TTC_CUDA(cudaMemcpyAsync(dptr[i], src[i], in_bytes[i], cudaMemcpyHostToDevice, h->in_stream));
    for (int c = 0; c < nslice; ++c) {
        const size_t i0 = (size_t)c * per, cnt = (N - i0 < per) ? N - i0 : per;
        for (int i = 0; i < 9; ++i)
            TTC_CUDA(cudaMemcpyAsync(dptr[i] + i0 * per_inst_in[i], static_cast<const unsigned char*>(src[i]) + i0 * per_inst_in[i],
                                     cnt * per_inst_in[i], cudaMemcpyHostToDevice, h->in_stream));
        TTC_CUDA(cudaEventRecord(h->ev_in[c], h->in_stream));
        TTC_CUDA(cudaStreamWaitEvent(st, h->ev_in[c], 0));
        if ((s = launch_layer(h, &din, T, reinterpret_cast<float*>(dev_out[0]), reinterpret_cast<float*>(dev_out[1]),
                              reinterpret_cast<int32_t*>(dev_out[2]), st, (long long)i0, (long long)cnt))) {
            cudaDeviceSynchronize();
            return s;
        }
        TTC_CUDA(cudaEventRecord(h->ev_done[c], st));
        TTC_CUDA(cudaStreamWaitEvent(h->out_stream, h->ev_done[c], 0));
        for (int i = 0; i < 3; ++i)
            if (host_out[i])
                TTC_CUDA(cudaMemcpyAsync(static_cast<unsigned char*>(host_out[i]) + i0 * per_inst_out[i],
                                         dev_out[i] + i0 * per_inst_out[i], cnt * per_inst_out[i], cudaMemcpyDeviceToHost,
                                         h->out_stream));
    }
    TTC_CUDA(cudaStreamSynchronize(h->out_stream));
    TTC_CUDA(cudaStreamSynchronize(st));
    TTC_CUDA(cudaStreamSynchronize(h->in_stream));
    return TTC_OK;
}

int ttc_lqr_solve_host(ttc_lqr_handle* h, const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                       const ttc_operand* R, const ttc_operand* x0, int32_t H, float* K, float* P, float* x,
                       float* u, int32_t* info, uint32_t flags)
{
    if (!h)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null handle");
    // alignment of host pointers is irrelevant; validate the rest through a relaxed copy
    if (H < 1 || H > h->cfg.max_horizon)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "H=%d outside [1, max_horizon=%d]", H, h->cfg.max_horizon);
    if (flags & ~(TTC_OUT_FIRST_ONLY | TTC_OUT_BF16))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "unknown flag bits 0x%x", flags);
    TTC_CUDA(cudaSetDevice(h->cfg.device));
    { int sp = ensure_host_pipeline(h); if (sp) return sp; }
    const int n = h->cfg.n, m = h->cfg.m;
    const long long N = h->N, b0 = h->cfg.batch[0], b1 = h->cfg.batch[1], b2 = h->cfg.batch[2];
    const bool first = (flags & TTC_OUT_FIRST_ONLY) != 0;
    const ttc_operand* in[5] = {A, B, Q, R, x0};
    const char* names[5] = {"A", "B", "Q", "R", "x0"};
    const size_t elems[5] = {(size_t)n * n, (size_t)n * m, (size_t)n * n, (size_t)m * m, (size_t)n};
    ttc_operand dev[5];
    size_t in_bytes[5] = {0, 0, 0, 0, 0};
    for (int i = 0; i < 5; ++i) {
        dev[i].ptr = nullptr; dev[i].dtype = TTC_F32; dev[i].reserved = 0;
        dev[i].bstride[0] = dev[i].bstride[1] = dev[i].bstride[2] = 0;
        if (!in[i] || !in[i]->ptr) {
            if (i == 4 && !x && !u)
                continue;
            return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s is null", names[i]);
        }
        if (in[i]->dtype != TTC_F32 && !(in[i]->dtype == TTC_BF16 && (i == 2 || i == 4)))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s: dtype %d not supported", names[i], in[i]->dtype);
        size_t extent = elems[i];
        for (int d = 0; d < 3; ++d) {
            if (in[i]->bstride[d] < 0)
                return fail(TTC_STATUS_INVALID_ARGUMENT, "operand %s: negative stride", names[i]);
            extent += (size_t)(h->cfg.batch[d] - 1) * (size_t)in[i]->bstride[d];
        }
        in_bytes[i] = extent * (in[i]->dtype == TTC_BF16 ? 2 : 4);
        int s = ensure(h->st_in[i], in_bytes[i]);
        if (s) return s;
        dev[i] = *in[i];
        dev[i].ptr = h->st_in[i].ptr;
    }
    void* host_out[5] = {K, P, x, u, info};
    const size_t esz = (flags & TTC_OUT_BF16) ? 2 : sizeof(float);     // K, P, x, u as bfloat16 halve the copy-out
    const size_t per_out[5] = {                        // bytes per instance
        esz * (size_t)H * m * n, esz * (size_t)(first ? 1 : H + 1) * n * n,
        esz * (size_t)(H + 1) * n, esz * (size_t)(first ? 1 : H) * m, sizeof(int32_t)};
    void* dev_out[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    size_t total_bytes = 0;
    for (int i = 0; i < 5; ++i) {
        total_bytes += in_bytes[i];
        if (host_out[i]) {
            int s = ensure(h->st_out[i], per_out[i] * (size_t)N);
            if (s) return s;
            dev_out[i] = h->st_out[i].ptr;
            total_bytes += per_out[i] * (size_t)N;
        }
    }

    // ---- slices of the token dimension: copy in, solve and copy out overlap across slices
    int nslice = 1;
    if (total_bytes >= ((size_t)64 << 20) && b2 >= 256) {
        nslice = (int)(b2 / 128 < kMaxSlices ? b2 / 128 : kMaxSlices);
        for (int i = 0; i < 5 && nslice > 1; ++i) {    // per-token operands must have separable rows
            if (!dev[i].ptr || in[i]->bstride[2] == 0)
                continue;
            const long long s1 = in[i]->bstride[1], s2 = in[i]->bstride[2];
            if (s2 < (long long)elems[i] || (b1 > 1 && s1 != 0 && s1 < (b2 - 1) * s2 + (long long)elems[i]))
                nslice = 1;
        }
    }
    long long tslice = (b2 + nslice - 1) / nslice;
    tslice = (tslice + 15) / 16 * 16;
    // few bytes per instance and step: the solve, not the link, sets the pace (a problem bound by its copies is better
    // off with the shortest slices, whose first copy-in and last copy-out are all that stays exposed)
    const bool solve_bound = (double)total_bytes < 64.0 * n * (double)N * H;
    long long edge = 0;                                // tokens of one round of the grid (0: unknown)
    if (nslice > 1 && solve_bound && n == m && (n == 16 || n == 32 || n == 64)) {
        // The kernels behind these shapes run a persistent grid over work items of a few tokens of one head.  A slice
        // whose items do not fill a whole number of rounds of that grid leaves SMs idle in its last round (a slice
        // of 128 tokens x 32 heads is 128 items for 148 CTAs of the n = 64 kernel), so prefer the slice length that
        // fills its rounds best, among those that are at least 128 tokens and keep the slice count within the limit.
        const int item_tokens = n == 64 ? 32 : n == 32 ? 4 : 8;
        const long long grid = (long long)h->sm_count * (n == 64 ? 1 : n == 32 ? 3 : 4);
        const double round_tokens = (double)(grid * item_tokens) / (double)(b0 * b1);      // tokens per head in one round
        auto fill = [&](long long t) {
            const double rounds = std::ceil((double)((t + item_tokens - 1) / item_tokens * item_tokens) / round_tokens - 1e-9);
            return (double)t / (rounds * round_tokens);
        };
        long long best = tslice;
        double best_fill = fill(tslice);
        for (int j = 1; j <= 8; ++j) {
            const long long step = item_tokens > 16 ? item_tokens : 16;
            const long long t = (long long)(j * round_tokens) / step * step;
            if (t < 128 || t >= b2 || (b2 + t - 1) / t > kMaxSlices)
                continue;
            if (fill(t) > best_fill + 0.03) {
                best = t;
                best_fill = fill(t);
            }
        }
        tslice = best;
        const long long step = item_tokens > 16 ? item_tokens : 16;
        edge = (long long)round_tokens / step * step;
    }
    nslice = (int)((b2 + tslice - 1) / tslice);
    // slice boundaries; a solve-bound pipeline starts and ends with a short slice (one round of the grid, 128 tokens
    // at least): the first copy-in and the last copy-out are the only copies that nothing overlaps
    long long cut[kMaxSlices + 1];
    for (int c = 0; c <= nslice; ++c)
        cut[c] = (c * tslice < b2) ? c * tslice : b2;
    if (nslice > 2 && edge >= 128 && tslice >= 2 * edge) {
        const long long mid = b2 - 2 * edge;
        const int nmid = (int)((mid + tslice - 1) / tslice);
        if (mid > 0 && nmid + 2 <= kMaxSlices) {
            nslice = nmid + 2;
            cut[0] = 0;
            for (int c = 0; c < nmid; ++c)
                cut[c + 1] = edge + c * tslice;
            cut[nmid + 1] = b2 - edge;
            cut[nmid + 2] = b2;
        }
    }

    h->last_launches = 0;
    { int se = clear_device_error(h, h->host_stream); if (se) return se; }
    for (int i = 0; i < 5; ++i)                        // operands shared along the token dimension: whole, once
        if (dev[i].ptr && (nslice == 1 || in[i]->bstride[2] == 0))
            TTC_CUDA(cudaMemcpyAsync(h->st_in[i].ptr, in[i]->ptr, in_bytes[i], cudaMemcpyHostToDevice, h->in_stream));
    for (int c = 0; c < nslice; ++c) {
        const long long t0 = cut[c], tc = cut[c + 1] - cut[c];
        if (nslice > 1)
            for (int i = 0; i < 5; ++i) {
                if (!dev[i].ptr || in[i]->bstride[2] == 0)
                    continue;
                const size_t es = in[i]->dtype == TTC_BF16 ? 2 : 4;
                const long long s0 = in[i]->bstride[0], s1 = in[i]->bstride[1], s2 = in[i]->bstride[2];
                const size_t width = ((size_t)(tc - 1) * s2 + elems[i]) * es;
                const size_t rows = (s1 == 0) ? 1 : (size_t)b1;
                const size_t pitch = rows > 1 ? (size_t)s1 * es : width;
                for (long long i0 = 0; i0 < (s0 == 0 ? 1 : b0); ++i0) {
                    const size_t off = ((size_t)i0 * s0 + (size_t)t0 * s2) * es;
                    if (rows > 1 && pitch <= h->max_pitch) {
                        TTC_CUDA(cudaMemcpy2DAsync(static_cast<char*>(h->st_in[i].ptr) + off, pitch,
                                                   static_cast<const char*>(in[i]->ptr) + off, pitch, width, rows,
                                                   cudaMemcpyHostToDevice, h->in_stream));
                    } else {                           // one row, or rows further apart than a 2D copy allows
                        for (size_t rr = 0; rr < rows; ++rr)
                            TTC_CUDA(cudaMemcpyAsync(static_cast<char*>(h->st_in[i].ptr) + off + rr * pitch,
                                                     static_cast<const char*>(in[i]->ptr) + off + rr * pitch, width,
                                                     cudaMemcpyHostToDevice, h->in_stream));
                    }
                }
            }
        TTC_CUDA(cudaEventRecord(h->ev_in[c], h->in_stream));
        TTC_CUDA(cudaStreamWaitEvent(h->host_stream, h->ev_in[c], 0));
        int s = solve_window(h, &dev[0], &dev[1], &dev[2], &dev[3], dev[4].ptr ? &dev[4] : nullptr, H,
                             (float*)dev_out[0], (float*)dev_out[1], (float*)dev_out[2], (float*)dev_out[3],
                             (int32_t*)dev_out[4], flags, h->host_stream, t0, tc);
        if (s) {
            cudaDeviceSynchronize();
            return s;
        }
        TTC_CUDA(cudaEventRecord(h->ev_done[c], h->host_stream));
        TTC_CUDA(cudaStreamWaitEvent(h->out_stream, h->ev_done[c], 0));
        for (int i = 0; i < 5; ++i) {
            if (!host_out[i])
                continue;
            if (nslice == 1) {
                TTC_CUDA(cudaMemcpyAsync(host_out[i], dev_out[i], per_out[i] * (size_t)N, cudaMemcpyDeviceToHost, h->out_stream));
            } else {                                   // rows = (sequence, head), one run of tc instances per row
                const size_t off = (size_t)t0 * per_out[i], pitch = (size_t)b2 * per_out[i];
                const size_t rows = (size_t)(b0 * b1), width = (size_t)tc * per_out[i];
                if (rows > 1 && pitch <= h->max_pitch) {
                    TTC_CUDA(cudaMemcpy2DAsync(static_cast<char*>(host_out[i]) + off, pitch,
                                               static_cast<const char*>(dev_out[i]) + off, pitch, width, rows,
                                               cudaMemcpyDeviceToHost, h->out_stream));
                } else {                               // a 2D copy cannot express a pitch above the device's limit
                    for (size_t rr = 0; rr < rows; ++rr)
                        TTC_CUDA(cudaMemcpyAsync(static_cast<char*>(host_out[i]) + off + rr * pitch,
                                                 static_cast<const char*>(dev_out[i]) + off + rr * pitch, width,
                                                 cudaMemcpyDeviceToHost, h->out_stream));
                }
            }
        }
    }
    TTC_CUDA(cudaStreamSynchronize(h->out_stream));
    TTC_CUDA(cudaStreamSynchronize(h->host_stream));
    if (h->last_kernel == TTC_KERNEL_RICCATI_UMMA) {   // a bounded wait that ran out in ANY slice leaves the word set
        int flag = 0;
        TTC_CUDA(cudaMemcpy(&flag, static_cast<int*>(h->ws_E.ptr) + 1, sizeof(int), cudaMemcpyDeviceToHost));
        if (flag)
            return fail(TTC_STATUS_CUDA_ERROR, "a bounded wait inside the kernel ran out: the outputs are not valid");
    }
    return TTC_OK;
}

} // extern "C"

extern "C" int ttc_lqr_measure_fp32_peak(int32_t device, double* tflops_scalar, double* tflops_packed)
{
    if (!tflops_scalar || !tflops_packed)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null result pointer");
    int ndev = 0;
    TTC_CUDA(cudaGetDeviceCount(&ndev));
    if (device < 0 || device >= ndev)
        return fail(TTC_STATUS_CUDA_ERROR, "device %d not present (%d devices)", device, ndev);
    TTC_CUDA(cudaSetDevice(device));
    int sms = 0;
    TTC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    float* sink = nullptr;
    TTC_CUDA(cudaMalloc(&sink, sizeof(float) * probe::THREADS));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    const int iters = 8192, blocks = 2 * sms;
    double best[2] = {0.0, 0.0};
    for (int variant = 0; variant < 2 && e == cudaSuccess; ++variant)
        for (int rep = 0; rep < 6 && e == cudaSuccess; ++rep) {          // rep 0 warms up
            cudaEventRecord(e0, 0);
            if (variant == 0)
                probe::fma_chain_kernel<false><<<blocks, probe::THREADS>>>(iters, 1.0f, sink);
            else
                probe::fma_chain_kernel<true><<<blocks, probe::THREADS>>>(iters, 1.0f, sink);
            cudaEventRecord(e1, 0);
            e = cudaEventSynchronize(e1);
            float ms = 0.f;
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
            if (e == cudaSuccess && rep > 0 && ms > 0.f) {
                const double tf = probe::launch_flops(blocks, iters) / (ms * 1e-3) / 1e12;
                if (tf > best[variant]) best[variant] = tf;
            }
        }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    if (e != cudaSuccess)
        return fail(TTC_STATUS_CUDA_ERROR, "fp32 peak measurement: %s", cudaGetErrorString(e));
    *tflops_scalar = best[0];
    *tflops_packed = best[1];
    return TTC_OK;
}

extern "C" int ttc_lqr_selftest_bounded_wait(int32_t device, int32_t poll_limit, int32_t* timed_out)
{
    if (!timed_out)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null result pointer");
    if (poll_limit < 1 || poll_limit > (1 << 20))
        return fail(TTC_STATUS_INVALID_ARGUMENT, "poll_limit=%d outside [1, 2^20]", poll_limit);
    int ndev = 0;
    TTC_CUDA(cudaGetDeviceCount(&ndev));
    if (device < 0 || device >= ndev)
        return fail(TTC_STATUS_CUDA_ERROR, "device %d not present (%d devices)", device, ndev);
    TTC_CUDA(cudaSetDevice(device));
    int* flag = nullptr;
    TTC_CUDA(cudaMalloc(&flag, sizeof(int)));
    cudaError_t e = cudaMemset(flag, 0, sizeof(int));
    if (e == cudaSuccess) {
        umma64::bounded_wait_selftest_kernel<<<1, 32>>>(poll_limit, flag);
        e = cudaGetLastError();
    }
    int host = 0;
    if (e == cudaSuccess)
        e = cudaMemcpy(&host, flag, sizeof(int), cudaMemcpyDeviceToHost);
    cudaFree(flag);
    if (e != cudaSuccess)
        return fail(TTC_STATUS_CUDA_ERROR, "bounded-wait self test: %s", cudaGetErrorString(e));
    *timed_out = host;
    return TTC_OK;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free P_0 / u_0 solve for callers that must not allocate device memory (allocator
// callbacks, plugins whose host owns all device memory, real-time loops).  Same kernels as the
// TTC_SCAN first-only path of ttc_lqr_solve; the per-instance scratch (P_1 and a status word)
// sits in a fixed array inside the library image instead of a cudaMalloc'd workspace.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[TTC_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_dev_ptr[kMaxDevices] = {};   // device address of g_noalloc_scratch, per device ordinal
int g_noalloc_sm_count[kMaxDevices] = {};

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address: the
// address each device gave the array is looked up once per device, with that device current.
int noalloc_scratch_for_device(int device, void** ptr, int* sm_count)
{
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_dev_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p)
            return fail(TTC_STATUS_CUDA_ERROR, "cudaGetSymbolAddress(scratch) on device %d: %s", device,
                        cudaGetErrorString(e));
        int major = 0, sms = 0;
        TTC_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        TTC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        if (major != 10)
            return fail(TTC_STATUS_CUDA_ERROR, "device %d is not an sm_100 device", device);
        g_noalloc_sm_count[device] = sms;
        g_noalloc_dev_ptr[device] = p;
    }
    *ptr = g_noalloc_dev_ptr[device];
    *sm_count = g_noalloc_sm_count[device];
    return TTC_OK;
}
} // namespace

extern "C" int ttc_lqr_solve_first_noalloc(int32_t n, int32_t m, const int64_t batch[3], int32_t device,
                                           const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                                           const ttc_operand* R, const ttc_operand* x0, int32_t H, float* P0,
                                           float* u0, int32_t* info, void* cuda_stream)
{
    if (n < 1 || n > 64 || m < 1 || m > 64)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "n=%d, m=%d outside [1, 64]", n, m);
    if (!batch)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "null batch");
    if (H < 1 || H > 65536)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "H=%d outside [1, 65536]", H);
    if (device < 0 || device >= kMaxDevices)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "device %d outside [0, %d)", device, kMaxDevices);
    long long N = 1;
    for (int d = 0; d < 3; ++d) {
        if (batch[d] < 1 || batch[d] > (1ll << 31))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "batch[%d]=%lld out of range", d, (long long)batch[d]);
        N *= batch[d];
        if (N > (1ll << 31))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "more than 2^31 instances");
    }
    const size_t p1_bytes = ((size_t)N * n * n * sizeof(float) + 255) & ~(size_t)255;
    const size_t need = p1_bytes + (size_t)N * sizeof(int);
    if (need > (size_t)TTC_NOALLOC_SCRATCH_BYTES)
        return fail(TTC_STATUS_INVALID_ARGUMENT,
                    "allocation-free solve: %lld instances of n=%d need %zu bytes of scratch but the built-in "
                    "array holds %u; split the batch or use ttc_lqr_solve",
                    N, n, need, (unsigned)TTC_NOALLOC_SCRATCH_BYTES);
    int s;
    if ((s = check_operand("A", A, false, false))) return s;
    if ((s = check_operand("B", B, false, false))) return s;
    if ((s = check_operand("Q", Q, true, false))) return s;
    if ((s = check_operand("R", R, false, false))) return s;
    if ((s = check_operand("x0", x0, true, u0 == nullptr))) return s;
    if (!P0 && !u0 && !info)
        return fail(TTC_STATUS_INVALID_ARGUMENT, "no output requested");
    const void* outs[3] = {P0, u0, info};
    for (int i = 0; i < 3; ++i)
        if (outs[i] && (reinterpret_cast<uintptr_t>(outs[i]) & 15u))
            return fail(TTC_STATUS_INVALID_ARGUMENT, "an output pointer is not 16-byte aligned");
    int ndev = 0;
    TTC_CUDA(cudaGetDeviceCount(&ndev));
    if (device >= ndev)
        return fail(TTC_STATUS_CUDA_ERROR, "device %d not present (%d devices)", device, ndev);
    TTC_CUDA(cudaSetDevice(device));
    void* scratch = nullptr;
    int sm_count = 0;
    if ((s = noalloc_scratch_for_device(device, &scratch, &sm_count))) return s;

    SolveParams p;
    p.n = n; p.m = m; p.H = H;
    p.b0 = batch[0]; p.b1 = batch[1]; p.b2 = batch[2]; p.N = N;
    p.t0 = 0; p.tcount = batch[2];
    p.A = to_dev(A); p.B = to_dev(B); p.Q = to_dev(Q); p.R = to_dev(R); p.x0 = to_dev(x0);
    p.Qf = to_dev(nullptr);
    p.r = to_dev(nullptr);
    p.r_count = 0;
    p.K = nullptr; p.P = P0; p.x = nullptr; p.u = u0; p.info = info;
    p.Kws = nullptr;
    p.kff = nullptr; p.pvec = nullptr;
    p.first_only = 1;
    p.out_bf16 = 0;
    float* p1 = static_cast<float*>(scratch);
    int* flags = reinterpret_cast<int*>(static_cast<unsigned char*>(scratch) + p1_bytes);
    int launches = 0;
    cudaError_t e = launch_scan_path(p, p1, flags, /*pfull=*/0, sm_count, static_cast<cudaStream_t>(cuda_stream),
                                     &launches);
    if (e != cudaSuccess)
        return fail(TTC_STATUS_CUDA_ERROR, "allocation-free solve launch: %s", cudaGetErrorString(e));
    return TTC_OK;
}
