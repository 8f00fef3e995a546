// C ABI of the CERAR library: plan life-cycle, round state machine, counters,
// argument checking, and the launches of the data-path kernels.
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/cerar.h"
#include "kernels.cuh"
#include "plan.hpp"

namespace cerar {
}

struct cerar_plan {
    cerar::HostPlan host;
    // device copies (fp32): U_i as the c x c encode matrix, R_i as the (L+1) x c decode matrix
    float* d_U = nullptr;
    float* d_R = nullptr;
    int* d_status = nullptr;
    // copy streams and events of the host-buffer entry point (created with the plan)
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
    cudaEvent_t ev_start = nullptr, ev_h2d[3] = {nullptr, nullptr, nullptr}, ev_comp[3] = {nullptr, nullptr, nullptr},
                ev_d2h[3] = {nullptr, nullptr, nullptr};
    int device = -1;
    int num_sms = 0;
    bool on_device = false;
    // diagnostics cache
    bool info_done = false;
    cerar_plan_info_t info{};
    // state machine and counters
    int encoded = 0;
    int rounds_done = 0;
    int64_t cur_d = 0;
    uint64_t bytes_forwarded = 0;
    uint64_t launches = 0;
    int kernel_mode = 0;
};

namespace {

thread_local std::string g_err;

cerar_status_t fail(cerar_status_t s, const std::string& msg) {
    g_err = msg;
    return s;
}

cerar_status_t cuda_fail(cudaError_t e, const char* what) {
    g_err = std::string(what) + ": " + cudaGetErrorString(e);
    return CERAR_ERR_CUDA;
}

cerar_status_t upload(cerar_plan* P) {
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || count == 0) {
        cudaGetLastError();     // clear the sticky "no device" error
        return CERAR_OK;        // host-only plan
    }
    const int N = P->host.N, c = P->host.c, L = P->host.L;
    if ((e = cudaGetDevice(&P->device)) != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, P->device)) != cudaSuccess) return cuda_fail(e, "cudaGetDeviceProperties");
    P->num_sms = prop.multiProcessorCount;
    std::vector<float> hU((size_t)N * c * c), hR((size_t)N * (L + 1) * c);
    for (int i = 0; i < N; ++i) {
        for (size_t t = 0; t < (size_t)c * c; ++t) hU[(size_t)i * c * c + t] = (float)P->host.U[i][t];
        for (size_t t = 0; t < (size_t)(L + 1) * c; ++t) hR[(size_t)i * (L + 1) * c + t] = (float)P->host.R[i][t];
    }
    for (float v : hU) if (!std::isfinite(v)) return fail(CERAR_ERR_SINGULAR, "an encoder entry overflows fp32");
    for (float v : hR) if (!std::isfinite(v)) return fail(CERAR_ERR_SINGULAR, "a decoder entry overflows fp32");
    if ((e = cudaMalloc(&P->d_U, hU.size() * sizeof(float))) != cudaSuccess) return cuda_fail(e, "cudaMalloc U");
    if ((e = cudaMalloc(&P->d_R, hR.size() * sizeof(float))) != cudaSuccess) return cuda_fail(e, "cudaMalloc R");
    if ((e = cudaMalloc(&P->d_status, sizeof(int))) != cudaSuccess) return cuda_fail(e, "cudaMalloc status");
    if ((e = cudaMemcpy(P->d_U, hU.data(), hU.size() * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess)
        return cuda_fail(e, "upload U");
    if ((e = cudaMemcpy(P->d_R, hR.data(), hR.size() * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess)
        return cuda_fail(e, "upload R");
    if ((e = cudaMemset(P->d_status, 0, sizeof(int))) != cudaSuccess) return cuda_fail(e, "memset status");
    if ((e = cudaStreamCreateWithFlags(&P->s_h2d, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e, "stream");
    if ((e = cudaStreamCreateWithFlags(&P->s_d2h, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e, "stream");
    if ((e = cudaEventCreateWithFlags(&P->ev_start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "event");
    for (int b = 0; b < 3; ++b) {
        if ((e = cudaEventCreateWithFlags(&P->ev_h2d[b], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "event");
        if ((e = cudaEventCreateWithFlags(&P->ev_comp[b], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "event");
        if ((e = cudaEventCreateWithFlags(&P->ev_d2h[b], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "event");
    }
    P->on_device = true;
    return CERAR_OK;
}

cerar_status_t finish_create(cerar_plan* P, bool host_only, cerar_plan_t** out) {
    if (!host_only) {
        cerar_status_t st = upload(P);
        if (st != CERAR_OK) { cerar_plan_destroy(P); return st; }
    }
    *out = P;
    return CERAR_OK;
}

// cerar_allreduce_sim runs all rounds in one launch up to this workspace size (half of the 126 MB L2)
constexpr size_t kOneLaunchRoundsBytes = (size_t)64 << 20;

cerar_status_t check_data_call(const cerar_plan* P, int64_t d, int64_t* p_out) {
    if (!P) return fail(CERAR_ERR_INVALID_ARG, "plan is NULL");
    if (!P->on_device) return fail(CERAR_ERR_CUDA, "plan has no device copies (no CUDA device, or host_only)");
    if (d <= 0 || d % P->host.c != 0) return fail(CERAR_ERR_SHAPE, "d must be a positive multiple of c");
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != P->device)
        return fail(CERAR_ERR_CUDA, "the device the plan was created on must be current");
    *p_out = d / P->host.c;
    return CERAR_OK;
}

}  // namespace

extern "C" {

const char* cerar_status_string(cerar_status_t s) {
    switch (s) {
        case CERAR_OK: return "ok";
        case CERAR_ERR_INVALID_ARG: return "invalid argument";
        case CERAR_ERR_SHAPE: return "bad shape";
        case CERAR_ERR_SINGULAR: return "singular or non-finite design";
        case CERAR_ERR_NOT_CONVERGED: return "design did not meet its constraint";
        case CERAR_ERR_STATE: return "call out of order";
        case CERAR_ERR_CUDA: return "CUDA error";
        case CERAR_ERR_NOMEM: return "out of memory";
        case CERAR_ERR_TIMEOUT: return "device-side wait timed out";
        case CERAR_ERR_TOO_LARGE: return "size beyond a fixed capacity";
        case CERAR_ERR_BOUNDS: return "checked build: address outside its buffer";
    }
    return "unknown status";
}

const char* cerar_last_error(void) { return g_err.c_str(); }

int cerar_build_is_checked(void) {
#ifdef CERAR_BOUNDS_CHECK
    return 1;
#else
    return 0;
#endif
}

// for the library's other translation units
void cerar_internal_set_error(const char* msg) { g_err = msg ? msg : ""; }
// device ordinal the plan's fp32 copies live on, or -1 for a plan without device copies
int cerar_internal_plan_device(const cerar_plan_t* P) { return (P && P->on_device) ? P->device : -1; }

cerar_status_t cerar_plan_create_ex(int N, int c, cerar_construction_t kind, double param,
                                    const cerar_options_t* opt, cerar_plan_t** out) {
    if (!out) return fail(CERAR_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (N < 2 || c < N || c > 512) return fail(CERAR_ERR_INVALID_ARG, "need 2 <= N <= c <= 512");
    cerar_options_t o;
    std::memset(&o, 0, sizeof(o));
    if (opt) o = *opt;
    cerar_plan* P = new (std::nothrow) cerar_plan();
    if (!P) return fail(CERAR_ERR_NOMEM, "plan allocation failed");
    std::string err;
    int st = cerar::BUILD_INVALID;
    std::vector<double> Bdef;
    const double* B = o.B;
    if (!B && kind != CERAR_VANDERMONDE) {
        Bdef = cerar::default_base_matrix(N, c, o.seed);
        B = Bdef.data();
    }
    switch (kind) {
        case CERAR_VANDERMONDE: st = cerar::build_vandermonde(N, c, param, o.h, P->host, err); break;
        case CERAR_EPSILON: st = cerar::build_epsilon(N, c, param, B, o.h, P->host, err); break;
        case CERAR_KAPPA:
            st = cerar::build_kappa(N, c, param, B, o.h, o.eps_init, o.als_iters, o.als_tol, P->host, err);
            break;
        default: err = "unknown construction"; break;
    }
    if (st != cerar::BUILD_OK) {
        delete P;
        return fail((cerar_status_t)st, err);
    }
    return finish_create(P, o.host_only != 0, out);
}

cerar_status_t cerar_plan_create(int N, int c, cerar_construction_t kind, double param, cerar_plan_t** out) {
    return cerar_plan_create_ex(N, c, kind, param, nullptr, out);
}

cerar_status_t cerar_plan_create_custom(int N, int c, const double* U, const double* R, int host_only,
                                        cerar_plan_t** out) {
    if (!out) return fail(CERAR_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (N < 2 || c < N || c > 512) return fail(CERAR_ERR_INVALID_ARG, "need 2 <= N <= c <= 512");
    if (!U || !R) return fail(CERAR_ERR_INVALID_ARG, "U or R is NULL");
    cerar_plan* P = new (std::nothrow) cerar_plan();
    if (!P) return fail(CERAR_ERR_NOMEM, "plan allocation failed");
    const int L = c + N - 2;
    P->host.N = N; P->host.c = c; P->host.L = L; P->host.kind = 3;
    P->host.U.resize(N); P->host.R.resize(N);
    for (int i = 0; i < N; ++i) {
        P->host.U[i].assign(U + (size_t)i * c * c, U + (size_t)(i + 1) * c * c);
        P->host.R[i].assign(R + (size_t)i * (L + 1) * c, R + (size_t)(i + 1) * (L + 1) * c);
        for (double v : P->host.U[i]) if (!std::isfinite(v)) { delete P; return fail(CERAR_ERR_SINGULAR, "non-finite U"); }
        for (double v : P->host.R[i]) if (!std::isfinite(v)) { delete P; return fail(CERAR_ERR_SINGULAR, "non-finite R"); }
    }
    return finish_create(P, host_only != 0, out);
}

void cerar_plan_destroy(cerar_plan_t* P) {
    if (!P) return;
    if (P->on_device || P->d_U || P->d_R || P->d_status) {
        cudaFree(P->d_U); cudaFree(P->d_R); cudaFree(P->d_status);
        if (P->s_h2d) cudaStreamDestroy(P->s_h2d);
        if (P->s_d2h) cudaStreamDestroy(P->s_d2h);
        if (P->ev_start) cudaEventDestroy(P->ev_start);
        for (int b = 0; b < 3; ++b) {
            if (P->ev_h2d[b]) cudaEventDestroy(P->ev_h2d[b]);
            if (P->ev_comp[b]) cudaEventDestroy(P->ev_comp[b]);
            if (P->ev_d2h[b]) cudaEventDestroy(P->ev_d2h[b]);
        }
    }
    delete P;
}

cerar_status_t cerar_plan_get_U(const cerar_plan_t* P, int worker, double* out) {
    if (!P || !out || worker < 0 || worker >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "bad argument");
    std::memcpy(out, P->host.U[worker].data(), P->host.U[worker].size() * sizeof(double));
    return CERAR_OK;
}

cerar_status_t cerar_plan_get_R(const cerar_plan_t* P, int worker, double* out) {
    if (!P || !out || worker < 0 || worker >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "bad argument");
    std::memcpy(out, P->host.R[worker].data(), P->host.R[worker].size() * sizeof(double));
    return CERAR_OK;
}

cerar_status_t cerar_plan_info(cerar_plan_t* P, cerar_plan_info_t* out) {
    if (!P || !out) return fail(CERAR_ERR_INVALID_ARG, "bad argument");
    if (!P->info_done) {
        cerar_plan_info_t& I = P->info;
        I.N = P->host.N; I.c = P->host.c; I.L = P->host.L;
        I.construction = P->host.kind; I.param = P->host.param;
        I.phi = (P->host.phi_closed >= 0) ? P->host.phi_closed : cerar::phi_direct(P->host);
        I.kappa_U_max = cerar::kappa_U_max(P->host);
        I.kappa_M_max = cerar::kappa_M_max(P->host);
        I.inv_residual_max = P->host.inv_residual_max;
        double mu = 0, mr = 0;
        for (const auto& m : P->host.U) for (double v : m) mu = std::fmax(mu, std::fabs(v));
        for (const auto& m : P->host.R) for (double v : m) mr = std::fmax(mr, std::fabs(v));
        I.abs_U_max = mu; I.abs_R_max = mr;
        I.als_iters_done = P->host.als_iters_done;
        P->info_done = true;
    }
    P->info.on_device = P->on_device ? 1 : 0;
    *out = P->info;
    return CERAR_OK;
}

cerar_status_t cerar_design_gamma(int N, int c, const double* B, uint64_t seed, const double* h, double* gamma_out) {
    if (!gamma_out || N < 2 || c < N) return fail(CERAR_ERR_INVALID_ARG, "need 2 <= N <= c and an output pointer");
    std::vector<double> Bdef, hdef;
    if (!B) { Bdef = cerar::default_base_matrix(N, c, seed); B = Bdef.data(); }
    if (!h) { hdef = cerar::default_nodes(c); h = hdef.data(); }
    for (int i = 0; i < N * c; ++i) if (!std::isfinite(B[i])) return fail(CERAR_ERR_INVALID_ARG, "B is not finite");
    for (int i = 0; i < c; ++i) if (!std::isfinite(h[i])) return fail(CERAR_ERR_INVALID_ARG, "h is not finite");
    *gamma_out = cerar::k_limit_gamma(N, c, B, h);
    return CERAR_OK;
}

cerar_status_t cerar_design_optimize_h(int N, int c, const double* B, uint64_t seed, double* h, int use_start,
                                       int sweeps, int grid, double* gamma_out, int* moves_out) {
    if (!h || N < 2 || c < N) return fail(CERAR_ERR_INVALID_ARG, "need 2 <= N <= c and a buffer for h");
    if (sweeps < 1 || grid < 3 || grid > 1025) return fail(CERAR_ERR_INVALID_ARG, "need sweeps >= 1 and 3 <= grid <= 1025");
    std::vector<double> Bdef;
    if (!B) { Bdef = cerar::default_base_matrix(N, c, seed); B = Bdef.data(); }
    for (int i = 0; i < N * c; ++i) if (!std::isfinite(B[i])) return fail(CERAR_ERR_INVALID_ARG, "B is not finite");
    if (!use_start) {
        const std::vector<double> h0 = cerar::default_nodes(c);
        for (int j = 0; j < c; ++j) h[j] = h0[j];
    }
    bool any = false;
    for (int j = 0; j < c; ++j) {
        if (!std::isfinite(h[j])) return fail(CERAR_ERR_INVALID_ARG, "h is not finite");
        any = any || h[j] != 0.0;
    }
    if (!any) return fail(CERAR_ERR_INVALID_ARG, "the start h is zero");
    const double g = cerar::optimize_h(N, c, B, h, sweeps, grid, moves_out);
    if (gamma_out) *gamma_out = g;
    return CERAR_OK;
}

int64_t cerar_padded_length(const cerar_plan_t* P, int64_t d) {
    if (!P || d <= 0) return 0;
    const int64_t q = 4 * (int64_t)P->host.c;
    return (d + q - 1) / q * q;
}

size_t cerar_workspace_bytes(const cerar_plan_t* P, int64_t d) {
    if (!P || d <= 0 || d % P->host.c != 0) return 0;
    return (size_t)4 * P->host.N * (size_t)(P->host.c + P->host.N) * (size_t)(d / P->host.c);
}

cerar_status_t cerar_encode(cerar_plan_t* P, const float* grads, int64_t grads_stride, float* ws, int64_t d,
                            cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!grads || !ws) return fail(CERAR_ERR_INVALID_ARG, "grads or ws is NULL");
    if (grads_stride < d) return fail(CERAR_ERR_SHAPE, "grads_stride < d");
    const int N = P->host.N, c = P->host.c;
    cerar::ContractArgs a{};
    a.in = grads; a.in_wstride = grads_stride; a.in_rstride = p;
    a.out = ws + (int64_t)N * p; a.out_wstride = (int64_t)(c + N) * p; a.out_rstride = p;
    a.coef = P->d_U; a.K = c; a.J = c; a.skip_row = 1 << 30; a.skip_count = 0;
    a.N = N; a.p = p; a.scale = 1.0f; a.status = P->d_status;
    cudaError_t e = cerar::launch_contract(a, P->kernel_mode, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "encode launch");
    P->encoded = 1; P->rounds_done = 0; P->cur_d = d; P->bytes_forwarded = 0;
    return CERAR_OK;
}

cerar_status_t cerar_ring_round(cerar_plan_t* P, float* ws, int64_t d, int k, cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws) return fail(CERAR_ERR_INVALID_ARG, "ws is NULL");
    if (!P->encoded || d != P->cur_d) return fail(CERAR_ERR_STATE, "encode (with the same d) must come first");
    if (k != P->rounds_done + 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "rounds must run in order 1..L");
    cerar::RoundArgs a{ws, p, P->host.N, P->host.c, k, 0};
    a.status = P->d_status;
    cudaError_t e = cerar::launch_round(a, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "round launch");
    P->rounds_done = k;
    P->bytes_forwarded += (uint64_t)4 * (uint64_t)p;
    return CERAR_OK;
}

cerar_status_t cerar_ring_rounds(cerar_plan_t* P, float* ws, int64_t d, int k_first, int k_last,
                                 cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws) return fail(CERAR_ERR_INVALID_ARG, "ws is NULL");
    if (!P->encoded || d != P->cur_d) return fail(CERAR_ERR_STATE, "encode (with the same d) must come first");
    if (k_first != P->rounds_done + 1 || k_last < k_first || k_last > P->host.L)
        return fail(CERAR_ERR_STATE, "rounds must run in order 1..L");
    cerar::RoundArgs a{ws, p, P->host.N, P->host.c, k_first, 0};
    a.status = P->d_status;
    cudaError_t e = cerar::launch_rounds_multi(a, k_last, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rounds launch");
    P->rounds_done = k_last;
    P->bytes_forwarded += (uint64_t)4 * (uint64_t)p * (uint64_t)(k_last - k_first + 1);
    return CERAR_OK;
}

cerar_status_t cerar_decode(cerar_plan_t* P, const float* ws, float* out, int64_t out_stride, int64_t d,
                            float scale, cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !out) return fail(CERAR_ERR_INVALID_ARG, "ws or out is NULL");
    if (out_stride < d) return fail(CERAR_ERR_SHAPE, "out_stride < d");
    if (!P->encoded || d != P->cur_d || P->rounds_done != P->host.L)
        return fail(CERAR_ERR_STATE, "decode needs encode and all L rounds");
    const int N = P->host.N, c = P->host.c, L = P->host.L;
    cerar::ContractArgs a{};
    a.in = ws; a.in_wstride = (int64_t)(c + N) * p; a.in_rstride = p;
    a.out = out; a.out_wstride = out_stride; a.out_rstride = p;
    a.coef = P->d_R; a.K = L + 1; a.J = c; a.skip_row = L; a.skip_count = 1;     // y_{L+1} sits in slot L+1
    a.N = N; a.p = p; a.scale = scale; a.status = P->d_status;
    cudaError_t e = cerar::launch_contract(a, P->kernel_mode, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "decode launch");
    const float* ws_end = ws + (size_t)N * (size_t)(c + N) * (size_t)p;
    if (out + (size_t)(N - 1) * out_stride + d > ws && out < ws_end)
        P->encoded = 0;     // decoded in place: the observations are gone
    return CERAR_OK;
}

cerar_status_t cerar_allreduce_sim(cerar_plan_t* P, const float* grads, int64_t grads_stride, float* out,
                                   int64_t out_stride, float* ws, int64_t d, float scale, cerar_stream_t stream) {
    cerar_status_t st = cerar_encode(P, grads, grads_stride, ws, d, stream);
    if (st != CERAR_OK) return st;
    // One launch for all rounds (one warp per worker, messages handed on through shared memory as well
    // as stored) wherever that kernel applies at full width: it measured faster than one launch per
    // round at every shape tried (from 1.2 times at d = 2^30 to 10 times where the launches dominate).
    const size_t one_launch_limit = cerar::g_tune_rounds_one_launch_mb > 0
                                        ? (size_t)cerar::g_tune_rounds_one_launch_mb << 20 : kOneLaunchRoundsBytes;
    const int64_t p_sim = d / P->host.c;
    bool one_launch = cerar_workspace_bytes(P, d) <= one_launch_limit;
    if (cerar::g_tune_rounds_one_launch_mb == 0 && P->host.N <= 32)
        one_launch = one_launch || p_sim <= 65536 || p_sim % 4 == 0;
    if (cerar::g_tune_rounds_one_launch_off) one_launch = false;
    if (one_launch) {
        if ((st = cerar_ring_rounds(P, ws, d, 1, P->host.L, stream)) != CERAR_OK) return st;
    } else {
        for (int k = 1; k <= P->host.L; ++k)
            if ((st = cerar_ring_round(P, ws, d, k, stream)) != CERAR_OK) return st;
    }
    return cerar_decode(P, ws, out, out_stride, d, scale, stream);
}

cerar_status_t cerar_allreduce_sim_host(cerar_plan_t* P, const float* h_grads, int64_t h_grads_stride,
                                        float* h_out, int64_t h_out_stride, float* ws, int64_t d, float scale,
                                        cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!h_grads || !h_out || !ws) return fail(CERAR_ERR_INVALID_ARG, "NULL buffer");
    if (h_grads_stride < d || h_out_stride < d) return fail(CERAR_ERR_SHAPE, "stride < d");
    const int N = P->host.N, c = P->host.c;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    // Positions are independent, so the job is cut into slices of ps positions that flow
    // through three slice-sized workspaces carved out of ws: the H2D copy of slice i+1 and
    // the D2H copy of slice i-1 (two copy streams, PCIe is full duplex) overlap the kernels
    // of slice i, which run in place on `stream`.
    int64_t ps = p;
    if (p >= 3 * 262144) {
        int64_t nsl = p / 1048576;
        if (nsl < 3) nsl = 3;
        if (nsl > 64) nsl = 64;
        ps = ((p + nsl - 1) / nsl + 127) / 128 * 128;
    }
    const int64_t nslices = (p + ps - 1) / ps;
    const int nbuf = nslices >= 3 ? 3 : 1;
    const int64_t slot_floats = (int64_t)N * (c + N) * ps;      // one slice workspace
    if ((e = cudaEventRecord(P->ev_start, s)) != cudaSuccess) return cuda_fail(e, "event record");
    if ((e = cudaStreamWaitEvent(P->s_h2d, P->ev_start, 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
    if ((e = cudaStreamWaitEvent(P->s_d2h, P->ev_start, 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
    for (int64_t i = 0; i < nslices; ++i) {
        const int b = (int)(i % nbuf);
        const int64_t q0 = i * ps;
        const int64_t pl = (p - q0 < ps) ? (p - q0) : ps;      // positions in this slice
        float* wsl = ws + b * slot_floats;
        const int64_t wstride = (int64_t)(c + N) * pl;
        float* drows = wsl + (int64_t)N * pl;
        if (i >= nbuf && (e = cudaStreamWaitEvent(P->s_h2d, P->ev_d2h[b], 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
        for (int w = 0; w < N; ++w) {
            e = cudaMemcpy2DAsync(drows + w * wstride, (size_t)pl * 4, h_grads + w * h_grads_stride + q0, (size_t)p * 4,
                                  (size_t)pl * 4, (size_t)c, cudaMemcpyHostToDevice, P->s_h2d);
            if (e != cudaSuccess) return cuda_fail(e, "H2D copy");
        }
        if ((e = cudaEventRecord(P->ev_h2d[b], P->s_h2d)) != cudaSuccess) return cuda_fail(e, "event record");
        if ((e = cudaStreamWaitEvent(s, P->ev_h2d[b], 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
        st = cerar_allreduce_sim(P, drows, wstride, drows, wstride, wsl, (int64_t)c * pl, scale, stream);
        if (st != CERAR_OK) return st;
        if ((e = cudaEventRecord(P->ev_comp[b], s)) != cudaSuccess) return cuda_fail(e, "event record");
        if ((e = cudaStreamWaitEvent(P->s_d2h, P->ev_comp[b], 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
        for (int w = 0; w < N; ++w) {
            e = cudaMemcpy2DAsync(h_out + w * h_out_stride + q0, (size_t)p * 4, drows + w * wstride, (size_t)pl * 4,
                                  (size_t)pl * 4, (size_t)c, cudaMemcpyDeviceToHost, P->s_d2h);
            if (e != cudaSuccess) return cuda_fail(e, "D2H copy");
        }
        if ((e = cudaEventRecord(P->ev_d2h[b], P->s_d2h)) != cudaSuccess) return cuda_fail(e, "event record");
    }
    // the caller's stream resumes when the last results are on the host
    for (int b = 0; b < nbuf; ++b)
        if ((e = cudaStreamWaitEvent(s, P->ev_d2h[b], 0)) != cudaSuccess) return cuda_fail(e, "stream wait");
    // counters describe the whole job, not the last slice
    P->cur_d = d;
    P->bytes_forwarded = (uint64_t)4 * (uint64_t)p * (uint64_t)P->host.L;
    return CERAR_OK;
}

// ---------------------------------------------------------------- one worker per GPU
size_t cerar_rank_workspace_bytes(const cerar_plan_t* P, int64_t d) {
    if (!P || d <= 0 || d % P->host.c != 0) return 0;
    return (size_t)4 * (size_t)(P->host.c + P->host.N + 1) * (size_t)(d / P->host.c);
}

cerar_status_t cerar_rank_round_slots(const cerar_plan_t* P, int k, int* slot_prev, int* slot_cancel, int* slot_add,
                                      int* slot_land) {
    if (!P || !slot_prev || !slot_cancel || !slot_add || !slot_land) return fail(CERAR_ERR_INVALID_ARG, "bad argument");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_INVALID_ARG, "round index outside 1..L");
    cerar::rank_round_slots(P->host.N, P->host.c, k, slot_prev, slot_cancel, slot_add, slot_land);
    return CERAR_OK;
}

cerar_status_t cerar_rank_encode(cerar_plan_t* P, int rank, const float* grad, float* ws, int64_t d,
                                 cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!grad || !ws) return fail(CERAR_ERR_INVALID_ARG, "grad or ws is NULL");
    const int N = P->host.N, c = P->host.c;
    if (rank < 0 || rank >= N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    cerar::ContractArgs a{};
    // one worker per call: the worker strides are never stepped, but keep them what they would be
    a.in = grad; a.in_wstride = (int64_t)c * p; a.in_rstride = p;
    a.out = ws + (int64_t)(N + 1) * p; a.out_wstride = (int64_t)(c + N + 1) * p; a.out_rstride = p;
    a.coef = P->d_U + (size_t)rank * c * c; a.K = c; a.J = c; a.skip_row = 1 << 30; a.skip_count = 0;
    a.N = 1; a.p = p; a.scale = 1.0f; a.status = P->d_status;
    cudaError_t e = cerar::launch_contract(a, P->kernel_mode, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank encode launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_round(cerar_plan_t* P, int rank, const float* ws, float* peer_ws, int64_t d, int k,
                                cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !peer_ws) return fail(CERAR_ERR_INVALID_ARG, "ws or peer_ws is NULL");
    if (ws == peer_ws) return fail(CERAR_ERR_INVALID_ARG, "peer_ws must be the next worker's workspace, not this one's");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    cerar::RankRoundArgs a{};
    a.ws = ws; a.peer_ws = peer_ws; a.p = p; a.N = P->host.N; a.c = P->host.c; a.k = k;
    cudaError_t e = cerar::launch_rank_round(a, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank round launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_round_msg(cerar_plan_t* P, int rank, const float* ws, float* msg, int64_t d, int k,
                                    cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !msg) return fail(CERAR_ERR_INVALID_ARG, "ws or msg is NULL");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    cerar::RankRoundArgs a{};
    a.ws = ws; a.peer_ws = msg; a.p = p; a.N = P->host.N; a.c = P->host.c; a.k = k; a.to_message = 1;
    cudaError_t e = cerar::launch_rank_round(a, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank round (message) launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_round_msg_bf16(cerar_plan_t* P, int rank, const float* ws, uint16_t* msg, int64_t d, int k,
                                         cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !msg) return fail(CERAR_ERR_INVALID_ARG, "ws or msg is NULL");
    if (reinterpret_cast<uintptr_t>(msg) & 1u) return fail(CERAR_ERR_INVALID_ARG, "msg must be 2-byte aligned");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    cerar::RankRoundArgs a{};
    a.ws = ws; a.peer_ws = reinterpret_cast<float*>(msg); a.p = p; a.N = P->host.N; a.c = P->host.c; a.k = k;
    a.to_message = 2;
    cudaError_t e = cerar::launch_rank_round(a, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank round (bfloat16 message) launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_recv_bf16(cerar_plan_t* P, int rank, float* ws, const uint16_t* msg, int64_t d, int k,
                                    cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !msg) return fail(CERAR_ERR_INVALID_ARG, "ws or msg is NULL");
    if (reinterpret_cast<uintptr_t>(msg) & 1u) return fail(CERAR_ERR_INVALID_ARG, "msg must be 2-byte aligned");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    int sp, sc, sa, sl;
    cerar::rank_round_slots(P->host.N, P->host.c, k, &sp, &sc, &sa, &sl);
    cudaError_t e = cerar::launch_rank_recv_bf16(ws + (int64_t)sl * p, msg, p, P->num_sms, (cudaStream_t)stream,
                                                 &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank receive (bfloat16 message) launch");
    return CERAR_OK;
}

size_t cerar_fp8_message_bytes(const cerar_plan_t* P, int64_t d) {
    if (!P || d <= 0 || d % P->host.c != 0) return 0;
    return cerar::fp8_message_bytes(d / P->host.c);
}

cerar_status_t cerar_rank_round_msg_fp8(cerar_plan_t* P, int rank, const float* ws, void* msg, int64_t d, int k,
                                        cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !msg) return fail(CERAR_ERR_INVALID_ARG, "ws or msg is NULL");
    if (reinterpret_cast<uintptr_t>(msg) & 15u) return fail(CERAR_ERR_INVALID_ARG, "msg must be 16-byte aligned");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    cerar::RankRoundArgs a{};
    a.ws = ws; a.peer_ws = nullptr; a.p = p; a.N = P->host.N; a.c = P->host.c; a.k = k; a.to_message = 3;
    cudaError_t e = cerar::launch_rank_round_fp8(a, msg, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank round (8-bit message) launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_recv_fp8(cerar_plan_t* P, int rank, float* ws, const void* msg, int64_t d, int k,
                                   cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !msg) return fail(CERAR_ERR_INVALID_ARG, "ws or msg is NULL");
    if (reinterpret_cast<uintptr_t>(msg) & 15u) return fail(CERAR_ERR_INVALID_ARG, "msg must be 16-byte aligned");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    if (k < 1 || k > P->host.L) return fail(CERAR_ERR_STATE, "round index outside 1..L");
    int sp, sc, sa, sl;
    cerar::rank_round_slots(P->host.N, P->host.c, k, &sp, &sc, &sa, &sl);
    cudaError_t e = cerar::launch_rank_recv_fp8(ws + (int64_t)sl * p, msg, p, P->num_sms, (cudaStream_t)stream,
                                                &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank receive (8-bit message) launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_decode(cerar_plan_t* P, int rank, const float* ws, float* out, int64_t d, float scale,
                                 cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !out) return fail(CERAR_ERR_INVALID_ARG, "ws or out is NULL");
    const int N = P->host.N, c = P->host.c, L = P->host.L;
    if (rank < 0 || rank >= N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    cerar::ContractArgs a{};
    a.in = ws; a.in_wstride = (int64_t)(c + N + 1) * p; a.in_rstride = p;
    a.out = out; a.out_wstride = (int64_t)c * p; a.out_rstride = p;
    // y_1..y_L sit in slots 0..L-1, y_{L+1} = delta_c in slot N+c = L+2; slots L and L+1 are spent deltas
    a.coef = P->d_R + (size_t)rank * (L + 1) * c; a.K = L + 1; a.J = c; a.skip_row = L; a.skip_count = 2;
    a.N = 1; a.p = p; a.scale = scale; a.status = P->d_status;
    cudaError_t e = cerar::launch_contract(a, P->kernel_mode, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "rank decode launch");
    return CERAR_OK;
}

namespace {
// Positions per tile of the fused rounds: small enough that a short job still has a few tiles
// per resident block, large enough that polling and publishing two counters per tile and round
// stays a few per cent of the tile's memory time.
int64_t ring_tile_positions(int64_t p) {
    if (cerar::g_tune_ring_tile > 0) return (int64_t)cerar::g_tune_ring_tile;
    return p >= ((int64_t)1 << 23) ? 4 * CERAR_RING_TILE : CERAR_RING_TILE;
}
}  // namespace

int64_t cerar_ring_tiles(const cerar_plan_t* P, int64_t d) {
    if (!P || d <= 0 || d % P->host.c != 0) return 0;
    const int64_t p = d / P->host.c;
    const int64_t tile = ring_tile_positions(p);
    return (p + tile - 1) / tile;
}

namespace {
cerar_status_t ring_fused_common(cerar_plan_t* P, int64_t d, int64_t* p_out) {
    cerar_status_t st = check_data_call(P, d, p_out);
    if (st != CERAR_OK) return st;
    if (P->host.N > cerar::RING_MAX_WORKERS) return fail(CERAR_ERR_INVALID_ARG, "more workers than one launch can serve");
    return CERAR_OK;
}
void ring_fused_fill(cerar::RingFusedArgs& a, const cerar_plan_t* P, int64_t p, unsigned epoch) {
    a.N = P->host.N; a.c = P->host.c; a.p = p;
    a.tile = ring_tile_positions(p); a.ntiles = (p + a.tile - 1) / a.tile;
    a.base = epoch * (unsigned)(P->host.L + 1);
    a.status = P->d_status;
    a.limit_ns = (unsigned long long)(cerar::g_tune_ring_wait_ms > 0 ? cerar::g_tune_ring_wait_ms : 2000) * 1000000ull;
}
}  // namespace

cerar_status_t cerar_ring_rounds_fused_local(cerar_plan_t* P, float* const* ws, unsigned* counters, int64_t d,
                                             unsigned epoch, cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = ring_fused_common(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !counters) return fail(CERAR_ERR_INVALID_ARG, "ws or counters is NULL");
    const int N = P->host.N;
    cerar::RingFusedArgs a{};
    ring_fused_fill(a, P, p, epoch);
    bool vec = (p % 4 == 0);
    for (int i = 0; i < N; ++i) {
        if (!ws[i]) return fail(CERAR_ERR_INVALID_ARG, "a workspace pointer is NULL");
        for (int j = 0; j < i; ++j) if (ws[i] == ws[j]) return fail(CERAR_ERR_INVALID_ARG, "two workers share a workspace");
        vec = vec && ((reinterpret_cast<uintptr_t>(ws[i]) & 15u) == 0);
    }
    a.vec = vec ? 1 : 0;
    for (int i = 0; i < N; ++i) {
        const int nx = (i + 1) % N, pv = (i + N - 1) % N;
        a.ws[i] = ws[i]; a.peer_ws[i] = ws[nx];
        a.landed_local[i] = counters + (size_t)(2 * i) * a.ntiles;
        a.freed_local[i] = counters + (size_t)(2 * i + 1) * a.ntiles;
        a.landed_next[i] = counters + (size_t)(2 * nx) * a.ntiles;
        a.freed_prev[i] = counters + (size_t)(2 * pv + 1) * a.ntiles;
    }
    cudaError_t e = cerar::launch_ring_rounds(a, N, true, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "fused ring rounds launch");
    return CERAR_OK;
}

cerar_status_t cerar_rank_rounds_fused(cerar_plan_t* P, int rank, const float* ws, float* peer_ws,
                                       const unsigned* landed_local, const unsigned* freed_local,
                                       unsigned* landed_next, unsigned* freed_prev, int64_t d, unsigned epoch,
                                       cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = ring_fused_common(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!ws || !peer_ws || !landed_local || !freed_local || !landed_next || !freed_prev)
        return fail(CERAR_ERR_INVALID_ARG, "NULL buffer");
    if (ws == peer_ws) return fail(CERAR_ERR_INVALID_ARG, "peer_ws must be the next worker's workspace, not this one's");
    if (rank < 0 || rank >= P->host.N) return fail(CERAR_ERR_INVALID_ARG, "rank outside 0..N-1");
    cerar::RingFusedArgs a{};
    ring_fused_fill(a, P, p, epoch);
    a.vec = ((p % 4 == 0) && ((reinterpret_cast<uintptr_t>(ws) & 15u) == 0) &&
             ((reinterpret_cast<uintptr_t>(peer_ws) & 15u) == 0)) ? 1 : 0;
    a.ws[0] = ws; a.peer_ws[0] = peer_ws;
    a.landed_local[0] = landed_local; a.freed_local[0] = freed_local;
    a.landed_next[0] = landed_next; a.freed_prev[0] = freed_prev;
    cudaError_t e = cerar::launch_ring_rounds(a, 1, false, P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "fused rank rounds launch");
    return CERAR_OK;
}

cerar_status_t cerar_allreduce_fused(cerar_plan_t* P, const float* grads, int64_t grads_stride, float* out,
                                     int64_t out_stride, int64_t d, float scale, cerar_stream_t stream) {
    int64_t p;
    cerar_status_t st = check_data_call(P, d, &p);
    if (st != CERAR_OK) return st;
    if (!grads || !out) return fail(CERAR_ERR_INVALID_ARG, "grads or out is NULL");
    if (grads_stride < d || out_stride < d) return fail(CERAR_ERR_SHAPE, "stride < d");
    const int N = P->host.N, c = P->host.c;
    if (!cerar::fused_supported(N, c))
        return fail(CERAR_ERR_INVALID_ARG, "the on-chip path needs c <= 32 (a multiple of 4, or 5, 6) and N (c+N) small "
                                           "enough for shared memory; use cerar_allreduce_sim");
    cudaError_t e = cerar::launch_fused(grads, grads_stride, out, out_stride, P->d_U, P->d_R, N, c, p, scale,
                                        P->num_sms, (cudaStream_t)stream, &P->launches);
    if (e != cudaSuccess) return cuda_fail(e, "fused launch");
    // the L rounds ran (on chip): the logical message bytes are the same
    P->encoded = 0; P->rounds_done = P->host.L; P->cur_d = d;
    P->bytes_forwarded = (uint64_t)4 * (uint64_t)p * (uint64_t)P->host.L;
    return CERAR_OK;
}

int cerar_fused_supported(const cerar_plan_t* P) {
    return (P && cerar::fused_supported(P->host.N, P->host.c)) ? 1 : 0;
}

cerar_status_t cerar_get_counters(const cerar_plan_t* P, cerar_counters_t* out) {
    if (!P || !out) return fail(CERAR_ERR_INVALID_ARG, "bad argument");
    const int64_t p = P->cur_d / (P->host.c ? P->host.c : 1);
    out->encoded = P->encoded;
    out->rounds_done = P->rounds_done;
    out->bytes_forwarded_per_worker = P->bytes_forwarded;
    out->bytes_forwarded_last_round = P->rounds_done > 0 ? (uint64_t)4 * p : 0;
    out->bytes_stored_per_worker = (uint64_t)4 * p * (uint64_t)(P->host.c + P->host.N);
    out->bytes_gradient = (uint64_t)4 * (uint64_t)P->cur_d;
    return CERAR_OK;
}

uint64_t cerar_launch_count(const cerar_plan_t* P) { return P ? P->launches : 0; }

int cerar_set_kernel_mode(cerar_plan_t* P, int mode) {
    if (!P) return -1;
    int old = P->kernel_mode;
    if (mode >= 0 && mode <= 3) P->kernel_mode = mode;
    return old;
}

cerar_status_t cerar_device_status(cerar_plan_t* P, cerar_stream_t stream) {
    if (!P) return fail(CERAR_ERR_INVALID_ARG, "plan is NULL");
    if (!P->on_device) return fail(CERAR_ERR_CUDA, "plan has no device copies");
    int flag = 0;
    cudaError_t e = cudaMemcpyAsync(&flag, P->d_status, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "status read");
    if (flag != 0) {
        cudaMemsetAsync(P->d_status, 0, sizeof(int), (cudaStream_t)stream);
        if (flag == cerar::STATUS_BOUNDS)
            return fail(CERAR_ERR_BOUNDS, "checked build: a kernel formed an address outside its buffer (the access was skipped)");
        return fail(CERAR_ERR_TIMEOUT, "a kernel gave up on a bounded wait");
    }
    return CERAR_OK;
}

cerar_status_t cerar_selftest_wait_timeout(cerar_plan_t* P, int limit_ms, cerar_stream_t stream) {
    if (!P) return fail(CERAR_ERR_INVALID_ARG, "plan is NULL");
    if (!P->on_device) return fail(CERAR_ERR_CUDA, "plan has no device copies");
    if (limit_ms < 1 || limit_ms > 1000) return fail(CERAR_ERR_INVALID_ARG, "limit_ms must be in 1..1000");
    cudaError_t e = cerar::launch_wait_timeout_selftest(P->d_status, (unsigned long long)limit_ms * 1000000ull,
                                                        (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "selftest launch");
    ++P->launches;
    return CERAR_OK;
}

int cerar_set_tuning(const char* name, int value) {
    if (!name) return -1;
    std::string n(name);
    if (n == "kc") cerar::g_tune_kc = value;
    else if (n == "stages") cerar::g_tune_stages = value;
    else if (n == "jt") cerar::g_tune_jt = value;
    else if (n == "slabs") cerar::g_tune_slabs = value;
    else if (n == "tc_kc") cerar::g_tune_tc_kc = value;
    else if (n == "tc_stages") cerar::g_tune_tc_stages = value;
    else if (n == "tc_variant") cerar::g_tune_tc_variant = value;
    else if (n == "ring_wait_ms") cerar::g_tune_ring_wait_ms = value;
    else if (n == "pdl_off") cerar::g_tune_pdl_off = value;
    else if (n == "serpentine_off") cerar::g_tune_serpentine_off = value;
    else if (n == "tc_min_c") cerar::g_tune_tc_min_c = value;
    else if (n == "tc_epi") cerar::g_tune_tc_epi = value;
    else if (n == "tc_unaligned_off") cerar::g_tune_tc_unaligned_off = value;
    else if (n == "tc_split") cerar::g_tune_tc_split = value;
    else if (n == "staged_unaligned_off") cerar::g_tune_staged_unaligned_off = value;
    else if (n == "round_split") cerar::g_tune_round_split = value;
    else if (n == "checked_shrink") cerar::g_tune_checked_shrink = value;
    else if (n == "rounds_one_launch_off") cerar::g_tune_rounds_one_launch_off = value;
    else if (n == "rounds_one_launch_mb") cerar::g_tune_rounds_one_launch_mb = value;
    else if (n == "rounds_multi_form") cerar::g_tune_rounds_multi_form = value;
    else if (n == "rounds_coop_shape") cerar::g_tune_rounds_coop_shape = value;
    else if (n == "rounds_hints") cerar::g_tune_rounds_hints = value;
    else if (n == "ring_tile") cerar::g_tune_ring_tile = (value / 4) * 4;
    else return -1;
    return 0;
}

}  // extern "C"
