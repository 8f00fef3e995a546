// Whole protocol on chip for small N (c+N): a CTA of N warps carries 64 positions
// through encode, all L rounds and decode with the (c+N) slots of every worker in shared
// memory; thread (w, t) plays worker w for positions 2t, 2t+1 of the tile.  Global memory
// is touched twice per element (read the gradients, write the results) instead of
// 8c+3N-8 row passes; the ring hand-offs of Algorithm 1 are stores into the neighbour's
// slot in shared memory (two CTA barriers per round), not in HBM, so this path is reported
// separately from the HBM pipeline.  The arithmetic (order of the FMAs, cancel-then-add
// in the rounds, scale at the end) is the one of the FMA kernels: results are identical.
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace {

constexpr int FUSED_TP = 32;               // threads per worker (one warp), two positions each
constexpr int FUSED_PP = 2 * FUSED_TP;     // positions per CTA pass

template <int C>
__device__ __forceinline__ void fma_row(float2 (&acc)[C], const float* coef_row, float2 x) {
    if constexpr (C % 4 == 0) {
#pragma unroll
        for (int j4 = 0; j4 < C / 4; ++j4) {
            const float4 u = *reinterpret_cast<const float4*>(coef_row + 4 * j4);
            ptx::fma2(acc[4 * j4 + 0].x, acc[4 * j4 + 0].y, u.x, x.x, x.y);
            ptx::fma2(acc[4 * j4 + 1].x, acc[4 * j4 + 1].y, u.y, x.x, x.y);
            ptx::fma2(acc[4 * j4 + 2].x, acc[4 * j4 + 2].y, u.z, x.x, x.y);
            ptx::fma2(acc[4 * j4 + 3].x, acc[4 * j4 + 3].y, u.w, x.x, x.y);
        }
    } else {
#pragma unroll
        for (int j = 0; j < C; ++j) {
            const float u = coef_row[j];
            ptx::fma2(acc[j].x, acc[j].y, u, x.x, x.y);
        }
    }
}

// shared memory: U (N*c*c) | R (N*(L+1)*c) | state: N*(c+N) rows of FUSED_PP floats
template <int C>
__global__ void __launch_bounds__(FUSED_TP * 16)
fused_kernel(const float* __restrict__ grads, int64_t grads_stride, float* __restrict__ out, int64_t out_stride,
             const float* __restrict__ Ucoef, const float* __restrict__ Rcoef, int N, int64_t p, float scale) {
    extern __shared__ __align__(16) float smem_f[];
    const int c = C, L = c + N - 2, slots = c + N;
    float* Us = smem_f;
    float* Rs = Us + (((size_t)N * c * c + 3) / 4) * 4;                 // every block starts 16-byte aligned
    float* state = Rs + (((size_t)N * (L + 1) * c + 3) / 4) * 4;
    for (int i = threadIdx.x; i < N * c * c; i += blockDim.x) Us[i] = Ucoef[i];
    for (int i = threadIdx.x; i < N * (L + 1) * c; i += blockDim.x) Rs[i] = Rcoef[i];
    __syncthreads();
    const int w = threadIdx.x / FUSED_TP, t = threadIdx.x % FUSED_TP;
    const int wn = (w + 1 == N) ? 0 : w + 1;
    // this thread's column of worker w (mine) and of the ring neighbour w+1 (next): slot s at [s * FUSED_TP]
    float2* mine = reinterpret_cast<float2*>(state) + (size_t)w * slots * FUSED_TP + t;
    float2* next = reinterpret_cast<float2*>(state) + (size_t)wn * slots * FUSED_TP + t;
    const float* Uw = Us + (size_t)w * c * c;
    const float* Rw = Rs + (size_t)w * (L + 1) * c;
    const bool vec_ok = (p % 2 == 0) && ((grads_stride % 2) == 0) && ((out_stride % 2) == 0) &&
                        ((reinterpret_cast<uintptr_t>(grads) & 7u) == 0) && ((reinterpret_cast<uintptr_t>(out) & 7u) == 0);
    const float* gbase = grads + (int64_t)w * grads_stride + 2 * t;
    float* obase = out + (int64_t)w * out_stride + 2 * t;
    constexpr bool PREFETCH = (C <= 16);      // keep the next tile's inputs in registers during the rounds
    float2 x[C];
    auto load_tile = [&](int64_t q0) {
        const int64_t q = q0 + 2 * t;
        const bool v0 = q < p, v1 = q + 1 < p;
        const float* gw = gbase + q0;
#pragma unroll
        for (int l = 0; l < C; ++l) {
            if (vec_ok && v1) x[l] = *reinterpret_cast<const float2*>(gw + (int64_t)l * p);
            else { x[l].x = v0 ? gw[(int64_t)l * p] : 0.f; x[l].y = v1 ? gw[(int64_t)l * p + 1] : 0.f; }
        }
    };
    const int64_t step = (int64_t)gridDim.x * FUSED_PP;
    int64_t q0 = (int64_t)blockIdx.x * FUSED_PP;
    if (PREFETCH && q0 < p) load_tile(q0);
    for (; q0 < p; q0 += step) {
        const int64_t q = q0 + 2 * t;
        const bool v0 = q < p, v1 = q + 1 < p;
        // ---- encode: delta_{w,j} = sum_l U_w[l][j] g_w[l]
        {
            if (!PREFETCH) load_tile(q0);
            float2 acc[C];
#pragma unroll
            for (int j = 0; j < C; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll
            for (int l = 0; l < C; ++l) fma_row<C>(acc, Uw + l * C, x[l]);
#pragma unroll
            for (int j = 0; j < C; ++j) mine[(N + j) * FUSED_TP] = acc[j];
        }
        if (PREFETCH && q0 + step < p) load_tile(q0 + step);       // in flight during the rounds and decode
        __syncthreads();
        // ---- rounds 1..L: x_{w,k} = (y_{w,k-1} - delta_{w,k-N}) + delta_{w,k} -> slot k-1 of worker w+1
        for (int k = 1; k <= L; ++k) {
            float2 y = make_float2(0.f, 0.f), dc = make_float2(0.f, 0.f), da = make_float2(0.f, 0.f);
            if (k >= 2) y = mine[(k - 2) * FUSED_TP];
            const bool has_cancel = (k - 1) >= N;
            if (has_cancel) dc = mine[(k - 1) * FUSED_TP];
            if (k <= c) da = mine[(N - 1 + k) * FUSED_TP];
            // the landing slot is the neighbour's cancel operand of this same round: everybody reads first
            if (has_cancel) __syncthreads();
            next[(k - 1) * FUSED_TP] = make_float2((y.x - dc.x) + da.x, (y.y - dc.y) + da.y);
            __syncthreads();
        }
        // ---- decode: g_hat_w[l] = scale * sum_m R_w[m][l] y_{w,m+1}; y_{L+1} sits in slot L+1
        {
            float2 acc[C];
#pragma unroll
            for (int j = 0; j < C; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll 4
            for (int m = 0; m <= L; ++m) fma_row<C>(acc, Rw + m * C, mine[((m < L) ? m : L + 1) * FUSED_TP]);
            float* ow = obase + q0;
#pragma unroll
            for (int j = 0; j < C; ++j) {
                const float2 o = make_float2(acc[j].x * scale, acc[j].y * scale);
                if (vec_ok && v1) *reinterpret_cast<float2*>(ow + (int64_t)j * p) = o;
                else { if (v0) ow[(int64_t)j * p] = o.x; if (v1) ow[(int64_t)j * p + 1] = o.y; }
            }
        }
        __syncthreads();       // the next tile's encode overwrites the D slots
    }
}

template <int C>
cudaError_t launch_c(const float* grads, int64_t gs, float* out, int64_t os, const float* U, const float* R, int N,
                     int64_t p, float scale, int num_sms, size_t smem, cudaStream_t s) {
    auto kern = fused_kernel<C>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, FUSED_TP * N, smem)) != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    int64_t blocks = (p + FUSED_PP - 1) / FUSED_PP;
    const int64_t cap = (int64_t)num_sms * occ;
    if (blocks > cap) blocks = cap;
    kern<<<(unsigned)blocks, FUSED_TP * N, smem, s>>>(grads, gs, out, os, U, R, N, p, scale);
    return cudaGetLastError();
}

}  // namespace

size_t fused_smem_bytes(int N, int c) {
    const int L = c + N - 2;
    return ((((size_t)N * c * c + 3) / 4) * 4 + (((size_t)N * (L + 1) * c + 3) / 4) * 4 +
            (size_t)N * (c + N) * FUSED_PP) * 4;
}

bool fused_supported(int N, int c) {
    if (N > 16 || c > 32 || ((c % 4) != 0 && c != 5 && c != 6)) return false;
    return fused_smem_bytes(N, c) <= 200 * 1024;
}

cudaError_t launch_fused(const float* grads, int64_t gs, float* out, int64_t os, const float* U, const float* R, int N,
                         int c, int64_t p, float scale, int num_sms, cudaStream_t s, uint64_t* launches) {
    if (!fused_supported(N, c)) return cudaErrorInvalidConfiguration;
    const size_t smem = fused_smem_bytes(N, c);
    cudaError_t e;
    switch (c) {
        case 4: e = launch_c<4>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 5: e = launch_c<5>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 6: e = launch_c<6>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 8: e = launch_c<8>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 12: e = launch_c<12>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 16: e = launch_c<16>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 20: e = launch_c<20>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 24: e = launch_c<24>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 28: e = launch_c<28>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        case 32: e = launch_c<32>(grads, gs, out, os, U, R, N, p, scale, num_sms, smem, s); break;
        default: return cudaErrorInvalidConfiguration;
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
