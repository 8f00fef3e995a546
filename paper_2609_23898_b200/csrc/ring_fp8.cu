// 8-bit ring messages for the one-worker-per-GPU form: the sender forms message k in binary32
// (same arithmetic as rank_round_kernel), and per tile of CERAR_FP8_TILE positions puts on the wire
// one power-of-two scale 2^e (binary32) and one e4m3 code per position (x 2^-e rounded to nearest,
// ties to even); e is the smallest integer with max|x| 2^-e <= 448, the format's largest value.
// The receiver expands codes and scales into the binary32 landing slot.  A quarter of the bytes of
// a binary32 message cross the transport (plus 4 bytes per 1024 positions).
//
// Message buffer layout (device memory, 16-byte aligned): p codes, padding up to a multiple of 16
// bytes, then ceil(p / tile) binary32 scales.
#include <cuda_fp8.h>

#include "../../include/cerar.h"
#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace {

constexpr int TILE = CERAR_FP8_TILE;          // positions per scale: 256 threads x 4 positions
static_assert(TILE == 1024, "one block of 256 threads, four positions each");

__device__ __forceinline__ float term(const float* row, int64_t q) { return row ? row[q] : 0.f; }

// e of the tile from its largest magnitude (bit pattern of a non-negative binary32 number)
__device__ __forceinline__ int scale_exponent(float amax) {
    const unsigned b = __float_as_uint(amax);
    const int ef = (int)(b >> 23);
    if (b == 0u || ef == 255) return 0;                    // zeros (or non-finite data): scale 1
    if (ef == 0) return -100;                              // subnormal maximum: the smallest scale
    // amax = m 2^E with m in [0.5, 1): E = ef - 126, and m <= 0.875 iff the fraction of 1.f is <= 0.75
    const int E = ef - 126;
    int e = ((b & 0x7FFFFFu) <= 0x600000u) ? E - 9 : E - 8;
    return e < -100 ? -100 : (e > 100 ? 100 : e);
}
__device__ __forceinline__ float pow2(int e) { return __uint_as_float((unsigned)(e + 127) << 23); }

__device__ __forceinline__ float e4m3_value(unsigned code) {
    const unsigned E = (code >> 3) & 15u, M = code & 7u;
    const float mag = E ? (float)(8u + M) * pow2((int)E - 10) : (float)M * pow2(-9);
    return (code & 0x80u) ? -mag : mag;
}

__global__ void __launch_bounds__(256) rank_round_fp8_kernel(const RankRoundArgs a, unsigned char* codes, float* scales,
                                                             int64_t ntiles) {
    __shared__ float red[8];
    __shared__ int e_sh;
    ptx::grid_dependency_wait();
    const float* prev = a.slot_prev >= 0 ? a.ws + (int64_t)a.slot_prev * a.p : nullptr;
    const float* cancel = a.slot_cancel >= 0 ? a.ws + (int64_t)a.slot_cancel * a.p : nullptr;
    const float* add = a.slot_add >= 0 ? a.ws + (int64_t)a.slot_add * a.p : nullptr;
    const bool vec = (a.p % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.ws) & 15u) == 0);
    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t q0 = t * TILE + 4 * (int64_t)threadIdx.x;
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (vec && q0 + 3 < a.p) {
            float4 y = make_float4(0.f, 0.f, 0.f, 0.f), dc = y, da = y;
            if (prev) y = *reinterpret_cast<const float4*>(prev + q0);
            if (cancel) dc = *reinterpret_cast<const float4*>(cancel + q0);
            if (add) da = *reinterpret_cast<const float4*>(add + q0);
            x[0] = (y.x - dc.x) + da.x; x[1] = (y.y - dc.y) + da.y; x[2] = (y.z - dc.z) + da.z; x[3] = (y.w - dc.w) + da.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (q0 + j < a.p) x[j] = (term(prev, q0 + j) - term(cancel, q0 + j)) + term(add, q0 + j);
        }
        float m = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            float mm = red[0];
#pragma unroll
            for (int w = 1; w < 8; ++w) mm = fmaxf(mm, red[w]);
            const int e = scale_exponent(mm);
            e_sh = e;
            scales[t] = pow2(e);
        }
        __syncthreads();
        const float inv = pow2(-e_sh);
        unsigned pk = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            pk |= (unsigned)__nv_cvt_float_to_fp8(x[j] * inv, __NV_SATFINITE, __NV_E4M3) << (8 * j);
        if (q0 + 3 < a.p && (reinterpret_cast<uintptr_t>(codes) & 3u) == 0) {
            *reinterpret_cast<unsigned*>(codes + q0) = pk;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (q0 + j < a.p) codes[q0 + j] = (unsigned char)(pk >> (8 * j));
        }
        __syncthreads();                                   // red / e_sh are reused by the next tile
    }
}

__global__ void __launch_bounds__(256) rank_recv_fp8_kernel(float* slot, const unsigned char* codes, const float* scales,
                                                            int64_t p, int64_t ntiles) {
    ptx::grid_dependency_wait();
    const bool vec = (p % 4 == 0) && ((reinterpret_cast<uintptr_t>(slot) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(codes) & 3u) == 0);
    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const float sc = scales[t];
        const int64_t q0 = t * TILE + 4 * (int64_t)threadIdx.x;
        if (vec && q0 + 3 < p) {
            const unsigned pk = *reinterpret_cast<const unsigned*>(codes + q0);
            *reinterpret_cast<float4*>(slot + q0) = make_float4(e4m3_value(pk & 255u) * sc, e4m3_value((pk >> 8) & 255u) * sc,
                                                                e4m3_value((pk >> 16) & 255u) * sc, e4m3_value(pk >> 24) * sc);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (q0 + j < p) slot[q0 + j] = e4m3_value(codes[q0 + j]) * sc;
        }
    }
}

}  // namespace

size_t fp8_scales_offset(int64_t p) { return (size_t)((p + 15) / 16 * 16); }
size_t fp8_message_bytes(int64_t p) { return fp8_scales_offset(p) + 4 * (size_t)((p + TILE - 1) / TILE); }

cudaError_t launch_rank_round_fp8(RankRoundArgs a, void* msg, int num_sms, cudaStream_t s, uint64_t* launches) {
    if (a.p <= 0) return cudaSuccess;
    rank_round_slots(a.N, a.c, a.k, &a.slot_prev, &a.slot_cancel, &a.slot_add, &a.slot_land);
    const int64_t ntiles = (a.p + TILE - 1) / TILE;
    int64_t blocks = ntiles;
    const int64_t cap = (int64_t)num_sms * 16;
    if (blocks > cap) blocks = cap;
    unsigned char* codes = static_cast<unsigned char*>(msg);
    float* scales = reinterpret_cast<float*>(codes + fp8_scales_offset(a.p));
    cudaError_t e = launch_pdl(rank_round_fp8_kernel, dim3((unsigned)blocks), dim3(256), 0, s, a, codes, scales, ntiles);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

cudaError_t launch_rank_recv_fp8(float* slot, const void* msg, int64_t p, int num_sms, cudaStream_t s, uint64_t* launches) {
    if (p <= 0) return cudaSuccess;
    const int64_t ntiles = (p + TILE - 1) / TILE;
    int64_t blocks = ntiles;
    const int64_t cap = (int64_t)num_sms * 16;
    if (blocks > cap) blocks = cap;
    const unsigned char* codes = static_cast<const unsigned char*>(msg);
    const float* scales = reinterpret_cast<const float*>(codes + fp8_scales_offset(p));
    cudaError_t e = launch_pdl(rank_recv_fp8_kernel, dim3((unsigned)blocks), dim3(256), 0, s, slot, codes, scales, p, ntiles);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
