// One worker's side of a ring round, for the one-worker-per-GPU form of the protocol.
//
// The worker's own state is a (c+N+1) x p fp32 matrix: slot k-1 receives message k
// (k = 1..L), slot N+j holds delta_{i,j} (j = 1..c).  Compared with the single-GPU
// layout there is one more row, so that the slot a neighbour writes in round k
// (k-1) is never a slot its owner reads in the same round (k-2: the previous message,
// k: the delta to cancel, N+k: the delta to add).  Rounds therefore need no finer
// ordering between neighbours than "round k starts when round k-1 is finished on
// both sides" (Algorithm 1 has the same structure: send, receive, then update).
//
// The message x_{i,k} = (y_{i,k-1} - delta_{i,k-N}) + delta_{i,k} (the terms that exist, in
// the order of Algorithm 1: cancel, then add) is stored straight into the neighbour's
// landing slot through `peer_ws`, which may be a peer-mapped pointer into another
// GPU's memory: plain coalesced 16-byte stores, no TMA and no multicast.
#include <cuda_bf16.h>

#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace {

template <typename VT> __device__ __forceinline__ VT vz();
template <> __device__ __forceinline__ float4 vz<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float vz<float>() { return 0.f; }
__device__ __forceinline__ float comb(float y, float dc, float da) { return (y - dc) + da; }
__device__ __forceinline__ float4 comb(float4 y, float4 dc, float4 da) {
    return make_float4((y.x - dc.x) + da.x, (y.y - dc.y) + da.y, (y.z - dc.z) + da.z, (y.w - dc.w) + da.w);
}

template <typename VT>
__global__ void __launch_bounds__(256) rank_round_kernel(const RankRoundArgs a) {
    constexpr int VW = sizeof(VT) / 4;
    const int64_t nv = a.p / VW;
    ptx::grid_dependency_wait();
    const VT* ws = reinterpret_cast<const VT*>(a.ws);
    VT* land = reinterpret_cast<VT*>(a.peer_ws) + (int64_t)a.slot_land * nv;
    const VT* prev = ws + (int64_t)a.slot_prev * nv;
    const VT* cancel = ws + (int64_t)a.slot_cancel * nv;
    const VT* add = ws + (int64_t)a.slot_add * nv;
    const bool has_prev = a.slot_prev >= 0, has_cancel = a.slot_cancel >= 0, has_add = a.slot_add >= 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += (int64_t)gridDim.x * blockDim.x) {
        VT y = vz<VT>(), dc = vz<VT>(), da = vz<VT>();
        if (has_prev) y = prev[v];
        if (has_cancel) dc = cancel[v];
        if (has_add) da = add[v];
        land[v] = comb(y, dc, da);
    }
}

// The same message, rounded to bfloat16 (nearest, ties to even) by its sender and left in a 2-byte
// buffer for the transport: half the bytes on the wire.  The worker's own arithmetic stays binary32.
__device__ __forceinline__ unsigned short bf16_bits(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float bf16_value(unsigned short b) { return __uint_as_float((unsigned)b << 16); }

template <typename VT>
__global__ void __launch_bounds__(256) rank_round_bf16_kernel(const RankRoundArgs a) {
    constexpr int VW = sizeof(VT) / 4;
    const int64_t nv = a.p / VW;
    ptx::grid_dependency_wait();
    const VT* ws = reinterpret_cast<const VT*>(a.ws);
    const VT* prev = ws + (int64_t)a.slot_prev * nv;
    const VT* cancel = ws + (int64_t)a.slot_cancel * nv;
    const VT* add = ws + (int64_t)a.slot_add * nv;
    const bool has_prev = a.slot_prev >= 0, has_cancel = a.slot_cancel >= 0, has_add = a.slot_add >= 0;
    unsigned short* out = reinterpret_cast<unsigned short*>(a.peer_ws);
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += (int64_t)gridDim.x * blockDim.x) {
        VT y = vz<VT>(), dc = vz<VT>(), da = vz<VT>();
        if (has_prev) y = prev[v];
        if (has_cancel) dc = cancel[v];
        if (has_add) da = add[v];
        const VT x = comb(y, dc, da);
        if constexpr (VW == 4) {
            uint2 pk;
            pk.x = (unsigned)bf16_bits(x.x) | ((unsigned)bf16_bits(x.y) << 16);
            pk.y = (unsigned)bf16_bits(x.z) | ((unsigned)bf16_bits(x.w) << 16);
            reinterpret_cast<uint2*>(out)[v] = pk;
        } else {
            out[v] = bf16_bits(x);
        }
    }
}

// Receiver's side: the bfloat16 message that arrived becomes the binary32 content of the landing slot.
template <int VW>
__global__ void __launch_bounds__(256) rank_recv_bf16_kernel(float* slot, const unsigned short* msg, int64_t p) {
    const int64_t nv = p / VW;
    ptx::grid_dependency_wait();
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += (int64_t)gridDim.x * blockDim.x) {
        if constexpr (VW == 4) {
            const uint2 pk = reinterpret_cast<const uint2*>(msg)[v];
            reinterpret_cast<float4*>(slot)[v] = make_float4(bf16_value((unsigned short)(pk.x & 0xFFFFu)), bf16_value((unsigned short)(pk.x >> 16)),
                                                             bf16_value((unsigned short)(pk.y & 0xFFFFu)), bf16_value((unsigned short)(pk.y >> 16)));
        } else {
            slot[v] = bf16_value(msg[v]);
        }
    }
}

}  // namespace

void rank_round_slots(int N, int c, int k, int* slot_prev, int* slot_cancel, int* slot_add, int* slot_land) {
    *slot_prev = (k >= 2) ? k - 2 : -1;        // y_{i,k-1}: message k-1, received in the round before
    *slot_cancel = (k > N) ? k : -1;           // delta_{i,k-N} sits in slot N + (k-N)
    *slot_add = (k <= c) ? N + k : -1;         // delta_{i,k}
    *slot_land = k - 1;                        // in the neighbour's workspace
}

cudaError_t launch_rank_round(RankRoundArgs a, int num_sms, cudaStream_t s, uint64_t* launches) {
    if (a.p <= 0) return cudaSuccess;
    rank_round_slots(a.N, a.c, a.k, &a.slot_prev, &a.slot_cancel, &a.slot_add, &a.slot_land);
    if (a.to_message) a.slot_land = 0;          // the message goes to a buffer of its own, for a transport to send
    const bool vec = (a.p % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.ws) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(a.peer_ws) & 15u) == 0);
    const int64_t nv = vec ? a.p / 4 : a.p;
    int64_t blocks = (nv + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 16;         // grid-stride beyond 16 resident-size waves
    if (blocks > cap) blocks = cap;
    cudaError_t e;
    if (a.to_message == 2) {
        const bool vec2 = (a.p % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.ws) & 15u) == 0) &&
                          ((reinterpret_cast<uintptr_t>(a.peer_ws) & 7u) == 0);
        e = vec2 ? launch_pdl(rank_round_bf16_kernel<float4>, dim3((unsigned)blocks), dim3(256), 0, s, a)
                 : launch_pdl(rank_round_bf16_kernel<float>, dim3((unsigned)((a.p + 255) / 256 < cap ? (a.p + 255) / 256 : cap)),
                              dim3(256), 0, s, a);
    } else
    e = vec ? launch_pdl(rank_round_kernel<float4>, dim3((unsigned)blocks), dim3(256), 0, s, a)
            : launch_pdl(rank_round_kernel<float>, dim3((unsigned)blocks), dim3(256), 0, s, a);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

cudaError_t launch_rank_recv_bf16(float* slot, const unsigned short* msg, int64_t p, int num_sms, cudaStream_t s,
                                  uint64_t* launches) {
    if (p <= 0) return cudaSuccess;
    const bool vec = (p % 4 == 0) && ((reinterpret_cast<uintptr_t>(slot) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(msg) & 7u) == 0);
    const int64_t nv = vec ? p / 4 : p;
    int64_t blocks = (nv + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 16;
    if (blocks > cap) blocks = cap;
    cudaError_t e = vec ? launch_pdl(rank_recv_bf16_kernel<4>, dim3((unsigned)blocks), dim3(256), 0, s, slot, msg, p)
                        : launch_pdl(rank_recv_bf16_kernel<1>, dim3((unsigned)blocks), dim3(256), 0, s, slot, msg, p);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
