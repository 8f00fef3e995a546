// All L ring rounds of a worker in ONE launch, ordered against its neighbours tile by tile.
//
// cerar_rank_round needs a barrier between rounds.  Here a worker's kernel runs through
// rounds 1..L by itself and synchronises with its two neighbours per tile of `tile`
// positions through two counters per tile, both polled in LOCAL memory and written by
// the neighbour (over NVLink when the neighbour is another GPU):
//   landed[t]   written by the previous worker after it stored message k for tile t into
//               this worker's workspace: value base + k
//   freed[t]    written by the next worker after it finished round k on tile t, i.e. after
//               it read the slot that this worker's message k+1 will overwrite: base + k
// Round k of tile t waits for landed[t] >= base + k-1 and freed[t] >= base + k-1, computes
// x = (y_{k-1} - delta_{k-N}) + delta_k, stores it into the next worker's slot k-1 (plain
// 16-byte stores through peer_ws), then publishes landed (to the next worker) and freed
// (to the previous one) with a system-scope release.  Dependencies only point to smaller
// k, and every block walks its tiles in the same order for every round, so the kernels of
// the N workers cannot wait on one another in a cycle as long as they all run.  `base`
// grows by L+1 per aggregation, so the counters are never reset.
//
// With one worker per GPU every GPU launches this kernel for its own worker.  On ONE GPU
// the N workers are emulated by one cooperative launch (blockIdx.y = worker), which
// guarantees that all blocks are resident: separate launches that wait on one another
// must not share a GPU.
//
// Every wait is bounded (limit_ns); a wait that runs out sets the status word, which all
// other waits watch, so the whole grid leaves within about one limit.
#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace {

__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(unsigned* p, unsigned v) {
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_relaxed_status(const int* p) {
    int v;
    asm volatile("ld.relaxed.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// true when *flag >= want (counters only grow; the difference is taken modulo 2^32)
__device__ __forceinline__ bool wait_counter(const unsigned* flag, unsigned want, const int* status,
                                             unsigned long long limit_ns) {
    if ((int)(ld_acquire_sys(flag) - want) >= 0) return true;
    const unsigned long long t0 = ptx::global_ns();
    for (;;) {
        for (int i = 0; i < 32; ++i)
            if ((int)(ld_acquire_sys(flag) - want) >= 0) return true;
        if (ld_relaxed_status(status) != 0) return false;          // somebody else gave up: so do we
        if (ptx::global_ns() - t0 > limit_ns) return false;
    }
}

__device__ __forceinline__ float4 comb4(float4 y, float4 dc, float4 da) {
    return make_float4((y.x - dc.x) + da.x, (y.y - dc.y) + da.y, (y.z - dc.z) + da.z, (y.w - dc.w) + da.w);
}

__global__ void __launch_bounds__(256) ring_rounds_kernel(const RingFusedArgs a) {
    const int wi = blockIdx.y;                       // index into the workers this launch serves
    const float* ws = a.ws[wi];
    float* peer = a.peer_ws[wi];
    const unsigned* landed = a.landed_local[wi];
    const unsigned* freed = a.freed_local[wi];
    unsigned* landed_next = a.landed_next[wi];
    unsigned* freed_prev = a.freed_prev[wi];
    const int N = a.N, c = a.c, L = c + N - 2;
    const int64_t p = a.p;
    __shared__ int ok_s;
    for (int k = 1; k <= L; ++k) {
        int sp, sc, sa, sl;
        sp = (k >= 2) ? k - 2 : -1;
        sc = (k > N) ? k : -1;
        sa = (k <= c) ? N + k : -1;
        sl = k - 1;
        for (int64_t t = blockIdx.x; t < a.ntiles; t += gridDim.x) {
            if (threadIdx.x == 0) {
                bool ok = ld_relaxed_status(a.status) == 0;
                if (ok && k >= 2) {
                    ok = wait_counter(landed + t, a.base + (unsigned)(k - 1), a.status, a.limit_ns) &&
                         wait_counter(freed + t, a.base + (unsigned)(k - 1), a.status, a.limit_ns);
                    if (!ok) atomicCAS(a.status, 0, 4);
                }
                ok_s = ok ? 1 : 0;
            }
            __syncthreads();
            const bool ok = ok_s != 0;
            __syncthreads();                          // ok_s is rewritten for the next tile
            if (!ok) return;                          // uniform over the block
            const int64_t q0 = t * a.tile;
            const int64_t q1 = (q0 + a.tile < p) ? q0 + a.tile : p;
            if (a.vec) {
                const int64_t pv = p / 4;
                const float4* w4 = reinterpret_cast<const float4*>(ws);
                float4* l4 = reinterpret_cast<float4*>(peer) + (int64_t)sl * pv;
                for (int64_t v = q0 / 4 + threadIdx.x; v < q1 / 4; v += blockDim.x) {
                    float4 y = make_float4(0.f, 0.f, 0.f, 0.f), dc = y, da = y;
                    // .cg loads: a slot is read again two rounds after the neighbour has overwritten it,
                    // and this kernel never ends in between, so nothing may be served from this SM's L1
                    if (sp >= 0) y = __ldcg(w4 + (int64_t)sp * pv + v);
                    if (sc >= 0) dc = __ldcg(w4 + (int64_t)sc * pv + v);
                    if (sa >= 0) da = __ldcg(w4 + (int64_t)sa * pv + v);
                    l4[v] = comb4(y, dc, da);
                }
            } else {
                float* l1 = peer + (int64_t)sl * p;
                for (int64_t q = q0 + threadIdx.x; q < q1; q += blockDim.x) {
                    float y = 0.f, dc = 0.f, da = 0.f;
                    if (sp >= 0) y = __ldcg(ws + (int64_t)sp * p + q);
                    if (sc >= 0) dc = __ldcg(ws + (int64_t)sc * p + q);
                    if (sa >= 0) da = __ldcg(ws + (int64_t)sa * p + q);
                    l1[q] = (y - dc) + da;
                }
            }
            __syncthreads();                          // all stores of the tile are issued
            if (threadIdx.x == 0) {
                __threadfence_system();               // ... and visible before the counters move
                st_release_sys(landed_next + t, a.base + (unsigned)k);
                st_release_sys(freed_prev + t, a.base + (unsigned)k);
            }
        }
    }
    // the launch is complete only when the last message has landed here too (decode comes next)
    for (int64_t t = blockIdx.x; t < a.ntiles; t += gridDim.x) {
        if (threadIdx.x == 0 && ld_relaxed_status(a.status) == 0 &&
            !wait_counter(landed + t, a.base + (unsigned)L, a.status, a.limit_ns))
            atomicCAS(a.status, 0, 4);
    }
}

}  // namespace

int g_tune_ring_wait_ms = 0, g_tune_ring_tile = 0;

cudaError_t launch_ring_rounds(const RingFusedArgs& a, int nworkers, bool cooperative, int num_sms, cudaStream_t s,
                               uint64_t* launches) {
    if (a.p <= 0 || nworkers <= 0) return cudaSuccess;
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ring_rounds_kernel, 256, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (per_sm > 8) per_sm = 8;
    int64_t gx = (int64_t)per_sm * num_sms / nworkers;      // all workers' blocks resident at once
    if (gx < 1) return cudaErrorCooperativeLaunchTooLarge;   // more workers than resident blocks
    if (gx > a.ntiles) gx = a.ntiles;
    dim3 grid((unsigned)gx, (unsigned)nworkers);
    if (cooperative) {
        void* args[] = {const_cast<RingFusedArgs*>(&a)};
        e = cudaLaunchCooperativeKernel((const void*)ring_rounds_kernel, grid, dim3(256), args, 0, s);
    } else {
        ring_rounds_kernel<<<grid, 256, 0, s>>>(a);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
