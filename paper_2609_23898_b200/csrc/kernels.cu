// CUDA kernels of the CERAR data path for sm_100a.
//
//  contract_ref_kernel     plain per-position contraction, any p and alignment
//  contract_staged_kernel  warp-specialised contraction: one producer warp streams
//                          row tiles into shared memory with bulk async copies
//                          (cp.async.bulk + mbarrier), consumer warps run the FMA
//                          register tile; used for encode and decode
//  round_kernel            one ring round for all workers: fused cancel + add +
//                          hand-off store into the neighbour's landing slot
#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace {

constexpr int REF_MAX_J = 512;

using namespace ptx;

// ------------------------------------------------------------------ reference contraction
__global__ void contract_ref_kernel(const ContractArgs a) {
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int w = blockIdx.y;
    grid_dependency_wait();
    if (q >= a.p) return;
    float acc[REF_MAX_J];
    for (int j = 0; j < a.J; ++j) acc[j] = 0.f;
    const float* in = a.in + (int64_t)w * a.in_wstride + q;
    const float* cf = a.coef + (size_t)w * a.K * a.J;
    for (int k = 0; k < a.K; ++k) {
        const int row = (k < a.skip_row) ? k : k + a.skip_count;
        float x = 0.f;
        if (CERAR_RANGE_OK(in + (int64_t)row * a.in_rstride, 4, a.in_range, a.status)) x = in[(int64_t)row * a.in_rstride];
        for (int j = 0; j < a.J; ++j) acc[j] = fmaf(cf[(size_t)k * a.J + j], x, acc[j]);
    }
    float* out = a.out + (int64_t)w * a.out_wstride + q;
    for (int j = 0; j < a.J; ++j)
        if (CERAR_RANGE_OK(out + (int64_t)j * a.out_rstride, 4, a.out_range, a.status)) out[(int64_t)j * a.out_rstride] = acc[j] * a.scale;
}

// ------------------------------------------------------------------ tiled contraction, any alignment
//
// For shapes whose rows do not start on 16-byte boundaries (p not a multiple of 4), where
// neither vector loads nor bulk copies apply.  A block stages all K input rows of its TP
// positions in shared memory with plain coalesced 4-byte loads, then every thread (one
// position) forms the J outputs eight at a time from shared memory; the coefficients sit
// in shared memory too, padded to a multiple of 8 columns so that they are read as two
// 16-byte broadcasts per input row.  All inputs of the tile are read before its first
// output is stored, so in-place use stays safe.
__global__ void __launch_bounds__(256) contract_tile_kernel(const ContractArgs a) {
    extern __shared__ __align__(16) float tile_smem[];
    const int TP = blockDim.x;
    const int Jpad = (a.J + 7) / 8 * 8;
    float* coef_s = tile_smem;                        // K x Jpad
    float* in_s = tile_smem + (size_t)a.K * Jpad;     // K x TP
    const int w = blockIdx.y;
    const int64_t q = (int64_t)blockIdx.x * TP + threadIdx.x;
    const float* cf = a.coef + (size_t)w * a.K * a.J;
    for (int idx = threadIdx.x; idx < a.K * Jpad; idx += TP) {
        const int k = idx / Jpad, j = idx - k * Jpad;
        coef_s[idx] = (j < a.J) ? cf[(size_t)k * a.J + j] : 0.f;
    }
    grid_dependency_wait();                           // the coefficients above are constants of the plan
    if (q < a.p) {
        const float* in = a.in + (int64_t)w * a.in_wstride + q;
        for (int k = 0; k < a.K; ++k) {
            const int row = (k < a.skip_row) ? k : k + a.skip_count;
            in_s[(size_t)k * TP + threadIdx.x] =
                CERAR_RANGE_OK(in + (int64_t)row * a.in_rstride, 4, a.in_range, a.status) ? in[(int64_t)row * a.in_rstride] : 0.f;
        }
    }
    __syncthreads();
    if (q >= a.p) return;
    float* out = a.out + (int64_t)w * a.out_wstride + q;
    for (int jc = 0; jc < a.J; jc += 8) {
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        for (int k = 0; k < a.K; ++k) {
            const float x = in_s[(size_t)k * TP + threadIdx.x];
            const float4 c0 = *reinterpret_cast<const float4*>(coef_s + (size_t)k * Jpad + jc);
            const float4 c1 = *reinterpret_cast<const float4*>(coef_s + (size_t)k * Jpad + jc + 4);
            acc[0] = fmaf(c0.x, x, acc[0]); acc[1] = fmaf(c0.y, x, acc[1]);
            acc[2] = fmaf(c0.z, x, acc[2]); acc[3] = fmaf(c0.w, x, acc[3]);
            acc[4] = fmaf(c1.x, x, acc[4]); acc[5] = fmaf(c1.y, x, acc[5]);
            acc[6] = fmaf(c1.z, x, acc[6]); acc[7] = fmaf(c1.w, x, acc[7]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (jc + j < a.J && CERAR_RANGE_OK(out + (int64_t)(jc + j) * a.out_rstride, 4, a.out_range, a.status))
                out[(int64_t)(jc + j) * a.out_rstride] = acc[j] * a.scale;
    }
}

// ------------------------------------------------------------------ staged contraction
//
// grid = (CTAs per worker, N).  CTA (b, w) walks tiles b, b+gridDim.x, ... of
// worker w.  A tile is tile_p = slabs*PV*128 consecutive positions; it is
// streamed through shared memory in chunks of KC input rows.  Every consumer
// thread owns 4*PV positions x JT outputs; all K inputs of a tile are consumed
// before its outputs are stored, which makes in-place use (outputs overwriting
// input rows) safe: tiles are disjoint in positions.
//
// shared memory: [full[stages], empty[stages] mbarriers | coef K x Jpad | stages x KC x tile_p]
//
// UNAL: rows that do not start on 16-byte boundaries (p not a multiple of 4, offset buffers).  A row's bulk
// copy then starts at the 16-byte boundary below its first element and the row sits in shared memory with
// the same offset of 0..3 floats (row pitch tile_p + 4); a thread takes the positions lane, lane + 32, ... of
// its 128 (instead of four consecutive ones), so that shared-memory reads and global stores of single
// floats are conflict-free and coalesced.
template <int PV, int JT, int MAXW, bool UNAL>
__global__ void __launch_bounds__(32 * (MAXW + 1), 1)
contract_staged_kernel(const __grid_constant__ ContractArgs a) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int CW = a.slabs * a.jgroups;                 // consumer warps; warp CW is the producer
    const int Jpad = a.jgroups * JT;
    const int stages = a.stages, KC = a.KC, tile_p = a.tile_p;
    const int pitch = tile_p + (UNAL ? 4 : 0);          // floats between rows of a stage
    const int nkc = (a.K + KC - 1) / KC;
    const int w = blockIdx.y;

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);
    // (barriers take a whole number of 128-byte lines)
    float* coef_s = reinterpret_cast<float*>(smem_raw + ((2 * stages * 8 + 127) / 128) * 128);
    float* stage_s = coef_s + (((size_t)a.K * Jpad + 31) / 32) * 32;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8u * stages;
    const uint32_t stage0 = smem_u32(stage_s);
    const uint32_t stage_bytes = (uint32_t)KC * pitch * 4u;

    // set-up (the only CTA-wide barrier, before any bounded wait)
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, CW);
        }
        mbar_init_fence();
    }
    {
        const float* cf = a.coef + (size_t)w * a.K * a.J;
        for (int idx = threadIdx.x; idx < a.K * Jpad; idx += blockDim.x) {
            const int k = idx / Jpad, j = idx - k * Jpad;
            coef_s[idx] = (j < a.J) ? cf[(size_t)k * a.J + j] : 0.f;
        }
    }
    __syncthreads();
    // everything above reads only the plan's constant coefficients: it may overlap the tail of the
    // kernel before this one; the data rows may not
    grid_dependency_wait();

    uint32_t it = 0;            // chunk counter, same sequence in producer and consumers
    bool failed = false;

    if (warp == CW) {
        // ---------------- producer warp
        const float* in_w = a.in + (int64_t)w * a.in_wstride;
        for (int64_t t = blockIdx.x; t < a.tiles_per_worker && !failed; t += gridDim.x) {
            const int64_t q0 = t * tile_p;
            const int64_t rem = a.p - q0;
            const uint32_t valid = (uint32_t)(rem < tile_p ? rem : tile_p);
            for (int kc = 0; kc < nkc; ++kc, ++it) {
                const uint32_t s = it % stages, ph = (it / stages) & 1u;
                if (!mbar_wait_bounded(empty0 + 8u * s, ph ^ 1u)) { failed = true; break; }
                const int k0 = kc * KC;
                const int kcount = (a.K - k0 < KC) ? (a.K - k0) : KC;
                if constexpr (UNAL) {
                    uint32_t total = 0;
                    for (int r = lane; r < kcount; r += 32) {
                        const int k = k0 + r;
                        const int row = (k < a.skip_row) ? k : k + a.skip_count;
                        const uintptr_t first = reinterpret_cast<uintptr_t>(in_w + (int64_t)row * a.in_rstride + q0);
                        total += (uint32_t)((first & 15u) + valid * 4u + 15u) & ~15u;
                    }
                    total = __reduce_add_sync(0xffffffffu, total);
                    if (lane == 0) mbar_arrive_expect_tx(full0 + 8u * s, total);
                    __syncwarp();
                    for (int r = lane; r < kcount; r += 32) {
                        const int k = k0 + r;
                        const int row = (k < a.skip_row) ? k : k + a.skip_count;
                        const uintptr_t first = reinterpret_cast<uintptr_t>(in_w + (int64_t)row * a.in_rstride + q0);
                        const uint32_t bytes = (uint32_t)((first & 15u) + valid * 4u + 15u) & ~15u;
                        // (checked build: the row proper is checked, not the up to 12 bytes around it that share its
                        // 16-byte groups; a skipped copy leaves its bytes outstanding and the consumers' wait runs out)
                        if (CERAR_RANGE_OK(reinterpret_cast<const void*>(first), valid * 4u, a.in_range, a.status))
                            bulk_load(stage0 + s * stage_bytes + (uint32_t)r * pitch * 4u,
                                      reinterpret_cast<const void*>(first & ~(uintptr_t)15), bytes, full0 + 8u * s);
                    }
                } else {
                    if (lane == 0) mbar_arrive_expect_tx(full0 + 8u * s, (uint32_t)kcount * valid * 4u);
                    __syncwarp();
                    for (int r = lane; r < kcount; r += 32) {
                        const int k = k0 + r;
                        const int row = (k < a.skip_row) ? k : k + a.skip_count;
                        // (checked build: a copy that is skipped leaves its bytes outstanding, so the consumers' wait
                        // runs out and the launch ends with both codes' worth of evidence in the status word)
                        if (CERAR_RANGE_OK(in_w + (int64_t)row * a.in_rstride + q0, valid * 4u, a.in_range, a.status))
                            bulk_load(stage0 + s * stage_bytes + (uint32_t)r * tile_p * 4u,
                                      in_w + (int64_t)row * a.in_rstride + q0, valid * 4u, full0 + 8u * s);
                    }
                }
            }
        }
        if (failed) {
            if (lane == 0) atomicExch(a.status, 1);
            // let copies that were already issued land before the CTA retires
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < 1000000ull) { }
        }
    } else {
        // ---------------- consumer warps
        const int jg = warp % a.jgroups, slab = warp / a.jgroups;
        const float* coef_w = coef_s + jg * JT;
        uint32_t pos[PV];
#pragma unroll
        for (int v = 0; v < PV; ++v)     // first position of this thread in vector group v (UNAL: its four are 32 apart)
            pos[v] = UNAL ? (uint32_t)((slab * PV + v) * 128 + lane) : (uint32_t)(((slab * PV + v) * 32 + lane) * 4);
        float* out_w = a.out + (int64_t)w * a.out_wstride;
        const float* in_w = a.in + (int64_t)w * a.in_wstride;
        for (int64_t t = blockIdx.x; t < a.tiles_per_worker && !failed; t += gridDim.x) {
            const int64_t q0 = t * tile_p;
            const int64_t rem = a.p - q0;
            const uint32_t valid = (uint32_t)(rem < tile_p ? rem : tile_p);
            float acc[JT][PV * 4];
#pragma unroll
            for (int j = 0; j < JT; ++j)
#pragma unroll
                for (int e = 0; e < PV * 4; ++e) acc[j][e] = 0.f;
            for (int kc = 0; kc < nkc; ++kc, ++it) {
                const uint32_t s = it % stages, ph = (it / stages) & 1u;
                if (!mbar_wait_bounded(full0 + 8u * s, ph)) { failed = true; break; }
                const int k0 = kc * KC;
                const int kcount = (a.K - k0 < KC) ? (a.K - k0) : KC;
                const float* st = stage_s + (size_t)s * KC * pitch;
                const float* cfa = coef_w + (size_t)k0 * Jpad;
#pragma unroll 2
                for (int kk = 0; kk < kcount; ++kk, cfa += Jpad) {
                    float4 x[PV];
                    if constexpr (UNAL) {
                        const int k = k0 + kk;
                        const int row = (k < a.skip_row) ? k : k + a.skip_count;
                        const uint32_t sh = (uint32_t)((reinterpret_cast<uintptr_t>(in_w + (int64_t)row * a.in_rstride + q0) >> 2) & 3u);
#pragma unroll
                        for (int v = 0; v < PV; ++v) {
                            const float* xr = st + (size_t)kk * pitch + sh + pos[v];
                            x[v] = make_float4(xr[0], xr[32], xr[64], xr[96]);
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < PV; ++v)
                            x[v] = *reinterpret_cast<const float4*>(st + (size_t)kk * tile_p + pos[v]);
                    }
#pragma unroll
                    for (int j4 = 0; j4 < JT / 4; ++j4) {
                        const float4 cc = *reinterpret_cast<const float4*>(cfa + 4 * j4);
                        const float cj[4] = {cc.x, cc.y, cc.z, cc.w};
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                            for (int v = 0; v < PV; ++v) {
                                const int j = j4 * 4 + jj;
                                fma2(acc[j][v * 4 + 0], acc[j][v * 4 + 1], cj[jj], x[v].x, x[v].y);
                                fma2(acc[j][v * 4 + 2], acc[j][v * 4 + 3], cj[jj], x[v].z, x[v].w);
                            }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8u * s);
            }
            if (failed) break;
#pragma unroll
            for (int j = 0; j < JT; ++j) {
                const int jj = jg * JT + j;
                if (jj < a.J) {
                    float* orow = out_w + (int64_t)jj * a.out_rstride + q0;
#pragma unroll
                    for (int v = 0; v < PV; ++v) {
                        if constexpr (UNAL) {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (pos[v] + 32u * e < valid && CERAR_RANGE_OK(orow + pos[v] + 32 * e, 4, a.out_range, a.status))
                                    orow[pos[v] + 32 * e] = acc[j][v * 4 + e] * a.scale;
                        } else if (pos[v] < valid && CERAR_RANGE_OK(orow + pos[v], 16, a.out_range, a.status)) {
                            float4 o;
                            o.x = acc[j][v * 4 + 0] * a.scale;
                            o.y = acc[j][v * 4 + 1] * a.scale;
                            o.z = acc[j][v * 4 + 2] * a.scale;
                            o.w = acc[j][v * 4 + 3] * a.scale;
                            *reinterpret_cast<float4*>(orow + pos[v]) = o;
                        }
                    }
                }
            }
        }
        if (failed && lane == 0) atomicExch(a.status, 1);
    }
}

// ------------------------------------------------------------------ ring round
//
// Round k for all workers and one (vector of) position(s) per thread:
//   x_{i,k} = (y_{i,k-1} - delta_{i,k-N}) + delta_{i,k}    (terms that exist)
// read from slots k-2, k-1 and N-1+k of worker i, stored into slot k-1 of
// worker i+1.  Slot k-1 of worker i+1 is also that worker's cancel operand, so a
// thread walks the ring downwards (i = N-1 .. 0) and keeps worker 0's operand in
// a register: every slot is read before the same thread overwrites it, and no
// other thread touches this position.
template <typename VT> __device__ __forceinline__ VT vzero();
template <> __device__ __forceinline__ float vzero<float>() { return 0.f; }
template <> __device__ __forceinline__ float4 vzero<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ float combine(float y, float dc, float da) { return (y - dc) + da; }
__device__ __forceinline__ float4 combine(float4 y, float4 dc, float4 da) {
    return make_float4((y.x - dc.x) + da.x, (y.y - dc.y) + da.y, (y.z - dc.z) + da.z, (y.w - dc.w) + da.w);
}

// One round k for the position vector at `base` (all N workers), as described above.
template <typename VT, int WG>
__device__ __forceinline__ void round_body(VT* base, int64_t pv, int64_t wstride, int N, int c, int k, Range range, int* status) {
    const bool has_prev = k >= 2, has_cancel = (k - 1) >= N, has_add = k <= c;
    const int64_t off_prev = (int64_t)(k - 2) * pv, off_land = (int64_t)(k - 1) * pv,
                  off_add = (int64_t)(N - 1 + k) * pv;
    VT carry = vzero<VT>();
    if (has_cancel && CERAR_RANGE_OK(base + off_land, sizeof(VT), range, status)) carry = base[off_land];   // worker 0's delta_{0,k-N}
    for (int i0 = N - 1; i0 >= 0; i0 -= WG) {
        VT y[WG], dc[WG], da[WG];
#pragma unroll
        for (int g = 0; g < WG; ++g) {
            const int i = i0 - g;
            y[g] = dc[g] = da[g] = vzero<VT>();
            if (i >= 0) {
                const VT* wb = base + (int64_t)i * wstride;
                if (has_prev && CERAR_RANGE_OK(wb + off_prev, sizeof(VT), range, status)) y[g] = wb[off_prev];
                if (has_cancel) dc[g] = (i == 0) ? carry : CERAR_RANGE_OK(wb + off_land, sizeof(VT), range, status) ? wb[off_land] : vzero<VT>();
                if (has_add && CERAR_RANGE_OK(wb + off_add, sizeof(VT), range, status)) da[g] = wb[off_add];
            }
        }
#pragma unroll
        for (int g = 0; g < WG; ++g) {
            const int i = i0 - g;
            if (i >= 0) {
                const int dst = (i + 1 == N) ? 0 : i + 1;
                if (CERAR_RANGE_OK(base + (int64_t)dst * wstride + off_land, sizeof(VT), range, status))
                    base[(int64_t)dst * wstride + off_land] = combine(y[g], dc[g], da[g]);
            }
        }
    }
}

template <typename VT, int WG>
__global__ void __launch_bounds__(256) round_kernel(const RoundArgs a) {
    constexpr int VW = sizeof(VT) / 4;
    const int64_t nv = a.p / VW;
    // Even rounds walk the positions downwards: what the round before wrote last is read first,
    // while it is still in L2 (measured: +0.7 % at p = 2.2e7, +3 % at p = 4e6, nothing lost below).
    const int64_t blk = a.reverse ? (int64_t)gridDim.x - 1 - blockIdx.x : (int64_t)blockIdx.x;
    const int64_t v = blk * blockDim.x + threadIdx.x;
    // Programmatic dependent launch: this grid may be scheduled while the grid before it drains and
    // touches memory only after that grid has completed.  (Letting the NEXT grid in early, with an
    // explicit trigger at the top, gained nothing and cost 8 % at N = 16, c = 128.)
    grid_dependency_wait();
    if (v >= nv) return;
    const int64_t pv = a.p / VW;                               // row pitch in vectors
    round_body<VT, WG>(reinterpret_cast<VT*>(a.ws) + v, pv, (int64_t)(a.c + a.N) * pv, a.N, a.c, a.k, a.range, a.status);
}

// The same round for few positions (the grid above would leave SMs idle and every thread with N / 4
// dependent groups of loads): thread (v, q) takes workers 4q .. 4q+3 of position vector v, the
// 256 / ceil(N/4) vectors of a block are contiguous.  The slot a message lands in is the cancel
// operand of the worker it belongs to, which another thread of the same block reads: all loads,
// one block barrier, then all stores.  Same operations in the same order per element as round_body.
__global__ void __launch_bounds__(256) round_split_kernel(const RoundArgs a, int groups) {
    const int64_t nv = a.p / 4;
    const int pvb = blockDim.x / groups;                       // position vectors per block
    const int64_t blk = a.reverse ? (int64_t)gridDim.x - 1 - blockIdx.x : (int64_t)blockIdx.x;
    const int q = threadIdx.x / pvb;
    const int64_t v = blk * pvb + (threadIdx.x - q * pvb);
    const int N = a.N, c = a.c, k = a.k;
    const bool has_prev = k >= 2, has_cancel = (k - 1) >= N, has_add = k <= c;
    const int64_t wstride = (int64_t)(c + N) * nv;
    const int64_t off_prev = (int64_t)(k - 2) * nv, off_land = (int64_t)(k - 1) * nv, off_add = (int64_t)(N - 1 + k) * nv;
    float4* base = reinterpret_cast<float4*>(a.ws) + v;
    const bool active = v < nv && q < groups;
    float4 x[4];
    grid_dependency_wait();
    if (active) {
        float4 y[4], dc[4], da[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int i = 4 * q + g;
            y[g] = dc[g] = da[g] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < N) {
                const float4* wb = base + (int64_t)i * wstride;
                if (has_prev && CERAR_RANGE_OK(wb + off_prev, 16, a.range, a.status)) y[g] = wb[off_prev];
                if (has_cancel && CERAR_RANGE_OK(wb + off_land, 16, a.range, a.status)) dc[g] = wb[off_land];
                if (has_add && CERAR_RANGE_OK(wb + off_add, 16, a.range, a.status)) da[g] = wb[off_add];
            }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) x[g] = combine(y[g], dc[g], da[g]);
    }
    __syncthreads();
    if (active) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int i = 4 * q + g;
            float4* dstp = base + (int64_t)((i + 1 == N) ? 0 : i + 1) * wstride + off_land;
            if (i < N && CERAR_RANGE_OK(dstp, 16, a.range, a.status)) *dstp = x[g];
        }
    }
}

// Rounds k .. k_last in one launch, one THREAD per position vector: the thread owns its positions
// for all N workers, and a round touches nothing else, so it simply runs the rounds one after the
// other (its own stores are visible to its own later loads).  Latency-bound (L dependent rounds
// of N / WG dependent groups each); kept for N > 32, which the warp-per-worker kernel below cannot
// hold in one block.  Groups of 8 workers, 8-byte accesses and fewer resident threads were measured
// and are slower.
template <typename VT, int WG>
__global__ void __launch_bounds__(256) rounds_multi_kernel(const RoundArgs a, int k_last) {
    constexpr int VW = sizeof(VT) / 4;
    const int64_t nv = a.p / VW;
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();
    if (v >= nv) return;
    const int64_t pv = a.p / VW;
    VT* base = reinterpret_cast<VT*>(a.ws) + v;
    for (int k = a.k; k <= k_last; ++k) round_body<VT, WG>(base, pv, (int64_t)(a.c + a.N) * pv, a.N, a.c, k, a.range, a.status);
}

// The same rounds k .. k_last in one launch with one WARP per worker: a block of N warps owns 32 PV
// vectors of positions, warp i plays worker i.  The message of a round is stored into the neighbour's
// slot (as always) and handed to the neighbour's warp through shared memory, so a round costs one
// block barrier instead of a trip to memory, and the operands of the next DIST rounds (which do not
// depend on this one) are already on their way when the barrier is reached.  Hazard: the slot a
// message lands in holds the delta its owner cancels in that very round; every thread therefore
// reads its cancel operand at least one round early (before the barrier that precedes the store),
// never after.  Measured on B200 (rounds of N=8, c=32, d=2^28, in the metric's bytes): DIST 1
// 8.2 TB/s, DIST 2 10.4, DIST 3 and 4 9.7; one launch per round 7.2.  Keeping the deltas that are
// cancelled N rounds later in a register ring (N <= 8, loop unrolled by N) instead of reading them
// again: 6.8-7.0 TB/s (100-200 registers per thread), rejected.
// L2 residency hints for the one-launch rounds: a delta is read twice, N rounds apart (added, then
// cancelled): the first read asks L2 to keep the line, the second lets it go; a stored message is not
// read again before the decode.
__device__ __forceinline__ uint64_t policy_keep() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float4 ld_keep(const float4* p, uint64_t pol) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ float ld_keep(const float* p, uint64_t pol) {
    float v;
    asm volatile("ld.global.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(v) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ float4 ld_last_use(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ float ld_last_use(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(float* p, float v) { __stcs(p, v); }

template <typename VT, int PV, int DIST, int MAXT>
__global__ void __launch_bounds__(MAXT) rounds_coop_kernel(const RoundArgs a, int k_last) {
    extern __shared__ float4 coop_smem[];
    VT* hand = reinterpret_cast<VT*>(coop_smem);                // [2][N][PV][32]
    constexpr int VW = sizeof(VT) / 4;
    const int i = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = a.N, c = a.c;
    const int64_t pv = a.p / VW;
    const int64_t v0 = (int64_t)blockIdx.x * (32 * PV) + lane;  // this lane's vectors: v0 + 32 j
    bool live[PV];
#pragma unroll
    for (int j = 0; j < PV; ++j) live[j] = v0 + 32 * j < pv;
    const int64_t wstride = (int64_t)(c + N) * pv;
    const int dst = (i + 1 == N) ? 0 : i + 1;
    VT* own = reinterpret_cast<VT*>(a.ws) + (int64_t)i * wstride + v0;
    VT* nxt = reinterpret_cast<VT*>(a.ws) + (int64_t)dst * wstride + v0;
    grid_dependency_wait();
    int k = a.k;
    const bool hints = a.hints != 0;                            // set by the launcher
    const uint64_t pol = policy_keep();
    // operands of rounds k .. k+DIST-1 (index t = rounds ahead); absent terms are zero
    VT y[PV], da[DIST][PV], dc[DIST][PV];
#pragma unroll
    for (int j = 0; j < PV; ++j) {
        y[j] = vzero<VT>();
        if (live[j] && k >= 2 && CERAR_RANGE_OK(own + (int64_t)(k - 2) * pv + 32 * j, sizeof(VT), a.range, a.status)) y[j] = own[(int64_t)(k - 2) * pv + 32 * j];
#pragma unroll
        for (int t = 0; t < DIST; ++t) {
            const int kt = k + t;
            da[t][j] = dc[t][j] = vzero<VT>();
            if (live[j] && kt <= k_last) {
                if (kt <= c && CERAR_RANGE_OK(own + (int64_t)(N - 1 + kt) * pv + 32 * j, sizeof(VT), a.range, a.status)) da[t][j] = hints ? ld_keep(own + (int64_t)(N - 1 + kt) * pv + 32 * j, pol) : own[(int64_t)(N - 1 + kt) * pv + 32 * j];
                if (kt - 1 >= N && CERAR_RANGE_OK(own + (int64_t)(kt - 1) * pv + 32 * j, sizeof(VT), a.range, a.status)) dc[t][j] = hints ? ld_last_use(own + (int64_t)(kt - 1) * pv + 32 * j) : own[(int64_t)(kt - 1) * pv + 32 * j];
            }
        }
    }
    __syncthreads();
    for (; k <= k_last; ++k) {
        VT* hb = hand + (size_t)(k & 1) * N * (32 * PV);
#pragma unroll
        for (int j = 0; j < PV; ++j) {
            const VT x = combine(y[j], dc[0][j], da[0][j]);
            if (live[j] && CERAR_RANGE_OK(nxt + (int64_t)(k - 1) * pv + 32 * j, sizeof(VT), a.range, a.status)) {
                if (hints) st_stream(nxt + (int64_t)(k - 1) * pv + 32 * j, x); else nxt[(int64_t)(k - 1) * pv + 32 * j] = x;
            }
            hb[(dst * PV + j) * 32 + lane] = x;
        }
        // shift the operand queue and fetch round k + DIST (its slots are not written before that round)
        const int kn = k + DIST;
#pragma unroll
        for (int j = 0; j < PV; ++j) {
#pragma unroll
            for (int t = 0; t + 1 < DIST; ++t) { da[t][j] = da[t + 1][j]; dc[t][j] = dc[t + 1][j]; }
            da[DIST - 1][j] = dc[DIST - 1][j] = vzero<VT>();
            if (live[j] && kn <= k_last) {
                if (kn <= c && CERAR_RANGE_OK(own + (int64_t)(N - 1 + kn) * pv + 32 * j, sizeof(VT), a.range, a.status)) da[DIST - 1][j] = hints ? ld_keep(own + (int64_t)(N - 1 + kn) * pv + 32 * j, pol) : own[(int64_t)(N - 1 + kn) * pv + 32 * j];
                if (kn - 1 >= N && CERAR_RANGE_OK(own + (int64_t)(kn - 1) * pv + 32 * j, sizeof(VT), a.range, a.status)) dc[DIST - 1][j] = hints ? ld_last_use(own + (int64_t)(kn - 1) * pv + 32 * j) : own[(int64_t)(kn - 1) * pv + 32 * j];
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < PV; ++j) y[j] = hb[(i * PV + j) * 32 + lane];
    }
}

// Nothing ever arrives on this barrier: the bounded wait runs out after limit_ns and the
// kernel reports it through the status word, exactly as the pipelined kernels would.
__global__ void wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        mbar_init_fence();
        if (!mbar_wait_bounded(smem_u32(&bar), 0, limit_ns)) atomicExch(status, 3);
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <int PV, int JT, int MAXW, bool UNAL>
cudaError_t launch_staged(ContractArgs& a, int num_sms, cudaStream_t s) {
    auto kern = contract_staged_kernel<PV, JT, MAXW, UNAL>;
    const int Jpad = a.jgroups * JT;
    const size_t bar_bytes = ((2 * (size_t)a.stages * 8 + 127) / 128) * 128;
    const size_t coef_bytes = (((size_t)a.K * Jpad + 31) / 32) * 32 * 4;
    const size_t smem = bar_bytes + coef_bytes + (size_t)a.stages * a.KC * (a.tile_p + (UNAL ? 4 : 0)) * 4;
    {   // per device and cheap: set on every launch rather than cached
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int threads = 32 * (a.slabs * a.jgroups + 1);
    int occ = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    int64_t per_worker = ((int64_t)num_sms * occ) / a.N;
    if (per_worker < 1) per_worker = 1;
    if (per_worker > a.tiles_per_worker) per_worker = a.tiles_per_worker;
    dim3 grid((unsigned)per_worker, (unsigned)a.N);
    return launch_pdl(kern, grid, dim3(threads), smem, s, a);
}

}  // namespace

// Tuning knobs (0 = default), settable through the C ABI for experiments.
int g_tune_round_split = 0;
int g_tune_staged_unaligned_off = 0;
int g_tune_checked_shrink = 0;   // checked build, tests only: the extents that stores are checked against end this many floats early
int g_tune_kc = 0, g_tune_stages = 0, g_tune_jt = 0, g_tune_slabs = 0, g_tune_pdl_off = 0, g_tune_serpentine_off = 0,
    g_tune_rounds_one_launch_off = 0, g_tune_rounds_one_launch_mb = 0, g_tune_rounds_multi_form = 0, g_tune_rounds_coop_shape = 0, g_tune_rounds_hints = 0;

cudaError_t launch_contract(ContractArgs a, int mode, int num_sms, cudaStream_t s, uint64_t* launches) {
    if (a.p <= 0 || a.N <= 0) return cudaSuccess;
    a.in_range = Range{a.in, a.in + (int64_t)(a.N - 1) * a.in_wstride + (int64_t)(a.K + a.skip_count - 1) * a.in_rstride + a.p};
    a.out_range = Range{a.out, a.out + (int64_t)(a.N - 1) * a.out_wstride + (int64_t)(a.J - 1) * a.out_rstride + a.p -
                                   g_tune_checked_shrink};
    bool can_stage = (a.p % 4 == 0) && aligned16(a.in) && aligned16(a.out) && (a.in_wstride % 4 == 0) &&
                     (a.out_wstride % 4 == 0) && (a.in_rstride % 4 == 0) && (a.out_rstride % 4 == 0);
    if (mode == KERNEL_TC && !tc_eligible(a)) return cudaErrorInvalidValue;
    // automatic choice: the FMA kernel is HBM-bound below c ~ 24; from there on only the tensor cores keep up
    if (mode == KERNEL_TC || (mode == KERNEL_AUTO && tc_eligible(a))) {
        return launch_contract_tc(a, num_sms, s, launches);
    }
    // rows that are not 16-byte aligned: the same kernel with realigned bulk copies, for the small c that the
    // tensor-core kernel leaves (tuning: staged_unaligned_off = 1 sends them to the tiled plain-load kernel)
    const bool unal_staged = !can_stage && !g_tune_staged_unaligned_off && a.J <= 64;
    if (mode == KERNEL_STAGED && !can_stage && !unal_staged) return cudaErrorInvalidValue;
    bool use_staged = (can_stage || unal_staged) && mode != KERNEL_REF;
    if (use_staged) {
        // register tile: 8 outputs x 8 positions per thread where J allows it (more resident
        // warps than 16 x 8), 4 x 8 otherwise; as many position slabs as the warp budget
        // allows; stages of about 64 KB (values measured best on B200 for c = 8..24)
        int JT = g_tune_jt ? g_tune_jt : ((a.J % 8 == 0 && a.J >= 16) ? 8 : 4);
        // decode at c = 16 (19-31 input rows): 4 outputs per thread and twice the warps per output group, measured inside
        // the pipeline: +4 % at p = 2^20, +10 % at p = 2^22 (the encode loses 5 % with it and keeps 8)
        if (!g_tune_jt && a.J == 16 && a.K > a.J) JT = 4;
        if (unal_staged && JT != 8) JT = 4;
        // c = 20 (the paper's 8-GPU configuration), decode: all 20 outputs of 4 positions in one
        // thread, so that the data is read from shared memory once instead of by five warps
        // (+7 % measured; neutral for encode, worse for c = 12 and for c padded up to 20)
        if (!g_tune_jt && a.J == 20 && a.K > a.J && !unal_staged) JT = 20;
        const int PV = (JT == 20) ? 1 : 2;
        a.jgroups = (a.J + JT - 1) / JT;
        const int maxw = (JT == 16 || JT == 20) ? 8 : 16;
        if (a.jgroups > maxw) {
            use_staged = false;
        } else {
            int slabs = g_tune_slabs ? g_tune_slabs : maxw / a.jgroups;
            if (slabs > 8) slabs = 8;
            if (slabs < 1) slabs = 1;
            while (slabs > 1 && slabs * a.jgroups > maxw) --slabs;
            a.slabs = slabs;
            a.tile_p = slabs * PV * 128;
            a.KC = g_tune_kc ? g_tune_kc : 16;
            if (!g_tune_kc) {
                const int fit = (64 * 1024) / (a.tile_p * 4);
                if (a.KC > fit) a.KC = fit < 2 ? 2 : fit;
            }
            if (a.KC > a.K) a.KC = a.K;
            // three stages; two for c <= 8 (a tile is one or two chunks): measured inside the pipeline at c = 8, +4..+7 %
            // for both contractions (at c = 16, where the decode has three or four chunks per tile, two stages cost it 10-25 %)
            a.stages = g_tune_stages ? g_tune_stages : (a.J <= 8 ? 2 : 3);
            a.tiles_per_worker = (int)((a.p + a.tile_p - 1) / a.tile_p);
            a.total_tiles = (int64_t)a.tiles_per_worker * a.N;
            // shared memory must fit: shrink the pipeline, then give up
            auto smem_of = [&](int st) {
                return ((2 * (size_t)st * 8 + 127) / 128) * 128 + (((size_t)a.K * a.jgroups * JT + 31) / 32) * 128 +
                       (size_t)st * a.KC * a.tile_p * 4;
            };
            while (a.stages > 2 && smem_of(a.stages) > 200 * 1024) --a.stages;
            if (smem_of(a.stages) > 220 * 1024) use_staged = false;
            if (use_staged) {
                cudaError_t e;
                if (!can_stage) {       // rows that are not 16-byte aligned
                    if (JT == 8) e = launch_staged<2, 8, 16, true>(a, num_sms, s);
                    else e = launch_staged<2, 4, 16, true>(a, num_sms, s);
                } else if (JT == 20) e = launch_staged<1, 20, 8, false>(a, num_sms, s);
                else if (JT == 16) e = launch_staged<2, 16, 8, false>(a, num_sms, s);
                else if (JT == 8) e = launch_staged<2, 8, 16, false>(a, num_sms, s);
                else e = launch_staged<2, 4, 16, false>(a, num_sms, s);
                if (e == cudaSuccess && launches) ++*launches;
                return e;
            }
        }
    }
    if (mode == KERNEL_STAGED) return cudaErrorInvalidConfiguration;
    if (mode != KERNEL_REF) {
        // unaligned rows: positions tiled through shared memory with plain loads
        int tp = 256;
        size_t smem = ((size_t)a.K * ((a.J + 7) / 8 * 8) + (size_t)a.K * tp) * sizeof(float);
        while (smem > 200 * 1024 && tp > 32) { tp /= 2; smem = ((size_t)a.K * ((a.J + 7) / 8 * 8) + (size_t)a.K * tp) * sizeof(float); }
        if (smem <= 200 * 1024) {
            cudaError_t es = cudaFuncSetAttribute(contract_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (es != cudaSuccess) return es;
            dim3 grid((unsigned)((a.p + tp - 1) / tp), (unsigned)a.N);
            es = launch_pdl(contract_tile_kernel, grid, dim3(tp), smem, s, a);
            if (es == cudaSuccess && launches) ++*launches;
            return es;
        }
    }
    if (a.J > REF_MAX_J) return cudaErrorInvalidValue;
    const int threads = 128;
    dim3 grid((unsigned)((a.p + threads - 1) / threads), (unsigned)a.N);
    { cudaError_t el = launch_pdl(contract_ref_kernel, grid, dim3(threads), 0, s, a); if (el != cudaSuccess) return el; }
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

cudaError_t launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, cudaStream_t s) {
    wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status, limit_ns);
    return cudaGetLastError();
}

cudaError_t launch_round(const RoundArgs& a_in, cudaStream_t s, uint64_t* launches) {
    if (a_in.p <= 0) return cudaSuccess;
    RoundArgs a = a_in;
    a.range = Range{a.ws, a.ws + (int64_t)a.N * (a.c + a.N) * a.p - g_tune_checked_shrink};
    a.reverse = (a.k % 2 == 0 && !g_tune_serpentine_off) ? 1 : 0;
    const int threads = 256;
    cudaError_t e;
    if (a.p % 4 == 0 && aligned16(a.ws)) {
        const int64_t nv = a.p / 4;
        const unsigned blocks = (unsigned)((nv + threads - 1) / threads);
        const int groups = (a.N + 3) / 4;
        // Fewer blocks than SMs and more than 4 workers: one thread per group of 4 workers.  Measured on B200
        // over N = 8, 16, 32 and c = 8 .. 128: +10 .. +70 % up to p = 131072, -1 .. -8 % at p = 262144, 0 .. +7 %
        // at p = 524288, nothing from 2^20 on (tuning: 1 = never, 2 = always)
        const bool split = g_tune_round_split ? g_tune_round_split == 2 : (blocks <= 148);
        if (split && groups >= 2 && groups <= 8) {
            const int pvb = threads / groups;
            e = launch_pdl(round_split_kernel, dim3((unsigned)((nv + pvb - 1) / pvb)), dim3(pvb * groups), 0, s, a, groups);
            if (e == cudaSuccess && launches) ++*launches;
            return e;
        }
        // plain loads and stores, 4 workers in flight per thread: streaming cache hints (also with an L2
        // evict_last policy on the message stores: -1..-4 %), 512-thread blocks and 8 workers per group were
        // all measured and are not faster at d = 1.4e9
        e = launch_pdl(round_kernel<float4, 4>, dim3(blocks), dim3(threads), 0, s, a);
    } else {
        e = launch_pdl(round_kernel<float, 4>, dim3((unsigned)((a.p + threads - 1) / threads)), dim3(threads), 0, s, a);
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

cudaError_t launch_rounds_multi(const RoundArgs& a_in, int k_last, cudaStream_t s, uint64_t* launches) {
    RoundArgs a = a_in;
    a.range = Range{a.ws, a.ws + (int64_t)a.N * (a.c + a.N) * a.p - g_tune_checked_shrink};
    // L2 residency hints (measured: +6..+13 % at N = 8, +1..+4 % at N = 16, -1..-4 % at N = 4, where the
    // delta to cancel is still in L2 anyway); tuning: 1 = off, 2 = on
    a.hints = g_tune_rounds_hints ? (g_tune_rounds_hints == 2) : (a.N >= 8);
    if (a.p <= 0 || k_last < a.k) return cudaSuccess;
    // this form is latency-bound (L dependent rounds per thread): spread a small job over all SMs
    // with narrower accesses and smaller blocks rather than leave most of them idle
    int threads = 256;
    const bool vec = (a.p % 4 == 0 && aligned16(a.ws));
    if (a.N <= 32 && g_tune_rounds_multi_form != 1) {
        // float4 per lane once that still gives every SM a few blocks; single floats below
        const bool v4 = vec && (a.p / 128 >= 148 * 2) && g_tune_rounds_multi_form != 3;
        const int64_t pv = v4 ? a.p / 4 : a.p;
        // two vectors per lane where that still leaves every SM two blocks (measured: +2 .. +15 % on most
        // shapes); tuning: 1 / 2 force one / two
        int PVr = !v4 ? 1 : g_tune_rounds_coop_shape ? g_tune_rounds_coop_shape : (a.p / 256 >= 148 * 2 ? 2 : 1);
        if ((size_t)2 * a.N * 32 * PVr * 16 > 48 * 1024) PVr = 1;   // the hand-off tiles stay within the default 48 KB
        const unsigned blocks = (unsigned)((pv + 32 * PVr - 1) / (32 * PVr));
        const size_t smem = (size_t)2 * a.N * 32 * PVr * (v4 ? 16 : 4);
        const dim3 blk(32 * a.N);
        cudaError_t ec;
#define COOP(VT, PV) (a.N > 16 ? launch_pdl(rounds_coop_kernel<VT, PV, 2, 1024>, dim3(blocks), blk, smem, s, a, k_last) \
                               : launch_pdl(rounds_coop_kernel<VT, PV, 2, 512>, dim3(blocks), blk, smem, s, a, k_last))
        ec = !v4 ? COOP(float, 1) : PVr == 2 ? COOP(float4, 2) : COOP(float4, 1);
#undef COOP
        if (ec == cudaSuccess && launches) ++*launches;
        return ec;
    }
    bool use_vec = vec;
    if (vec && a.p / 4 >= (int64_t)148 * 256 * 4) threads = 256;
    else if (vec && a.p / 4 >= (int64_t)148 * 64 * 4) threads = 64;
    else { use_vec = false; threads = (a.p >= (int64_t)148 * 128 * 2) ? 128 : 64; }
    cudaError_t e;
    if (use_vec) {
        const int64_t nv = a.p / 4;
        e = launch_pdl(rounds_multi_kernel<float4, 4>, dim3((unsigned)((nv + threads - 1) / threads)), dim3(threads), 0, s,
                       a, k_last);
    } else {
        e = launch_pdl(rounds_multi_kernel<float, 4>, dim3((unsigned)((a.p + threads - 1) / threads)), dim3(threads), 0,
                       s, a, k_last);
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
