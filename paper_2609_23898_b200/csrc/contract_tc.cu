// Tensor-core contraction for encode / decode at large c (sm_100a: TMA + tcgen05 + TMEM).
//
//   out[j][q] = scale * sum_k coef[k][j] * in[k][q],   j < J (= c),  k < K rows,  q < p
//
// is a skinny GEMM with M = positions (128 per tile), N = J, K = input rows.  At
// c >= 32 the FP32 FMA pipe cannot keep up with HBM (c/4 flop per byte), so the
// products run on the 5th-generation tensor cores as 3 x TF32: every fp32 value
// is split into hi = tf32(x) and lo = tf32(x - hi) and
//   x*y ~ lo_x*hi_y + hi_x*lo_y + hi_x*hi_y           (relative error ~ 2^-22),
// accumulated in fp32 in tensor memory.
//
// One CTA of 11 warps per SM, persistent over the 128-position tiles of one worker:
//   warp 0      producer: one TMA load per chunk ([KC rows] x [128 positions], row-major)
//   warps 6-9   splitter: thread = position; reads its column of the chunk from shared
//               memory, splits it, and writes hi | lo into tensor memory (tcgen05.st),
//               where they are the A operand (rows = positions, columns = k)
//   warps 1,10  MMA issuers (one lane each, even / odd tiles, so that one can issue while
//               the other drains): tcgen05.mma kind::tf32, A from TMEM, B = the
//               coefficient matrix (hi and lo copies) resident in shared memory,
//               M=128, N=Npad, K=8 per instruction; warp 1 owns the TMEM allocation
//   warps 2-5   epilogue: tcgen05.ld of the accumulator, scale, transpose through a
//               shared-memory tile, one TMA store per 32 output rows
// So the data tile is read from shared memory exactly once, and global memory is
// touched only by TMA in rows of 512 contiguous bytes.  Every wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>

#include "kernels.cuh"
#include "tc_common.cuh"

namespace cerar {
namespace {

constexpr int TILE_M = 128;          // positions per tile = UMMA M
constexpr int NUM_THREADS = 32 * 11;
constexpr int OUT_ROWS = 32;         // output rows per TMA store

using namespace tc;

struct TcParams {
    int K_rows;        // physical input rows that carry data; rows beyond read as zero (TMA fill)
    int K_pad;         // K_rows rounded up to a multiple of KC
    int stages;        // shared-memory stages of raw chunks
    int NA;            // A (hi|lo) chunk buffers in tensor memory
    int Npad;          // J rounded up to 32
    int tmem_cols;     // power of two >= 2*Npad + NA*2*KC
};

// shared memory (1024-aligned): B_hi | B_lo | raw stages | 2 output tiles | barriers | tmem slot
template <int KC>
__global__ void __launch_bounds__(NUM_THREADS, 1)
contract_tc_kernel(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_out,
                   const __grid_constant__ ContractArgs a, const __grid_constant__ TcParams tp) {
    extern __shared__ unsigned char smem_dyn[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.y;
    const int stages = tp.stages, NA = tp.NA, Npad = tp.Npad, K_pad = tp.K_pad;
    const int nkc = K_pad / KC;
    const int nblk = Npad / 32;
    const uint32_t NAh = (uint32_t)NA / 2u;      // A buffers per MMA issuer

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* smem_al = smem_dyn + (smem_base - smem_u32(smem_dyn));
    const uint32_t b_bytes = (uint32_t)K_pad * Npad * 4u;            // one of B_hi / B_lo
    constexpr uint32_t chunk_bytes = (uint32_t)KC * TILE_M * 4u;
    constexpr uint32_t out_bytes = (uint32_t)OUT_ROWS * TILE_M * 4u;
    const uint32_t bhi_u32 = smem_base, blo_u32 = smem_base + b_bytes;
    const uint32_t raw_u32 = smem_base + 2u * b_bytes;
    const uint32_t out_u32 = raw_u32 + (uint32_t)stages * chunk_bytes;
    const uint32_t bar_u32 = out_u32 + 2u * out_bytes;
    const uint32_t raw_full = bar_u32, raw_empty = raw_full + 8u * stages;
    const uint32_t a_full = raw_empty + 8u * stages, a_empty = a_full + 8u * NA;
    const uint32_t acc_full = a_empty + 8u * NA, acc_empty = acc_full + 16u;
    const uint32_t out_full = acc_empty + 16u, out_free = out_full + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_al + (out_free + 16u - smem_base));
    const float* raw_s = reinterpret_cast<const float*>(smem_al + (raw_u32 - smem_base));
    float* out_s = reinterpret_cast<float*>(smem_al + (out_u32 - smem_base));

    // ---------------- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(raw_full + 8u * s, 1); mbar_init(raw_empty + 8u * s, 4); }
        for (int b = 0; b < NA; ++b) { mbar_init(a_full + 8u * b, 4); mbar_init(a_empty + 8u * b, 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full + 8u * b, 1); mbar_init(acc_empty + 8u * b, 4);
            mbar_init(out_full + 8u * b, 4); mbar_init(out_free + 8u * b, 1);
        }
        mbar_init_fence();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)tp.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {
        // coefficients of this worker as the tensor core's B operand (tf32 hi and lo copies)
        split_coefficients(a, w, K_pad, Npad, reinterpret_cast<uint32_t*>(smem_al),
                           reinterpret_cast<uint32_t*>(smem_al + b_bytes));
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // the set-up above reads only the plan's constant coefficients and may overlap the tail of the
    // kernel before this one in the stream; the data may not be touched before that kernel is done
    grid_dependency_wait();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t a_col0 = 2u * (uint32_t)Npad;            // A buffers start after the two accumulators

    const int64_t ntiles = a.tiles_per_worker;
    bool failed = false;

    if (warp == 0) {
        // ================= producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x) {
                const int q0 = (int)(t * TILE_M);
                for (int kc = 0; kc < nkc; ++kc, ++it) {
                    const uint32_t s = it % stages, ph = (it / stages) & 1u;
                    if (!mbar_wait_bounded(raw_empty + 8u * s, ph ^ 1u)) { failed = true; break; }
                    mbar_arrive_expect_tx(raw_full + 8u * s, chunk_bytes);
                    tma_load_3d(raw_u32 + s * chunk_bytes, &tmap_in, q0, kc * KC, w, raw_full + 8u * s);
                }
            }
        }
    } else if (warp == 1 || warp == 10) {
        // ================= MMA issuers: issuer m takes tiles m, m+2, ... into accumulator m
        if (lane == 0) {
            const uint32_t m = (warp == 1) ? 0u : 1u;
            // instruction descriptor: D=f32, A=B=tf32, A from TMEM (K-major), B MN-major, N=Npad, M=128
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) |
                                   ((uint32_t)(Npad >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
            const uint32_t b_lbo = (uint32_t)K_pad * 128u;
            const uint64_t bhi0 = make_desc(bhi_u32, b_lbo, 512u), blo0 = make_desc(blo_u32, b_lbo, 512u);
            const uint32_t d_tmem = tmem_base + m * (uint32_t)Npad;
            uint32_t tc = m;
            for (int64_t t = blockIdx.x + (int64_t)m * gridDim.x; t < ntiles && !failed; t += 2 * (int64_t)gridDim.x, tc += 2) {
                const uint32_t aph = (tc >> 1) & 1u;
                if (!mbar_wait_bounded(acc_empty + 8u * m, aph ^ 1u)) { failed = true; break; }
                tc_fence_after();
                for (int kc = 0; kc < nkc; ++kc) {
                    const uint32_t seq = (tc >> 1) * (uint32_t)nkc + (uint32_t)kc;
                    const uint32_t ab = m * NAh + seq % NAh, ph = (seq / NAh) & 1u;
                    if (!mbar_wait_bounded(a_full + 8u * ab, ph)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t a_hi = tmem_base + a_col0 + ab * (2u * KC), a_lo = a_hi + KC;
                    int ksteps = KC / 8;
                    const int rows_left = tp.K_rows - kc * KC;               // rows with data in this chunk
                    if (rows_left < KC) ksteps = (rows_left + 7) / 8;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        // descriptor start address advances by 8 rows x 128 B (in 16-byte units)
                        const uint64_t boff = (uint64_t)(((kc * KC + ks * 8) * 128) >> 4);
                        tc_mma_tf32_ts(d_tmem, a_lo + ks * 8u, bhi0 + boff, idesc, (kc | ks) != 0);
                        tc_mma_tf32_ts(d_tmem, a_hi + ks * 8u, blo0 + boff, idesc, 1u);
                        tc_mma_tf32_ts(d_tmem, a_hi + ks * 8u, bhi0 + boff, idesc, 1u);
                    }
                    tc_commit(a_empty + 8u * ab);      // the A buffer is free once these MMAs have read it
                }
                if (failed) break;
                tc_commit(acc_full + 8u * m);          // the accumulator is complete
            }
        }
    } else if (warp < 6) {
        // ================= epilogue (warps 2..5; TMEM lanes 32*(warp%4) ..)
        const int qd = warp & 3;
        const int pos = qd * 32 + lane;
        uint32_t tc = 0, oc = 0;
        for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++tc) {
            const uint32_t buf = tc & 1u, aph = (tc >> 1) & 1u;
            if (!warp_wait(acc_full + 8u * buf, aph)) { failed = true; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + buf * (uint32_t)Npad;
            for (int nb = 0; nb < nblk; ++nb, ++oc) {
                float v[32];
                tc_ld32(taddr + (uint32_t)nb * 32u, v);
                if (nb == nblk - 1) {
                    // everything is in registers: hand the accumulator back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty + 8u * buf);
                }
                const uint32_t ob = oc & 1u, oph = (oc >> 1) & 1u;
                if (!warp_wait(out_free + 8u * ob, oph ^ 1u)) { failed = true; break; }
                float* o = out_s + (size_t)ob * (OUT_ROWS * TILE_M) + pos;
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j * TILE_M] = v[j] * a.scale;
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(out_full + 8u * ob);
                if (warp == 2 && lane == 0) {
                    if (!mbar_wait_bounded(out_full + 8u * ob, oph)) {
                        failed = true;
                    } else {
                        // rows beyond J and positions beyond p are clipped by the tensor map
                        tma_store_3d(&tmap_out, (int)(t * TILE_M), nb * OUT_ROWS, w, out_u32 + ob * out_bytes);
                        bulk_commit();
                        if (oc >= 1) {                 // the store before this one has read its tile: free it
                            bulk_wait_read_1();
                            mbar_arrive(out_free + 8u * (ob ^ 1u));
                        }
                    }
                }
                if (warp == 2) failed = __any_sync(0xffffffffu, failed ? 1 : 0) != 0;
                if (failed) break;
            }
        }
        if (warp == 2 && lane == 0) bulk_wait_all();   // all output has left shared memory and is written
    } else {
        // ================= splitter (warps 6..9): thread = position
        const int qd = warp & 3;
        const int pos = qd * 32 + lane;
        uint32_t it = 0, tc = 0;
        for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++tc) {
            for (int kc = 0; kc < nkc; ++kc, ++it) {
                const uint32_t s = it % stages, ph = (it / stages) & 1u;
                // A buffers are split between the two MMA issuers: tile parity picks the half
                const uint32_t seq = (tc >> 1) * (uint32_t)nkc + (uint32_t)kc;
                const uint32_t ab = (tc & 1u) * NAh + seq % NAh, pa = (seq / NAh) & 1u;
                if (!warp_wait(raw_full + 8u * s, ph)) { failed = true; break; }
                const float* col = raw_s + (size_t)s * (KC * TILE_M) + pos;
                uint32_t hi[KC], lo[KC];
#pragma unroll
                for (int k = 0; k < KC; ++k) {
                    const float x = col[k * TILE_M];
                    hi[k] = tf32_bits(x);
                    lo[k] = tf32_bits(x - __uint_as_float(hi[k]));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(raw_empty + 8u * s);        // the values are in registers
                if (!warp_wait(a_empty + 8u * ab, pa ^ 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t ta = tmem_base + ((uint32_t)(qd * 32) << 16) + a_col0 + ab * (2u * KC);
#pragma unroll
                for (int k8 = 0; k8 < KC / 8; ++k8) {
                    tc_st8(ta + 8u * k8, hi + 8 * k8);
                    tc_st8(ta + KC + 8u * k8, lo + 8 * k8);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full + 8u * ab);
            }
        }
    }

    if (failed) {
        if (lane == 0) atomicExch(a.status, 2);
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) { }      // let async work that is in flight finish
    }
    // ---------------- tear-down: every warp arrives here (all waits above are bounded)
    // (only now may the next kernel of the stream be scheduled next to this CTA: blocks that arrive
    // early and wait for this grid to finish were measured to slow it down by 10 %)
    grid_dependents_may_launch();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tp.tmem_cols) : "memory");
    }
}

template <int KC>
cudaError_t launch_kc(const CUtensorMap& tin, const CUtensorMap& tout, const ContractArgs& a, const TcParams& tp,
                      size_t smem, dim3 grid, cudaStream_t s) {
    auto kern = contract_tc_kernel<KC>;
    {   // per device and cheap: set on every launch rather than cached
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    return launch_pdl(kern, grid, dim3(NUM_THREADS), smem, s, tin, tout, a, tp);
}

}  // namespace

int g_tune_tc_kc = 0, g_tune_tc_stages = 0, g_tune_tc_variant = 0;

bool tc_eligible(const ContractArgs& a) {
    if (a.J < 32 || a.J > 128) return false;      // N = J padded to 32; two coefficient copies must fit in smem
    if (a.p % 4 != 0 || a.p >= (int64_t)1 << 31) return false;
    if ((reinterpret_cast<uintptr_t>(a.in) & 15u) || (a.in_rstride % 4) || (a.in_wstride % 4)) return false;
    if ((reinterpret_cast<uintptr_t>(a.out) & 15u) || (a.out_rstride % 4) || (a.out_wstride % 4)) return false;
    return get_encode_fn() != nullptr;
}

cudaError_t launch_contract_tc(ContractArgs a, int num_sms, cudaStream_t s, uint64_t* launches) {
    TcParams tp;
    tp.K_rows = a.K + a.skip_count;                         // decode: physical rows that are not part of Y
    tp.Npad = ((a.J + 31) / 32) * 32;
    // rows per chunk: as few padded rows as possible, then as large as possible, with at
    // least 3 stages in the shared memory that the two coefficient copies leave
    const size_t budget = 227 * 1024 - 1024;
    const int cands[4] = {40, 32, 24, 16};
    int best_kc = 0, best_pad = 1 << 30, best_stages = 0;
    for (int ci = 0; ci < 4; ++ci) {
        const int kc = cands[ci];
        if (g_tune_tc_kc && kc != g_tune_tc_kc) continue;
        if (2 * tp.Npad + 2 * 2 * kc > 512) continue;       // two accumulators + at least two A buffers
        const int kpad = ((tp.K_rows + kc - 1) / kc) * kc;
        const size_t fixed_c = 1024 + 2 * (size_t)kpad * tp.Npad * 4 + 2 * OUT_ROWS * TILE_M * 4 + 512;
        const size_t stage_c = (size_t)kc * TILE_M * 4;
        if (fixed_c + 3 * stage_c > budget) continue;
        int st = (int)((budget - fixed_c) / stage_c);
        if (st > 8) st = 8;
        if (g_tune_tc_stages && g_tune_tc_stages < st) st = g_tune_tc_stages;
        if (st < 2) continue;
        if (kpad < best_pad) { best_pad = kpad; best_kc = kc; best_stages = st; }
    }
    if (!best_kc) return cudaErrorInvalidConfiguration;
    const int KC = best_kc;
    tp.K_pad = best_pad;
    tp.stages = best_stages;
    tp.NA = (512 - 2 * tp.Npad) / (2 * KC);
    if (tp.NA > 4) tp.NA = 4;
    tp.NA -= tp.NA % 2;                                   // one half per MMA issuer
    tp.tmem_cols = 32;
    while (tp.tmem_cols < 2 * tp.Npad + tp.NA * 2 * KC) tp.tmem_cols *= 2;
    const size_t smem = 1024 + 2 * (size_t)tp.K_pad * tp.Npad * 4 + (size_t)tp.stages * KC * TILE_M * 4 +
                        2 * OUT_ROWS * TILE_M * 4 + 512;

    CUtensorMap tin, tout;
    if (!make_map(&tin, a.in, a.p, tp.K_rows, a.N, a.in_rstride, a.in_wstride, TILE_M, KC)) return cudaErrorInvalidValue;
    if (!make_map(&tout, a.out, a.p, a.J, a.N, a.out_rstride, a.out_wstride, TILE_M, OUT_ROWS)) return cudaErrorInvalidValue;

    a.tiles_per_worker = (int)((a.p + TILE_M - 1) / TILE_M);
    int64_t per_worker = num_sms / a.N;
    if (per_worker < 1) per_worker = 1;
    if (per_worker > a.tiles_per_worker) per_worker = a.tiles_per_worker;
    dim3 grid((unsigned)per_worker, (unsigned)a.N);
    cudaError_t e;
    switch (KC) {
        case 40: e = launch_kc<40>(tin, tout, a, tp, smem, grid, s); break;
        case 32: e = launch_kc<32>(tin, tout, a, tp, smem, grid, s); break;
        case 24: e = launch_kc<24>(tin, tout, a, tp, smem, grid, s); break;
        default: e = launch_kc<16>(tin, tout, a, tp, smem, grid, s); break;
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
