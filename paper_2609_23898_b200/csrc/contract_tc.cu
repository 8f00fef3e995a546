// Tensor-core contraction for encode / decode at large c (sm_100a: TMA + tcgen05 + TMEM).
//
//   out[j][q] = scale * sum_k coef[k][j] * in[k][q],   j < J (= c),  k < K rows,  q < p
//
// is a skinny GEMM with M = positions (128 per tile), N = J, K = input rows.  At
// c >= 32 the FP32 FMA pipe cannot keep up with HBM (c/4 flop per byte), so the
// products run on the 5th-generation tensor cores as 3 x TF32: every fp32 value
// is split into hi = tf32(x) and lo = tf32(x - hi) and
//   x*y ~ hi_x*hi_y + lo_x*hi_y + hi_x*lo_y           (relative error ~ 2^-22),
// accumulated in fp32 in tensor memory.
//
// Roles in a CTA of 10 warps (one CTA per SM, persistent over the tiles of one worker):
//   warp 0      producer: TMA loads of [KC rows x 128 positions] chunks (swizzled 32 x KC boxes)
//   warp 1      MMA issuer (one lane): tcgen05.mma kind::tf32, M=128, N=Npad, K=8; owns TMEM
//   warps 2-5   epilogue: tcgen05.ld of the accumulator, scale, coalesced stores
//   warps 6-9   splitter: rewrite a landed chunk as hi (in place) and lo (second buffer)
// Both operands are "MN-major": positions (A) and outputs j (B) are the contiguous
// dimension in shared memory, which is exactly how the data lies in HBM (no transpose).
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>

#include "kernels.cuh"

namespace cerar {
namespace {

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;
constexpr int TILE_M = 128;          // positions per tile = UMMA M
constexpr int NSPLIT = 4;            // splitter warps
constexpr int NUM_THREADS = 32 * (6 + NSPLIT);

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int u, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(u), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float tf32_rna(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// Shared-memory matrix descriptor for an MN-major 32-bit operand.  The only layout
// the tensor core accepts for that case is the 128-byte swizzle with 32-byte atoms:
// rows of 128 bytes (32 fp32 along M/N) at a 128-byte pitch along K, and inside every
// group of 4 rows the 32-byte chunk index is XOR-ed with (row & 3) -- the pattern TMA
// writes with CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B.  lbo = byte distance between
// consecutive 32-element blocks along M/N, sbo = between consecutive 4-row groups.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;          // descriptor version for sm_100
    d |= (uint64_t)1 << 61;          // 128-byte swizzle, 32-byte atom
    return d;
}

#ifdef CERAR_TC_DEBUG
__device__ float g_dbg[1 << 16];
#endif

struct TcParams {
    int K_rows;        // input rows that carry data (tensor-map rows); rows beyond read as zero
    int K_pad;         // K_rows rounded up to KC
    int KC;            // rows per pipeline stage (multiple of 8)
    int stages;
    int Npad;          // J rounded up to 32
    int tmem_cols;     // power of two >= 2*Npad
    int dbg;
};

// shared memory: [1024-aligned] B_hi | B_lo | stages x (raw/hi chunk, lo chunk) | barriers | tmem slot
template <int DUMMY>
__global__ void __launch_bounds__(NUM_THREADS, 1)
contract_tc_kernel(const __grid_constant__ CUtensorMap tmap4, const __grid_constant__ CUtensorMap tmap3,
                   const __grid_constant__ ContractArgs a, const __grid_constant__ TcParams tp) {
    extern __shared__ unsigned char smem_dyn[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.y;
    const int KC = tp.KC, stages = tp.stages, Npad = tp.Npad, K_pad = tp.K_pad;
    const int nkc = K_pad / KC;
    const int nblk = Npad / 32;

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* smem_al = smem_dyn + (smem_base - smem_u32(smem_dyn));
    const uint32_t b_bytes = (uint32_t)K_pad * Npad * 4u;            // one of B_hi / B_lo
    const uint32_t chunk_bytes = (uint32_t)KC * TILE_M * 4u;         // one of hi / lo chunk
    const uint32_t bhi_u32 = smem_base, blo_u32 = smem_base + b_bytes;
    const uint32_t stage_u32 = smem_base + 2u * b_bytes;             // 1024-aligned: K_pad % 8 == 0
    const uint32_t bar_u32 = stage_u32 + (uint32_t)stages * 2u * chunk_bytes;
    // barriers: raw_full[s], lo_full[s], empty[s], acc_full[2], acc_empty[2]
    const uint32_t raw_full = bar_u32, lo_full = bar_u32 + 8u * stages, empty = bar_u32 + 16u * stages;
    const uint32_t acc_full = bar_u32 + 24u * stages, acc_empty = acc_full + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_al + (bar_u32 - smem_base) + 24u * stages + 32u);

    // ---------------- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(raw_full + 8u * s, 1);
            mbar_init(lo_full + 8u * s, 1);
            mbar_init(empty + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full + 8u * b, 1);
            mbar_init(acc_empty + 8u * b, 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)tp.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {
        // coefficients of this worker, split into tf32 hi / lo, written in the swizzled
        // MN-major layout: block nb (32 outputs) | row k (128 B) | 32-byte chunk ^ (k & 3)
        const float* cf = a.coef + (size_t)w * a.K * a.J;
        float* bhi = reinterpret_cast<float*>(smem_al);
        float* blo = reinterpret_cast<float*>(smem_al + b_bytes);
        for (int idx = threadIdx.x; idx < K_pad * Npad; idx += blockDim.x) {
            const int k = idx / Npad, j = idx - k * Npad;
            // physical input row k -> coefficient row (the row at skip_row is not part of Y: zero)
            int src = -1;
            if (k < a.skip_row) src = k; else if (k > a.skip_row) src = k - 1;
            float v = 0.f;
            if (src >= 0 && src < a.K && j < a.J) v = cf[(size_t)src * a.J + j];
            const float hi = tf32_rna(v);
            const float lo = tf32_rna(v - hi);
            const int nb = j >> 5, jj = j & 31;
            const int off = nb * (K_pad * 32) + k * 32 + ((((jj >> 3) ^ (k & 3)) << 3) | (jj & 7));
            bhi[off] = hi;
            blo[off] = lo;
        }
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
#ifdef CERAR_TC_DEBUG
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        const float* bh = reinterpret_cast<const float*>(smem_al);
        for (int i = threadIdx.x; i < K_pad * Npad && i < 8192; i += blockDim.x) g_dbg[8192 + i] = bh[i];   // B_hi
        if (threadIdx.x == 0) { g_dbg[20000] = __uint_as_float(tmem_base); g_dbg[20001] = (float)stages; g_dbg[20002] = (float)K_pad; }
    }
#endif

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
                    if (!mbar_wait_bounded(empty + 8u * s, ph ^ 1u)) { failed = true; break; }
                    mbar_arrive_expect_tx(raw_full + 8u * s, chunk_bytes);
                    const uint32_t dst = stage_u32 + s * 2u * chunk_bytes;
                    if ((int64_t)q0 + TILE_M <= a.p) {
                        // whole tile: one 4-D box = 4 blocks of 32 positions x KC rows (the smem layout of 4 boxes)
                        tma_load_4d(dst, &tmap4, 0, kc * KC, q0 >> 5, w, raw_full + 8u * s);
                    } else {
                        // ragged last tile: position-bounded 3-D boxes, zero-filled beyond p
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            tma_load_3d(dst + (uint32_t)b * KC * 128u, &tmap3, q0 + 32 * b, kc * KC, w, raw_full + 8u * s);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer
        if (lane == 0) {
            // instruction descriptor: D=f32, A=B=tf32, both MN-major, N=Npad, M=128
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) |
                                   ((uint32_t)(Npad >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
            const uint32_t a_lbo = (uint32_t)KC * 128u, b_lbo = (uint32_t)K_pad * 128u;
            uint32_t it = 0, tc = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++tc) {
                const uint32_t buf = tc & 1u, aph = (tc >> 1) & 1u;
                if (!mbar_wait_bounded(acc_empty + 8u * buf, aph ^ 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)Npad;
                for (int kc = 0; kc < nkc; ++kc, ++it) {
                    const uint32_t s = it % stages, ph = (it / stages) & 1u;
                    if (!mbar_wait_bounded(lo_full + 8u * s, ph)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t hi_u32 = stage_u32 + s * 2u * chunk_bytes, lo_u32 = hi_u32 + chunk_bytes;
                    int ksteps = KC / 8;
                    const int rows_left = tp.K_rows - kc * KC;               // rows with data in this chunk
                    if (rows_left < KC) ksteps = (rows_left + 7) / 8;
                    for (int ks = 0; ks < ((tp.dbg & 4) ? 0 : ksteps); ++ks) {
                        const uint64_t ahi = make_desc(hi_u32 + ks * 1024u, a_lbo, 512u);
                        const uint64_t alo = make_desc(lo_u32 + ks * 1024u, a_lbo, 512u);
                        const uint32_t boff = (uint32_t)(kc * KC + ks * 8) * 128u;
                        const uint64_t bhi = make_desc(bhi_u32 + boff, b_lbo, 512u);
                        const uint64_t blo = make_desc(blo_u32 + boff, b_lbo, 512u);
                        tc_mma_tf32(d_tmem, alo, bhi, idesc, (kc | ks) != 0);
                        tc_mma_tf32(d_tmem, ahi, blo, idesc, 1u);
                        tc_mma_tf32(d_tmem, ahi, bhi, idesc, 1u);
                    }
                    tc_commit(empty + 8u * s);         // the stage is free once these MMAs have read it
                }
                if (failed) break;
                tc_commit(acc_full + 8u * buf);        // the accumulator is complete
            }
        }
    } else if (warp < 6) {
        // ================= epilogue (warps 2..5; TMEM lanes 32*(warp%4) ..)
        const int qd = warp & 3;
        float* out_w = a.out + (int64_t)w * a.out_wstride;
        uint32_t tc = 0;
        for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++tc) {
            const uint32_t buf = tc & 1u, aph = (tc >> 1) & 1u;
            if (!mbar_wait_bounded(acc_full + 8u * buf, aph)) { failed = true; break; }
            tc_fence_after();
            const int64_t pos = t * TILE_M + qd * 32 + lane;
            const bool in_range = pos < a.p;
            const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + buf * (uint32_t)Npad;
            for (int nb = 0; nb < nblk; ++nb) {
                float v[32];
                tc_ld32(taddr + (uint32_t)nb * 32u, v);
                if (nb == nblk - 1) {
                    // everything is in registers: hand the accumulator back before storing
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty + 8u * buf);
                }
#ifdef CERAR_TC_DEBUG
                if (blockIdx.x == 0 && blockIdx.y == 0 && tc == 0 && nb == 0)
                    for (int j = 0; j < 32; ++j) g_dbg[(qd * 32 + lane) * 32 + j] = v[j];      // [0, 4096): D tile
#endif
                if (in_range && !(tp.dbg & 2)) {
                    float* o = out_w + (int64_t)(nb * 32) * a.out_rstride + pos;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (nb * 32 + j < a.J) o[(int64_t)j * a.out_rstride] = v[j] * a.scale;
                }
            }
        }
    } else {
        // ================= splitter (warps 6..): every warp owns whole chunks (chunk it -> warp it % NSPLIT),
        // so several chunks are being split at once; hi is written in place, lo to the second buffer
        const int sw = warp - 6;
        const int n4 = KC * TILE_M / 4;             // float4 per chunk
        uint32_t it = 0;
        for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x) {
            for (int kc = 0; kc < nkc; ++kc, ++it) {
                if ((int)(it % NSPLIT) != sw) continue;
                const uint32_t s = it % stages, ph = (it / stages) & 1u;
                if (!mbar_wait_bounded(raw_full + 8u * s, ph)) { failed = true; break; }
                float4* hi = reinterpret_cast<float4*>(smem_al + (stage_u32 - smem_base) + (size_t)s * 2u * chunk_bytes);
                float4* lo = reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(hi) + chunk_bytes);
                if (!(tp.dbg & 1)) {
                    // 4 independent float4 per lane and step: loads first, then the stores
                    for (int i0 = lane; i0 < n4; i0 += 128) {
                        float4 x[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) x[u] = hi[i0 + 32 * u];          // n4 is a multiple of 128
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            float4 h, l;
                            h.x = tf32_rna(x[u].x); l.x = tf32_rna(x[u].x - h.x);
                            h.y = tf32_rna(x[u].y); l.y = tf32_rna(x[u].y - h.y);
                            h.z = tf32_rna(x[u].z); l.z = tf32_rna(x[u].z - h.z);
                            h.w = tf32_rna(x[u].w); l.w = tf32_rna(x[u].w - h.w);
                            hi[i0 + 32 * u] = h;
                            lo[i0 + 32 * u] = l;
                        }
                    }
                }
#ifdef CERAR_TC_DEBUG
                if (blockIdx.x == 0 && blockIdx.y == 0 && it == 0) {
                    const float* hf = reinterpret_cast<const float*>(hi);
                    for (int i = lane; i < KC * TILE_M; i += 32) g_dbg[4096 + i] = hf[i];          // [4096, 4096+2048): hi chunk 0
                }
#endif
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(lo_full + 8u * s);
            }
        }
    }

    if (failed) {
        if (lane == 0) atomicExch(a.status, 2);
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) { }      // let async work that is in flight finish
    }
    // ---------------- tear-down: every warp arrives here (all waits above are bounded)
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tp.tmem_cols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

int g_tune_tc_kc = 0, g_tune_tc_stages = 0, g_tune_tc_dbg = 0;

bool tc_eligible(const ContractArgs& a) {
    if (a.J < 32 || a.J > 128) return false;      // N = J padded to 32; two coefficient copies must fit in smem
    if (a.p % 4 != 0 || a.p >= (int64_t)1 << 31) return false;
    if ((reinterpret_cast<uintptr_t>(a.in) & 15u) || (a.in_rstride % 4) || (a.in_wstride % 4)) return false;
    if (a.in_rstride != a.p) return false;
    return get_encode_fn() != nullptr;
}

cudaError_t launch_contract_tc(ContractArgs a, int num_sms, cudaStream_t s, uint64_t* launches) {
    TcParams tp;
    const bool has_skip = a.skip_row < a.K;                 // decode: one physical row is not part of Y
    tp.K_rows = a.K + (has_skip ? 1 : 0);
    tp.Npad = ((a.J + 31) / 32) * 32;
    tp.dbg = g_tune_tc_dbg;
    tp.tmem_cols = 32;
    while (tp.tmem_cols < 2 * tp.Npad) tp.tmem_cols *= 2;
    // rows per stage: as few padded rows as possible, then as large as possible, with at
    // least NSPLIT stages in the shared memory that the two coefficient copies leave
    const size_t budget = 225 * 1024;
    const int cands[4] = {40, 32, 24, 16};
    int best_kc = 0, best_pad = 1 << 30, best_stages = 0;
    for (int ci = 0; ci < 4; ++ci) {
        const int kc = cands[ci];
        if (g_tune_tc_kc && kc != g_tune_tc_kc) continue;
        const int kpad = ((tp.K_rows + kc - 1) / kc) * kc;
        const size_t fixed_c = 1024 + 2 * (size_t)kpad * tp.Npad * 4 + 256;
        const size_t stage_c = 2 * (size_t)kc * TILE_M * 4;
        if (fixed_c + NSPLIT * stage_c > budget) continue;
        int st = (int)((budget - fixed_c) / stage_c);
        if (st > 12) st = 12;
        if (g_tune_tc_stages && g_tune_tc_stages < st) st = g_tune_tc_stages;
        st -= st % NSPLIT;
        if (st < NSPLIT) continue;
        if (kpad < best_pad) { best_pad = kpad; best_kc = kc; best_stages = st; }
    }
    if (!best_kc) return cudaErrorInvalidConfiguration;
    // Chunk i is split by warp i % NSPLIT and lives in stage i % stages.  With stages a
    // multiple of NSPLIT the two uses of a stage that follow each other belong to the same
    // warp, so a warp never waits on a barrier phase that is more than one step ahead.
    tp.KC = best_kc;
    tp.K_pad = best_pad;
    tp.stages = best_stages;
    const size_t chunk_bytes = (size_t)tp.KC * TILE_M * 4;
    const size_t fixed = 1024 + 2 * (size_t)tp.K_pad * tp.Npad * 4 + 256;
    const int stages = tp.stages;
    const size_t smem = fixed + (size_t)stages * 2 * chunk_bytes + (size_t)stages * 24;

    // Tensor maps over the input.  tmap3: (positions, rows, workers), boxes of 32 positions x KC
    // rows, bounded by p (ragged last tile).  tmap4: (32 positions, rows, blocks of 32 positions,
    // workers) over the whole blocks only: one box brings a whole 128-position chunk.
    CUtensorMap tmap3, tmap4;
    {
        cuuint64_t gdim[3] = {(cuuint64_t)a.p, (cuuint64_t)tp.K_rows, (cuuint64_t)a.N};
        cuuint64_t gstr[2] = {(cuuint64_t)a.in_rstride * 4, (cuuint64_t)a.in_wstride * 4};
        cuuint32_t box[3] = {32, (cuuint32_t)tp.KC, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = get_encode_fn()(&tmap3, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(a.in), gdim, gstr,
                                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t nblocks = (cuuint64_t)(a.p / 32) > 0 ? (cuuint64_t)(a.p / 32) : 1;
        cuuint64_t gdim[4] = {32, (cuuint64_t)tp.K_rows, nblocks, (cuuint64_t)a.N};
        cuuint64_t gstr[3] = {(cuuint64_t)a.in_rstride * 4, 128, (cuuint64_t)a.in_wstride * 4};
        cuuint32_t box[4] = {32, (cuuint32_t)tp.KC, 4, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = get_encode_fn()(&tmap4, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(a.in), gdim, gstr,
                                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }

    auto kern = contract_tc_kernel<0>;
    static thread_local size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    a.tiles_per_worker = (int)((a.p + TILE_M - 1) / TILE_M);
    int64_t per_worker = num_sms / a.N;
    if (per_worker < 1) per_worker = 1;
    if (per_worker > a.tiles_per_worker) per_worker = a.tiles_per_worker;
    dim3 grid((unsigned)per_worker, (unsigned)a.N);
    kern<<<grid, NUM_THREADS, smem, s>>>(tmap4, tmap3, a, tp);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

#ifdef CERAR_TC_DEBUG
extern "C" int cerar_debug_fetch(float* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, g_dbg, (size_t)n * 4);
}
#endif

}  // namespace cerar
