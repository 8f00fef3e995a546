// tcgen05 / TMA helpers shared by the tensor-core contraction kernels (sm_100a).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.cuh"
#include "ptx.cuh"

namespace cerar {
namespace tc {

using namespace ptx;

// whole-warp wait with one outcome for all lanes (the .sync.aligned tcgen05 instructions
// that follow need the warp converged)
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait_bounded(bar, parity) ? 1 : 0) != 0;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
        ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// Hardware barrier `id` among `count` threads (whole warps); the second form also ORs a flag over them.
__device__ __forceinline__ void bar_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ bool bar_red_or(uint32_t id, uint32_t count, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.b32 q, %3, 0;\n bar.red.or.pred p, %1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(r) : "r"(id), "r"(count), "r"((uint32_t)flag) : "memory");
    return r != 0;
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One k-step (8 rows) of the 3 x TF32 product, A in tensor memory, B through a shared-memory descriptor:
// D (+)= A_lo B_hi, D += A_hi B_lo, D += A_hi B_hi, issued back to
// back from one asm statement.  An issuing thread cannot start a tcgen05.mma more often than every ~54 clk
// (measured; the pipe takes 16 clk for M128 N32 K8), and whatever integer work sits between two of them adds
// to that, so the operands are prepared before the burst.
__device__ __forceinline__ void tc_mma_tf32_ts_x3(uint32_t tmem_d, uint32_t tmem_a_hi, uint32_t tmem_a_lo, uint64_t bhi,
                                                  uint64_t blo, uint32_t idesc, uint32_t accumulate_first) {
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.b32 p, %6, 0;\n setp.eq.b32 q, 0, 0;\n"
        " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%2], %3, %5, p;\n"
        " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %4, %5, q;\n"
        " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %3, %5, q;\n}\n"
        ::"r"(tmem_d), "r"(tmem_a_hi), "r"(tmem_a_lo), "l"(bhi), "l"(blo), "r"(idesc), "r"(accumulate_first) : "memory");
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
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
// fp32 -> tf32 (10 explicit mantissa bits), round to nearest, ties away from zero
// (two integer instructions; cvt.rna.tf32.f32 gives the same bits in one, but runs on the slow conversion pipe:
// the whole contraction measured 35 % slower with it)
__device__ __forceinline__ uint32_t tf32_bits(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }

// Shared-memory matrix descriptor for an MN-major 32-bit operand.  The only layout
// the tensor core accepts for that case is the 128-byte swizzle with 32-byte atoms:
// rows of 128 bytes (32 fp32 along N) at a 128-byte pitch along K, and inside every
// group of 4 rows the 32-byte chunk index is XOR-ed with (row & 3).  lbo = byte
// distance between consecutive 32-element blocks along N, sbo = between 4-row groups.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;          // descriptor version for sm_100
    d |= (uint64_t)1 << 61;          // 128-byte swizzle, 32-byte atom
    return d;
}


// 16 accumulator columns of this warp's 32 TMEM lanes
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st4(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                   "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
}
// N consecutive columns (N a multiple of 4) with as few instructions as possible
template <int N>
__device__ __forceinline__ void tc_st_cols(uint32_t taddr, const uint32_t* v) {
    if constexpr (N >= 16) { tc_st16(taddr, v); tc_st_cols<N - 16>(taddr + 16u, v + 16); }
    else if constexpr (N >= 8) { tc_st8(taddr, v); tc_st_cols<N - 8>(taddr + 8u, v + 8); }
    else if constexpr (N >= 4) { tc_st4(taddr, v); tc_st_cols<N - 4>(taddr + 4u, v + 4); }
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
// instruction descriptor: D = f32, A = B = tf32, A from TMEM (K-major), B MN-major, N = n, M = 128
__device__ __forceinline__ uint32_t idesc_tf32_ts(uint32_t n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// Worker w's K x J coefficient matrix, split into tf32 hi / lo copies, in the only layout the
// tensor core takes for an MN-major 32-bit B operand (128-byte swizzle with 32-byte atoms):
// block nb (32 outputs) | row k (128 B) | 32-byte chunk ^ (k & 3).  Physical input rows that are
// not part of the contraction (a.skip_row ..) and the padding up to K_pad x Npad are zero.
// All threads of the CTA take part; the caller fences (async proxy) and synchronises.
__device__ __forceinline__ void split_coefficients(const ContractArgs& a, int w, int K_pad, int Npad, uint32_t* bhi,
                                                   uint32_t* blo) {
    const float* cf = a.coef + (size_t)w * a.K * a.J;
    for (int idx = threadIdx.x; idx < K_pad * Npad; idx += blockDim.x) {
        const int k = idx / Npad, j = idx - k * Npad;
        int src = -1;                      // physical input row k -> coefficient row
        if (k < a.skip_row) src = k; else if (k >= a.skip_row + a.skip_count) src = k - a.skip_count;
        float v = 0.f;
        if (src >= 0 && src < a.K && j < a.J) v = cf[(size_t)src * a.J + j];
        const uint32_t hi = tf32_bits(v);
        const uint32_t lo = tf32_bits(v - __uint_as_float(hi));
        const int nb = j >> 5, jj = j & 31;
        const int off = nb * (K_pad * 32) + k * 32 + ((((jj >> 3) ^ (k & 3)) << 3) | (jj & 7));
        bhi[off] = hi;
        blo[off] = lo;
    }
}

// ---- host side: tensor maps over [N workers][rows][p positions] fp32 arrays
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
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

// box = box_cols positions x box_rows rows of one worker; positions beyond p and rows
// beyond `rows` read as zero and are not written
inline bool make_map(CUtensorMap* m, const float* base, int64_t p, int rows, int N, int64_t rstride, int64_t wstride,
                     int box_cols, int box_rows) {
    cuuint64_t gdim[3] = {(cuuint64_t)p, (cuuint64_t)rows, (cuuint64_t)N};
    cuuint64_t gstr[2] = {(cuuint64_t)rstride * 4, (cuuint64_t)wstride * 4};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return get_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), gdim, gstr, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace cerar
