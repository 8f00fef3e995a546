// Tensor-core contraction for encode / decode at large c (sm_100a: TMA + tcgen05 + TMEM).
//
//   out[j][q] = scale * sum_k coef[k][j] * in[k][q],   j < J (= c),  k < K rows,  q < p
//
// is a skinny GEMM with M = positions, N = J, K = input rows.  From c ~ 24 on the FP32 FMA pipe
// cannot keep up with HBM (c/4 flop per byte), so the products run on the 5th-generation
// tensor cores as 3 x TF32: every fp32 value is split into hi = tf32(x), lo = tf32(x - hi) and
//   x*y ~ lo_x*hi_y + hi_x*lo_y + hi_x*hi_y           (relative error ~ 2^-22),
// accumulated in fp32 in tensor memory.
//
// A tile is HALVES UMMA tiles of M = 128 positions ("halves").  HALVES = 2 (c <= 64): global
// memory is read and written in rows of 1 KB, which HBM serves measurably better than 512 B;
// half h belongs to the MMA issuers of half h for the whole run.  HALVES = 1 (c <= 128): the
// four accumulators of two halves would not leave room for the A operand in the 512 TMEM
// columns, and two coefficient copies of c = 128 leave shared memory for 128-position stages
// only.
//
// One CTA of 21 warps per SM.  The tiles of all workers form one list that is cut into one
// contiguous range per CTA, so every SM is busy whatever N is; a range that crosses a worker
// boundary is processed in two segments (the coefficients are per worker).
//   warp 0        producer: one TMA load per chunk ([KC rows] x [tile positions])
//   warps 11-18   splitter: thread = position; the two warps of a lane quadrant take one half of
//                 the chunk's rows each, for every half of the tile (or, with two halves and two
//                 or more chunks per tile, all rows of one half each); values are split into
//                 tf32 hi | lo and written to tensor memory (tcgen05.st), where they are
//                 the A operand of their half: shared memory is read once per element
//   warps 1, 2    MMA issuers (one lane each) for half 0 / 1, even tiles; warps 19, 20 the
//                 same for the odd tiles (an issuing thread is limited by its own instruction
//                 stream, not by the tensor pipe; at c = 32 warps 1, 2 take all tiles):
//                 tcgen05.mma kind::tf32, A from TMEM, B = the coefficients (hi and lo
//                 copies) in shared memory, M=128, N=Npad, K=8; two accumulators per half,
//                 so that the epilogue of one tile overlaps the products of the next;
//                 warp 1 owns the TMEM allocation
//   warps 3-10    epilogue: tcgen05.ld, scale, transpose through a shared-memory tile, one TMA
//                 store per 32 output rows.  One group of four warps per tile parity, each with
//                 a tile of its own and a hardware barrier inside the group (no polling between
//                 the warps); one group for all tiles at 128 output columns; or, on request,
//                 all eight warps on every tile (16 of every 32 rows per warp, two tiles handed
//                 round with mbarriers)
// Rows that do not start on 16-byte boundaries run the same kernel with UNAL = true: per-row bulk
// copies instead of tensor-map copies (see the kernel).
// Every wait is bounded; a wait that runs out sets the status word and the CTA leaves
// through the common exit, where tensor memory is freed.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <type_traits>

#include "kernels.cuh"
#include "tc_common.cuh"

namespace cerar {
namespace {

using namespace tc;

constexpr int HALF_M = 128;              // UMMA M
constexpr int OUT_ROWS = 32;             // output rows per TMA store
constexpr int NUM_WARPS = 21;
constexpr int NUM_THREADS = 32 * NUM_WARPS;
constexpr int WARP_EPI0 = 3, WARP_SPLIT0 = 11, WARP_MMA2 = 19;

struct PairParams {
    int K_rows;        // physical input rows that carry data; rows beyond read as zero (TMA fill)
    int K_pad;         // K_rows rounded up to a multiple of KC
    int stages;        // shared-memory stages of raw chunks
    int NAh;           // A (hi|lo) chunk buffers per half in tensor memory
    int Npad;          // J rounded up to 32
    int tmem_cols;     // power of two >= HALVES * (2*Npad + NAh*2*KC)
    int four_issuers;  // 1: every half has one issuer per accumulator (even / odd tiles)
    int epi_groups;      // group epilogue: 2 = one group per tile parity, 1 = one group for all tiles (one output tile less)
    int split_by_half; // two halves per tile: 1 = each splitter warp takes all rows of ONE half (one hand-off per chunk), 0 = half of the rows of both
    int group_epilogue;  // 1: each group of four epilogue warps works on tiles of its own (hardware barriers inside the group)
    int64_t tiles_per_worker;
    int64_t total_tiles;
};

// shared memory (1024-aligned): B_hi | B_lo | raw stages | 2 output tiles | barriers | tmem slot
template <int KC, int HALVES, bool UNAL>
__global__ void __launch_bounds__(NUM_THREADS, 1)
contract_tc_kernel(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_out,
                   const __grid_constant__ ContractArgs a, const __grid_constant__ PairParams tp) {
    constexpr int TILE_W = HALVES * HALF_M;      // positions per tile
    // UNAL: rows that do not start on 16-byte boundaries (p not a multiple of 4, or an unaligned buffer).
    // Tensor-map copies cannot address them, so every row of a chunk comes in with a 1-D bulk copy of its
    // own that starts at the 16-byte boundary below the row's first element; the row sits in shared memory
    // with the same offset (0..3 floats) it has in global memory, which the splitter adds when it reads.
    // Output rows are laid out with THEIR offsets, so that the 16-byte aligned middle of a row leaves with
    // one bulk store and the up to three elements on either side with plain stores.
    constexpr int PITCH = TILE_W + (UNAL ? 4 : 0);   // floats between rows of a stage and of an output tile
    extern __shared__ unsigned char smem_dyn[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = tp.stages, Npad = tp.Npad, K_pad = tp.K_pad;
    const uint32_t NAh = (uint32_t)tp.NAh;
    const int nkc = K_pad / KC;
    const int nblk = Npad / 32;
    static_assert(KC % 8 == 0, "a chunk is a whole number of k-steps");
    constexpr int KG = KC / 2;           // rows of a chunk per splitter warp of a quadrant (a multiple of 4)

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* smem_al = smem_dyn + (smem_base - smem_u32(smem_dyn));
    const uint32_t b_bytes = (uint32_t)K_pad * Npad * 4u;            // one of B_hi / B_lo
    constexpr uint32_t chunk_bytes = (uint32_t)KC * PITCH * 4u;
    constexpr uint32_t out_bytes = (uint32_t)OUT_ROWS * PITCH * 4u;
    const uint32_t bhi_u32 = smem_base, blo_u32 = smem_base + b_bytes;
    const uint32_t raw_u32 = smem_base + 2u * b_bytes;
    const uint32_t out_u32 = raw_u32 + (uint32_t)stages * chunk_bytes;
    const uint32_t bar_u32 = out_u32 + (uint32_t)tp.epi_groups * out_bytes;
    const uint32_t raw_full = bar_u32, raw_empty = raw_full + 8u * stages;
    // "A buffer filled": one barrier per (half, tile parity, buffer), so that each has ONE waiter
    // (the issuer of that half and parity) who sees all of its phases in order; a barrier that two
    // issuers took turns on could be two phases ahead of one of them, which a parity wait cannot tell
    const uint32_t a_full = raw_empty + 8u * stages;                 // [half][parity][NAh]
    const uint32_t a_empty = a_full + 16u * HALVES * NAh;            // [half][NAh]
    const uint32_t acc_full = a_empty + 8u * HALVES * NAh;           // [half][2]
    const uint32_t acc_empty = acc_full + 32u;
    const uint32_t out_full = acc_empty + 32u, out_free = out_full + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_al + (out_free + 16u - smem_base));
    const float* raw_s = reinterpret_cast<const float*>(smem_al + (raw_u32 - smem_base));
    float* out_s = reinterpret_cast<float*>(smem_al + (out_u32 - smem_base));

    // ---------------- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(raw_full + 8u * s, 1); mbar_init(raw_empty + 8u * s, 8); }
        for (uint32_t b = 0; b < 2u * HALVES * NAh; ++b) mbar_init(a_full + 8u * b, (HALVES == 2 && tp.split_by_half) ? 4 : 8);
        for (uint32_t b = 0; b < HALVES * NAh; ++b) mbar_init(a_empty + 8u * b, 1);
        for (int b = 0; b < 2 * HALVES; ++b) { mbar_init(acc_full + 8u * b, 1); mbar_init(acc_empty + 8u * b, tp.group_epilogue ? 4 : 8); }
        for (int b = 0; b < 2; ++b) { mbar_init(out_full + 8u * b, 8); mbar_init(out_free + 8u * b, 1); }
        mbar_init_fence();
    }
    if (warp == 1) tc_alloc(smem_u32(tmem_slot), (uint32_t)tp.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t a_col0 = 2u * HALVES * (uint32_t)Npad;   // A buffers start after the accumulators (two per half)

    // this CTA's contiguous range of the tile list (worker-major), cut at worker boundaries
    const int64_t T = tp.tiles_per_worker;
    const int64_t g_begin = tp.total_tiles * blockIdx.x / gridDim.x;
    const int64_t g_end = tp.total_tiles * (blockIdx.x + 1) / gridDim.x;
    const int w_first = (int)(g_begin / T);
    const int w_last = g_end > g_begin ? (int)((g_end - 1) / T) : w_first - 1;

    bool failed = false;
    uint32_t it = 0, tc = 0, oc = 0;      // chunks, tiles and output blocks this CTA has gone through (all roles count alike)
    uint32_t afull_ph = 0;                // issuers: next phase parity of their "filled" barriers, bit = 4 * parity + buffer

    for (int w = w_first; w <= w_last; ++w) {
        const int64_t t_begin = (w == w_first) ? g_begin - (int64_t)w * T : 0;
        const int64_t t_end = (w == w_last) ? g_end - (int64_t)w * T : T;
        {
            // coefficients of this worker as the tensor core's B operand (tf32 hi and lo copies)
            split_coefficients(a, w, K_pad, Npad, reinterpret_cast<uint32_t*>(smem_al),
                               reinterpret_cast<uint32_t*>(smem_al + b_bytes));
            fence_proxy_async_smem();
        }
        __syncthreads();
        // up to here only the plan's constant coefficients were read: that may overlap the tail of the
        // kernel before this one in the stream; the data may not be touched before that kernel is done
        if (w == w_first) grid_dependency_wait();

        if (failed) {
            // a wait of this warp ran out in an earlier segment: only keep the CTA barriers company
        } else if (warp == 0) {
            // ================= producer
            if constexpr (UNAL) {
                // one bulk copy per row, issued by the lanes in parallel; lane 0 announces their total first
                const uintptr_t in_w = reinterpret_cast<uintptr_t>(a.in + (int64_t)w * a.in_wstride);
                for (int64_t t = t_begin; t < t_end && !failed; ++t) {
                    const int64_t q0 = t * TILE_W;
                    const uint32_t valid = (uint32_t)(a.p - q0 < TILE_W ? a.p - q0 : TILE_W);
                    for (int kc = 0; kc < nkc; ++kc, ++it) {
                        const uint32_t s = it % stages, ph = (it / stages) & 1u;
                        if (!warp_wait(raw_empty + 8u * s, ph ^ 1u)) { failed = true; break; }
                        uint32_t bytes[(KC + 31) / 32];
                        uintptr_t src[(KC + 31) / 32];
                        uint32_t total = 0;
#pragma unroll
                        for (int rr = 0; rr < (KC + 31) / 32; ++rr) {
                            const int r = rr * 32 + lane, row = kc * KC + r;
                            bytes[rr] = 0;
                            if (r < KC && row < tp.K_rows) {
                                const uintptr_t first = in_w + ((uintptr_t)row * (uintptr_t)a.in_rstride + (uintptr_t)q0) * 4u;
                                src[rr] = first & ~(uintptr_t)15;
                                bytes[rr] = (uint32_t)((first - src[rr]) + valid * 4u + 15u) & ~15u;
                                if (!CERAR_RANGE_OK(reinterpret_cast<const void*>(first), valid * 4u, a.in_range, a.status)) bytes[rr] = 0;
                            }
                            total += bytes[rr];
                        }
                        total = __reduce_add_sync(0xffffffffu, total);
                        if (lane == 0) mbar_arrive_expect_tx(raw_full + 8u * s, total);
                        __syncwarp();
#pragma unroll
                        for (int rr = 0; rr < (KC + 31) / 32; ++rr)
                            if (bytes[rr])
                                bulk_load(raw_u32 + s * chunk_bytes + (uint32_t)(rr * 32 + lane) * (PITCH * 4u),
                                          reinterpret_cast<const void*>(src[rr]), bytes[rr], raw_full + 8u * s);
                    }
                }
            } else if (lane == 0) {
                for (int64_t t = t_begin; t < t_end && !failed; ++t) {
                    const int q0 = (int)(t * TILE_W);
                    for (int kc = 0; kc < nkc; ++kc, ++it) {
                        const uint32_t s = it % stages, ph = (it / stages) & 1u;
                        if (!mbar_wait_bounded(raw_empty + 8u * s, ph ^ 1u)) { failed = true; break; }
                        mbar_arrive_expect_tx(raw_full + 8u * s, chunk_bytes);
                        tma_load_3d(raw_u32 + s * chunk_bytes, &tmap_in, q0, kc * KC, w, raw_full + 8u * s);
                    }
                }
            }
        } else if (warp == 1 || warp == 2 || warp >= WARP_MMA2) {
            // ================= MMA issuer of half m: accumulators 2m, 2m+1 alternate by tile.
            // With four issuers, warps 1, 2 take the even tiles and warps 19, 20 the odd ones
            // (an issuing thread is limited by its own instruction stream, not by the tensor pipe).
            const bool odd_only = warp >= WARP_MMA2;
            const uint32_t m = (uint32_t)(odd_only ? warp - WARP_MMA2 : warp - 1);
            if (lane == 0 && m < (uint32_t)HALVES && (tp.four_issuers || !odd_only)) {
                const uint32_t idesc = idesc_tf32_ts((uint32_t)Npad);
                const uint32_t b_lbo = (uint32_t)K_pad * 128u;
                const uint64_t bhi0 = make_desc(bhi_u32, b_lbo, 512u), blo0 = make_desc(blo_u32, b_lbo, 512u);
                for (int64_t t = t_begin; t < t_end && !failed; ++t, ++tc) {
                    const uint32_t buf = tc & 1u, aph = (tc >> 1) & 1u;
                    if (tp.four_issuers && (buf != 0u) != odd_only) continue;
                    const uint32_t d_tmem = tmem_base + (2u * m + buf) * (uint32_t)Npad;
                    if (!mbar_wait_bounded(acc_empty + 8u * (2u * m + buf), aph ^ 1u)) { failed = true; break; }
                    tc_fence_after();
                    for (int kc = 0; kc < nkc; ++kc) {
                        const uint32_t seq = tc * (uint32_t)nkc + (uint32_t)kc;
                        const uint32_t b = seq % NAh, ab = m * NAh + b;
                        const uint32_t bit = 4u * buf + b, ph = (afull_ph >> bit) & 1u;
                        if (!mbar_wait_bounded(a_full + 8u * ((2u * m + buf) * NAh + b), ph)) { failed = true; break; }
                        afull_ph ^= 1u << bit;
                        tc_fence_after();
                        const uint32_t a_hi = tmem_base + a_col0 + ab * (2u * KC), a_lo = a_hi + KC;
                        const int rows_left = tp.K_rows - kc * KC;               // rows with data in this chunk
                        // descriptor start address: 8 rows x 128 B = 64 units of 16 bytes per k-step
                        const uint64_t bh = bhi0 + (uint64_t)(kc * KC * 8), bl = blo0 + (uint64_t)(kc * KC * 8);
                        if (rows_left >= KC) {
#pragma unroll
                            for (int ks = 0; ks < KC / 8; ++ks)
                                tc_mma_tf32_ts_x3(d_tmem, a_hi + ks * 8u, a_lo + ks * 8u, bh + (uint64_t)(ks * 64),
                                                  bl + (uint64_t)(ks * 64), idesc, ks ? 1u : (uint32_t)(kc != 0));
                        } else {
                            const int ksteps = (rows_left + 7) / 8;
                            for (int ks = 0; ks < ksteps; ++ks)
                                tc_mma_tf32_ts_x3(d_tmem, a_hi + ks * 8u, a_lo + ks * 8u, bh + (uint64_t)(ks * 64),
                                                  bl + (uint64_t)(ks * 64), idesc, (uint32_t)((kc | ks) != 0));
                        }
                        tc_commit(a_empty + 8u * ab);      // the A buffer is free once these MMAs have read it
                    }
                    if (failed) break;
                    tc_commit(acc_full + 8u * (2u * m + buf));          // the accumulator is complete
                }
            }
        } else if (warp < WARP_SPLIT0) {
            // ================= epilogue (TMEM lanes 32*(warp%4) ..; group g takes rows 16g..16g+15 of every 32)
            const int qd = warp & 3, g = (warp - WARP_EPI0) >> 2;
            const int pos = qd * 32 + lane;
            if (tp.group_epilogue) {
                // Group g (four warps, one per TMEM lane quadrant) owns the tiles of parity g, i.e. accumulator
                // buffer g of every half, and an output tile of its own: the two groups never wait for one
                // another, and inside a group a hardware barrier orders "tile filled" -> TMA store -> "store has
                // read the tile" (no polling).  The next accumulator block is fetched from tensor memory before
                // the group waits for its previous store.
                const bool elected = ((warp - WARP_EPI0) & 3) == 0 && lane == 0;
                auto run = [&](auto rows_c) {
                    constexpr int R = decltype(rows_c)::value;          // output rows per block and store
                    float* o = out_s + (size_t)g * (R * PITCH) + pos;
                    const int nb_e = Npad / R;
                    bool pending = false, stop = false;
                    for (int64_t t = t_begin; t < t_end && !stop; ++t, ++tc) {
                        const uint32_t buf = tc & 1u;
                        if (tp.epi_groups == 2 ? buf != (uint32_t)g : g != 0) continue;
                        const uint32_t aph = (tc >> 1) & 1u;
                        for (int nb = 0; nb < nb_e && !stop; ++nb) {
#pragma unroll
                            for (int h = 0; h < HALVES; ++h) {
                                const uint32_t acc = 2u * h + buf;
                                if (nb == 0 && !failed && !warp_wait(acc_full + 8u * acc, aph)) failed = true;
                                tc_fence_after();
                                float v[R];
                                if (!failed) {
                                    const uint32_t ta = tmem_base + ((uint32_t)(qd * 32) << 16) + acc * (uint32_t)Npad + (uint32_t)(nb * R);
                                    if constexpr (R == 32) tc_ld32(ta, v); else tc_ld16(ta, v);
                                } else {
#pragma unroll
                                    for (int j = 0; j < R; ++j) v[j] = 0.f;
                                }
                                if (nb == nb_e - 1) {
                                    tc_fence_before();
                                    __syncwarp();
                                    if (lane == 0) mbar_arrive(acc_empty + 8u * acc);
                                }
                                if (h == 0) {
                                    if ((UNAL ? ((warp - WARP_EPI0) & 3) == 0 : elected) && pending) bulk_wait_read_0();   // the group's tile is free again
                                    if (bar_red_or(1u + (uint32_t)g, 128u, failed)) { failed = true; stop = true; break; }
                                }
                                if constexpr (UNAL) {
                                    const uint32_t o0 = (uint32_t)((reinterpret_cast<uintptr_t>(a.out + (int64_t)w * a.out_wstride) >> 2) +
                                                                   (uint64_t)(t * TILE_W) + (uint64_t)(nb * R) * (uint64_t)a.out_rstride);
                                    const uint32_t os = (uint32_t)(a.out_rstride & 3);
#pragma unroll
                                    for (int j = 0; j < R; ++j) o[j * PITCH + h * HALF_M + (int)((o0 + (uint32_t)j * os) & 3u)] = v[j] * a.scale;
                                } else {
#pragma unroll
                                    for (int j = 0; j < R; ++j) o[j * PITCH + h * HALF_M] = v[j] * a.scale;
                                }
                            }
                            if (stop) break;
                            fence_proxy_async_smem();
                            bar_sync(1u + (uint32_t)g, 128u);
                            if constexpr (UNAL) {
                                // lane j of the group's first warp stores row j: the aligned middle with a bulk copy, the rest plainly
                                if (((warp - WARP_EPI0) & 3) == 0) {
                                    const int j = nb * R + lane;
                                    const int64_t q0 = t * TILE_W;
                                    const int valid = (int)(a.p - q0 < TILE_W ? a.p - q0 : TILE_W);
                                    if (lane < R && j < a.J) {
                                        float* dst = a.out + (int64_t)w * a.out_wstride + (int64_t)j * a.out_rstride + q0;
                                        const int sh = (int)((reinterpret_cast<uintptr_t>(dst) >> 2) & 3u);
                                        const float* srow = out_s + (size_t)g * (R * PITCH) + (size_t)lane * PITCH + sh;   // element 0 of the row
                                        int head = (4 - sh) & 3;
                                        if (head > valid) head = valid;
                                        const int body = (valid - head) & ~3;
                                        if (CERAR_RANGE_OK(dst, (size_t)valid * 4u, a.out_range, a.status)) {
                                            if (body > 0)
                                                bulk_store(dst + head, smem_u32(srow + head), (uint32_t)body * 4u);
                                            for (int e = 0; e < head; ++e) dst[e] = srow[e];
                                            for (int e = head + body; e < valid; ++e) dst[e] = srow[e];
                                        }
                                    }
                                    bulk_commit();
                                    pending = true;
                                }
                            } else if (elected) {
                                tma_store_3d(&tmap_out, (int)(t * TILE_W), nb * R, w, out_u32 + (uint32_t)g * (uint32_t)(R * PITCH * 4));
                                bulk_commit();
                                pending = true;
                            }
                        }
                    }
                };
                run(std::integral_constant<int, OUT_ROWS>{});
            } else
            for (int64_t t = t_begin; t < t_end && !failed; ++t, ++tc) {
                const uint32_t buf = tc & 1u, aph = (tc >> 1) & 1u;
                for (int nb = 0; nb < nblk && !failed; ++nb, ++oc) {
                    const uint32_t ob = oc & 1u, oph = (oc >> 1) & 1u;
                    if (!warp_wait(out_free + 8u * ob, oph ^ 1u)) { failed = true; break; }
                    float* o = out_s + (size_t)ob * (OUT_ROWS * TILE_W) + (size_t)(g * 16) * TILE_W + pos;
#pragma unroll
                    for (int h = 0; h < HALVES; ++h) {
                        const uint32_t acc = 2u * h + buf;
                        if (nb == 0 && !warp_wait(acc_full + 8u * acc, aph)) { failed = true; break; }
                        tc_fence_after();
                        float v[16];
                        tc_ld16(tmem_base + ((uint32_t)(qd * 32) << 16) + acc * (uint32_t)Npad + (uint32_t)(nb * 32 + g * 16), v);
                        if (nb == nblk - 1) {
                            // this warp's part of the accumulator is in registers: hand it back
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(acc_empty + 8u * acc);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) o[j * TILE_W + h * HALF_M] = v[j] * a.scale;
                    }
                    if (failed) break;
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(out_full + 8u * ob);
                    if (warp == WARP_EPI0) {
                        if (lane == 0) {
                            if (!mbar_wait_bounded(out_full + 8u * ob, oph)) {
                                failed = true;
                            } else {
                                // rows beyond J and positions beyond p are clipped by the tensor map
                                tma_store_3d(&tmap_out, (int)(t * TILE_W), nb * OUT_ROWS, w, out_u32 + ob * out_bytes);
                                bulk_commit();
                                if (oc >= 1) {                 // the store before this one has read its tile: free it
                                    bulk_wait_read_1();
                                    mbar_arrive(out_free + 8u * (ob ^ 1u));
                                }
                            }
                        }
                        failed = __any_sync(0xffffffffu, failed ? 1 : 0) != 0;
                    }
                }
            }
        } else {
            // ================= splitter (TMEM lanes 32*(warp%4) ..; group g takes rows [g*KG, (g+1)*KG) of the chunk)
            const int qd = warp & 3, g = (warp - WARP_SPLIT0) >> 2;
            const int pos = qd * 32 + lane;
            const int r0 = g * KG;
            if (HALVES == 2 && tp.split_by_half) {
                // warp group g writes half g: all rows of the chunk in two batches of KG, one wait for the A buffer
                // and one hand-off to the issuer per chunk (every warp still meets every chunk, so no barrier is
                // ever a phase ahead of a waiter)
                const int h = g;
                for (int64_t t = t_begin; t < t_end && !failed; ++t, ++tc) {
                    for (int kc = 0; kc < nkc && !failed; ++kc, ++it) {
                        const uint32_t s = it % stages, ph = (it / stages) & 1u;
                        const uint32_t seq = tc * (uint32_t)nkc + (uint32_t)kc;
                        const uint32_t abi = seq % NAh, pa = (seq / NAh) & 1u;
                        if (!warp_wait(raw_full + 8u * s, ph)) { failed = true; break; }
                        const float* colh = raw_s + (size_t)s * (KC * PITCH) + pos + h * HALF_M;
                        const int rows_left = tp.K_rows - kc * KC;
                        const int kround = ((rows_left < KC ? rows_left : KC) + 7) / 8 * 8;
                        const uint32_t ab = (uint32_t)h * NAh + abi;
#pragma unroll
                        for (int b = 0; b < 2; ++b) {
                            const int rb = b * KG;
                            const int kuse = kround - rb;
                            uint32_t sh0 = 0, shs = 0;
                            if constexpr (UNAL) {
                                shs = (uint32_t)(a.in_rstride & 3);
                                sh0 = (uint32_t)((reinterpret_cast<uintptr_t>(a.in + (int64_t)w * a.in_wstride) >> 2) + (uint64_t)(t * TILE_W) +
                                                 (uint64_t)(kc * KC + rb) * (uint64_t)a.in_rstride);
                            }
                            uint32_t hi[KG], lo[KG];
#pragma unroll
                            for (int k = 0; k < KG; ++k) {
                                hi[k] = lo[k] = 0u;
                                if ((k & ~3) < kuse && (!UNAL || rb + k < rows_left)) {
                                    const float x = colh[(rb + k) * PITCH + (UNAL ? (int)((sh0 + (uint32_t)k * shs) & 3u) : 0)];
                                    hi[k] = tf32_bits(x);
                                    lo[k] = tf32_bits(x - __uint_as_float(hi[k]));
                                }
                            }
                            if (b == 1) {
                                __syncwarp();
                                if (lane == 0) mbar_arrive(raw_empty + 8u * s);        // this warp has all it needs of the chunk
                            } else {
                                if (!warp_wait(a_empty + 8u * ab, pa ^ 1u)) { failed = true; break; }
                                tc_fence_after();
                            }
                            const uint32_t ta = tmem_base + ((uint32_t)(qd * 32) << 16) + a_col0 + ab * (2u * KC) + (uint32_t)rb;
                            if (kuse > 0) {
                                tc_st_cols<KG>(ta, hi);
                                tc_st_cols<KG>(ta + KC, lo);
                            }
                        }
                        if (failed) break;
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(a_full + 8u * ((2u * (uint32_t)h + (tc & 1u)) * NAh + abi));
                    }
                }
            } else
            for (int64_t t = t_begin; t < t_end && !failed; ++t, ++tc) {
                for (int kc = 0; kc < nkc && !failed; ++kc, ++it) {
                    const uint32_t s = it % stages, ph = (it / stages) & 1u;
                    const uint32_t seq = tc * (uint32_t)nkc + (uint32_t)kc;
                    const uint32_t abi = seq % NAh, pa = (seq / NAh) & 1u;
                    if (!warp_wait(raw_full + 8u * s, ph)) { failed = true; break; }
                    const float* col = raw_s + (size_t)s * (KC * PITCH) + (size_t)r0 * PITCH + pos;
                    // UNAL: offset (in floats, mod 4) of the first element of row r0 of this chunk, and its step per row
                    uint32_t sh0 = 0, shs = 0;
                    if constexpr (UNAL) {
                        shs = (uint32_t)(a.in_rstride & 3);
                        sh0 = (uint32_t)((reinterpret_cast<uintptr_t>(a.in + (int64_t)w * a.in_wstride) >> 2) + (uint64_t)(t * TILE_W) +
                                         (uint64_t)(kc * KC + r0) * (uint64_t)a.in_rstride);
                    }
                    // rows of this chunk that some product reads (the last chunk may be short): rounded up
                    // to the k-step, rows beyond the data are zero (TMA fill)
                    const int rows_left = tp.K_rows - kc * KC;
                    const int kuse = ((rows_left < KC ? rows_left : KC) + 7) / 8 * 8 - r0;   // relative to r0
#pragma unroll
                    for (int h = 0; h < HALVES; ++h) {
                        uint32_t hi[KG], lo[KG];
#pragma unroll
                        for (int k = 0; k < KG; ++k) {
                            hi[k] = lo[k] = 0u;
                            if ((k & ~3) < kuse && (!UNAL || r0 + k < rows_left)) {     // (a tensor-map load fills rows beyond the data with zeros)
                                const float x = col[k * PITCH + h * HALF_M + (UNAL ? (int)((sh0 + (uint32_t)k * shs) & 3u) : 0)];
                                hi[k] = tf32_bits(x);
                                lo[k] = tf32_bits(x - __uint_as_float(hi[k]));
                            }
                        }
                        if (h == HALVES - 1) {
                            __syncwarp();
                            if (lane == 0) mbar_arrive(raw_empty + 8u * s);        // the whole chunk is in registers
                        }
                        const uint32_t ab = (uint32_t)h * NAh + abi;
                        if (!warp_wait(a_empty + 8u * ab, pa ^ 1u)) { failed = true; break; }
                        tc_fence_after();
                        const uint32_t ta = tmem_base + ((uint32_t)(qd * 32) << 16) + a_col0 + ab * (2u * KC) + (uint32_t)r0;
                        if (kuse > 0) {                        // uniform over the warp; rows beyond the data are zeros
                            tc_st_cols<KG>(ta, hi);
                            tc_st_cols<KG>(ta + KC, lo);
                        }
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(a_full + 8u * ((2u * (uint32_t)h + (tc & 1u)) * NAh + abi));
                    }
                }
            }
        }
        // ---------------- end of segment: all products that read these coefficients are done
        // (the epilogue has waited for every accumulator) before the next worker's overwrite them
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    if ((warp == WARP_EPI0 || warp == WARP_EPI0 + 4) && (UNAL || lane == 0)) bulk_wait_all();   // all output has left shared memory and is written
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
        tc_dealloc(tmem_base, (uint32_t)tp.tmem_cols);
    }
}

template <int KC, int HALVES, bool UNAL>
cudaError_t launch_kc(const CUtensorMap& tin, const CUtensorMap& tout, const ContractArgs& a, const PairParams& tp,
                      size_t smem, int grid, cudaStream_t s) {
    auto kern = contract_tc_kernel<KC, HALVES, UNAL>;
    {   // per device and cheap: set on every launch rather than cached
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    return launch_pdl(kern, dim3((unsigned)grid), dim3(NUM_THREADS), smem, s, tin, tout, a, tp);
}

template <int HALVES, bool UNAL>
cudaError_t launch_halves(int KC, const CUtensorMap& tin, const CUtensorMap& tout, const ContractArgs& a,
                          const PairParams& tp, size_t smem, int grid, cudaStream_t s) {
    switch (KC) {
        case 40: return launch_kc<40, HALVES, UNAL>(tin, tout, a, tp, smem, grid, s);
        case 32: return launch_kc<32, HALVES, UNAL>(tin, tout, a, tp, smem, grid, s);
        case 24: return launch_kc<24, HALVES, UNAL>(tin, tout, a, tp, smem, grid, s);
        default: return launch_kc<16, HALVES, UNAL>(tin, tout, a, tp, smem, grid, s);
    }
}

// Rows per chunk (0 if nothing fits): as few chunks as possible, then as few padded rows as
// possible, with at least 3 stages in the shared memory that the coefficient copies and the
// output tiles leave and at least two A buffers per half in the tensor memory that the
// accumulators leave.
int choose_chunk(const ContractArgs& a, int halves, PairParams* tp, int out_tiles = 2, bool unal = false) {
    const int tile_w = halves * HALF_M + (unal ? 4 : 0);      // row pitch in shared memory
    tp->K_rows = a.K + a.skip_count;                        // decode: physical rows that are not part of Y
    tp->Npad = ((a.J + 31) / 32) * 32;
    const size_t budget = 227 * 1024 - 1024;
    const int cands[4] = {40, 32, 24, 16};
    int best_kc = 0, best_pad = 1 << 30, best_stages = 0, best_nk = 1 << 30;
    for (int ci = 0; ci < 4; ++ci) {
        const int kc = cands[ci];
        if (g_tune_tc_kc && kc != g_tune_tc_kc) continue;
        if (halves * (2 * tp->Npad + 2 * 2 * kc) > 512) continue;
        const int kpad = ((tp->K_rows + kc - 1) / kc) * kc;
        const size_t fixed_c = 1024 + 2 * (size_t)kpad * tp->Npad * 4 + out_tiles * (size_t)OUT_ROWS * tile_w * 4 + 512;
        const size_t stage_c = (size_t)kc * tile_w * 4;
        if (fixed_c + 3 * stage_c > budget) continue;
        int st = (int)((budget - fixed_c) / stage_c);
        if (st > 8) st = 8;
        if (g_tune_tc_stages && g_tune_tc_stages < st) st = g_tune_tc_stages;
        if (st < 2) continue;
        // fewest chunks first (every chunk costs a round of barrier hand-offs), then fewest padded rows
        const int nk = kpad / kc;
        if (nk < best_nk || (nk == best_nk && kpad < best_pad)) { best_nk = nk; best_pad = kpad; best_kc = kc; best_stages = st; }
        // The one measured exception: 64 input rows into 64 output columns on tiles of 256 positions (the encode at
        // c = 64) runs 8-9 % faster on three chunks of 24 rows than on two of 32 (inside the pipeline, N = 4, 8, 16;
        // the neighbouring shapes c = 56, 60 and the decode do not).
        if (!g_tune_tc_kc && halves == 2 && tp->K_rows == 64 && tp->Npad == 64 && kc == 24) {
            best_nk = 0; best_pad = kpad; best_kc = kc; best_stages = st;     // nothing after it in the list beats nk = 0
        }
    }
    tp->K_pad = best_pad;
    tp->stages = best_stages;
    return best_kc;
}

}  // namespace

int g_tune_tc_kc = 0, g_tune_tc_stages = 0, g_tune_tc_variant = 0, g_tune_tc_min_c = 0, g_tune_tc_epi = 0, g_tune_tc_unaligned_off = 0, g_tune_tc_split = 0;

// Rows that start on 16-byte boundaries everywhere: what tensor-map copies need.
static bool rows_aligned(const ContractArgs& a) {
    if (a.p % 4 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(a.in) & 15u) || (a.in_rstride % 4) || (a.in_wstride % 4)) return false;
    if ((reinterpret_cast<uintptr_t>(a.out) & 15u) || (a.out_rstride % 4) || (a.out_wstride % 4)) return false;
    return true;
}

bool tc_eligible(const ContractArgs& a) {
    // N = J padded to 32 (rows beyond J are clipped by the output map); measured against the FMA kernel
    // on B200: +40 % at c = 28, +5 % at c = 24, -15 % at c = 20.  Two coefficient copies must fit in smem.
    // Rows that are not 16-byte aligned run the same kernel with per-row bulk copies (no tensor maps); the
    // alternative there is the tiled plain-load kernel, so the tensor cores take over from a smaller c.
    const bool aligned = rows_aligned(a);
    // (measured at unaligned p against the tiled kernel: c = 32 2.4-2.7 -> 4.9-5.4 TB/s, c = 64 1.1 -> 4.7-5.5; up to
    // c = 16 the staged FMA kernel's realigning form is ahead: 5.6-5.9 against 3.7-3.9 TB/s at c = 16; at c = 20 the
    // tensor cores are: 4.2 against 3.6-3.9)
    const int min_c = g_tune_tc_min_c > 0 ? g_tune_tc_min_c : (aligned ? 24 : 17);
    if (a.J < min_c || a.J > 128) return false;
    if (a.p >= (int64_t)1 << 31) return false;
    if (!aligned && g_tune_tc_unaligned_off) return false;
    return get_encode_fn() != nullptr;
}

cudaError_t launch_contract_tc(ContractArgs a, int num_sms, cudaStream_t s, uint64_t* launches) {
    // tiles of 256 positions where four accumulators fit next to the A operand (c <= 64) and the
    // coefficient copies leave room for 256-position stages; tc_variant 1 forces tiles of 128
    PairParams tp;
    const bool unal = !rows_aligned(a);
    int halves = (a.J <= 64 && g_tune_tc_variant != 1) ? 2 : 1;
    int KC = choose_chunk(a, halves, &tp, 2, unal);
    if (!KC && halves == 2) { halves = 1; KC = choose_chunk(a, halves, &tp, 2, unal); }
    if (!KC) return cudaErrorInvalidConfiguration;
    const int tile_w = halves * HALF_M;
    const int pitch = tile_w + (unal ? 4 : 0);
    tp.NAh = (512 - 2 * halves * tp.Npad) / (halves * 2 * KC);
    if (tp.NAh > 4) tp.NAh = 4;
    // Issuers per half: one per accumulator (even / odd tiles).  An issuing thread needs 150-160 clk per product
    // inside this kernel (a lone thread in an empty SM: 54), so one thread per half holds a tile for 12 x 160 clk
    // of the ~2400 a tile of 256 positions may take.  Measured on B200 (medians of interleaved runs, group
    // epilogue): encode +7 % at c = 32, +16 % at c = 24, +34 % at c = 28; c = 48, 56: +4..+15 %; c = 40, 64: 0..+4 %.
    // (With the eight-warp epilogue of earlier versions a second issuer cost 10-15 % at 64 columns.)
    // The exception, measured inside the pipeline (whole steps: encode, rounds, decode, as bench.py runs them, at config
    // 3's full size) is c = 32: one issuer per half with the group epilogue, encode 6.15 against 5.85 TB/s, decode 5.95
    // against 5.90.  (Back to back, in loops of one kernel under the power cap, the same shape prefers the second
    // pair by 7 %: what counts is the kernel between the launches it runs between.)
    tp.four_issuers = a.J == 32 ? 0 : 1;
    if (g_tune_tc_variant == 2) tp.four_issuers = 0;
    if (g_tune_tc_variant == 3) tp.four_issuers = 1;
    // Epilogue form, measured on B200 (medians of interleaved runs, c = 24 .. 128, one issuer per accumulator): a
    // group of four warps per tile parity with hardware barriers is ahead of all eight warps on every tile by
    // 3-10 % for most shapes and never behind inside the pipeline, so it is the default; tc_epi = 2 selects the
    // eight-warp form.  Unaligned rows are stored row by row, which only the group form does.
    tp.group_epilogue = 1;
    if (g_tune_tc_epi) tp.group_epilogue = g_tune_tc_epi == 2 ? 0 : 1;
    if (unal) tp.group_epilogue = 1;
    // With 128 output columns the two coefficient copies leave 46-64 KB for the input stages: one group for
    // all tiles needs one output tile less, which buys one or two stages (measured: encode +3 %, decode +7 % at
    // c = 128, nothing at c = 112, -14 % for the encode at c = 80).  tc_epi 3 / 4 force one / two groups.
    tp.epi_groups = (tp.group_epilogue && halves == 1 && tp.Npad > 96) ? 1 : 2;
    if (tp.group_epilogue && g_tune_tc_epi >= 3) tp.epi_groups = g_tune_tc_epi == 3 ? 1 : 2;
    if (tp.epi_groups == 1) {                           // the stages chosen again with what that frees
        KC = choose_chunk(a, halves, &tp, 1, unal);
        tp.NAh = (512 - 2 * halves * tp.Npad) / (halves * 2 * KC);
        if (tp.NAh > 4) tp.NAh = 4;
    }
    // Two halves per tile: the two splitter warps of a lane quadrant either take half of a chunk's rows each, for
    // both halves, or all rows of one half each: then a warp waits for one A buffer and hands over once per chunk
    // instead of twice.  Measured on B200 where a tile has two or more chunks: c = 40, 48: +9 % (encode), +12 %
    // (decode); c = 56: +7 % / -1 %; c = 64: -1 % / +22 %; with one chunk per tile (c <= 32) it is neutral, +-2 %.
    // tc_split forces it off (2) or on (1).
    tp.split_by_half = (halves == 2 && tp.K_pad / KC >= 2) ? 1 : 0;
    if (g_tune_tc_split) tp.split_by_half = (halves == 2 && g_tune_tc_split == 1) ? 1 : 0;
    tp.tmem_cols = 32;
    while (tp.tmem_cols < halves * (2 * tp.Npad + tp.NAh * 2 * KC)) tp.tmem_cols *= 2;
    const size_t smem = 1024 + 2 * (size_t)tp.K_pad * tp.Npad * 4 + (size_t)tp.stages * KC * pitch * 4 +
                        (size_t)tp.epi_groups * OUT_ROWS * pitch * 4 + 512;

    CUtensorMap tin, tout;
    if (unal) {
        memset(&tin, 0, sizeof tin);      // no tensor maps: every row travels with a 1-D bulk copy of its own
        memset(&tout, 0, sizeof tout);
    } else {
        if (!make_map(&tin, a.in, a.p, tp.K_rows, a.N, a.in_rstride, a.in_wstride, tile_w, KC)) return cudaErrorInvalidValue;
        if (!make_map(&tout, a.out, a.p, a.J, a.N, a.out_rstride, a.out_wstride, tile_w, OUT_ROWS)) return cudaErrorInvalidValue;
    }

    tp.tiles_per_worker = (a.p + tile_w - 1) / tile_w;
    tp.total_tiles = tp.tiles_per_worker * a.N;
    int grid = num_sms;
    if ((int64_t)grid > tp.total_tiles) grid = (int)tp.total_tiles;
    cudaError_t e = unal ? (halves == 2 ? launch_halves<2, true>(KC, tin, tout, a, tp, smem, grid, s)
                                        : launch_halves<1, true>(KC, tin, tout, a, tp, smem, grid, s))
                         : (halves == 2 ? launch_halves<2, false>(KC, tin, tout, a, tp, smem, grid, s)
                                        : launch_halves<1, false>(KC, tin, tout, a, tp, smem, grid, s));
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace cerar
