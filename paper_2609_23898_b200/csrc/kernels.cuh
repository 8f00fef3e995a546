// Device kernels of the CERAR data path and their launch descriptors (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace cerar {

// Checked build (-DCERAR_BOUNDS_CHECK, libcerar_checked.so): every address that the kernels of the in-HBM
// pipeline form for a plain load, a plain store or a 1-D bulk copy is compared with the extent of
// the buffer it belongs to.  An address outside is recorded in the plan's status word (STATUS_BOUNDS;
// the first offender wins) and the access is skipped, so nothing faults; cerar_device_status then
// reports CERAR_ERR_BOUNDS.  The release build compiles the checks away.  Tensor-map (TMA) copies need no
// check of this kind: the hardware clips them at the extents in the map, which are the buffer's own.
constexpr int STATUS_BOUNDS = 16;
struct Range {            // [lo, hi) in floats
    const float* lo;
    const float* hi;
};
#ifdef CERAR_BOUNDS_CHECK
__device__ __forceinline__ bool range_ok(const void* p, size_t bytes, Range r, int* status) {
    const char* b = static_cast<const char*>(p);
    if (b >= reinterpret_cast<const char*>(r.lo) && b + bytes <= reinterpret_cast<const char*>(r.hi)) return true;
    atomicCAS(status, 0, STATUS_BOUNDS);
    return false;
}
#define CERAR_RANGE_OK(p, bytes, r, status) ::cerar::range_ok((p), (bytes), (r), (status))
#else
#define CERAR_RANGE_OK(p, bytes, r, status) true
#endif

// A skinny contraction out[j][q] = scale * sum_k coef[k][j] * in[row(k)][q] over
// positions q in [0, p), for N workers.  Encoding (Delta_i = G_i U_i) and
// decoding (G_hat_i = Y_i R_i) are both of this form.
struct ContractArgs {
    const float* in;        // worker 0, row 0
    int64_t in_wstride;     // floats between workers
    int64_t in_rstride;     // floats between rows
    float* out;
    int64_t out_wstride;
    int64_t out_rstride;
    const float* coef;      // device: worker i's K x J row-major matrix at coef + i*K*J
    int K, J;
    int skip_row;           // input row index r >= skip_row reads physical row r + skip_count
    int skip_count;         // physical rows skip_row .. skip_row+skip_count-1 are not inputs (0 = none)
    int N;
    int64_t p;
    float scale;
    int* status;            // device word; set non-zero when a bounded wait gives up
    // staged kernel only
    int KC, stages, slabs, jgroups, tile_p;
    int tiles_per_worker;
    int64_t total_tiles;
    Range in_range, out_range;   // extents of the two buffers (filled in by the launcher; read by the checked build)
};

struct RoundArgs {
    float* ws;              // workspace, worker i at ws + i*(c+N)*p
    int64_t p;
    int N, c, k;            // round k in 1..L
    int reverse;            // round_kernel: 1 = blocks walk the positions downwards (set by the launcher)
    int hints;              // rounds_coop_kernel: 1 = L2 residency hints on the delta rows (set by the launcher)
    int* status;            // device word of the plan
    Range range;            // extent of the workspace (filled in by the launcher; read by the checked build)
};

// One worker's ring round in the one-worker-per-GPU layout ((c+N+1) x p per worker).
struct RankRoundArgs {
    const float* ws;        // this worker's workspace
    float* peer_ws;         // the next worker's workspace (may be peer-mapped memory of another GPU)
    int64_t p;
    int N, c, k;            // round k in 1..L
    int slot_prev, slot_cancel, slot_add, slot_land;   // filled in by the launcher (-1 = term absent)
    int to_message;         // 1: peer_ws is a plain p-float message buffer (row 0), not a workspace;
                            // 2: a buffer of p bfloat16 values (the message rounded to nearest-even)
};

// All L rounds of up to RING_MAX_WORKERS workers in one launch (blockIdx.y = index into the arrays).
constexpr int RING_MAX_WORKERS = 32;
struct RingFusedArgs {
    const float* ws[RING_MAX_WORKERS];            // the worker's own workspace ((c+N+1) x p)
    float* peer_ws[RING_MAX_WORKERS];             // the next worker's workspace (may be peer memory)
    const unsigned* landed_local[RING_MAX_WORKERS];   // per tile: last message that has landed here
    const unsigned* freed_local[RING_MAX_WORKERS];    // per tile: last round the next worker has finished
    unsigned* landed_next[RING_MAX_WORKERS];      // the next worker's landed counters (written here)
    unsigned* freed_prev[RING_MAX_WORKERS];       // the previous worker's freed counters (written here)
    int N, c;
    int64_t p;
    int64_t tile, ntiles;                          // positions per tile (a multiple of 4), tiles per worker
    unsigned base;                                 // counters of this aggregation are base + k
    int vec;                                       // 1: p % 4 == 0 and 16-byte aligned workspaces
    int* status;
    unsigned long long limit_ns;
};

enum { KERNEL_AUTO = 0, KERNEL_REF = 1, KERNEL_STAGED = 2, KERNEL_TC = 3 };

// Returns cudaSuccess or the launch error.  *launches is incremented by the
// number of kernels launched.
cudaError_t launch_contract(ContractArgs a, int mode, int num_sms, cudaStream_t s, uint64_t* launches);
// Tensor-core (tcgen05, 3 x TF32) contraction; tc_eligible says whether the shape fits it.
bool tc_eligible(const ContractArgs& a);
cudaError_t launch_contract_tc(ContractArgs a, int num_sms, cudaStream_t s, uint64_t* launches);
// Tuning knobs (0 = default), settable through cerar_set_tuning.
extern int g_tune_kc, g_tune_stages, g_tune_jt, g_tune_slabs, g_tune_tc_kc, g_tune_tc_stages, g_tune_tc_variant,
           g_tune_ring_wait_ms, g_tune_ring_tile, g_tune_pdl_off, g_tune_serpentine_off, g_tune_tc_min_c, g_tune_tc_epi, g_tune_tc_unaligned_off, g_tune_tc_split, g_tune_staged_unaligned_off, g_tune_round_split, g_tune_checked_shrink,
           g_tune_rounds_one_launch_off, g_tune_rounds_one_launch_mb, g_tune_rounds_multi_form, g_tune_rounds_coop_shape, g_tune_rounds_hints;
cudaError_t launch_round(const RoundArgs& a, cudaStream_t s, uint64_t* launches);
// Rounds a.k .. k_last in one launch (for states that are cache-resident anyway).
cudaError_t launch_rounds_multi(const RoundArgs& a, int k_last, cudaStream_t s, uint64_t* launches);
// Slots of the per-worker layout that round k reads (-1 = term absent) and the landing slot
// in the neighbour's workspace; the one definition that launcher and callers share.
void rank_round_slots(int N, int c, int k, int* slot_prev, int* slot_cancel, int* slot_add, int* slot_land);
cudaError_t launch_rank_round(RankRoundArgs a, int num_sms, cudaStream_t s, uint64_t* launches);
cudaError_t launch_rank_recv_bf16(float* slot, const unsigned short* msg, int64_t p, int num_sms, cudaStream_t s,
                                  uint64_t* launches);
// 8-bit messages (e4m3 codes + one power-of-two scale per CERAR_FP8_TILE positions); msg is 16-byte aligned
size_t fp8_message_bytes(int64_t p);
cudaError_t launch_rank_round_fp8(RankRoundArgs a, void* msg, int num_sms, cudaStream_t s, uint64_t* launches);
cudaError_t launch_rank_recv_fp8(float* slot, const void* msg, int64_t p, int num_sms, cudaStream_t s, uint64_t* launches);
// cooperative = true when the launch serves workers that wait on one another (all on this GPU).
cudaError_t launch_ring_rounds(const RingFusedArgs& a, int nworkers, bool cooperative, int num_sms, cudaStream_t s,
                               uint64_t* launches);
// A kernel whose bounded wait is made to run out (nothing arrives on its barrier).
cudaError_t launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, cudaStream_t s);
// Whole protocol in one launch with the slots in shared memory (small N (c+N) only).
bool fused_supported(int N, int c);
cudaError_t launch_fused(const float* grads, int64_t grads_stride, float* out, int64_t out_stride, const float* U,
                         const float* R, int N, int c, int64_t p, float scale, int num_sms, cudaStream_t s,
                         uint64_t* launches);

// Launch with programmatic stream serialization (programmatic dependent launch): the kernel may be
// scheduled while the previous kernel of the stream is still draining, so it must execute
// ptx::grid_dependency_wait() before its first access to global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_tune_pdl_off ? 0 : 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace cerar
