// Tensor-core FP16 GEMM for sm_100a with CTA pairs and 256x512 output tiles (paper section 3.3:
// FP16 operands, FP32 accumulation, FP16 on the store; same fused epilogue as the other kernels).
//
// Same machinery as the 256x256 CTA-pair kernel (tcgen05.mma.cta_group::2, TMA-fed ring, bounded
// waits, no TMA multicast), but a cluster holds TWO 256x256 accumulators side by side - all 512
// columns of tensor memory - and feeds both from one stream of A: per 64-deep k-block a CTA loads
// its 128 rows of A once and its 128-column halves of two B blocks, 48 KB instead of 2 x 32 KB.
// That is a quarter fewer operand bytes from L2 to the SMs, and a wave of 74 such tiles touches
// fewer distinct panels per flop, so less comes from DRAM.  The price: with tensor memory full
// the epilogue of a tile is not overlapped with the next tile's main loop (it runs on two sets of
// four warps, one accumulator each).
//
// Measured on B200 (4096x12288x12288, 1000 W cap): DRAM traffic 1.06 GB per launch against 1.24 GB,
// L2->SM traffic 7.3 GB against 9.7 GB, tensor pipe 90 % of active cycles against 98 %.  With the
// stores of the epilogue coalesced through shared memory: burst rate level (1440 TFLOP/s),
// seconds-long rate 1225-1234 against 1212-1216 for K = 12288, 1160-1165 against 1200-1207 for
// K = 4096 (the exposed epilogue weighs more on short tiles); used for the long-K products of the
// training step it changes the step time by less than the run-to-run spread.  It is therefore
// never chosen automatically: MPT_GEMM_FORCE_PAIR512 selects it.
//
// Roles in each CTA (320 threads): warp 0 TMA producer, warp 1 MMA issuer (leader CTA only; both
// CTAs' warp 1 take part in the paired tensor-memory allocation), warps 2-9 epilogue.  Barriers:
//   full[s]   in the leader: 1 arrival (expect_tx for both CTAs' bytes) + the bytes of both CTAs' loads
//   empty[s]  in each CTA: tcgen05.commit multicast to both CTAs when the MMAs have read stage s
//   accf      in each CTA: tcgen05.commit multicast when a unit's accumulators are complete
//   acce      in the leader: 16 arrivals, one per epilogue warp of both CTAs
// Work units: every cluster first takes the same number of 256x512 tiles; the tiles left over for
// a last, partly filled round are cut into 256x256 units (one accumulator) so that the last round
// takes about half as long.  Every other unit of a cluster walks K downwards (see the 256x256
// kernel).  Every mbarrier wait is bounded (see tc_ptx.cuh).
#include <cuda.h>

#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

namespace pair512 {

static constexpr int CTA_M = 128;          // rows per CTA (256 per pair)
static constexpr int ACC_N = 256;          // columns per accumulator (one MMA instruction: N = 256)
static constexpr int TILE_N = 512;         // columns per tile (two accumulators)
static constexpr int CTA_N = 128;          // columns of each B block this CTA loads
static constexpr int BLOCK_K = 64, UMMA_K = 16;
static constexpr int STAGES = 4;
static constexpr int A_STAGE_BYTES = CTA_M * BLOCK_K * 2;   // 16 KB
static constexpr int B_STAGE_BYTES = CTA_N * BLOCK_K * 2;   // 16 KB per B block
static constexpr int STAGE_BYTES = A_STAGE_BYTES + 2 * B_STAGE_BYTES;
static constexpr int MN_BOX_BYTES = 64 * BLOCK_K * 2;
static constexpr int TMEM_COLS = 512;
static constexpr int NUM_THREADS = 320;
static constexpr int EPI_STAGE_BYTES = 32 * kEpiStagePitch;                 // per epilogue warp
static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256 + 8 * EPI_STAGE_BYTES;

// instruction descriptor: FP32 accumulate, operand majors, N = 256, M = 256
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn)
{
    return (1u << 4) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(ACC_N >> 3) << 17) |
           ((uint32_t)((2 * CTA_M) >> 4) << 24);
}

struct Params {
    int M, N, K;
    uint16_t *C;
    int ldc;
    const uint16_t *mask;
    int ldmask;
    int relu;
    uint32_t *nonfinite_flag;
    uint32_t *status;
    int tiles_m, tiles_n, group_m;   // tiles of 256 rows x 512 columns
    int full_units, num_units;       // units [0, full_units) are whole tiles, the rest are 256-column halves
};

struct Unit {
    int mb;          // row block (256 rows)
    int col0;        // first output column
    int width;       // 512 (two accumulators) or 256 (one)
};

__device__ __forceinline__ void tile_coords(const Params &p, int tile, int &mb, int &nb)
{
    // groups of group_m row blocks, row block fastest inside a group
    int per_group = p.group_m * p.tiles_n;
    int g = tile / per_group;
    int first_m = g * p.group_m;
    int gsz = min(p.group_m, p.tiles_m - first_m);
    int r = tile - g * per_group;
    mb = first_m + r % gsz;
    nb = r / gsz;
}

__device__ __forceinline__ Unit unit_of(const Params &p, int u)
{
    Unit w;
    int nb;
    if (u < p.full_units) {
        tile_coords(p, u, w.mb, nb);
        w.col0 = nb * TILE_N;
        w.width = (p.N - w.col0 > ACC_N) ? TILE_N : ACC_N;     // a ragged right edge that fits one accumulator
    } else {
        const int h = u - p.full_units;
        tile_coords(p, p.full_units + (h >> 1), w.mb, nb);
        w.col0 = nb * TILE_N + (h & 1) * ACC_N;
        w.width = ACC_N;
    }
    return w;
}

__device__ __forceinline__ void report(const Params &p, volatile uint32_t *abort_flag, uint32_t code)
{
    *abort_flag = 1u;
    if (p.status) atomicCAS(p.status, 0u, code | 0xC0u | ((uint32_t)blockIdx.x << 8));
}

template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gemm_tc3(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p)
{
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    const uint32_t accf_bar = bars + 8u * (2 * STAGES), acce_bar = bars + 8u * (2 * STAGES + 1);
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(base_ptr + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 2));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
    const bool leader = rank == 0;
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_units = p.num_units;
    const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accf_bar, 1);
        mbar_init(acce_bar, 16);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // paired allocation: the same warp of both CTAs executes it
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                            // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();      // everything above ran beside the tail of the preceding kernel; global memory is touched below

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t issued = 0, s = 0, ph = 0;
            bool ok = true;
            int t = 0;
            for (int u = pair_id; u < num_units && ok; u += num_pairs, t++) {
                const Unit w = unit_of(p, u);
                const bool down = (t & 1) != 0;                            // every other unit walks K downwards
                const bool two = w.width == TILE_N;
                const int m0 = w.mb * (2 * CTA_M) + (int)rank * CTA_M;    // this CTA's rows of A
                const int n0 = w.col0 + (int)rank * CTA_N;                // this CTA's columns of the first B block
                const uint32_t tx_bytes = 2u * (uint32_t)(A_STAGE_BYTES + (two ? 2 : 1) * B_STAGE_BYTES);
                for (int kb = 0; kb < nkb; kb++, issued++, s = (s + 1 == STAGES) ? 0 : s + 1, ph ^= (s == 0)) {
                    if (!mbar_try_wait(empty_bar(s), ph ^ 1u) && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        if (!*abort_flag) report(p, abort_flag, KERR_WAIT_EMPTY);
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + s * STAGE_BYTES, sb0 = sa + A_STAGE_BYTES, sb1 = sb0 + B_STAGE_BYTES;
                    const uint32_t lead_full = mapa_u32(full_bar(s), 0);
                    if (leader) mbar_arrive_expect_tx(full_bar(s), tx_bytes);
                    const int k0 = (down ? nkb - 1 - kb : kb) * BLOCK_K;
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < CTA_M / 64; j++) tma_load_2d_pair(sa + j * MN_BOX_BYTES, &tmA, m0 + 64 * j, k0, lead_full);
                    } else {
                        tma_load_2d_pair(sa, &tmA, k0, m0, lead_full);
                    }
                    if (B_MN) {
                        tma_load_2d_pair(sb0, &tmB, n0, k0, lead_full);
                        tma_load_2d_pair(sb0 + MN_BOX_BYTES, &tmB, n0 + 64, k0, lead_full);
                        if (two) {
                            tma_load_2d_pair(sb1, &tmB, n0 + ACC_N, k0, lead_full);
                            tma_load_2d_pair(sb1 + MN_BOX_BYTES, &tmB, n0 + ACC_N + 64, k0, lead_full);
                        }
                    } else {
                        tma_load_2d_pair(sb0, &tmB, k0, n0, lead_full);
                        if (two) tma_load_2d_pair(sb1, &tmB, k0, n0 + ACC_N, lead_full);
                    }
                }
            }
            if (!ok && leader) {
                // let the copies already in flight land before the CTA exits (bounded)
                uint32_t first = issued > (uint32_t)STAGES ? issued - STAGES : 0;
                for (uint32_t i = first; i < issued; i++) {
                    unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_bar(i % STAGES), (i / STAGES) & 1u) && global_ns() - t0 < 1000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer (leader only)
        if (leader && lane == 0) {
            constexpr uint32_t idesc = make_idesc(A_MN, B_MN);
            // descriptor halves: only the start address (low word) changes with stage and k
            constexpr uint32_t KSTEP_A = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            constexpr uint32_t KSTEP_B = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            const uint32_t a_hi = desc_hi(1024), b_hi = desc_hi(1024);
            const uint32_t a_lo0 = desc_lo(base, A_MN ? MN_BOX_BYTES : 16);
            const uint32_t b_lo0 = desc_lo(base + A_STAGE_BYTES, B_MN ? MN_BOX_BYTES : 16);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int t = 0;
            for (int u = pair_id; u < num_units && ok; u += num_pairs, t++) {
                const Unit w = unit_of(p, u);
                const bool two = w.width == TILE_N;
                // the accumulators are free once the epilogues of the previous unit have read them
                if (!mbar_try_wait(acce_bar, (uint32_t)(t & 1) ^ 1u) && !mbar_wait(acce_bar, (uint32_t)(t & 1) ^ 1u, abort_flag)) {
                    if (!*abort_flag) report(p, abort_flag, KERR_WAIT_ACC_FREE);
                    ok = false;
                    break;
                }
                tc_fence_after();
                uint32_t acc = 0;                          // first MMA of a unit overwrites the accumulators
                for (int kb = 0; kb < nkb; kb++) {
                    if (!mbar_try_wait(full_bar(s), ph) && !mbar_wait(full_bar(s), ph, abort_flag)) {
                        if (!*abort_flag) report(p, abort_flag, KERR_WAIT_FULL);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t alo = a_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
                    const uint32_t blo = b_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
                    // the four k-steps of one accumulator back to back, then those of the other
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; k++)
                        tc_mma_f16_pair(tmem_base, desc_join(alo + k * KSTEP_A, a_hi), desc_join(blo + k * KSTEP_B, b_hi), idesc,
                                        k == 0 ? acc : 1u);
                    if (two) {
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; k++)
                            tc_mma_f16_pair(tmem_base + ACC_N, desc_join(alo + k * KSTEP_A, a_hi),
                                            desc_join(blo + (uint32_t)(B_STAGE_BYTES >> 4) + k * KSTEP_B, b_hi), idesc,
                                            k == 0 ? acc : 1u);
                    }
                    acc = 1;
                    tc_commit_pair(empty_bar(s), 3);        // both CTAs' producers may refill stage s
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit_pair(accf_bar, 3);        // both CTAs' epilogues may read the accumulators
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (both CTAs)
        const int q = warp & 3;                    // tensor-memory lane quadrant this warp may access
        const int set = (warp - 2) >> 2;           // which accumulator (512-wide unit) or which half (256-wide unit)
        bool ok = true;
        int t = 0;
        for (int u = pair_id; u < num_units && ok; u += num_pairs, t++) {
            const Unit w = unit_of(p, u);
            const bool got = mbar_wait(accf_bar, (uint32_t)(t & 1), abort_flag);
            if (!__all_sync(0xFFFFFFFFu, got)) {
                if (!*abort_flag && lane == 0) report(p, abort_flag, KERR_WAIT_ACC);
                ok = false;
                break;
            }
            tc_fence_after();
            bool bad = false;
            // 512-wide unit: set s drains accumulator s (8 chunks of 32 columns); 256-wide: 4 chunks each
            const int nch = w.width == TILE_N ? ACC_N / 32 : ACC_N / 64;
            const int cbase = w.width == TILE_N ? set * ACC_N : set * (ACC_N / 2);
            const int row0 = w.mb * (2 * CTA_M) + (int)rank * CTA_M + q * 32;
            uint8_t *stage = base_ptr + STAGES * STAGE_BYTES + 256 + (warp - 2) * EPI_STAGE_BYTES;
#pragma unroll 1
            for (int c = 0; c < nch; c++) {
                uint32_t r[32];
                tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(cbase + c * 32), r);
                tc_wait_ld();
                const int col0 = w.col0 + cbase + c * 32;
                if (col0 < p.N)      // warp-uniform
                    epilogue_store32_coalesced(r, stage, p.C, p.ldc, p.mask, p.ldmask, row0, col0, p.M, p.N, p.relu != 0, bad);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_u32(acce_bar, 0));
            if (p.nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(p.nonfinite_flag, 1u);
        }
    }

    // common exit: all waits above are bounded, so both CTAs of the pair arrive here; neither
    // may leave while the other can still touch its shared or tensor memory
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <bool A_MN, bool B_MN>
static cudaError_t launch_variant(const CUtensorMap &ta, const CUtensorMap &tb, Params p, cudaStream_t st)
{
    static int max_pairs_dev[kMaxDevices] = {};     // 0 = this device not configured yet
    auto kern = k_gemm_tc3<A_MN, B_MN>;
    const int dev = current_device_slot();
    if (dev < 0) return cudaErrorInvalidDevice;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_pairs_dev[dev] == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3(148, 1, 1);
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorLaunchOutOfResources;
        max_pairs_dev[dev] = n < 74 ? n : 74;
    }
    const int max_pairs = max_pairs_dev[dev];
    // every cluster takes tiles / pairs whole tiles; what is left over runs as 256-column halves
    const int tiles = p.tiles_m * p.tiles_n;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    const int full = (tiles / pairs) * pairs, rest = tiles - full;
    p.full_units = full;
    p.num_units = full + 2 * rest;
    const int grid_pairs = p.num_units < max_pairs ? p.num_units : max_pairs;
    cfg.gridDim = dim3(2 * grid_pairs, 1, 1);
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, ta, tb, p);
}

}  // namespace pair512

cudaError_t launch_gemm_tc3(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag,
                            uint32_t *status, cudaStream_t st)
{
    using namespace pair512;
    g_last_gemm_launches = 1;
    CUtensorMap ta, tb;
    bool ok;
    if (op == MPT_OP_WGRAD) ok = tc_encode_map(&ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, 64, BLOCK_K);
    else ok = tc_encode_map(&ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BLOCK_K, CTA_M);
    if (op == MPT_OP_FWD) ok = ok && tc_encode_map(&tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BLOCK_K, CTA_N);
    else ok = ok && tc_encode_map(&tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, 64, BLOCK_K);
    if (!ok) return cudaErrorInvalidValue;
    Params p;
    p.M = M; p.N = N; p.K = K;
    p.C = C; p.ldc = ldc;
    p.mask = mask; p.ldmask = ldmask;
    p.relu = relu ? 1 : 0;
    p.nonfinite_flag = nonfinite_flag;
    p.status = status;
    p.tiles_m = (M + 2 * CTA_M - 1) / (2 * CTA_M);
    p.tiles_n = (N + TILE_N - 1) / TILE_N;
    p.group_m = 8;
    p.full_units = p.num_units = 0;
    if (op == MPT_OP_FWD) return launch_variant<false, false>(ta, tb, p, st);
    if (op == MPT_OP_DGRAD) return launch_variant<false, true>(ta, tb, p, st);
    return launch_variant<true, true>(ta, tb, p, st);
}

}  // namespace mpt
