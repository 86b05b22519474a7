// Tensor-core FP16 GEMM for few output tiles and a long contraction (paper section 3.3: FP16
// operands, FP32 accumulation, one rounding to FP16 on the store; section 4.5's projection product
// 2048 x 1024 x 8192 is the type case: 32 tiles of 256 x 256 for 74 CTA pairs).
//
// A cluster of 2*S CTAs (S = 2 or 4 CTA pairs) computes ONE 256x256 output tile.  Pair g of the
// cluster runs the k-blocks [nkb*g/S, nkb*(g+1)/S) of the contraction with tcgen05.mma.cta_group::2
// exactly as the pair kernel does (TMA ring, accumulator in tensor memory).  The S partial
// accumulators are then added inside the cluster, through distributed shared memory, instead of
// through a scratch buffer in global memory and a second launch:
//   * pair g owns the 256/S output columns [g*W, (g+1)*W); its epilogue warp (q, set) owns rows
//     32q..32q+31 of its CTA and columns g*W + set*W/2 .. + W/2;
//   * when every pair's MMAs are complete (one cluster barrier; the operand ring is idle from
//     then on and is reused for the exchange), warp (q, set) of pair g reads from tensor memory
//     the columns that warp (q, set) of every other pair d owns, 32 at a time, parks them as raw
//     FP32 in a staging block of its own CTA and sends each 4 KB chunk with one bulk copy
//     (cp.async.bulk.shared::cluster.shared::cta, no multicast) to the CTA of pair d that holds
//     the same rows; the copy completes on an mbarrier of the receiving warp;
//   * each warp waits for its chunks as they arrive, adds the parts in ascending part order (own
//     part from tensor memory in its place: one FP32 rounding per add, the order the
//     scratch-buffer split uses), and applies the usual epilogue with coalesced stores.
// All pairs send and receive at once, every warp of the cluster takes part in the epilogue, and
// the result does not depend on timing.  The exchange is bound by the SM-to-SM network (about 2 us
// for the 64 KB each CTA sends and receives); the first chunk's epilogue runs under the second's
// transfer.  Measured on B200 (graph replay): 2048 x 1024 x 8192 27.5 us against 42-44 us with the
// parts going through global memory and a second launch.
// Every mbarrier wait is bounded (tc_ptx.cuh); the cluster barriers are reached by every thread
// because every wait before them is bounded.  If a wait does run out (status word set, the context
// is poisoned), a bulk copy may still be in flight when its CTAs leave; nothing reads its result.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>

#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

namespace quad {

static constexpr int CTA_M = 128;          // rows per CTA (256 per pair)
static constexpr int TILE_N = 256;         // columns per tile
static constexpr int CTA_N = 128;          // columns of B each CTA loads
static constexpr int BLOCK_K = 64, UMMA_K = 16;
static constexpr int STAGES = 7;
static constexpr int A_STAGE_BYTES = CTA_M * BLOCK_K * 2;   // 16 KB
static constexpr int B_STAGE_BYTES = CTA_N * BLOCK_K * 2;   // 16 KB
static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
static constexpr int MN_BOX_BYTES = 64 * BLOCK_K * 2;
static constexpr int TMEM_COLS = 256;      // one accumulator: a cluster computes one tile
static constexpr int EPI_WARPS = 8;        // two sets of four (tensor-memory lane quadrants)
static constexpr int THREADS = 64 + 32 * EPI_WARPS;
static constexpr int MAX_S = 4;
static constexpr int NUM_BARS = 2 * STAGES + 1 + (MAX_S - 1) * EPI_WARPS;   // a received block has 2 chunks for S = 2, 1 for S = 4
static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 8 * NUM_BARS + 16;

__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn)
{
    return (1u << 4) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(TILE_N >> 3) << 17) |
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
    int tiles_m, tiles_n;
};

__device__ __forceinline__ void report(const Params &p, volatile uint32_t *abort_flag, uint32_t code)
{
    *abort_flag = 1u;
    if (p.status) atomicCAS(p.status, 0u, code | 0x80u | ((uint32_t)blockIdx.x << 8));
}

// Trace build only (-DMPT_GEMM_TRACE): the first and the last CTA of the grid write the time (ns, low
// word) of the steps of their launch into words [64 + 16 * which + i] of the status array.
#ifdef MPT_GEMM_TRACE
#define TC4_STAMP(i)                                                                                   \
    do {                                                                                               \
        if (p.status && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))                              \
            p.status[64 + 16 * (blockIdx.x == 0 ? 0 : 1) + (i)] = (uint32_t)global_ns();               \
    } while (0)
#define TC4_CYC(i)                                                                                     \
    do {                                                                                               \
        if (p.status && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))                              \
            p.status[64 + 16 * (blockIdx.x == 0 ? 0 : 1) + (i)] = (uint32_t)clock64();                 \
    } while (0)
#else
#define TC4_STAMP(i) do { } while (0)
#define TC4_CYC(i) do { } while (0)
#endif

// S: CTA pairs per cluster = parts of the contraction.  W = 256 / S columns per pair, W / 2 per warp.
template <bool A_MN, bool B_MN, int S>
__global__ void __launch_bounds__(THREADS, 1)
k_gemm_tc4(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Params p)
{
    constexpr int W = TILE_N / S;               // columns a pair owns in the epilogue
    constexpr int WCOLS = W / 2;                // columns a warp owns: 64 (S = 2) or 32 (S = 4)
    constexpr int NCH = WCOLS / 32;             // 32-column chunks per warp and source
    constexpr int BLOCK_BYTES = 32 * WCOLS * 4; // one warp's block from one source: [chunk][float4 index 0..7][lane],
                                                // so that a warp's 16-byte stores and loads are 512 contiguous bytes
    constexpr int CHUNK_BYTES = BLOCK_BYTES / NCH;            // 32 rows x 32 columns of FP32: the unit of the exchange
    constexpr int RECV_BYTES = (S - 1) * EPI_WARPS * BLOCK_BYTES;
    static_assert((S - 1) * NCH <= MAX_S - 1, "one mbarrier per received chunk");
    constexpr int SEND_BYTES = RECV_BYTES;                    // staging of the blocks this CTA sends
    constexpr int EPI_STAGE_BYTES = 32 * kEpiStagePitch;      // per warp: FP16 block for the coalesced global stores
    static_assert(RECV_BYTES + SEND_BYTES + EPI_WARPS * EPI_STAGE_BYTES <= STAGES * STAGE_BYTES, "the blocks of the exchange must fit the ring");

    pdl_trigger();
    if (threadIdx.x == 32) { prefetch_tensormap(&tmA); prefetch_tensormap(&tmB); }
    if (threadIdx.x == 0) TC4_STAMP(0);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    const uint32_t accf_bar = bars + 8u * (2 * STAGES);
    auto recv_bar = [&](int slot, int w, int c) { return bars + 8u * (2 * STAGES + 1 + (slot * EPI_WARPS + w) * NCH + c); };
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(base_ptr + STAGES * STAGE_BYTES + 8 * NUM_BARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();       // 0 .. 2S-1
    const uint32_t half = rank & 1u;               // which 128 rows of the tile this CTA holds
    const int g = (int)(rank >> 1);                // pair index = part of the contraction
    const uint32_t lead_rank = rank & ~1u;         // the CTA of this pair that issues the MMAs
    const bool leader = half == 0;
    const int tile = blockIdx.x / (2 * S);
    const int mb = tile % p.tiles_m, nb = tile / p.tiles_m;
    const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;
    const int kb0 = (int)(((long long)nkb * g) / S), kb1 = (int)(((long long)nkb * (g + 1)) / S);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accf_bar, 1);
        for (int j = 0; j < S - 1; j++)
            for (int w = 0; w < EPI_WARPS; w++)
                for (int c = 0; c < NCH; c++) {
                    mbar_init(recv_bar(j, w, c), 1);
                    mbar_arrive_expect_tx(recv_bar(j, w, c), (uint32_t)CHUNK_BYTES);   // completes when the chunk has arrived
                }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // paired allocation: the same warp of both CTAs of a pair executes it
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                            // every CTA's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) TC4_STAMP(1);
    pdl_wait();      // global memory is touched below
    if (threadIdx.x == 0) TC4_STAMP(2);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (every CTA)
        if (lane == 0) {
            uint32_t issued = 0, s = 0, ph = 0;
            bool ok = true;
            const int m0 = mb * (2 * CTA_M) + (int)half * CTA_M;       // this CTA's rows of A
            const int n0 = nb * TILE_N + (int)half * CTA_N;            // this CTA's columns of B
            constexpr uint32_t tx_bytes = 2u * (uint32_t)STAGE_BYTES;
            for (int kb = kb0; kb < kb1; kb++, issued++, s = (s + 1 == STAGES) ? 0 : s + 1, ph ^= (s == 0)) {
                if (!mbar_try_wait(empty_bar(s), ph ^ 1u) && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                    if (!*abort_flag) report(p, abort_flag, KERR_WAIT_EMPTY);
                    ok = false;
                    break;
                }
                const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                const uint32_t lead_full = mapa_u32(full_bar(s), lead_rank);
                if (leader) mbar_arrive_expect_tx(full_bar(s), tx_bytes);
                const int k0 = kb * BLOCK_K;
                if (A_MN) {
#pragma unroll
                    for (int j = 0; j < CTA_M / 64; j++) tma_load_2d_pair(sa + j * MN_BOX_BYTES, &tmA, m0 + 64 * j, k0, lead_full);
                } else {
                    tma_load_2d_pair(sa, &tmA, k0, m0, lead_full);
                }
                if (B_MN) {
                    tma_load_2d_pair(sb, &tmB, n0, k0, lead_full);
                    tma_load_2d_pair(sb + MN_BOX_BYTES, &tmB, n0 + 64, k0, lead_full);
                } else {
                    tma_load_2d_pair(sb, &tmB, k0, n0, lead_full);
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
        __syncwarp();
        cluster_arrive();          // this warp has nothing more to put into the ring
    } else if (warp == 1) {
        // ------------------------------------------------------ MMA issuer (first CTA of each pair)
        if (leader && lane == 0) {
            constexpr uint32_t idesc = make_idesc(A_MN, B_MN);
            constexpr uint32_t KSTEP_A = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            constexpr uint32_t KSTEP_B = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            const uint32_t a_hi = desc_hi(1024), b_hi = desc_hi(1024);
            const uint32_t a_lo0 = desc_lo(base, A_MN ? MN_BOX_BYTES : 16);
            const uint32_t b_lo0 = desc_lo(base + A_STAGE_BYTES, B_MN ? MN_BOX_BYTES : 16);
            const uint16_t pair_mask = (uint16_t)(3u << lead_rank);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            uint32_t acc = 0;                          // the first MMA overwrites the accumulator
            for (int kb = kb0; kb < kb1; kb++) {
                if (!mbar_try_wait(full_bar(s), ph) && !mbar_wait(full_bar(s), ph, abort_flag)) {
                    if (!*abort_flag) report(p, abort_flag, KERR_WAIT_FULL);
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (kb == kb0) { TC4_STAMP(3); TC4_CYC(11); }
                const uint32_t alo = a_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
                const uint32_t blo = b_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; k++) {
                    tc_mma_f16_pair(tmem_base, desc_join(alo + k * KSTEP_A, a_hi), desc_join(blo + k * KSTEP_B, b_hi), idesc, acc);
                    acc = 1;
                }
                tc_commit_pair(empty_bar(s), pair_mask);     // both CTAs' producers may refill stage s
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (ok) tc_commit_pair(accf_bar, pair_mask);     // both CTAs' epilogue warps may read the accumulator
            TC4_STAMP(4);
            TC4_CYC(12);
        }
        __syncwarp();
        cluster_arrive();
    } else {
        // ------------------------------------------------- exchange and epilogue (every CTA, 8 warps)
        const int q = warp & 3;                   // tensor-memory lane quadrant this warp may read
        const int set = (warp - 2) >> 2;          // which half of a pair's columns
        const int w = set * 4 + q;                // index of this warp's blocks and barriers
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        bool ok = mbar_wait(accf_bar, 0u, abort_flag);
        if (!__all_sync(0xFFFFFFFFu, ok)) {
            if (!*abort_flag && lane == 0) report(p, abort_flag, KERR_WAIT_ACC);
            ok = false;
        }
        tc_fence_after();
        if (warp == 2 && lane == 0) TC4_STAMP(5);
        // the tensor core has read the ring through the async proxy; plain stores will now overwrite it
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        cluster_arrive();
        cluster_wait();            // every pair's MMAs are complete: no ring of the cluster is in use any more
        if (warp == 2 && lane == 0) TC4_STAMP(6);
        if (ok) {
            // send: the columns warp (q, set) of pair d owns, into its block for source g.  The values go
            // from tensor memory to a staging block of this CTA's ring and from there to the other CTA
            // with one bulk copy per block, which completes on the receiving warp's mbarrier.
#pragma unroll
            for (int dd = 1; dd < S; dd++) {
                const int d = (g + dd) % S;                       // start with the next pair: spreads the traffic
                const int slot = g < d ? g : g - 1;               // blocks of a receiver are ordered by source
                const uint32_t dst_rank = (uint32_t)(2 * d) + half;
                const uint32_t stage = base + (uint32_t)(RECV_BYTES + ((dd - 1) * EPI_WARPS + w) * BLOCK_BYTES);
#pragma unroll
                for (int c = 0; c < NCH; c++) {
                    uint32_t r[32];
                    tc_ld32(t_lane + (uint32_t)(d * W + set * WCOLS + c * 32), r);
                    tc_wait_ld();
#pragma unroll
                    for (int v = 0; v < 8; v++)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + (uint32_t)((c * 8 + v) * 512 + lane * 16)),
                                     "r"(r[4 * v]), "r"(r[4 * v + 1]), "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                                     : "memory");
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads what the lanes just wrote
                    __syncwarp();
                    if (lane == 0)
                        bulk_copy_to_cluster(mapa_u32(base + (uint32_t)((slot * EPI_WARPS + w) * BLOCK_BYTES + c * CHUNK_BYTES), dst_rank),
                                             stage + (uint32_t)(c * CHUNK_BYTES), (uint32_t)CHUNK_BYTES,
                                             mapa_u32(recv_bar(slot, w, c), dst_rank));
                }
            }
            if (warp == 2 && lane == 0) TC4_STAMP(7);
            // receive and finish this warp's own columns
            bool bad = false;
            {
#pragma unroll 1
                for (int c = 0; c < NCH && ok; c++) {
#pragma unroll
                    for (int j = 0; j < S - 1; j++) {
                        const bool got = mbar_wait_cluster(recv_bar(j, w, c), 0u, abort_flag);
                        if (!__all_sync(0xFFFFFFFFu, got)) {
                            if (!*abort_flag && lane == 0) report(p, abort_flag, KERR_WAIT_PARTIAL);
                            ok = false;
                        }
                    }
                    if (!ok) break;
                    if (c == 0 && warp == 2 && lane == 0) TC4_STAMP(8);
                    uint32_t r[32];
                    tc_ld32(t_lane + (uint32_t)(g * W + set * WCOLS + c * 32), r);
                    tc_wait_ld();
                    float sum[32];
                    // parts in ascending order, the own one (part g) in its place
#pragma unroll
                    for (int part = 0; part < S; part++) {
                        if (part == g) {
#pragma unroll
                            for (int e = 0; e < 32; e++) sum[e] = part == 0 ? __uint_as_float(r[e]) : __fadd_rn(sum[e], __uint_as_float(r[e]));
                        } else {
                            const int slot = part < g ? part : part - 1;
                            const float4 *src = (const float4 *)(base_ptr + (slot * EPI_WARPS + w) * BLOCK_BYTES + c * 4096) + lane;
#pragma unroll
                            for (int v = 0; v < 8; v++) {
                                const float4 x = src[v * 32];
                                if (part == 0) {
                                    sum[4 * v] = x.x; sum[4 * v + 1] = x.y; sum[4 * v + 2] = x.z; sum[4 * v + 3] = x.w;
                                } else {
                                    sum[4 * v] = __fadd_rn(sum[4 * v], x.x);
                                    sum[4 * v + 1] = __fadd_rn(sum[4 * v + 1], x.y);
                                    sum[4 * v + 2] = __fadd_rn(sum[4 * v + 2], x.z);
                                    sum[4 * v + 3] = __fadd_rn(sum[4 * v + 3], x.w);
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 32; e++) r[e] = __float_as_uint(sum[e]);
                    const int col0 = nb * TILE_N + g * W + set * WCOLS + c * 32;
                    epilogue_store32_coalesced(r, base_ptr + RECV_BYTES + SEND_BYTES + w * EPI_STAGE_BYTES, p.C, p.ldc, p.mask, p.ldmask,
                                               mb * (2 * CTA_M) + (int)half * CTA_M + q * 32, col0, p.M, p.N, p.relu != 0, bad);
                }
                if (p.nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(p.nonfinite_flag, 1u);
                if (warp == 2 && lane == 0) TC4_STAMP(9);
            }
        }
    }
    if (warp < 2) cluster_wait();      // completes the arrive these warps made above

    // common exit: no CTA may leave while another can still touch its shared or tensor memory
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x == 0) TC4_STAMP(10);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <bool A_MN, bool B_MN, int S>
static cudaError_t launch_variant(const CUtensorMap &ta, const CUtensorMap &tb, const Params &p, cudaStream_t st)
{
    static int max_clusters_dev[kMaxDevices] = {};     // 0 = this device not configured yet, < 0 = cannot run here
    auto kern = k_gemm_tc4<A_MN, B_MN, S>;
    const int dev = current_device_slot();
    if (dev < 0) return cudaErrorInvalidDevice;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2 * S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_clusters_dev[dev] == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3(2 * S * 16, 1, 1);
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return e;
        max_clusters_dev[dev] = n >= 1 ? n : -1;
    }
    if (max_clusters_dev[dev] < 0) return cudaErrorLaunchOutOfResources;
    cfg.gridDim = dim3((unsigned)(2 * S * p.tiles_m * p.tiles_n), 1, 1);
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, ta, tb, p);
}

}  // namespace quad

// How many clusters of 2*S CTAs of this kernel the current device holds at once (cached per device);
// 0 when that cannot be asked (no device): the caller then leaves the shape to the other kernels.
template <int S>
static int resident_clusters()
{
    static int cached[kMaxDevices] = {};        // 0 = not asked yet, < 0 = none
    const int dev = current_device_slot();
    if (dev < 0) return 0;
    if (cached[dev] == 0) {
        auto kern = quad::k_gemm_tc4<false, false, S>;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2 * S;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.blockDim = dim3(quad::THREADS, 1, 1);
        cfg.gridDim = dim3(2 * S * 16, 1, 1);
        cfg.dynamicSmemBytes = quad::SMEM_BYTES;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, quad::SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        cached[dev] = n >= 1 ? n : -1;
        if (const char *e = getenv("MPT_DEBUG_PLAN"))
            if (e[0] == '1') fprintf(stderr, "mpt: %d clusters of %d CTAs of the in-cluster split kernel fit this device\n", n, 2 * S);
    }
    return cached[dev] > 0 ? cached[dev] : 0;
}

// Parts of the contraction (CTA pairs per cluster) the in-cluster split would use; 0 = this kernel
// is not the one for the shape.  Few tiles and a long contraction.  Every cluster must be resident at
// once (the hardware would run more in rounds, correctly but at twice the time).  Measured on B200,
// launches replayed from a graph, microseconds for single-CTA kernel / two parts / four parts:
//   512x512x4096 (4 tiles)    20.8 / 14.8 / 11.8      1024x768x4096 (12 tiles)   21.9 / 15.9 / 13.2
//   1024x1024x4096 (16 tiles) 22.2 / 15.6 / 24.1      2048x1024x8192 (32 tiles)  41.8 / 27.5 / 52.1
//   1024x1024x1024 (16 tiles)  7.8 /  8.4 / 16.9      2304x1024x4096 (36 tiles)  24.2 / 30.8 / 38.4
// so: four parts when their clusters all fit and a part keeps 16 k-blocks, else two parts when those
// clusters fit (at most 32 tiles) and a part keeps 16 k-blocks.
int tc4_split_for(int M, int N, int K)
{
    // MPT_DISABLE_CLUSTER_SPLIT=1: leave these shapes to the other kernels (comparisons)
    static const bool off = [] { const char *e = getenv("MPT_DISABLE_CLUSTER_SPLIT"); return e && e[0] == '1'; }();
    if (off || M < 256 || N < 256) return 0;
    const long tiles = (long)((M + 255) / 256) * ((N + 255) / 256);
    const int nkb = (K + quad::BLOCK_K - 1) / quad::BLOCK_K;
    if (tiles > 32 || nkb < 32) return 0;
    if (nkb >= 64 && tiles <= 12 && tiles <= resident_clusters<4>()) return 4;
    if (tiles <= resident_clusters<2>()) return 2;
    return 0;
}

cudaError_t launch_gemm_tc4(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag,
                            uint32_t *status, cudaStream_t st, int split)
{
    using namespace quad;
    g_last_gemm_launches = 1;
    const int nkb = (K + BLOCK_K - 1) / BLOCK_K;
    if ((split != 2 && split != 4) || nkb < split) return cudaErrorInvalidValue;
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
    if (split == 2) {
        if (op == MPT_OP_FWD) return launch_variant<false, false, 2>(ta, tb, p, st);
        if (op == MPT_OP_DGRAD) return launch_variant<false, true, 2>(ta, tb, p, st);
        return launch_variant<true, true, 2>(ta, tb, p, st);
    }
    if (op == MPT_OP_FWD) return launch_variant<false, false, 4>(ta, tb, p, st);
    if (op == MPT_OP_DGRAD) return launch_variant<false, true, 4>(ta, tb, p, st);
    return launch_variant<true, true, 4>(ta, tb, p, st);
}

}  // namespace mpt
