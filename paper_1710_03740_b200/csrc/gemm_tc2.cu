// Tensor-core FP16 GEMM for sm_100a with CTA pairs (paper section 3.3: FP16 operands,
// FP32 accumulation, FP16 on the store; same fused epilogue as the single-CTA kernel).
//
// Two CTAs on neighbouring SMs form a cluster and compute one 256x256 output tile with
// tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16 per instruction).  Each CTA loads its
// own 128 rows of A and its own 128 columns of B (64 k per stage, 32 KB per stage and CTA),
// the tensor core reads both CTAs' shared memory, and each CTA's tensor memory receives the
// 128 x 256 accumulator block of its rows.  Compared with one CTA per 128x256 tile this
// moves a third fewer operand bytes from L2 to the SMs and leaves room for a 6-stage ring plus
// 32 KB in which the epilogue stages the output for bulk tensor stores.
//
// Roles in each CTA (192 threads): warp 0 TMA producer, warp 1 MMA issuer (only the
// leader CTA, rank 0, issues; both CTAs' warp 1 take part in the paired tensor-memory
// allocation), warps 2-5 epilogue (long products: 32 x 64 output boxes rounded into shared memory and
// written by cp.async.bulk.tensor stores; short ones and the special forms: per-lane stores).  Synchronisation:
//   full[s]   in the leader: 1 arrival (leader's expect_tx for both CTAs' bytes) + the bytes
//             of both CTAs' loads (the peer's loads signal the leader's barrier)
//   empty[s]  in each CTA: tcgen05.commit multicast to both CTAs when the MMAs have read stage s
//   accf[b]   in each CTA: tcgen05.commit multicast when a tile's accumulator is complete
//   acce[b]   in the leader: 8 arrivals, one per epilogue warp of both CTAs
// Work units: every cluster first takes the same number of full 256x256 tiles; the tiles left
// over for a last, partly filled round are cut into two 256x128 halves when that lets every
// half run at once (the last round then takes about half as long).  A half unit is the same
// pipeline with 64 columns of B per CTA and N = 128 instructions.
// No TMA multicast is used.  Every mbarrier wait is bounded (see tc_ptx.cuh).
#include <cuda.h>
#include <stdlib.h>

#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

namespace pair {


static constexpr int CTA_M = 128;          // rows per CTA (256 per pair)
static constexpr int TILE_N = 256;         // columns per pair tile
static constexpr int CTA_N = 128;          // columns of B each CTA loads
static constexpr int BLOCK_K = 64, UMMA_K = 16;
static constexpr int STAGES = 6;             // 7 stages are not faster inside the step; the seventh's 32 KB stage the output
static constexpr int EPI_BOX_BYTES = 32 * 64 * 2;          // one box of the output: 32 rows x 64 columns of FP16
static constexpr int EPI_BYTES = 8 * EPI_BOX_BYTES;        // two boxes for each of four epilogue warps
static constexpr int A_STAGE_BYTES = CTA_M * BLOCK_K * 2;   // 16 KB
static constexpr int B_STAGE_BYTES = CTA_N * BLOCK_K * 2;   // 16 KB
static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
static constexpr int MN_BOX_BYTES = 64 * BLOCK_K * 2;
static constexpr int TMEM_COLS = 512;
static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 + 256;

// instruction descriptor without the N field (N >> 3 goes to bits 17..22)
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn)
{
    return (1u << 4) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)((2 * CTA_M) >> 4) << 24);
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
    int tiles_m, tiles_n, group_m;   // pair tiles (256 rows x 256 columns)
    int full_units, num_units;       // units [0, full_units) are whole tiles, the rest are half tiles
    // split-K (few tiles, long contraction): every whole tile is cut into split_k units along K;
    // a unit leaves its raw FP32 accumulator in partial[part][M][ldp] and a second kernel adds the
    // parts in ascending order and applies the epilogue.  split_k == 1: off.
    int split_k;
    float *partial;
    int ldp;
    // tail split: the tiles left over for a last, partly filled round are cut into tail_split units
    // along K (full-width instructions, unlike the half-width units, which take as long as whole
    // ones); unit h of the tail leaves its raw FP32 accumulator in tail_partial[h][256][256] and
    // k_tail_reduce finishes those tiles.  tail_split == 1: off (half-width units instead).
    int tail_split;
    float *tail_partial;
    int tma_store;                   // output of whole and half tiles through shared memory and tensor stores
    int hint_a, hint_b;              // L2 eviction priority of the operand loads (0 normal, 1 last, 2 first)
    LstmEpi lstm;                    // read only by the LSTM instantiation of the kernel
};

struct Unit {
    int mb, nb;      // tile coordinates
    int n_off;       // first column of the unit inside its tile (0 or 128)
    int width;       // 256 (whole tile) or 128 (half)
    int part;        // K part (split-K)
    int kb0, kb1;    // k-blocks [kb0, kb1) of the contraction
    int tail_slot;   // >= 0: unit of the split tail, index of its 256x256 FP32 block; -1 otherwise
};

__device__ __forceinline__ void tile_coords(const Params &p, int tile, int &mb, int &nb)
{
    int per_group = p.group_m * p.tiles_n;
    int g = tile / per_group;
    int first_m = g * p.group_m;
    int gsz = min(p.group_m, p.tiles_m - first_m);
    int r = tile - g * per_group;
    mb = first_m + r % gsz;
    nb = r / gsz;
}

__device__ __forceinline__ Unit unit_of(const Params &p, int u, int nkb)
{
    Unit w;
    int tile = u;
    w.n_off = 0;
    w.width = TILE_N;
    w.part = 0;
    w.kb0 = 0;
    w.kb1 = nkb;
    w.tail_slot = -1;
    if (p.split_k > 1) {            // parts of one tile are neighbouring units: they run side by side
        tile = u / p.split_k;
        w.part = u - tile * p.split_k;
        w.kb0 = (int)(((long long)nkb * w.part) / p.split_k);
        w.kb1 = (int)(((long long)nkb * (w.part + 1)) / p.split_k);
    } else if (u >= p.full_units && p.tail_split > 1) {
        const int h = u - p.full_units;
        tile = p.full_units + h / p.tail_split;
        w.part = h - (tile - p.full_units) * p.tail_split;
        w.kb0 = (int)(((long long)nkb * w.part) / p.tail_split);
        w.kb1 = (int)(((long long)nkb * (w.part + 1)) / p.tail_split);
        w.tail_slot = h;
    } else if (u >= p.full_units) {
        const int h = u - p.full_units;
        tile = p.full_units + (h >> 1);
        w.n_off = (h & 1) * (TILE_N / 2);
        w.width = TILE_N / 2;
    }
    tile_coords(p, tile, w.mb, w.nb);
    return w;
}

__device__ __forceinline__ void report(const Params &p, volatile uint32_t *abort_flag, uint32_t code)
{
    *abort_flag = 1u;
    if (p.status) atomicCAS(p.status, 0u, code | 0x80u | ((uint32_t)blockIdx.x << 8));
}

// Epilogue width.  One set of four warps drains an accumulator in about 2.4 us, which hides behind
// the next tile's main loop when a CTA has many tiles.  With two sets, each taking half of the
// columns of a unit, the exposed epilogue of the last tile halves: launch-bound products gain
// (1024^3 -7 %, tiny-MLP step -12 %), long ones lose about 1.4 % (more warps polling under the power
// cap).  The gate epilogue (LSTM) does far more arithmetic per element and always uses two sets.
template <bool WIDE>
struct EpiCfg {
    static constexpr int SETS = WIDE ? 2 : 1;
    static constexpr int THREADS = 64 + 128 * SETS;
};

template <bool A_MN, bool B_MN, bool LSTM = false, bool WIDE = false>
__global__ void __launch_bounds__(EpiCfg<LSTM || WIDE>::THREADS, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
           const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmC, const Params p)
{
    pdl_trigger();
    if (threadIdx.x == 32) { prefetch_tensormap(&tmA); prefetch_tensormap(&tmB); prefetch_tensormap(&tmBh); prefetch_tensormap(&tmC); }
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t epi_stage = base + STAGES * STAGE_BYTES;        // 1024-byte aligned boxes for the output stores
    const uint32_t bars = epi_stage + EPI_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(base_ptr + STAGES * STAGE_BYTES + EPI_BYTES + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
    const bool leader = rank == 0;
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_units = p.num_units;
    const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; b++) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 8 * EpiCfg<LSTM || WIDE>::SETS); }
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
            int tt = 0;
            const uint64_t pol_a = l2_policy(p.hint_a), pol_b = l2_policy(p.hint_b);
            for (int u = pair_id; u < num_units && ok; u += num_pairs, tt++) {
                const Unit w = unit_of(p, u, nkb);
                // Every other unit of a cluster walks its k-blocks downwards: the operand panels a wave of
                // tiles has just finished with are the first ones the next wave asks for, while they are
                // still in L2 (a wave touches about 107 MB of panels, more than L2 keeps).  Measured on
                // 4096x12288x12288: DRAM reads 1.36 -> 1.14 GB per launch, sustained rate +1.5-2 %.
                const bool down = (tt & 1) != 0;
                const int cta_n = w.width >> 1;                            // columns of B this CTA loads
                const int m0 = w.mb * (2 * CTA_M) + (int)rank * CTA_M;    // this CTA's rows of A
                const int n0 = w.nb * TILE_N + w.n_off + (int)rank * cta_n;
                const uint32_t tx_bytes = 2u * (uint32_t)(A_STAGE_BYTES + cta_n * BLOCK_K * 2);
                for (int kb = w.kb0; kb < w.kb1; kb++, issued++, s = (s + 1 == STAGES) ? 0 : s + 1, ph ^= (s == 0)) {
                    if (!mbar_try_wait(empty_bar(s), ph ^ 1u) && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        if (!*abort_flag) report(p, abort_flag, KERR_WAIT_EMPTY);
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const uint32_t lead_full = mapa_u32(full_bar(s), 0);
                    if (leader) mbar_arrive_expect_tx(full_bar(s), tx_bytes);
                    const int k0 = (down ? (w.kb0 + w.kb1 - 1 - kb) : kb) * BLOCK_K;
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < CTA_M / 64; j++) tma_load_2d_pair_hint(sa + j * MN_BOX_BYTES, &tmA, m0 + 64 * j, k0, lead_full, pol_a);
                    } else {
                        tma_load_2d_pair_hint(sa, &tmA, k0, m0, lead_full, pol_a);
                    }
                    if (B_MN) {
                        tma_load_2d_pair_hint(sb, &tmB, n0, k0, lead_full, pol_b);
                        if (cta_n == CTA_N) tma_load_2d_pair_hint(sb + MN_BOX_BYTES, &tmB, n0 + 64, k0, lead_full, pol_b);
                    } else {
                        tma_load_2d_pair_hint(sb, cta_n == CTA_N ? &tmB : &tmBh, k0, n0, lead_full, pol_b);
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
            constexpr uint32_t idesc_base = make_idesc(A_MN, B_MN);
            // descriptor halves: only the start address (low word) changes with stage and k
            constexpr uint32_t KSTEP_A = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            constexpr uint32_t KSTEP_B = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            const uint32_t a_hi = desc_hi(1024), b_hi = desc_hi(1024);
            const uint32_t a_lo0 = desc_lo(base, A_MN ? MN_BOX_BYTES : 16);
            const uint32_t b_lo0 = desc_lo(base + A_STAGE_BYTES, B_MN ? MN_BOX_BYTES : 16);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int t = 0;
#ifdef MPT_GEMM_TRACE
            // Trace build only (python -m paper_1710_03740_b200.build --trace): the issuing thread of every
            // cluster records when it started, how many SM cycles its main loops took and how many
            // k-blocks it issued, into words [64 + 8 * cluster ...] of the status array, which the
            // caller must then size at 1024 words.
            const unsigned long long tr_t0 = global_ns();
            const long long tr_c0 = clock64();
            unsigned tr_kb = 0;
#endif
            for (int u = pair_id; u < num_units && ok; u += num_pairs, t++) {
                const Unit w = unit_of(p, u, nkb);
                const uint32_t idesc = idesc_base | ((uint32_t)(w.width >> 3) << 17);
                const int buf = t & 1;
                const uint32_t acc_ph = (t >> 1) & 1u;
                if (!mbar_try_wait(acce_bar(buf), acc_ph ^ 1u) && !mbar_wait(acce_bar(buf), acc_ph ^ 1u, abort_flag)) {
                    if (!*abort_flag) report(p, abort_flag, KERR_WAIT_ACC_FREE);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * TILE_N);
                uint32_t acc = 0;                          // first MMA of a tile overwrites the accumulator
                for (int kb = w.kb0; kb < w.kb1; kb++) {
                    if (!mbar_try_wait(full_bar(s), ph) && !mbar_wait(full_bar(s), ph, abort_flag)) {
                        if (!*abort_flag) report(p, abort_flag, KERR_WAIT_FULL);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t alo = a_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
                    const uint32_t blo = b_lo0 + s * (uint32_t)(STAGE_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; k++) {
                        tc_mma_f16_pair(d_tmem, desc_join(alo + k * KSTEP_A, a_hi), desc_join(blo + k * KSTEP_B, b_hi), idesc, acc);
                        acc = 1;
                    }
                    tc_commit_pair(empty_bar(s), 3);        // both CTAs' producers may refill stage s
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
#ifdef MPT_GEMM_TRACE
                    tr_kb++;
#endif
                }
                if (ok) tc_commit_pair(accf_bar(buf), 3);   // both CTAs' epilogues may read the accumulator
            }
#ifdef MPT_GEMM_TRACE
            if (p.status) {
                uint32_t *tr = p.status + 64 + 8 * pair_id;
                tr[0] = (uint32_t)tr_t0;
                tr[1] = (uint32_t)global_ns();
                tr[2] = (uint32_t)(clock64() - tr_c0);
                tr[3] = tr_kb;
                tr[4] = (uint32_t)t;
            }
#endif
        }
    } else {
        // ---------------------------------------------------------------- epilogue (both CTAs)
        const int q = warp & 3;
        bool ok = true;
        int t = 0;
        int boxes_sent = 0;          // tensor stores this warp has issued (lane 0 tracks their bulk groups)
        for (int u = pair_id; u < num_units && ok; u += num_pairs, t++) {
            const Unit w = unit_of(p, u, nkb);
            const int buf = t & 1;
            const uint32_t acc_ph = (t >> 1) & 1u;
            const bool got = mbar_wait(accf_bar(buf), acc_ph, abort_flag);
            if (!__all_sync(0xFFFFFFFFu, got)) {
                if (!*abort_flag && lane == 0) report(p, abort_flag, KERR_WAIT_ACC);
                ok = false;
                break;
            }
            tc_fence_after();
            const int row = w.mb * (2 * CTA_M) + (int)rank * CTA_M + q * 32 + lane;
            const bool row_ok = row < p.M;
            uint16_t *crow = p.C + (size_t)row * p.ldc;
            const uint16_t *mrow = p.mask ? p.mask + (size_t)row * p.ldmask : nullptr;
            bool bad = false;
            if constexpr (LSTM) {
                const int set = (warp - 2) >> 2, nch = w.width / 64;       // this set's half of the unit's columns
                epilogue_lstm_tile(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N + set * nch * 32), nch,
                                   w.nb * TILE_N + w.n_off + set * nch * 32, p.N, row, row_ok, crow, p.lstm);
            } else if (w.tail_slot >= 0) {
                // unit of the split tail: the raw 256x256 FP32 block of this part (all rows, all columns)
                float *prow = p.tail_partial + (size_t)w.tail_slot * (2 * CTA_M * TILE_N) +
                              (size_t)((int)rank * CTA_M + q * 32 + lane) * TILE_N;
                constexpr int NCH = TILE_N / 32 / EpiCfg<LSTM || WIDE>::SETS;
                const int set = (warp - 2) >> 2;
#pragma unroll 1
                for (int c = set * NCH; c < (set + 1) * NCH; c++) {
                    uint32_t r[32];
                    tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N + c * 32), r);
                    tc_wait_ld();
                    float4 *dst = (float4 *)(prow + c * 32);
#pragma unroll
                    for (int v = 0; v < 8; v++)
                        __stcg(dst + v, make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                    __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3])));
                }
            } else if (p.split_k > 1) {
                // raw FP32 partial sums of this unit; ldp is a multiple of 32, so a started chunk is whole
                float *prow = p.partial + ((size_t)w.part * p.M + row) * p.ldp;
                constexpr int NCH = TILE_N / 32 / EpiCfg<LSTM || WIDE>::SETS;
                const int set = (warp - 2) >> 2;
#pragma unroll 1
                for (int c = set * NCH; c < (set + 1) * NCH; c++) {
                    uint32_t r[32];
                    tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N + c * 32), r);
                    tc_wait_ld();
                    const int col0 = w.nb * TILE_N + c * 32;
                    if (row_ok && col0 < p.ldp) {
                        float4 *dst = (float4 *)(prow + col0);
#pragma unroll
                        for (int v = 0; v < 8; v++)
                            __stcg(dst + v, make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                        __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3])));
                    }
                }
            } else if (!(LSTM || WIDE) && p.tma_store) {
                // Output through shared memory and tensor stores: each lane rounds its row's 64 values of a box
                // (32 rows x 64 columns) into the swizzled layout the tensor map expects, one lane sends the box
                // with one bulk tensor store - whole 128-byte lines instead of 16-byte pieces of 32 different
                // rows per instruction.  Two boxes per warp: the store of one is read out while the next fills.
                const int nbox = w.width / 64;
                const int row0 = w.mb * (2 * CTA_M) + (int)rank * CTA_M + q * 32;
                uint32_t acc_bits = 0;
#pragma unroll 1
                for (int bx = 0; bx < nbox; bx++, boxes_sent++) {
                    const uint32_t box = epi_stage + (uint32_t)(((warp - 2) * 2 + (boxes_sent & 1)) * EPI_BOX_BYTES);
                    if (lane == 0 && boxes_sent >= 2) bulk_wait_group_read<1>();     // the store before last has left this box
                    __syncwarp();
                    const int colb = w.nb * TILE_N + w.n_off + bx * 64;
                    epilogue_box_store(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N + bx * 64), box, &tmC, row0,
                                       colb, p.M, p.N, p.relu != 0, mrow, row_ok, acc_bits);
                }
                bad |= nonfinite_any(acc_bits);
            } else {
                const int set = (warp - 2) >> 2, nch = w.width / 32 / EpiCfg<LSTM || WIDE>::SETS;   // this set's share of the columns
#pragma unroll 1
                for (int c = set * nch; c < (set + 1) * nch; c++) {
                    uint32_t r[32];
                    tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N + c * 32), r);
                    tc_wait_ld();
                    const int col0 = w.nb * TILE_N + w.n_off + c * 32;
                    if (row_ok && col0 < p.N) epilogue_store32(r, crow, mrow, col0, p.N, p.relu != 0, bad);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_u32(acce_bar(buf), 0));
            if (p.nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(p.nonfinite_flag, 1u);
        }
        if (lane == 0) bulk_wait_group_read<0>();      // shared memory must outlive the tensor stores that read it
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

// Finishes the tiles of the split tail: C = epilogue(part 0 + part 1 + ...) with the parts added in
// ascending order (one rounding per add), eight columns per thread.
__global__ void __launch_bounds__(256) k_tail_reduce(const Params p, int first_tile, int n_tiles)
{
    pdl_trigger();
    pdl_wait();
    constexpr int TILE_ELEMS = 2 * CTA_M * TILE_N;
    const size_t total = (size_t)n_tiles * (2 * CTA_M) * (TILE_N / 8);
    bool bad = false;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int ti = (int)(i / ((2 * CTA_M) * (TILE_N / 8)));
        const int rem = (int)(i - (size_t)ti * ((2 * CTA_M) * (TILE_N / 8)));
        const int r = rem / (TILE_N / 8), g = rem - r * (TILE_N / 8);
        int mb, nb;
        tile_coords(p, first_tile + ti, mb, nb);
        const int row = mb * (2 * CTA_M) + r, col = nb * TILE_N + g * 8;
        if (row >= p.M || col >= p.N) continue;
        const float *src = p.tail_partial + (size_t)ti * p.tail_split * TILE_ELEMS + (size_t)r * TILE_N + g * 8;
        float4 a = __ldcg((const float4 *)src), b = __ldcg((const float4 *)(src + 4));
        for (int sp = 1; sp < p.tail_split; sp++) {
            const float *q = src + (size_t)sp * TILE_ELEMS;
            const float4 c = __ldcg((const float4 *)q), d = __ldcg((const float4 *)(q + 4));
            a.x = __fadd_rn(a.x, c.x); a.y = __fadd_rn(a.y, c.y); a.z = __fadd_rn(a.z, c.z); a.w = __fadd_rn(a.w, c.w);
            b.x = __fadd_rn(b.x, d.x); b.y = __fadd_rn(b.y, d.y); b.z = __fadd_rn(b.z, d.z); b.w = __fadd_rn(b.w, d.w);
        }
        const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        for (int e = 0; e < 8 && col + e < p.N; e++) {
            float s = v[e];
            if (p.relu) s = (s > 0.0f || s != s) ? s : 0.0f;
            uint32_t h = (uint32_t)__half_as_ushort(__float2half_rn(s));
            if (p.mask) {
                const uint32_t mh = p.mask[(size_t)row * p.ldmask + col + e];
                if (!((mh & 0x8000u) == 0 && mh != 0 && mh <= 0x7C00u)) h = 0;
            }
            bad |= (h & 0x7C00u) == 0x7C00u;
            p.C[(size_t)row * p.ldc + col + e] = (uint16_t)h;
        }
    }
    if (p.nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(p.nonfinite_flag, 1u);
}

template <bool A_MN, bool B_MN, bool LSTM = false, bool WIDE = false>
static cudaError_t launch_variant(const CUtensorMap &ta, const CUtensorMap &tb, const CUtensorMap &tbh, const CUtensorMap &tc,
                                  Params p, cudaStream_t st)
{
    static int max_pairs_dev[kMaxDevices] = {};     // 0 = this device not configured yet
    auto kern = k_gemm_tc2<A_MN, B_MN, LSTM, WIDE>;
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
    cfg.blockDim = dim3(EpiCfg<LSTM || WIDE>::THREADS, 1, 1);
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
    // every cluster takes tiles / pairs whole tiles; what is left over is cut into halves when all
    // halves fit into one round
    const int tiles = p.tiles_m * p.tiles_n;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    int full = (tiles / pairs) * pairs, rest = tiles - full;
    if (2 * tiles <= max_pairs) { full = 0; rest = tiles; }   // too few tiles for the clusters: halves all the way
    if (p.split_k > 1) {
        p.full_units = tiles * p.split_k;
        p.num_units = tiles * p.split_k;
    } else if (p.tail_split > 1 && tiles > max_pairs && rest > 0 && 2 * rest <= max_pairs) {
        // the launcher passed the scratch size in tail_split's place: units of 256x256 floats it holds
        const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;
        int split = max_pairs / rest;
        if (split > 8) split = 8;
        while (split > 1 && (nkb / split < 8 || (long)rest * split > (long)p.tail_split)) split--;
        // the reduce launch and the FP32 round trip cost about 10 us: worth it only when the split saves
        // at least 96 k-blocks of main loop in the last round (4096^3 lost 5 % with it, K = 12288 gains)
        if ((long)nkb * (split - 1) / split < 96) split = 1;
        p.tail_split = split;
        if (split > 1) {
            p.full_units = full;
            p.num_units = full + rest * split;
        } else {
            p.full_units = full;
            p.num_units = full + 2 * rest;
        }
    } else if (rest > 0 && 2 * rest <= max_pairs) {
        p.tail_split = 1;
        p.full_units = full;
        p.num_units = full + 2 * rest;
    } else {
        p.tail_split = 1;
        p.full_units = tiles;
        p.num_units = tiles;
    }
    const int grid_pairs = p.num_units < max_pairs ? p.num_units : max_pairs;
    cfg.gridDim = dim3(2 * grid_pairs, 1, 1);
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, ta, tb, tbh, tc, p);
    if (e != cudaSuccess || p.split_k > 1 || p.tail_split <= 1) return e;
    const size_t work = (size_t)rest * (2 * CTA_M) * (TILE_N / 8);
    size_t blocks = (work + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    MPT_LAUNCH(k_tail_reduce, dim3((unsigned)blocks), dim3(256), 0, st, p, full, rest);
    g_last_gemm_launches = 2;
    return cudaGetLastError();
}

}  // namespace pair

bool tc2_gemm_preferred(int M, int N, int K)
{
    // Measured on B200 with launches replayed from a CUDA graph.  When all tiles run in one round either
    // way (at most 74 tiles of 256x256 = 148 of 128x256) both kernels spend the same time per k-block
    // (0.32 us) and the single-CTA kernel starts and ends about 1.7 us sooner (no cluster to place, no
    // paired allocation): 2048^3 16.4 against 18.2 us, 2048x2048x4096 26.7 against 28.3, 72 tiles with
    // K = 2048 18.8 against 19.3.  With more tiles than that the pair kernel wins (4096^3 100 against
    // 116 us: a third fewer operand bytes from L2, epilogues hidden behind the next tile).
    const long tiles = (long)((M + 255) / 256) * ((N + 255) / 256);
    const long nkb = (K + 63) / 64;
    return M >= 256 && N >= 256 && (tiles > 74 || (tiles >= 48 && nkb >= 256));
}

// Scratch the pair kernel would like for the split tail of a large product: one 256x256 FP32 block
// per unit of the last round (at most 74), when the tiles do not fill the last round.
size_t tc2_tail_ws_bytes(int M, int N, int K)
{
    const long tiles = (long)((M + 255) / 256) * ((N + 255) / 256);
    const int nkb = (K + pair::BLOCK_K - 1) / pair::BLOCK_K;
    if (tiles <= 74 || nkb < 16) return 0;
    const long rest = tiles % 74;
    if (rest == 0 || 2 * rest > 74) return 0;
    long split = 74 / rest;
    if (split > 8) split = 8;
    while (split > 1 && nkb / split < 8) split--;
    if ((long)nkb * (split - 1) / split < 96) split = 1;      // same rule as the launcher
    return split > 1 ? (size_t)(rest * split) * 256 * 256 * sizeof(float) : 0;
}

// Split factor for the pair kernel on outputs with few 256x256 tiles and a long contraction.
// Cost model in tensor-pipe cycles, same units as tc_gemm_plan: 512 cycles per 64-deep k-block of a
// pair tile, the exposed epilogue of the last unit, a launch, and for a split the reduce launch
// and the FP32 parts going to L2 and back (about 64 bytes per cycle and SM).  A part keeps at
// least 16 k-blocks; all units fit in one round of the 74 clusters.  Measured (graph replay):
// 2048x1024x8192 39-40 us split in two against 45 us as 64 half tiles; level with the single-CTA
// kernel's split there and a little behind it on 1024x1024x4096, hence the extra constant.  A
// variant in which the unit of a tile that finishes last adds the parts itself (no second launch)
// was slower: one warp per 32 rows cannot keep enough loads in flight (47-60 us).
void tc2_split_plan(int M, int N, int K, size_t ws_bytes, int *split_out, size_t *ws_needed, double *cost_out)
{
    const long tiles = (long)((M + 255) / 256) * ((N + 255) / 256);
    const int nkb = (K + pair::BLOCK_K - 1) / pair::BLOCK_K;
    const size_t ldp = ((size_t)N + 31) / 32 * 32;
    double best = 1e30;
    int best_s = 1;
    for (int s = 1; s <= 8; s++) {
        if (s > 1 && (nkb / s < 16 || tiles * s > 74)) break;
        const size_t need = s > 1 ? (size_t)s * M * ldp * 4 : 0;
        if (need > ws_bytes) break;
        const long rounds = (tiles * s + 73) / 74;
        double cost = rounds * ((double)nkb / s) * 512.0 + 8 * 400.0 + 14000.0;
        if (s > 1) cost += 8000.0 + (double)need * 2.0 / 148.0 / 64.0;    // cluster launch + second launch + partial traffic
        if (cost < best * 0.99) { best = cost; best_s = s; }
    }
    *split_out = best_s;
    if (ws_needed) *ws_needed = best_s > 1 ? (size_t)best_s * M * ldp * 4 : 0;
    if (cost_out) *cost_out = best;
}

cudaError_t launch_gemm_tc2(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag,
                            uint32_t *status, cudaStream_t st, const LstmEpi *lstm, void *splitk_ws, size_t splitk_ws_bytes)
{
    using namespace pair;
    g_last_gemm_launches = 1;
    CUtensorMap ta, tb, tbh;
    bool ok;
    if (op == MPT_OP_WGRAD) ok = tc_encode_map(&ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, 64, BLOCK_K);
    else ok = tc_encode_map(&ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BLOCK_K, CTA_M);
    if (op == MPT_OP_FWD) {
        // K-major B: one box of 128 rows per CTA for whole tiles, of 64 rows for half tiles
        ok = ok && tc_encode_map(&tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BLOCK_K, CTA_N);
        ok = ok && tc_encode_map(&tbh, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BLOCK_K, CTA_N / 2);
    } else {
        ok = ok && tc_encode_map(&tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, 64, BLOCK_K);
        tbh = tb;
    }
    CUtensorMap tcm;      // the output, in boxes of 32 rows x 64 columns
    ok = ok && tc_encode_map(&tcm, C, (uint64_t)M, (uint64_t)N, (uint64_t)ldc, 64, 32);
    if (!ok) return cudaErrorInvalidValue;
    Params p;
    p.M = M; p.N = N; p.K = K;
    p.C = C; p.ldc = ldc;
    // tensor stores of the output: whole groups of 8 columns only (the mask and the inf/NaN vote work on such groups);
    // MPT_TMA_STORE=0 selects the per-lane 16-byte stores for comparisons
    { const char *x = getenv("MPT_TMA_STORE"); p.tma_store = (N % 8 == 0) && (x ? atoi(x) != 0 : true); }
    p.mask = mask; p.ldmask = ldmask;
    p.relu = relu ? 1 : 0;
    p.nonfinite_flag = nonfinite_flag;
    p.status = status;
    p.tiles_m = (M + 2 * CTA_M - 1) / (2 * CTA_M);
    p.tiles_n = (N + TILE_N - 1) / TILE_N;
    // Row blocks per group of the tile order.  Consecutive waves of a group share its A panels; whether
    // those survive in L2 between waves depends on their size: with the short panels of a weight-gradient
    // product (K = batch = 4096: 2 MB each) 16 of them do, and DRAM reads of 12288x12288x4096 fall from
    // 1.01 GB (groups of 8) to 0.66 GB (0.77 / 0.82 / 1.00 / 1.57 GB with 12 / 24 / 32 / 4).  With long
    // panels nothing survives a wave, and 8 keeps the wave's own footprint smallest - unless the output has
    // no more than 16 row blocks: one group then spans all of M and no B panel is ever asked for twice
    // (4096x32000x12288: 5.6 -> 4.5 GB and 2.45 -> 2.30 ms; 4096x12288x32000: 6.5 -> 5.7 GB; the
    // large-MLP step 0.6 % faster).
    p.group_m = (K <= 6144 || p.tiles_m <= 16) ? 16 : 8;
    {
        // both operands "evict last" (see tma_load_2d_pair_hint); MPT_L2_HINT=<A digit><B digit> overrides for
        // comparisons: 0 normal, 1 evict last, 2 evict first
        const char *e = getenv("MPT_L2_HINT");
        p.hint_a = e && e[0] ? e[0] - '0' : 1;
        p.hint_b = e && e[0] && e[1] ? e[1] - '0' : 1;
    }
    p.full_units = p.num_units = 0;
    p.split_k = 1;
    p.partial = nullptr;
    p.ldp = (N + 31) / 32 * 32;
    p.tail_split = 1;
    p.tail_partial = nullptr;
    if (!lstm && splitk_ws && (((uintptr_t)splitk_ws) & 15) == 0) {
        int split = 1;
        tc2_split_plan(M, N, K, splitk_ws_bytes, &split, nullptr, nullptr);
        if (split > 1) {
            p.split_k = split;
            p.partial = (float *)splitk_ws;
        } else {
            // scratch for the split tail: launch_variant turns the capacity (in 256x256 FP32 blocks) into a split
            const size_t blocks = splitk_ws_bytes / ((size_t)2 * CTA_M * TILE_N * sizeof(float));
            if (blocks >= 2) {
                p.tail_split = (int)(blocks > 1024 ? 1024 : blocks);
                p.tail_partial = (float *)splitk_ws;
            }
        }
    }
    p.lstm = LstmEpi{};
    if (lstm) {
        if (op != MPT_OP_FWD || (N & 31) != 0) return cudaErrorInvalidValue;
        p.lstm = *lstm;
        return launch_variant<false, false, true>(ta, tb, tbh, tcm, p, st);
    }
    // two epilogue warp sets when a cluster's whole main loop is short (see EpiCfg)
    const long units = (long)p.tiles_m * p.tiles_n * p.split_k;
    const long kblocks = ((units + 73) / 74) * ((K + BLOCK_K - 1) / BLOCK_K / p.split_k);
    const bool wide = kblocks <= 160;
    cudaError_t e;
    if (op == MPT_OP_FWD) e = wide ? launch_variant<false, false, false, true>(ta, tb, tbh, tcm, p, st) : launch_variant<false, false>(ta, tb, tbh, tcm, p, st);
    else if (op == MPT_OP_DGRAD) e = wide ? launch_variant<false, true, false, true>(ta, tb, tbh, tcm, p, st) : launch_variant<false, true>(ta, tb, tbh, tcm, p, st);
    else e = wide ? launch_variant<true, true, false, true>(ta, tb, tbh, tcm, p, st) : launch_variant<true, true>(ta, tb, tbh, tcm, p, st);
    if (e != cudaSuccess || p.split_k == 1) return e;
    return launch_splitk_reduce(p.partial, p.split_k, M, N, p.ldp, C, ldc, relu, mask, ldmask, nonfinite_flag, st);
}

}  // namespace mpt
