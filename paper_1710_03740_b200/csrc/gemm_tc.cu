// Tensor-core FP16 GEMM for sm_100a (paper section 3.3: FP16 operands, FP32
// accumulation, FP16 on the store), with the point-wise work fused into the
// epilogue (ReLU, the ReLU-derivative mask of the backward pass, and the inf/NaN
// inspection of weight gradients of section 3.2).
//
// Structure: persistent kernel, one CTA per SM, 192 threads in three roles
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 128x64 (A) and 256x64 (B)
//               FP16 tiles into a 4-stage shared-memory ring (128-byte swizzle)
//   warp 1      MMA issuer: tcgen05.mma.kind::f16, 128x256x16 per instruction,
//               FP32 accumulators in tensor memory (2 x 256 columns, double buffered)
//   warps 2..5  epilogue: tcgen05.ld the accumulator, ReLU / mask / round to FP16 /
//               inspect, 128-bit stores to C
// Operand layouts are taken as stored (no transposed copies): a "K-major" operand has
// the contraction index contiguous, an "MN-major" operand has the output index
// contiguous; the forward product is K x K, dgrad is K x MN, wgrad is MN x MN.
// Ragged M, N, K are handled by TMA zero fill on loads and by predicated stores.
//
// Every wait on an mbarrier is bounded: after ~2 s the waiting role records an error
// word, raises a CTA-wide abort flag and all roles fall through to the common exit,
// which frees the tensor memory.
#include <cuda.h>

#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

static constexpr int BLOCK_M = 128, BLOCK_K = 64, UMMA_K = 16;
static constexpr int A_STAGE_BYTES = BLOCK_M * BLOCK_K * 2;  // 16 KB
static constexpr int MN_BOX_BYTES = 64 * BLOCK_K * 2;        // one 64(mn) x 64(k) box of an MN-major operand

// Tile width BN is 256 (four 48 KB stages) or, for outputs with too few 128x256 tiles to fill
// the SMs, 128 (six 32 KB stages) or 64 (eight 24 KB stages).  The two accumulator buffers take 2 * BN tensor-memory columns.
template <int BN>
struct TileCfg {
    static constexpr int B_STAGE_BYTES = BN * BLOCK_K * 2;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// Instruction descriptor, kind::f16: D = F32, A = B = F16, majors, N >> 3, M >> 4.
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn, int bn)
{
    return (1u << 4) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(bn >> 3) << 17) |
           ((uint32_t)(BLOCK_M >> 4) << 24);
}

struct TcParams {
    int M, N, K;
    uint16_t *C;
    int ldc;
    const uint16_t *mask;
    int ldmask;
    int relu;
    uint32_t *nonfinite_flag;
    uint32_t *status;  // may be null
    int tiles_m, tiles_n, group_m;
    // split-K: the contraction range of every tile is cut into split_k parts, each part is a
    // work unit that leaves its raw FP32 accumulator in `partial` [split_k][M][ldp]; a second
    // kernel adds the parts in a fixed order and applies the epilogue.  split_k == 1: off.
    int split_k;
    float *partial;
    int ldp;
    LstmEpi lstm;   // read only by the LSTM instantiations of the kernel
};

__device__ __forceinline__ void tile_coords(const TcParams &p, int tile, int &mb, int &nb)
{
    // groups of group_m row-blocks, row-block fastest inside a group: concurrently
    // running CTAs share B tiles and a bounded set of A tiles in L2
    int per_group = p.group_m * p.tiles_n;
    int g = tile / per_group;
    int first_m = g * p.group_m;
    int gsz = min(p.group_m, p.tiles_m - first_m);
    int r = tile - g * per_group;
    mb = first_m + r % gsz;
    nb = r / gsz;
}

__device__ __forceinline__ void report(const TcParams &p, volatile uint32_t *abort_flag, uint32_t code)
{
    *abort_flag = 1u;
    if (p.status) atomicCAS(p.status, 0u, code | ((uint32_t)blockIdx.x << 8));
}

// Epilogue width: one set of four warps, or two sets that each take half of the columns of a tile
// (launch-bound products and the LSTM gate epilogue; see the CTA-pair kernel for the measurements).
template <bool WIDE>
struct EpiCfg {
    static constexpr int SETS = WIDE ? 2 : 1;
    static constexpr int THREADS = 64 + 128 * SETS;
};

template <bool A_MN, bool B_MN, int BLOCK_N, bool LSTM = false, bool WIDE = false>
__global__ void __launch_bounds__(EpiCfg<LSTM || WIDE>::THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcParams p)
{
    pdl_trigger();
    if (threadIdx.x == 32) { prefetch_tensormap(&tmA); prefetch_tensormap(&tmB); }
    constexpr int STAGES = TileCfg<BLOCK_N>::STAGES;
    constexpr int STAGE_BYTES = TileCfg<BLOCK_N>::STAGE_BYTES;
    constexpr int TMEM_COLS = TileCfg<BLOCK_N>::TMEM_COLS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzled tiles need 1024-byte alignment
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + STAGES * STAGE_BYTES;
    // barrier words: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], then tmem slot + abort flag
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(base_ptr + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int num_units = num_tiles * p.split_k;   // unit u: tile u % num_tiles, contraction part u / num_tiles
    const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;
    // k-block range of contraction part `part` (32-bit arithmetic: nkb * split_k is far below 2^31)
    auto kb_begin = [&](int part) { return p.split_k == 1 ? part * nkb : (int)((unsigned)(nkb * part) / (unsigned)p.split_k); };
    auto unit_tile = [&](int u) { return p.split_k == 1 ? u : u % num_tiles; };
    auto unit_part = [&](int u) { return p.split_k == 1 ? 0 : u / num_tiles; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; b++) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4 * EpiCfg<LSTM || WIDE>::SETS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();      // everything above ran beside the tail of the preceding kernel; global memory is touched below

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t issued = 0, s = 0, ph = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
                int mb, nb;
                tile_coords(p, unit_tile(u), mb, nb);
                const int part = unit_part(u), kb1 = kb_begin(part + 1);
                const int m0 = mb * BLOCK_M, n0 = nb * BLOCK_N;
                for (int kb = kb_begin(part); kb < kb1; kb++, issued++, s = (s + 1 == STAGES) ? 0 : s + 1, ph ^= (s == 0)) {
                    if (!mbar_try_wait(empty_bar(s), ph ^ 1u) && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        if (!*abort_flag) report(p, abort_flag, KERR_WAIT_EMPTY);
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    mbar_arrive_expect_tx(full_bar(s), STAGE_BYTES);
                    const int k0 = kb * BLOCK_K;
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < BLOCK_M / 64; j++) tma_load_2d(sa + j * MN_BOX_BYTES, &tmA, m0 + 64 * j, k0, full_bar(s));
                    } else {
                        tma_load_2d(sa, &tmA, k0, m0, full_bar(s));
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < BLOCK_N / 64; j++) tma_load_2d(sb + j * MN_BOX_BYTES, &tmB, n0 + 64 * j, k0, full_bar(s));
                    } else {
                        tma_load_2d(sb, &tmB, k0, n0, full_bar(s));
                    }
                }
            }
            if (!ok) {
                // let the copies already in flight land before the CTA exits (bounded)
                uint32_t first = issued > (uint32_t)STAGES ? issued - STAGES : 0;
                for (uint32_t i = first; i < issued; i++) {
                    unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_bar(i % STAGES), (i / STAGES) & 1u) && global_ns() - t0 < 1000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(A_MN, B_MN, BLOCK_N);
            // descriptor halves: only the start address (low word) changes with stage and k.
            // K-major: 16 k = 32 bytes along the swizzled row; MN-major: 16 k-rows of 128 bytes.
            constexpr uint32_t KSTEP_A = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            constexpr uint32_t KSTEP_B = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
            const uint32_t a_hi = desc_hi(1024), b_hi = desc_hi(1024);
            const uint32_t a_lo0 = desc_lo(base, A_MN ? MN_BOX_BYTES : 16);
            const uint32_t b_lo0 = desc_lo(base + A_STAGE_BYTES, B_MN ? MN_BOX_BYTES : 16);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int t = 0;
            for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x, t++) {
                const int part = unit_part(u), kb0 = kb_begin(part), kb1 = kb_begin(part + 1);
                const int buf = t & 1;
                const uint32_t acc_ph = (t >> 1) & 1u;
                if (!mbar_try_wait(acce_bar(buf), acc_ph ^ 1u) && !mbar_wait(acce_bar(buf), acc_ph ^ 1u, abort_flag)) {
                    if (!*abort_flag) report(p, abort_flag, KERR_WAIT_ACC_FREE);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BLOCK_N);
                uint32_t acc = 0;                       // first MMA of a unit overwrites the accumulator
                for (int kb = kb0; kb < kb1; kb++) {
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
                        tc_mma_f16(d_tmem, desc_join(alo + k * KSTEP_A, a_hi), desc_join(blo + k * KSTEP_B, b_hi), idesc, acc);
                        acc = 1;
                    }
                    tc_commit(empty_bar(s));       // frees the stage when these MMAs have read it
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(accf_bar(buf));  // accumulator complete
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int q = warp & 3;                    // TMEM lane quadrant this warp may access
        bool ok = true;
        int t = 0;
        for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x, t++) {
            int mb, nb;
            tile_coords(p, unit_tile(u), mb, nb);
            const int part = unit_part(u);
            const int buf = t & 1;
            const uint32_t acc_ph = (t >> 1) & 1u;
            if (!mbar_wait(accf_bar(buf), acc_ph, abort_flag)) {
                if (!*abort_flag && lane == 0) report(p, abort_flag, KERR_WAIT_ACC);
                ok = false;
                break;
            }
            tc_fence_after();
            const int row = mb * BLOCK_M + q * 32 + lane;
            const bool row_ok = row < p.M;
            uint16_t *crow = p.C + (size_t)row * p.ldc;
            const uint16_t *mrow = p.mask ? p.mask + (size_t)row * p.ldmask : nullptr;
            bool bad = false;
            if constexpr (LSTM) {
                const int set = (warp - 2) >> 2;
                constexpr int NCH = BLOCK_N / 64;                          // this set's half of the tile's columns
                epilogue_lstm_tile(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BLOCK_N + set * NCH * 32), NCH,
                                   nb * BLOCK_N + set * NCH * 32, p.N, row, row_ok, crow, p.lstm);
            } else {
                // two register sets: the tensor-memory load of the next 32 columns is in flight while the
                // current ones are rounded and stored
                constexpr int NCHW = BLOCK_N / 32 / EpiCfg<LSTM || WIDE>::SETS;
                const int c_begin = ((warp - 2) >> 2) * NCHW, c_end = c_begin + NCHW;
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BLOCK_N);
                auto finish = [&](const uint32_t (&r)[32], int c) {
                    const int col0 = nb * BLOCK_N + c * 32;
                    if (p.split_k > 1) {
                        // raw FP32 partial sums; ldp is a multiple of 32, so a started chunk is always whole
                        if (row_ok && col0 < p.ldp) {
                            float4 *dst = (float4 *)(p.partial + ((size_t)part * p.M + row) * p.ldp + col0);
#pragma unroll
                            for (int v = 0; v < 8; v++)
                                dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                     __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                        }
                    } else if (row_ok && col0 < p.N) {
                        epilogue_store32(r, crow, mrow, col0, p.N, p.relu != 0, bad);
                    }
                };
                uint32_t ra[32], rb[32];
                tc_ld32(t_row + (uint32_t)(c_begin * 32), ra);
#pragma unroll 1
                for (int c = c_begin; c < c_end; c += 2) {
                    tc_wait_ld();
                    if (c + 1 < c_end) tc_ld32(t_row + (uint32_t)((c + 1) * 32), rb);
                    finish(ra, c);
                    if (c + 1 < c_end) {
                        tc_wait_ld();
                        if (c + 2 < c_end) tc_ld32(t_row + (uint32_t)((c + 2) * 32), ra);
                        finish(rb, c + 1);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));
            if (p.nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(p.nonfinite_flag, 1u);
        }
    }

    // common exit: every role gets here (all waits are bounded)
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// Second step of a split-K product: C = epilogue(partial[0] + partial[1] + ... ) with the parts
// added in ascending order (FP32, one rounding per add), eight columns per thread.
__global__ void __launch_bounds__(256) k_splitk_reduce(const float *__restrict__ partial, int split_k, int M, int N,
                                                       int ldp, uint16_t *__restrict__ C, int ldc, int relu,
                                                       const uint16_t *__restrict__ mask, int ldmask,
                                                       uint32_t *nonfinite_flag)
{
    pdl_trigger();
    pdl_wait();
    const int groups = (N + 7) / 8;
    const size_t total = (size_t)M * groups;
    bool bad = false;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int row = (int)(i / groups), col = (int)(i % groups) * 8;
        const float *src = partial + (size_t)row * ldp + col;
        float4 a = *(const float4 *)src, b = *(const float4 *)(src + 4);
        for (int sp = 1; sp < split_k; sp++) {
            const float *q = src + (size_t)sp * M * ldp;
            const float4 c = *(const float4 *)q, d = *(const float4 *)(q + 4);
            a.x += c.x; a.y += c.y; a.z += c.z; a.w += c.w;
            b.x += d.x; b.y += d.y; b.z += d.z; b.w += d.w;
        }
        const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        for (int e = 0; e < 8 && col + e < N; e++) {
            float s = v[e];
            if (relu) s = (s > 0.0f || s != s) ? s : 0.0f;
            uint32_t h = (uint32_t)__half_as_ushort(__float2half_rn(s));
            if (mask) {
                const uint32_t mh = mask[(size_t)row * ldmask + col + e];
                if (!((mh & 0x8000u) == 0 && mh != 0 && mh <= 0x7C00u)) h = 0;
            }
            bad |= (h & 0x7C00u) == 0x7C00u;
            C[(size_t)row * ldc + col + e] = (uint16_t)h;
        }
    }
    if (nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(nonfinite_flag, 1u);
}

thread_local int g_last_gemm_launches = 1;

cudaError_t launch_splitk_reduce(const float *partial, int split_k, int M, int N, int ldp, uint16_t *C, int ldc, bool relu,
                                 const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag, cudaStream_t st)
{
    const size_t work = (size_t)M * ((N + 7) / 8);
    size_t blocks = (work + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    MPT_LAUNCH(k_splitk_reduce, dim3((unsigned)blocks), dim3(256), 0, st, partial, split_k, M, N, ldp, C, ldc, relu ? 1 : 0, mask, ldmask,
               nonfinite_flag);
    g_last_gemm_launches = 2;
    return cudaGetLastError();
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    }
    return fn;
}

// 2-D FP16 tensor map over a row-major matrix [rows, cols] with pitch ld (elements);
// box = box_cols x box_rows, 128-byte swizzle, zero fill outside the matrix.
bool tc_encode_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                       uint32_t box_rows)
{
    EncodeTiledFn fn = get_encode();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool tc_gemm_supported(int op, int M, int N, int K, const void *A, int lda, const void *B, int ldb, const void *C,
                       int ldc, const void *mask, int ldmask)
{
    (void)op;
    if (M <= 0 || N <= 0 || K <= 0) return false;
    uintptr_t bits = (uintptr_t)A | (uintptr_t)B | (uintptr_t)C | (uintptr_t)mask;
    if (bits & 15) return false;
    if ((lda % 8) || (ldb % 8) || (ldc % 8) || (mask && (ldmask % 8))) return false;
    return true;
}

template <bool A_MN, bool B_MN, int BN, bool LSTM = false, bool WIDE = false>
static cudaError_t launch_variant(const CUtensorMap &ta, const CUtensorMap &tb, const TcParams &p, int grid,
                                  cudaStream_t st)
{
    static bool configured[kMaxDevices] = {};
    constexpr int SMEM_BYTES = TileCfg<BN>::SMEM_BYTES;
    auto kern = k_gemm_tc<A_MN, B_MN, BN, LSTM, WIDE>;
    const int dev = current_device_slot();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    MPT_LAUNCH(kern, dim3(grid), dim3(EpiCfg<LSTM || WIDE>::THREADS), SMEM_BYTES, st, ta, tb, p);
    return cudaGetLastError();
}

template <int BN>
static cudaError_t launch_bn(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                             TcParams p, cudaStream_t st)
{
    CUtensorMap ta, tb;
    bool ok;
    // A: stored [M,K] (K-major) for fwd/dgrad, stored [K,M] (MN-major) for wgrad
    if (op == MPT_OP_WGRAD) ok = tc_encode_map(&ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, 64, BLOCK_K);
    else ok = tc_encode_map(&ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BLOCK_K, BLOCK_M);
    // B: stored [N,K] (K-major) for fwd, stored [K,N] (MN-major) for dgrad/wgrad
    if (op == MPT_OP_FWD) ok = ok && tc_encode_map(&tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BLOCK_K, BN);
    else ok = ok && tc_encode_map(&tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, 64, BLOCK_K);
    if (!ok) return cudaErrorInvalidValue;
    p.tiles_m = (M + BLOCK_M - 1) / BLOCK_M;
    p.tiles_n = (N + BN - 1) / BN;
    p.group_m = 16;
    int units = p.tiles_m * p.tiles_n * p.split_k;
    int grid = units < 148 ? units : 148;
    cudaError_t e;
    // two epilogue warp sets when a CTA's whole main loop is short (see EpiCfg)
    const long kblocks = ((long)(units + 147) / 148) * ((K + BLOCK_K - 1) / BLOCK_K / p.split_k);
    const bool wide = kblocks <= 160;
    if (op == MPT_OP_FWD && p.lstm.c_out) e = launch_variant<false, false, BN, true>(ta, tb, p, grid, st);
    else if (op == MPT_OP_FWD) e = wide ? launch_variant<false, false, BN, false, true>(ta, tb, p, grid, st) : launch_variant<false, false, BN>(ta, tb, p, grid, st);
    else if (op == MPT_OP_DGRAD) e = wide ? launch_variant<false, true, BN, false, true>(ta, tb, p, grid, st) : launch_variant<false, true, BN>(ta, tb, p, grid, st);
    else e = wide ? launch_variant<true, true, BN, false, true>(ta, tb, p, grid, st) : launch_variant<true, true, BN>(ta, tb, p, grid, st);
    if (e != cudaSuccess || p.split_k == 1) return e;
    return launch_splitk_reduce(p.partial, p.split_k, M, N, p.ldp, p.C, p.ldc, p.relu != 0, p.mask, p.ldmask, p.nonfinite_flag, st);
}

// Tile width and split factor for the single-CTA kernel.  Cost model in tensor-pipe cycles: a
// 128x256 tile needs 512 cycles per 64-deep k-block; a 128x128 tile needs 256 but runs at about
// 0.6 of that rate (operand reads from shared memory bound it); measured per k-block: about 600
// and 437 cycles; a 128x64 tile takes as long as a 128x128 one per k-block (about 450: the A
// operand's shared-memory reads do not shrink with the tile), so it only pays when it fills more
// SMs or saves the second launch of a split.  The epilogue of a tile costs about 400 cycles per 32 columns and is exposed
// for the last tile of a CTA; a launch costs about 14000 cycles; a split adds a second, mostly
// overlapped launch (about 4000) and one FP32 write and read of the output per part, which
// stays in L2 (about 64 bytes per cycle and SM).  Calibrated with launches replayed from a CUDA
// graph on 2048x1024x8192, 1024x1024x4096, 512x256x4096 and the tiny-MLP products.  The split
// is only considered when a workspace is available.
void tc_gemm_plan(int M, int N, int K, size_t ws_bytes, int *bn_out, int *split_out, size_t *ws_needed, double *cost_out)
{
    const long tm = (M + BLOCK_M - 1) / BLOCK_M;
    const int nkb = (K + BLOCK_K - 1) / BLOCK_K;
    double best = 1e30;
    int best_bn = 256, best_s = 1;
    for (int bn : {256, 128, 64}) {
        if (bn < 256 && N <= bn) continue;
        const long tiles = tm * ((N + bn - 1) / bn);
        const double cyc = bn == 256 ? 600.0 : (bn == 128 ? 437.0 : 450.0);
        for (int s = 1; s <= 8; s++) {
            if (s > 1 && (nkb / s < 8)) break;
            const size_t need = s > 1 ? (size_t)s * M * (((size_t)N + 31) / 32 * 32) * 4 : 0;
            if (need > ws_bytes) break;
            const long rounds = (tiles * s + 147) / 148;
            double cost = rounds * ((double)nkb / s) * cyc + (bn / 32) * 400.0 + 14000.0;   // + exposed epilogue + launch
            if (s > 1) cost += 4000.0 + (double)need * 2.0 / 148.0 / 64.0;                  // second launch + partial traffic
            if (cost < best * 0.99) { best = cost; best_bn = bn; best_s = s; }
        }
    }
    *bn_out = best_bn;
    *split_out = best_s;
    if (ws_needed) *ws_needed = best_s > 1 ? (size_t)best_s * M * (((size_t)N + 31) / 32 * 32) * 4 : 0;
    if (cost_out) *cost_out = best;
}

bool tc_choose_pair(int M, int N, int K, size_t ws_bytes, size_t *ws_needed)
{
    if (ws_needed) *ws_needed = 0;
    if (tc2_gemm_preferred(M, N, K)) {
        if (ws_needed) *ws_needed = tc2_tail_ws_bytes(M, N, K);     // scratch for the split tail of the last round
        return true;
    }
    int bn, s1, s2;
    size_t need1 = 0, need2 = 0;
    double c1 = 0.0, c2 = 0.0;
    tc_gemm_plan(M, N, K, ws_bytes, &bn, &s1, &need1, &c1);
    if (M >= 256 && N >= 256) {
        tc2_split_plan(M, N, K, ws_bytes, &s2, &need2, &c2);
        if (s2 > 1 && c2 < c1) {
            if (ws_needed) *ws_needed = need2;
            return true;
        }
    }
    if (ws_needed) *ws_needed = need1;
    return false;
}

cudaError_t launch_gemm_tc(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                           uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag,
                           uint32_t *status, cudaStream_t st, float *splitk_ws, size_t splitk_ws_bytes, const LstmEpi *lstm)
{
    g_last_gemm_launches = 1;
    TcParams p;
    p.lstm = LstmEpi{};
    if (lstm) {   // gate epilogue: forward products only, never split (the epilogue needs the whole sum)
        if (op != MPT_OP_FWD || (N & 31) != 0) return cudaErrorInvalidValue;
        p.lstm = *lstm;
        splitk_ws = nullptr;
    }
    p.M = M; p.N = N; p.K = K;
    p.C = C; p.ldc = ldc;
    p.mask = mask; p.ldmask = ldmask;
    p.relu = relu ? 1 : 0;
    p.nonfinite_flag = nonfinite_flag;
    p.status = status;
    int bn = 256, split = 1;
    tc_gemm_plan(M, N, K, (splitk_ws && (((uintptr_t)splitk_ws) & 15) == 0) ? splitk_ws_bytes : 0, &bn, &split, nullptr);
    p.split_k = split;
    p.partial = splitk_ws;
    p.ldp = (N + 31) / 32 * 32;
    if (bn == 64 && !lstm) return launch_bn<64>(op, M, N, K, A, lda, B, ldb, p, st);
    if (bn <= 128) return launch_bn<128>(op, M, N, K, A, lda, B, ldb, p, st);
    return launch_bn<256>(op, M, N, K, A, lda, B, ldb, p, st);
}

}  // namespace mpt
