// Inline-PTX wrappers shared by the tensor-core GEMM kernels: mbarrier, TMA tensor loads,
// tcgen05 (MMA, commit, tensor-memory loads, fences) and the shared-memory matrix descriptor.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "mpt_common.cuh"

namespace mpt {

static constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

// Host: 2-D FP16 tensor map over a row-major matrix [rows, cols] with pitch ld (elements);
// box = box_cols x box_rows, 128-byte swizzle, zero fill outside the matrix.
bool tc_encode_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                   uint32_t box_rows);

// ----------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the CTA is aborting or the time limit expired.  The limit is
// an argument (default 2 s) so that a self-test can make a wait run out within a millisecond.
static __device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                              unsigned long long limit_ns = WAIT_LIMIT_NS)
{
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 127u) == 127u) {
            if (*abort_flag) return false;
            unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}

// Starts the fetch of a tensor map (a kernel parameter) into the TMA unit's descriptor cache, so that the
// first tensor load does not wait for it.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
#ifndef MPT_NO_TMAP_PREFETCH
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
#endif
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (tcgen05): start address, leading/stride byte
// offsets (all >> 4), descriptor version 1, 128-byte swizzle.
//   K-major  operand: rows of 128 bytes (64 k), 8-row groups 1024 bytes apart (stride offset);
//                     the leading offset is unused with swizzling.
//   MN-major operand: 64 k-rows of 128 bytes (64 mn) per box, 8-k groups 1024 bytes apart
//                     (stride offset), the next 64 mn one box (8192 bytes) further (leading offset).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

// The same descriptor split into its 32-bit halves: the low word holds the start address and
// the leading offset (advancing the address is a 32-bit add), the high word is constant.
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes)
{
    return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint32_t desc_hi(uint32_t sbo_bytes)
{
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ uint64_t desc_join(uint32_t lo, uint32_t hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}

// Rounds 32 FP32 sums to 16 words of two FP16 values each (element 2i in the low half), with the
// optional ReLU fused into the conversion: cvt.rn.relu turns a negative result into +0 and keeps NaN,
// which equals x > 0 ? x : +0 on the FP32 sum followed by the rounding (rounding is monotonic and
// keeps the sign).  One instruction per two elements.
__device__ __forceinline__ void round_pack32(const uint32_t (&r)[32], bool relu, uint32_t (&w)[16])
{
    if (relu) {
#pragma unroll
        for (int i = 0; i < 16; i++)
            asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(__uint_as_float(r[2 * i + 1])), "f"(__uint_as_float(r[2 * i])));
    } else {
#pragma unroll
        for (int i = 0; i < 16; i++)
            asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(__uint_as_float(r[2 * i + 1])), "f"(__uint_as_float(r[2 * i])));
    }
}
// ReLU-derivative mask on a word of two FP16 results: keep a half where the stored FP16 activation
// in the same half of mw is > 0 (sign clear, non-zero, not NaN).
__device__ __forceinline__ uint32_t mask_pair(uint32_t w, uint32_t mw)
{
    const uint32_t lo = mw & 0xFFFFu, hi = mw >> 16;
    if (!(lo != 0 && lo <= 0x7C00u)) w &= 0xFFFF0000u;
    if (!(hi != 0 && hi <= 0x7C00u)) w &= 0x0000FFFFu;
    return w;
}
// inf/NaN vote on words of two FP16 values: adding 0x0400 to an exponent field carries into bit 15
// of its half exactly when the field is all ones; acc collects the carries (test acc & 0x80008000).
__device__ __forceinline__ void nonfinite_acc(uint32_t w, uint32_t &acc) { acc |= (w & 0x7C007C00u) + 0x04000400u; }
__device__ __forceinline__ bool nonfinite_any(uint32_t acc) { return (acc & 0x80008000u) != 0; }

// Epilogue of one thread for 32 consecutive accumulator columns of its output row:
// optional ReLU on the FP32 sum, round to FP16, optional ReLU-derivative mask taken from a
// stored FP16 activation (keep where it is > 0), inf/NaN vote, 128-bit stores where the
// whole group of 8 lies inside the row, element stores on the ragged edge.
__device__ __forceinline__ void epilogue_store32(const uint32_t (&r)[32], uint16_t *crow, const uint16_t *mrow, int col0,
                                                 int N, bool relu, bool &bad)
{
    uint32_t w[16], acc = 0;
    round_pack32(r, relu, w);
#pragma unroll
    for (int g8 = 0; g8 < 4; g8++) {
        const int col = col0 + g8 * 8;
        if (col + 8 <= N) {
            if (mrow) {
                const uint4 mk = *(const uint4 *)(mrow + col);
                w[4 * g8] = mask_pair(w[4 * g8], mk.x);
                w[4 * g8 + 1] = mask_pair(w[4 * g8 + 1], mk.y);
                w[4 * g8 + 2] = mask_pair(w[4 * g8 + 2], mk.z);
                w[4 * g8 + 3] = mask_pair(w[4 * g8 + 3], mk.w);
            }
#pragma unroll
            for (int e = 0; e < 4; e++) nonfinite_acc(w[4 * g8 + e], acc);
            *(uint4 *)(crow + col) = make_uint4(w[4 * g8], w[4 * g8 + 1], w[4 * g8 + 2], w[4 * g8 + 3]);
        } else {
            for (int e = 0; e < 8 && col + e < N; e++) {
                uint32_t v = (e & 1) ? (w[4 * g8 + (e >> 1)] >> 16) : (w[4 * g8 + (e >> 1)] & 0xFFFFu);
                if (mrow) {
                    const uint32_t mh = mrow[col + e];
                    if (!(mh != 0 && mh <= 0x7C00u)) v = 0;
                }
                nonfinite_acc(v, acc);
                crow[col + e] = (uint16_t)v;
            }
        }
    }
    bad |= nonfinite_any(acc);
}

// The same epilogue for 32 consecutive accumulator columns of the 32 rows a warp owns, with the
// stores coalesced: each lane rounds its row's 32 values and parks them in a 32 x 32 FP16 block of
// shared memory (pitch 80 bytes: conflict-free for 16-byte accesses), then the warp writes the
// block out eight rows at a time, four lanes per row, 16 bytes per lane - 64 contiguous bytes per
// row instead of one 16-byte piece per row and instruction (a quarter of the memory transactions).
// The ReLU-derivative mask is read the same way.  stage: 32 * 80 bytes of shared memory owned by
// this warp.  row0: first of the warp's 32 rows; col0: a multiple of 32.
static constexpr int kEpiStagePitch = 80;
__device__ __forceinline__ void epilogue_store32_coalesced(const uint32_t (&r)[32], uint8_t *stage, uint16_t *C, int ldc,
                                                           const uint16_t *mask, int ldmask, int row0, int col0, int M, int N,
                                                           bool relu, bool &bad)
{
    const int lane = threadIdx.x & 31;
    uint4 *mine = (uint4 *)(stage + lane * kEpiStagePitch);
    {
        uint32_t w[16];
        round_pack32(r, relu, w);
#pragma unroll
        for (int g8 = 0; g8 < 4; g8++) mine[g8] = make_uint4(w[4 * g8], w[4 * g8 + 1], w[4 * g8 + 2], w[4 * g8 + 3]);
    }
    __syncwarp();
    const int piece = lane & 3, col = col0 + piece * 8;
    uint32_t acc = 0;
#pragma unroll
    for (int it = 0; it < 4; it++) {
        const int rr = it * 8 + (lane >> 2), row = row0 + rr;
        if (row < M && col < N) {
            const uint4 v = *(const uint4 *)(stage + rr * kEpiStagePitch + piece * 16);
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
            uint16_t *crow = C + (size_t)row * ldc;
            if (col + 8 <= N) {
                if (mask) {
                    const uint4 mk = *(const uint4 *)(mask + (size_t)row * ldmask + col);
                    w[0] = mask_pair(w[0], mk.x);
                    w[1] = mask_pair(w[1], mk.y);
                    w[2] = mask_pair(w[2], mk.z);
                    w[3] = mask_pair(w[3], mk.w);
                }
#pragma unroll
                for (int q = 0; q < 4; q++) nonfinite_acc(w[q], acc);
                *(uint4 *)(crow + col) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                for (int e = 0; e < 8 && col + e < N; e++) {
                    uint32_t x = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
                    if (mask) {
                        const uint32_t mh = mask[(size_t)row * ldmask + col + e];
                        if (!(mh != 0 && mh <= 0x7C00u)) x = 0;
                    }
                    nonfinite_acc(x, acc);
                    crow[col + e] = (uint16_t)x;
                }
            }
        }
    }
    bad |= nonfinite_any(acc);
    __syncwarp();    // the block may be overwritten by the next call
}

// LSTM gate arithmetic on FP32 values (sections 3.3, 4.5): one cell from its four pre-activations
// (bias already added).  Returns the FP16 bit patterns of the gate activations in act[4], the new
// cell state and the hidden state; h uses the STORED (rounded) cell state.
// The gate functions are evaluated with the hardware exp2 and reciprocal approximations (about
// 1e-6 relative error, three orders below the FP16 rounding of the stored result).  The epilogue
// runs beside the MMA stream and must not outlast a tile's main loop; its scarce resource is the
// special-function pipe (exp2, reciprocal and FP16<->FP32 conversions all issue there), so
// reciprocals are shared (1/a and 1/b from one reciprocal of a*b) and conversions are packed.
__device__ __forceinline__ float rcp_approx(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// tanh(x) for |x| below 1/16 (odd polynomial; the exp form cancels there), as a factor of |x|
__device__ __forceinline__ float tanh_small(float ax, float x2)
{
    return ax * (1.0f + x2 * (-0.33333334f + x2 * (0.13333334f + x2 * -0.053968254f)));
}
// The four gate values of one cell from its pre-activations: sigmoid(x) = 1/(1+exp(-x)) for
// i, f, o and tanh(x) = (1-e)/(1+e), e = exp(-2|x|), for g, with ONE reciprocal of the product of
// the four denominators.  Arguments of the sigmoids are clamped at -20 (sigmoid(-20) = 2e-9 rounds
// to zero in FP16 either way) so that the product stays below 2^127.
__device__ __forceinline__ void lstm_gates(const float (&pre)[4], float &gi, float &gf, float &gg, float &go)
{
    const float di = 1.0f + __expf(-fmaxf(pre[0], -20.0f));
    const float df = 1.0f + __expf(-fmaxf(pre[1], -20.0f));
    const float dq = 1.0f + __expf(-fmaxf(pre[3], -20.0f));
    const float ag = fabsf(pre[2]);
    const float eg = __expf(-2.0f * ag);
    const float dg = 1.0f + eg;
    const float pif = di * df, pgo = dg * dq;
    const float r = rcp_approx(pif * pgo);
    const float rif = r * pgo, rgo = r * pif;          // 1/(di*df), 1/(dg*dq)
    gi = rif * df;
    gf = rif * di;
    go = rgo * dg;
    const float big = (1.0f - eg) * (rgo * dq);
    gg = copysignf(ag < 0.0625f ? tanh_small(ag, ag * ag) : big, pre[2]);
    // NaN pre-activations must stay NaN (fmaxf drops them)
    if (pre[0] != pre[0]) gi = pre[0];
    if (pre[1] != pre[1]) gf = pre[1];
    if (pre[3] != pre[3]) go = pre[3];
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    const __half2 v = __floats2half2_rn(lo, hi);
    return *(const uint32_t *)&v;
}
// Two neighbouring cells at once: act[0..3] / act[4..7] are the FP16 gate activations of the two
// cells packed in pairs (i|f, g|o), c2 and h2 the two new cell and hidden states packed.  The
// hidden state uses the STORED (rounded) cell state.
__device__ __forceinline__ void lstm_cell_pair_math(const float (&pre0)[4], const float (&pre1)[4], float cp0, float cp1,
                                                    uint32_t (&act)[4], uint32_t &c2, uint32_t &h2)
{
    float gi0, gf0, gg0, go0, gi1, gf1, gg1, go1;
    lstm_gates(pre0, gi0, gf0, gg0, go0);
    lstm_gates(pre1, gi1, gf1, gg1, go1);
    act[0] = pack_f16x2(gi0, gf0);
    act[1] = pack_f16x2(gg0, go0);
    act[2] = pack_f16x2(gi1, gf1);
    act[3] = pack_f16x2(gg1, go1);
    const float c0 = __fadd_rn(__fmul_rn(gf0, cp0), __fmul_rn(gi0, gg0));
    const float c1 = __fadd_rn(__fmul_rn(gf1, cp1), __fmul_rn(gi1, gg1));
    const __half2 ch = __floats2half2_rn(c0, c1);
    c2 = *(const uint32_t *)&ch;
    const float s0 = __low2float(ch), s1 = __high2float(ch);
    const float a0 = fabsf(s0), a1 = fabsf(s1);
    const float e0 = __expf(-2.0f * a0), e1 = __expf(-2.0f * a1);
    const float d0 = 1.0f + e0, d1 = 1.0f + e1;
    const float r = rcp_approx(d0 * d1);
    float t0 = (1.0f - e0) * (r * d1), t1 = (1.0f - e1) * (r * d0);
    t0 = copysignf(a0 < 0.0625f ? tanh_small(a0, a0 * a0) : t0, s0);
    t1 = copysignf(a1 < 0.0625f ? tanh_small(a1, a1 * a1) : t1, s1);
    h2 = pack_f16x2(__fmul_rn(go0, t0), __fmul_rn(go1, t1));
}
// One cell on its own (CUDA-core kernel): the same arithmetic with the second lane idle.
__device__ __forceinline__ void lstm_cell_math(const float (&pre)[4], float c_prev, uint32_t (&act)[4], uint32_t &c16,
                                               uint32_t &h16)
{
    uint32_t a[4], c2, h2;
    lstm_cell_pair_math(pre, pre, c_prev, c_prev, a, c2, h2);
    act[0] = a[0] & 0xFFFFu; act[1] = a[0] >> 16; act[2] = a[1] & 0xFFFFu; act[3] = a[1] >> 16;
    c16 = c2 & 0xFFFFu;
    h16 = h2 & 0xFFFFu;
}

// Operands of the gate epilogue for one chunk of 32 gate-interleaved columns (8 whole cells) of
// one row: the bias values of the chunk (FP32 when the caller provides a converted copy, else
// FP16 bits in the first four vectors) and the eight previous cell states.
struct LstmChunkIn {
    uint4 b[8];
    uint4 cp;
};
__device__ __forceinline__ void lstm_fetch(LstmChunkIn &in, const LstmEpi &e, int row, int col0)
{
    in.cp = *(const uint4 *)(e.c_prev + (size_t)row * e.ldcp + (col0 >> 2));
    if (e.bias32) {
#pragma unroll
        for (int v = 0; v < 8; v++) in.b[v] = __ldg((const uint4 *)(e.bias32 + col0 + v * 4));
    } else {
#pragma unroll
        for (int g8 = 0; g8 < 4; g8++) in.b[g8] = __ldg((const uint4 *)(e.bias + col0 + g8 * 8));
    }
}

// Epilogue of one thread for 32 consecutive gate-interleaved accumulator columns (8 whole cells)
// of its output row: bias add, gate arithmetic, 128-bit stores of the activations (4), the
// cell state (1) and the hidden state (1).  col0 is a multiple of 32 and col0 + 32 <= 4H.
__device__ __forceinline__ void epilogue_lstm32(const uint32_t (&r)[32], const LstmChunkIn &in, uint16_t *arow, int row, int col0,
                                                const LstmEpi &e)
{
    const int j0 = col0 >> 2;
    const uint32_t cpw[4] = {in.cp.x, in.cp.y, in.cp.z, in.cp.w};
    uint32_t cw[4], hw[4];
    const bool f32bias = e.bias32 != nullptr;
#pragma unroll
    for (int g8 = 0; g8 < 4; g8++) {      // 8 columns = 2 cells
        float bias[8];
        if (f32bias) {
            const uint4 lo = in.b[2 * g8], hi = in.b[2 * g8 + 1];
            bias[0] = __uint_as_float(lo.x); bias[1] = __uint_as_float(lo.y); bias[2] = __uint_as_float(lo.z);
            bias[3] = __uint_as_float(lo.w); bias[4] = __uint_as_float(hi.x); bias[5] = __uint_as_float(hi.y);
            bias[6] = __uint_as_float(hi.z); bias[7] = __uint_as_float(hi.w);
        } else {
            const uint32_t bw[4] = {in.b[g8].x, in.b[g8].y, in.b[g8].z, in.b[g8].w};
#pragma unroll
            for (int v = 0; v < 4; v++) {
                const float2 f = __half22float2(*(const __half2 *)&bw[v]);
                bias[2 * v] = f.x; bias[2 * v + 1] = f.y;
            }
        }
        float pre0[4], pre1[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            pre0[q] = __fadd_rn(__uint_as_float(r[g8 * 8 + q]), bias[q]);
            pre1[q] = __fadd_rn(__uint_as_float(r[g8 * 8 + 4 + q]), bias[4 + q]);
        }
        const float2 cp = __half22float2(*(const __half2 *)&cpw[g8]);
        uint32_t act[4];
        lstm_cell_pair_math(pre0, pre1, cp.x, cp.y, act, cw[g8], hw[g8]);
        *(uint4 *)(arow + col0 + g8 * 8) = make_uint4(act[0], act[1], act[2], act[3]);
    }
    *(uint4 *)(e.c_out + (size_t)row * e.ldco + j0) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
    *(uint4 *)(e.h_out + (size_t)row * e.ldh + j0) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
}

// The whole gate epilogue of one thread for `nchunks` chunks of 32 accumulator columns starting at
// tensor-memory address taddr / output column col_base.  The global operands of chunk c+1 are
// requested before the arithmetic of chunk c, so their latency is hidden behind it.  Every lane
// runs the collective tensor-memory loads; only lanes whose row exists touch global memory.
__device__ __forceinline__ void epilogue_lstm_tile(uint32_t taddr, int nchunks, int col_base, int N, int row, bool row_ok,
                                                   uint16_t *arow, const LstmEpi &e)
{
    LstmChunkIn cur, nxt;
    cur.cp = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int v = 0; v < 8; v++) cur.b[v] = make_uint4(0, 0, 0, 0);
    nxt = cur;
    if (row_ok && col_base < N) lstm_fetch(cur, e, row, col_base);
#pragma unroll 1
    for (int c = 0; c < nchunks; c++) {
        uint32_t r[32];
        tc_ld32(taddr + (uint32_t)(c * 32), r);
        const int col0 = col_base + c * 32;
        const bool more = c + 1 < nchunks && row_ok && col0 + 32 < N;
        if (more) lstm_fetch(nxt, e, row, col0 + 32);
        tc_wait_ld();
        if (row_ok && col0 < N) epilogue_lstm32(r, cur, arow, row, col0, e);
        cur = nxt;
    }
}

// ------------------------------------------------------------ cluster / 2-CTA forms

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on an mbarrier that may live in the peer CTA (shared::cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// The two halves of cluster_sync_all, for threads that have work between arriving and waiting.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Wait on a local mbarrier whose arrivals come from other CTAs of the cluster together with plain
// stores into this CTA's shared memory: acquire at cluster scope makes those stores visible.
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
static __device__ __noinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                                      unsigned long long limit_ns = WAIT_LIMIT_NS)
{
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 127u) == 127u) {
            if (*abort_flag) return false;
            unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}
// 16-byte store into the shared memory of any CTA of the cluster (shared::cluster address from mapa)
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Bulk copy from this CTA's shared memory into the shared memory of a CTA of the cluster (no multicast;
// both shared::cluster addresses from mapa, all addresses and the size multiples of 16); the bytes are
// signalled on an mbarrier of the receiving CTA.
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t cluster_bar)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster),
                 "r"(src_cta), "r"(bytes), "r"(cluster_bar)
                 : "memory");
}
// TMA load whose completion bytes are signalled on an mbarrier of either CTA of the pair
// (no multicast: the data goes to the issuing CTA's own shared memory only)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t cluster_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar)
        : "memory");
}
// Tensor store of one box from this CTA's shared memory (layout as the tensor map's swizzle mode says) to
// global memory; parts of the box outside the tensor are not written.  x (the inner coordinate) times the
// element size must be a multiple of 16 bytes, and no coordinate may be negative.  Completion is tracked by
// the issuing thread's bulk groups.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until all but the N most recent bulk groups of this thread have finished READING shared memory
template <int N>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// Epilogue of one warp for one 32 x 64 box of the output (its 32 rows, 64 consecutive accumulator columns
// starting at tensor-memory address taddr): each lane rounds its row's values (optional ReLU fused, optional
// ReLU-derivative mask, inf/NaN vote into acc_bits - whole groups of 8 columns inside the matrix only, N must
// be a multiple of 8), parks them in `box` (4 KB of shared memory, 1024-byte aligned) in the 128-byte-swizzled
// layout of the output tensor map, and lane 0 sends the box with one tensor store and commits a bulk group
// (always, so that callers can count groups).  The caller makes sure the box is free (bulk_wait_group_read).
__device__ __forceinline__ void epilogue_box_store(uint32_t taddr, uint32_t box, const CUtensorMap *tmC, int row0, int colb,
                                                   int M, int N, bool relu, const uint16_t *mrow, bool row_ok,
                                                   uint32_t &acc_bits)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int h = 0; h < 2; h++) {
        uint32_t r[32], hw[16];
        tc_ld32(taddr + (uint32_t)(h * 32), r);
        tc_wait_ld();
        round_pack32(r, relu, hw);
        const int col0 = colb + h * 32;
        if (mrow && row_ok) {
#pragma unroll
            for (int g8 = 0; g8 < 4; g8++) {
                if (col0 + g8 * 8 + 8 <= N) {
                    const uint4 mk = *(const uint4 *)(mrow + col0 + g8 * 8);
                    hw[4 * g8] = mask_pair(hw[4 * g8], mk.x);
                    hw[4 * g8 + 1] = mask_pair(hw[4 * g8 + 1], mk.y);
                    hw[4 * g8 + 2] = mask_pair(hw[4 * g8 + 2], mk.z);
                    hw[4 * g8 + 3] = mask_pair(hw[4 * g8 + 3], mk.w);
                }
            }
        }
#pragma unroll
        for (int g8 = 0; g8 < 4; g8++) {
            // values outside the matrix are not stored (the tensor store clips) and must not vote
            if (row_ok && col0 + g8 * 8 + 8 <= N) {
#pragma unroll
                for (int e = 0; e < 4; e++) nonfinite_acc(hw[4 * g8 + e], acc_bits);
            }
            const uint32_t piece = (uint32_t)((h * 4 + g8) ^ (lane & 7));      // 128-byte swizzle
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box + (uint32_t)(lane * 128) + (piece << 4)),
                         "r"(hw[4 * g8]), "r"(hw[4 * g8 + 1]), "r"(hw[4 * g8 + 2]), "r"(hw[4 * g8 + 3])
                         : "memory");
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor store reads what the lanes wrote
    __syncwarp();
    if (lane == 0) {
        if (row0 < M && colb < N) tma_store_2d(tmC, box, colb, row0);
        bulk_commit_group();
    }
}

// The same load with an L2 eviction-priority hint (policy from l2_policy()).  Operand lines marked
// "evict last" outlive the output stores and the other kernels' streams in L2: inside the large-MLP step
// the products run 2-2.5 % faster with both operands marked (an operand one product has just read, or
// written, is often the next product's operand); "evict first" on the operand that is not reused by
// later waves made the step 6-8 % slower (the tiles of a wave that share a line do not ask for it at
// the same moment).  DRAM bytes of a single launch (measured with caches flushed) do not change.
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t cluster_bar,
                                                      uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar), "l"(policy)
        : "memory");
}
// kind 1: evict last, 2: evict first, else: evict normal
__device__ __forceinline__ uint64_t l2_policy(int kind)
{
    uint64_t pol;
    if (kind == 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    else if (kind == 2) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// commit of the pair's MMAs: arrives on the mbarrier at this offset in every CTA of `cta_mask`
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t cta_mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(cta_mask)
                 : "memory");
}

}  // namespace mpt
