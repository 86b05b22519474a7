// The optimizer step on one element of the FP32 master copy, shared by the single-GPU master pass
// and the data-parallel step.  Internal.
#pragma once

#include "mpt_common.cuh"

namespace mpt {

// gs: the loss-scaled gradient as FP32 (one FP16 value widened, or the FP32 sum of the replicas'
// values); inv: 1/S resp. 1/(S*R).
// One element; every operation rounded separately, in the order documented in mpt.h.
template <int KIND, bool WD>
__device__ __forceinline__ void opt1(float gs, float &w, float &s1, float &s2, float inv, float lr, float mu, float b2,
                                     float omb1, float omb2, float eps, float wd, float bc1, float bc2, float coef, bool &bad)
{
    float g = __fmul_rn(gs, inv);
    bad |= f32_nonfinite(g);
    g = __fmul_rn(g, coef);     // global-norm clipping coefficient (exactly 1.0f when clipping is off)
    if (WD) g = __fadd_rn(g, __fmul_rn(wd, w));
    float u;
    if (KIND == MPT_OPT_NESTEROV) {
        s1 = __fadd_rn(__fmul_rn(mu, s1), g);
        u = __fmul_rn(lr, __fadd_rn(g, __fmul_rn(mu, s1)));
    } else if (KIND == MPT_OPT_ADAGRAD) {
        s1 = __fadd_rn(s1, __fmul_rn(g, g));
        u = __fmul_rn(lr, __fdiv_rn(g, __fadd_rn(__fsqrt_rn(s1), eps)));
    } else if (KIND == MPT_OPT_ADAM) {
        s1 = __fadd_rn(__fmul_rn(mu, s1), __fmul_rn(omb1, g));
        s2 = __fadd_rn(__fmul_rn(b2, s2), __fmul_rn(omb2, __fmul_rn(g, g)));
        const float mh = __fdiv_rn(s1, bc1), vh = __fdiv_rn(s2, bc2);
        u = __fmul_rn(lr, __fdiv_rn(mh, __fadd_rn(__fsqrt_rn(vh), eps)));
    } else {  // SGD with weight decay: momentum iff s1 is in use (mu != 0)
        if (mu != 0.0f) {
            s1 = __fadd_rn(__fmul_rn(mu, s1), g);
            u = __fmul_rn(lr, s1);
        } else {
            u = __fmul_rn(lr, g);
        }
    }
    w = __fsub_rn(w, u);
}

}  // namespace mpt
