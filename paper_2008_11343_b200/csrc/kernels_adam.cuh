// Warmup phase: the fused Adam step on the worker-averaged gradient (Section 3.2).
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Warmup: Adam with bias correction on the worker-averaged gradient (Section 3.2).

struct AdamArgs {
    float* x; float* m; float* v;
    int64_t d; int n;
    float beta1, beta2, omb1, omb2, bc1, bc2, lr, eps, nf;
};

__device__ __forceinline__ void adam_elem(const AdamArgs& a, float gs, float& m, float& v, float& x) {
    const float gbar = __fdiv_rn(gs, a.nf);
    m = __fmaf_rn(a.beta1, m, __fmul_rn(a.omb1, gbar));
    v = __fmaf_rn(a.beta2, v, __fmul_rn(a.omb2, __fmul_rn(gbar, gbar)));
    const float mhat = __fdiv_rn(m, a.bc1);
    const float vhat = __fdiv_rn(v, a.bc2);
    x = __fsub_rn(x, __fdiv_rn(__fmul_rn(a.lr, mhat), __fadd_rn(__fsqrt_rn(vhat), a.eps)));
}

// One short-lived CTA per 1024 elements (one float4 per thread and stream): the n gradient
// loads of a thread are independent, and many small CTAs keep more of them in flight than a
// resident grid-stride loop does.
template <int GT>
__global__ void __launch_bounds__(kThreads)
k_warmup_adam(const __grid_constant__ GradPtrs G, const AdamArgs a)
{
    const int64_t j = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 4;
    if (j + 3 < a.d) {
        float4 m = ld_stream4(a.m + j);
        float4 v = ld_stream4(a.v + j);
        float4 x = ld_stream4(a.x + j);
        float4 gs = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int i = 0; i < a.n; ++i) {
            const float4 g = Grad<GT>::ld4(Grad<GT>::at(G.p[i], j), 0);
            gs.x = __fadd_rn(gs.x, g.x); gs.y = __fadd_rn(gs.y, g.y);
            gs.z = __fadd_rn(gs.z, g.z); gs.w = __fadd_rn(gs.w, g.w);
        }
        adam_elem(a, gs.x, m.x, v.x, x.x); adam_elem(a, gs.y, m.y, v.y, x.y);
        adam_elem(a, gs.z, m.z, v.z, x.z); adam_elem(a, gs.w, m.w, v.w, x.w);
        st_stream4(a.m + j, m);
        st_stream4(a.v + j, v);
        st_stream4(a.x + j, x);
    } else {
        // ragged tail (d not a multiple of 4): element by element
        for (int64_t e = j; e < a.d; ++e) {
            float gs = 0.f;
            for (int i = 0; i < a.n; ++i) gs = __fadd_rn(gs, Grad<GT>::ld1(G.p[i], e));
            float m = a.m[e], v = a.v[e], x = a.x[e];
            adam_elem(a, gs, m, v, x);
            APMS_STORE(a.m[e], m); APMS_STORE(a.v[e], v); APMS_STORE(a.x[e], x);
        }
    }
}

}  // namespace
