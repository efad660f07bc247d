// Momentum replacement and model update (Section 3.3 steps 5-6), the variants' update kernels,
// and the kernels that materialise errors and momentum for state reads.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Worker side again: the received chunk replaces the momentum (it stays in its compressed
// form) and the model moves with the frozen variance (Section 3.3 steps 5-6).
// One CTA per kApplyTile (4096) consecutive elements, whatever the chunk length.

constexpr int kApplyTile = 4096;
constexpr int kApplyU = kApplyTile / (kThreads * 4);

struct ApplyArgs {
    const uint32_t* Bbar; const float* Sbar; const float* den; float* x;     // den = sqrt(v) + eps, see k_make_den
    int64_t d; int64_t chunk; float lr;
    float inv_chunk;      // 1 / chunk in binary32 when there are fewer than 2^20 chunks (see div_small_quotient), else 0
};

// den = sqrt(v) + eps, the denominator of the model update while v is frozen.
__global__ void k_make_den(const float* __restrict__ v, float* __restrict__ den, int64_t d, float eps)
{
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x)
        APMS_STORE(den[j], __fadd_rn(__fsqrt_rn(v[j]), eps));
}

__global__ void __launch_bounds__(kThreads)
k_apply(const ApplyArgs a)
{
    const int64_t base = (int64_t)blockIdx.x * kApplyTile;
    const int64_t left = a.d - base;
    const int L = (int)(left < kApplyTile ? left : kApplyTile);
    const int64_t c0 = a.inv_chunk != 0.0f ? div_small_quotient(base, a.chunk, a.inv_chunk) : base / a.chunk;
    const uint32_t off0 = (uint32_t)(base - c0 * a.chunk);
    const uint32_t chunk32 = (uint32_t)a.chunk;
    const bool long_chunk = a.chunk >= kApplyTile;          // then a tile holds at most one chunk boundary: no division per access
    const uint32_t* __restrict__ bits = a.Bbar + base / 32;
    const float* __restrict__ v = a.den + base;
    float* __restrict__ x = a.x + base;
    const float* __restrict__ Sb = a.Sbar + c0;
    if (L == kApplyTile) {
        float4 vv[kApplyU], xx[kApplyU];
        uint32_t nib[kApplyU];
        float S[kApplyU];
#pragma unroll
        for (int u = 0; u < kApplyU; ++u) {
            const int k = (u * kThreads + threadIdx.x) * 4;
            vv[u] = ld_stream4(v + k);
            xx[u] = ld_stream4(x + k);
            nib[u] = bits[k >> 5] >> (k & 31);
            const uint32_t rel = off0 + (uint32_t)k;
            S[u] = Sb[long_chunk ? (rel >= chunk32 ? 1u : 0u) : rel / chunk32];
        }
#pragma unroll
        for (int u = 0; u < kApplyU; ++u) {
            const int k = (u * kThreads + threadIdx.x) * 4;
            const float cc = __fmul_rn(a.lr, S[u]);
            xx[u].x = apply_stored(xx[u].x, vv[u].x, nib[u] & 1u, cc);
            xx[u].y = apply_stored(xx[u].y, vv[u].y, nib[u] & 2u, cc);
            xx[u].z = apply_stored(xx[u].z, vv[u].z, nib[u] & 4u, cc);
            xx[u].w = apply_stored(xx[u].w, vv[u].w, nib[u] & 8u, cc);
            st_stream4(x + k, xx[u]);
        }
        return;
    }
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        const uint32_t rel = off0 + (uint32_t)k;
        const float S = Sb[long_chunk ? (rel >= chunk32 ? 1u : 0u) : rel / chunk32];
        const uint32_t nib = bits[k >> 5] >> (k & 31);
        const float cc = __fmul_rn(a.lr, S);
        if (k + 3 < L) {
            const float4 vv = ld_stream4(v + k);
            float4 xx = ld_stream4(x + k);
            xx.x = apply_stored(xx.x, vv.x, nib & 1u, cc);
            xx.y = apply_stored(xx.y, vv.y, nib & 2u, cc);
            xx.z = apply_stored(xx.z, vv.z, nib & 4u, cc);
            xx.w = apply_stored(xx.w, vv.w, nib & 8u, cc);
            st_stream4(x + k, xx);
        } else {
            for (int e = 0; e < 4 && k + e < L; ++e)
                APMS_STORE(x[k + e], apply_stored(x[k + e], v[k + e], (nib >> e) & 1u, cc));
        }
    }
}

// Steps 5-6 of the gradient-compressing variant (Section 5.3, item 4): the received chunk is a
// gradient ghat = +-Sbar; m <- b1 m + (1-b1) ghat stays binary32, the model moves with the new m.
struct ApplyGradArgs {
    const uint32_t* Bbar; const float* Sbar; const float* v; float* x; float* m;
    int64_t d; int64_t chunk; float lr, eps, beta1, omb1;
};

__global__ void __launch_bounds__(kThreads)
k_apply_gradient(const ApplyGradArgs a)
{
    const int64_t base = (int64_t)blockIdx.x * kApplyTile;
    const int64_t left = a.d - base;
    const int L = (int)(left < kApplyTile ? left : kApplyTile);
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        const int64_t j = base + k;
        const float S = a.Sbar[j / a.chunk];                       // chunks are multiples of 32: one scale per 4 elements
        const uint32_t nib = a.Bbar[j >> 5] >> (j & 31);
        if (k + 3 < L) {
            const float4 vv = ld_stream4(a.v + j);
            float4 xx = ld_stream4(a.x + j);
            float4 mm = ld_stream4(a.m + j);
            mm.x = __fmaf_rn(a.beta1, mm.x, __fmul_rn(a.omb1, bit_scale(nib & 1u, S)));
            mm.y = __fmaf_rn(a.beta1, mm.y, __fmul_rn(a.omb1, bit_scale(nib & 2u, S)));
            mm.z = __fmaf_rn(a.beta1, mm.z, __fmul_rn(a.omb1, bit_scale(nib & 4u, S)));
            mm.w = __fmaf_rn(a.beta1, mm.w, __fmul_rn(a.omb1, bit_scale(nib & 8u, S)));
            xx.x = apply_elem(xx.x, vv.x, mm.x, a.lr, a.eps);
            xx.y = apply_elem(xx.y, vv.y, mm.y, a.lr, a.eps);
            xx.z = apply_elem(xx.z, vv.z, mm.z, a.lr, a.eps);
            xx.w = apply_elem(xx.w, vv.w, mm.w, a.lr, a.eps);
            st_stream4(a.m + j, mm);
            st_stream4(a.x + j, xx);
        } else {
            for (int e = 0; e < 4 && k + e < L; ++e) {
                const float mn = __fmaf_rn(a.beta1, a.m[j + e], __fmul_rn(a.omb1, bit_scale((nib >> e) & 1u, S)));
                APMS_STORE(a.m[j + e], mn);
                APMS_STORE(a.x[j + e], apply_elem(a.x[j + e], a.v[j + e], mn, a.lr, a.eps));
            }
        }
    }
}

// "APMSqueeze (Uncompressed)" of Section 5.3 (item 3): v frozen, nothing compressed.  Every worker forms
// its local momentum, the momenta are averaged in worker order, the average is the new momentum:
//   m <- (1/n) sum_i (b1 m + (1-b1) g_i) ;  x <- x - lr m / (sqrt(v) + eps).
// The additions of +0 stand for the (zero) compression errors of the general step, so that a negative
// zero behaves as it does there.
struct UncompressedArgs {
    float* x; float* m; const float* v;
    int64_t d; int n;
    float beta1, omb1, lr, eps, nf;
};

__device__ __forceinline__ void uncompressed_elem(const UncompressedArgs& a, float acc, float& m, float v, float& x)
{
    m = __fadd_rn(__fdiv_rn(acc, a.nf), 0.0f);
    x = apply_elem(x, v, m, a.lr, a.eps);
}

template <int GT>
__global__ void __launch_bounds__(kThreads)
k_uncompressed(const __grid_constant__ GradPtrs G, const UncompressedArgs a)
{
    const int64_t j = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 4;
    if (j + 3 < a.d) {
        float4 m = ld_stream4(a.m + j);
        const float4 v = ld_stream4(a.v + j);
        float4 x = ld_stream4(a.x + j);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int i = 0; i < a.n; ++i) {
            const float4 g = Grad<GT>::ld4(Grad<GT>::at(G.p[i], j), 0);
            acc.x = __fadd_rn(acc.x, __fadd_rn(__fmaf_rn(a.beta1, m.x, __fmul_rn(a.omb1, g.x)), 0.0f));
            acc.y = __fadd_rn(acc.y, __fadd_rn(__fmaf_rn(a.beta1, m.y, __fmul_rn(a.omb1, g.y)), 0.0f));
            acc.z = __fadd_rn(acc.z, __fadd_rn(__fmaf_rn(a.beta1, m.z, __fmul_rn(a.omb1, g.z)), 0.0f));
            acc.w = __fadd_rn(acc.w, __fadd_rn(__fmaf_rn(a.beta1, m.w, __fmul_rn(a.omb1, g.w)), 0.0f));
        }
        uncompressed_elem(a, acc.x, m.x, v.x, x.x); uncompressed_elem(a, acc.y, m.y, v.y, x.y);
        uncompressed_elem(a, acc.z, m.z, v.z, x.z); uncompressed_elem(a, acc.w, m.w, v.w, x.w);
        st_stream4(a.m + j, m);
        st_stream4(a.x + j, x);
    } else {
        for (int64_t e = j; e < a.d; ++e) {
            float acc = 0.f;
            float m = a.m[e], x = a.x[e];
            for (int i = 0; i < a.n; ++i)
                acc = __fadd_rn(acc, __fadd_rn(__fmaf_rn(a.beta1, m, __fmul_rn(a.omb1, Grad<GT>::ld1(G.p[i], e))), 0.0f));
            uncompressed_elem(a, acc, m, a.v[e], x);
            APMS_STORE(a.m[e], m); APMS_STORE(a.x[e], x);
        }
    }
}

// ------------------------------------------------------------------------------------------
// State materialisation (parity, checkpoints): delta = z - (+-scale), m = +-Sbar.

__global__ void k_materialise_error(const float* __restrict__ z, const float* __restrict__ s,
                                    float* __restrict__ out, int64_t first, int64_t count, int64_t chunk)
{
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += (int64_t)gridDim.x * blockDim.x)
        out[j] = implied_error(z[first + j], s[(first + j) / chunk]);
}

__global__ void k_materialise_momentum(const uint32_t* __restrict__ bits, const float* __restrict__ S,
                                       float* __restrict__ out, int64_t first, int64_t count, int64_t chunk)
{
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = first + j;
        out[j] = bit_scale((bits[e >> 5] >> (e & 31)) & 1u, S[e / chunk]);
    }
}

}  // namespace
