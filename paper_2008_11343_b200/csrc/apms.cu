// APMSqueeze compressed-step library for B200 (sm_100a): kernels and C ABI.
//
// Data layout in HBM (one context, the n workers simulated as n buffer sets):
//   x, v            float[d]      model and (frozen) variance, one copy: every worker holds
//                                 the same x after every step (Algorithm 1 lines 10-11)
//   m32             float[d]      binary32 momentum; authoritative only during warmup, for the
//                                 first compressed step and after apms_set_state(M)
//   zbar            float[d]      the server's last compensated vector  zbar = avg + dbar_old
//   Bbar, Sbar      uint32[W], float[C]   the server's last message.  Together with zbar they
//                                 hold BOTH the shared momentum m = +-Sbar (Section 3.3 step 5)
//                                 and the server error dbar = zbar - (+-Sbar) (step 4)
//   z_i             n x float[d]  worker i's last compensated vector z_i = m_i + delta_i_old
//   B_i, s_i        n x uint32[W], n x float[C]   worker i's last message; its error is
//                                 delta_i = z_i - (+-s_i) (Section 3.3 step 2)
//
// Keeping z instead of delta removes the only intra-chunk dependency of the step (the error
// needs the chunk's scale, the scale needs the whole chunk): the subtraction delta = z - C[z]
// is performed, with the same single binary32 rounding, by the next step's read.  Every
// element of g_i and z_i is then read once and z_i written once per step, in one streaming
// pass, and nothing has to be held on chip across the chunk reduction.
//
// Arithmetic: explicit round-to-nearest intrinsics everywhere, so that the compiler can
// neither contract nor reorder; sums of squares in binary64 (products of binary32 values are
// exact in binary64, so only the order of the additions can differ from a sequential sum).

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#include <mutex>
#include <new>
#include <vector>

#include "apms.h"

namespace {

constexpr int kThreads = 256;            // threads per CTA in every kernel
constexpr int kWarps = kThreads / 32;
constexpr int kGroup = 128;              // elements one warp covers per 128-bit access (4 sign words)

// Tunables (defaults chosen by measurement on B200; override with -D to re-tune).
#ifndef APMS_WORKER_U
#define APMS_WORKER_U 4                  // 128-element groups in flight per warp, worker kernel
#endif
#ifndef APMS_SERVER_U
#define APMS_SERVER_U 2                  // the same for the server kernel
#endif
#ifndef APMS_WORKER_CTAS
#define APMS_WORKER_CTAS 3               // resident CTAs per SM the worker kernel is compiled for
#endif
#ifndef APMS_SERVER_CTAS
#define APMS_SERVER_CTAS 3
#endif

struct GradPtrs { const void* p[APMS_MAX_WORKERS]; };     // element type given by the kernel's GT template argument

// ------------------------------------------------------------------------------------------
// small device helpers

__device__ __forceinline__ float4 ld_stream4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st_stream4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

// Up to four consecutive floats starting at p[k]; elements at or past `len` read as 0.
__device__ __forceinline__ float4 ld4_checked(const float* p, int k, int len, bool streaming) {
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k + 3 < len) {
        r = streaming ? ld_stream4(p + k) : *reinterpret_cast<const float4*>(p + k);
    } else {
        if (k + 0 < len) r.x = p[k + 0];
        if (k + 1 < len) r.y = p[k + 1];
        if (k + 2 < len) r.z = p[k + 2];
    }
    return r;
}
__device__ __forceinline__ void st4_checked(float* p, int k, int len, float4 v) {
    if (k + 3 < len) {
        st_stream4(p + k, v);
    } else {
        if (k + 0 < len) p[k + 0] = v.x;
        if (k + 1 < len) p[k + 1] = v.y;
        if (k + 2 < len) p[k + 2] = v.z;
    }
}

// Gradient element types (apms_grad_type): binary32, bfloat16, binary16.  A 16-bit gradient is
// widened to binary32 exactly before its first use, so the arithmetic of a step does not change.
template <int GT> struct Grad;
template <> struct Grad<APMS_GRAD_F32> {
    static __device__ __forceinline__ const void* at(const void* p, int64_t e) { return (const float*)p + e; }
    static __device__ __forceinline__ float ld1(const void* p, int64_t e) { return ((const float*)p)[e]; }
    static __device__ __forceinline__ float4 ld4(const void* p, int k) { return ld_stream4((const float*)p + k); }
};
template <> struct Grad<APMS_GRAD_BF16> {
    static __device__ __forceinline__ const void* at(const void* p, int64_t e) { return (const uint16_t*)p + e; }
    static __device__ __forceinline__ float ld1(const void* p, int64_t e) { return __uint_as_float((uint32_t)((const uint16_t*)p)[e] << 16); }
    static __device__ __forceinline__ float4 ld4(const void* p, int k) {
        const uint2 r = __ldcs(reinterpret_cast<const uint2*>((const uint16_t*)p + k));
        return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                           __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
    }
};
template <> struct Grad<APMS_GRAD_F16> {
    static __device__ __forceinline__ const void* at(const void* p, int64_t e) { return (const __half*)p + e; }
    static __device__ __forceinline__ float ld1(const void* p, int64_t e) { return __half2float(((const __half*)p)[e]); }
    static __device__ __forceinline__ float4 ld4(const void* p, int k) {
        const uint2 r = __ldcs(reinterpret_cast<const uint2*>((const __half*)p + k));
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&r.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&r.y));
        return make_float4(a.x, a.y, b.x, b.y);
    }
};
// Up to four consecutive gradient elements starting at element k; elements at or past `len` read as 0.
template <int GT>
__device__ __forceinline__ float4 ld_grad4_checked(const void* p, int k, int len)
{
    if (k + 3 < len) return Grad<GT>::ld4(p, k);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k + 0 < len) r.x = Grad<GT>::ld1(p, k + 0);
    if (k + 1 < len) r.y = Grad<GT>::ld1(p, k + 1);
    if (k + 2 < len) r.z = Grad<GT>::ld1(p, k + 2);
    return r;
}

// +-s with the sign of the compressor: z >= 0 gives +s (so do +0 and -0), NaN gives -s.
__device__ __forceinline__ float signed_scale(float z, float s) { return (z >= 0.0f) ? s : -s; }
__device__ __forceinline__ float bit_scale(uint32_t bit, float s) { return bit ? s : -s; }

// Model update of one element with the frozen variance (Section 3.3 step 6).
__device__ __forceinline__ float apply_elem(float x, float v, float q, float lr, float eps) {
    return __fsub_rn(x, __fdiv_rn(__fmul_rn(lr, q), __fadd_rn(__fsqrt_rn(v), eps)));
}

// One element's contribution to a chunk's scale, and the scale from the sum.  The scale is the
// l2 norm of the chunk over sqrt(L) (Section 5.1 read with the paper's norm); the other reading
// of "magnitude", the mean of |z|, is kept as a switch: |z| = z * (+-1) is added by the same fma.
__device__ __forceinline__ void scale_accumulate(double& acc, float z, bool l1)
{
    const double zd = (double)z;
    acc = fma(zd, l1 ? copysign(1.0, zd) : zd, acc);
}
__device__ __forceinline__ float scale_from_sum(double total, double L, bool l1)
{
    return l1 ? (float)(total / L) : (float)sqrt(total / L);
}

// The compression error implied by a stored compensated value and its chunk's scale.
__device__ __forceinline__ float implied_error(float z, float s) { return __fsub_rn(z, signed_scale(z, s)); }

// Lane l of a warp holds the four sign bits (nibble) of elements 4l..4l+3 of a 128-element
// group.  Returns, in lanes 0, 8, 16, 24, the LSB-first sign word of elements 32*(l/8)...
__device__ __forceinline__ uint32_t pack_group_words(uint32_t nibble, int lane) {
    uint32_t w = nibble << (4 * (lane & 7));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    return w;
}

__device__ __forceinline__ double warp_sum(double a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_down_sync(0xffffffffu, a, o);
    return a;
}

// Fixed-order block sum (lane tree, then warps in order); result valid in thread 0.
__device__ __forceinline__ double block_sum(double a, double* smem) {
    a = warp_sum(a);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) smem[warp] = a;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += smem[w];
    }
    return t;
}

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
            a.m[e] = m; a.v[e] = v; a.x[e] = x;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Mapping of chunks to work items.  An item is one tile of one chunk (for one worker on the
// worker side).  Chunks up to kTileMax elements are one tile; longer chunks (the paper's own
// layout is chunk = d/n) are cut into tiles of kTileSplit elements whose binary64 partial sums
// of squares go to a scratch array and are added up, in tile order, by k_finalize_scales.
// A team of WPC warps works on an item: the whole CTA (WPC = 8) or, for short chunks, one warp
// (WPC = 1, eight items per CTA and no CTA-wide barrier).

constexpr int64_t kTileMax = 65536;
constexpr int64_t kTileSplit = 32768;
// A tile is given to a single warp (eight tiles per CTA, no CTA-wide barrier) whenever that
// still leaves at least kWarpTeamMinCtasPerSm CTAs per SM; small problems use one CTA per tile.
constexpr int kWarpTeamMinCtasPerSm = 6;

struct Tiling {
    int64_t d, chunk, tile;   // tile == chunk when P == 1
    int P;                    // tiles per chunk
    int64_t Pp;               // row stride of the partial-sum arrays (>= C * P)
    int l1 = 0;               // scale = mean |z| instead of ||z||_2 / sqrt(L)
};

struct Item { int64_t c; int p; int64_t base; int L; int Lc; };

__device__ __forceinline__ Item decode_item(const Tiling& t, int64_t chunk_tile)
{
    Item it;
    it.p = (t.P == 1) ? 0 : (int)(chunk_tile % t.P);
    it.c = (t.P == 1) ? chunk_tile : chunk_tile / t.P;
    const int64_t cbeg = it.c * t.chunk;
    const int64_t cend = (t.d - cbeg < t.chunk) ? t.d : cbeg + t.chunk;
    it.base = cbeg + (int64_t)it.p * t.tile;
    const int64_t left = cend - it.base;
    it.L = (int)(left < t.tile ? (left > 0 ? left : 0) : t.tile);
    it.Lc = (int)(cend - cbeg);
    return it;
}

template <int WPC>
__device__ __forceinline__ double team_sum(double a, double* smem)
{
    if (WPC == 1) return warp_sum(a);      // valid in lane 0
    return block_sum(a, smem);             // valid in thread 0
}

// ------------------------------------------------------------------------------------------
// Worker side: local momentum + error-compensated 1-bit compression (Section 3.3 steps 1-2).
// Items are ordered chunk-major, worker-minor, so that the n workers of one chunk run
// together and share that chunk's momentum bits through L2.

struct WorkerArgs {
    float* z;  int64_t dz;        // n x d compensated vectors, stride dz
    uint32_t* B; int64_t Wp;      // n x W sign words, stride Wp
    float* s;  int64_t Cp;        // n x C scales, stride Cp
    double* partial;              // n x Pp partial sums (only when P > 1)
    const float* m32;             // binary32 momentum (first step / forced)
    const uint32_t* Bbar; const float* Sbar;   // momentum as the server's last message
    Tiling t;
    int64_t items;                // C * P * ni
    int i0, ni;                   // this launch covers workers i0 .. i0+ni-1
    float beta1, omb1;
    int send_gradient;            // gradient-compressing variant: z = g_i + delta_i, the momentum is not read
};

template <bool M32, bool CHECKED>
__device__ __forceinline__ void worker_group(float beta1, float omb1, float* __restrict__ z, uint32_t* __restrict__ obits,
                                             int grp, int lane, int L, float s_old, float Sbar,
                                             float4 gv, float4 zv, float4 mv, uint32_t mw, double& acc, bool l1,
                                             bool send_gradient = false)
{
    const int k = grp * kGroup + lane * 4;
    float mm[4];
    if (M32) {
        mm[0] = mv.x; mm[1] = mv.y; mm[2] = mv.z; mm[3] = mv.w;
    } else {
        const uint32_t nib = mw >> (4 * (lane & 7));
#pragma unroll
        for (int e = 0; e < 4; ++e) mm[e] = bit_scale((nib >> e) & 1u, Sbar);
    }
    const float gg[4] = {gv.x, gv.y, gv.z, gv.w};
    const float zo[4] = {zv.x, zv.y, zv.z, zv.w};
    float zn[4];
    uint32_t nibble = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float mi = send_gradient ? gg[e]                                 // gradient variant: g_i itself is compensated
                                       : __fmaf_rn(beta1, mm[e], __fmul_rn(omb1, gg[e]));   // local momentum
        const float err = implied_error(zo[e], s_old);                          // delta_i (old)
        zn[e] = __fadd_rn(mi, err);                                             // compensated
        const bool valid = !CHECKED || (k + e < L);
        if (valid) {
            scale_accumulate(acc, zn[e], l1);
            nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
        }
    }
    const float4 out = make_float4(zn[0], zn[1], zn[2], zn[3]);
    if (CHECKED) st4_checked(z, k, L, out); else st_stream4(z + k, out);
    const uint32_t word = pack_group_words(nibble, lane);
    if ((lane & 7) == 0) {
        const int wk = grp * 4 + (lane >> 3);
        if (!CHECKED || wk * 32 < L) __stcs(obits + wk, word);     // streaming: a plain store here costs ~4 % of the kernel
    }
}

template <int GT, bool M32, int U, int WPC>
__global__ void __launch_bounds__(kThreads, APMS_WORKER_CTAS)
k_worker(const __grid_constant__ GradPtrs G, const WorkerArgs a)
{
    __shared__ double red[kWarps];
    constexpr int TEAMS = kWarps / WPC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t item = (int64_t)blockIdx.x * TEAMS + (WPC == 1 ? warp : 0);
    if (item >= a.items) return;                       // only in the last CTA of the WPC == 1 form
    const int ii = (int)(item % a.ni);
    const Item it = decode_item(a.t, item / a.ni);
    const int i = a.i0 + ii;
    const int L = it.L;
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], it.base);
    float* __restrict__ z = a.z + (int64_t)i * a.dz + it.base;
    const float* __restrict__ m32 = a.m32 + it.base;
    const uint32_t* __restrict__ mbits = a.Bbar + it.base / 32;
    uint32_t* __restrict__ obits = a.B + (int64_t)i * a.Wp + it.base / 32;
    float* sptr = a.s + (int64_t)i * a.Cp + it.c;
    const float s_old = *sptr;
    const float Sbar = M32 ? 0.0f : a.Sbar[it.c];
    const int full = L / kGroup;                  // groups with all 128 elements present
    const int ngroups = (L + kGroup - 1) / kGroup;
    double acc = 0.0;

    int g0 = (WPC == 1) ? 0 : warp;
    // fast path: U groups per warp per iteration, all loads issued before any use
    for (; g0 + WPC * (U - 1) < full; g0 += WPC * U) {
        float4 gv[U], zv[U], mv[U];
        uint32_t mw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int grp = g0 + WPC * u;
            const int k = grp * kGroup + lane * 4;
            gv[u] = Grad<GT>::ld4(g, k);
            zv[u] = ld_stream4(z + k);
            if (M32) mv[u] = *reinterpret_cast<const float4*>(m32 + k);
            else     mw[u] = mbits[grp * 4 + (lane >> 3)];
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            worker_group<M32, false>(a.beta1, a.omb1, z, obits, g0 + WPC * u, lane, L, s_old, Sbar,
                                     gv[u], zv[u], M32 ? mv[u] : make_float4(0, 0, 0, 0), M32 ? 0u : mw[u], acc, a.t.l1 != 0, a.send_gradient != 0);
    }
    // remainder: one group at a time, bounds-checked
    for (; g0 < ngroups; g0 += WPC) {
        const int k = g0 * kGroup + lane * 4;
        const float4 gv = ld_grad4_checked<GT>(g, k, L);
        const float4 zv = ld4_checked(z, k, L, true);
        float4 mv = make_float4(0, 0, 0, 0);
        uint32_t mw = 0;
        if (M32) mv = ld4_checked(m32, k, L, false);
        else if (k < L) mw = mbits[g0 * 4 + (lane >> 3)];
        worker_group<M32, true>(a.beta1, a.omb1, z, obits, g0, lane, L, s_old, Sbar, gv, zv, mv, mw, acc, a.t.l1 != 0, a.send_gradient != 0);
    }

    const double total = team_sum<WPC>(acc, red);
    if ((WPC == 1) ? (lane == 0) : (threadIdx.x == 0)) {
        if (a.t.P == 1) *sptr = scale_from_sum(total, (double)it.Lc, a.t.l1 != 0);    // ||z||_2 / sqrt(L)
        else a.partial[(int64_t)i * a.t.Pp + it.c * a.t.P + it.p] = total;
    }
}

// Worker side, fine-tiled form (steady state, chunk a multiple of kFineSub): one CTA per
// (worker, 4096-element tile), every load of the tile issued before the first use.  Short-lived
// CTAs that each touch 16 KiB of every stream once keep DRAM pages and the memory pipeline busier
// than long-running warps that each follow their own stream.
// Warp w owns the tile's groups 4w..4w+3 (kFineSub = 512 consecutive elements, all of one chunk),
// so its 16 momentum words are one 64-byte load handed round by shuffles, its 16 new sign words
// one 64-byte store, and its binary64 sum of squares one slot of a partial-sum array that
// k_finalize_fine adds up per chunk in element order: the kernel has no barrier at all.
// Launch order: runs of `run` consecutive tiles of one worker, then the same tiles of the next
// worker: every stream is read in long sequential pieces (measured: the longer the better for
// DRAM), while the momentum bits of a run (run * 512 bytes) stay in L2 for the other workers.

constexpr int kFineTile = 4096;           // 256 threads x 4 x (4 floats)
constexpr int kFineU = kFineTile / (kThreads * 4);
constexpr int kFineSub = kFineTile / kWarps;      // elements per warp = per partial sum
constexpr int kFineRunDefault = 4096;

struct WorkerFineArgs {
    float* z; int64_t dz;
    uint32_t* B; int64_t Wp;
    const float* s; int64_t Cp;       // the scales of the previous step (read only here)
    double* partial; int64_t Pp;      // ni rows of tiles * kWarps partial sums, row stride Pp
    const uint32_t* Bbar; const float* Sbar;
    int64_t d, chunk, tiles;
    int i0, ni, run;
    float beta1, omb1;
};

template <int GT, bool SENDG>          // SENDG: the gradient-compressing variant (no momentum is read)
__global__ void __launch_bounds__(kThreads, 4)
k_worker_fine(const __grid_constant__ GradPtrs G, const WorkerFineArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t per_stretch = (int64_t)a.ni * a.run;
    const int64_t stretch = (int64_t)blockIdx.x / per_stretch;
    const int rem = (int)((int64_t)blockIdx.x - stretch * per_stretch);
    const int ii = rem / a.run;
    const int64_t t = stretch * a.run + (rem - ii * a.run);
    if (t >= a.tiles) return;                                  // whole CTA: the last stretch may be short
    const int i = a.i0 + ii;
    const int64_t base = t * kFineTile + (int64_t)warp * kFineSub;     // this warp's 512 elements
    double* __restrict__ slot = a.partial + (int64_t)ii * a.Pp + t * kWarps + warp;
    const int64_t left = a.d - base;
    if (left <= 0) {                                           // past the end of the vector
        if (lane == 0) *slot = 0.0;
        return;
    }
    const int L = (int)(left < kFineSub ? left : kFineSub);
    const int64_t c = base / a.chunk;
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], base);
    float* __restrict__ z = a.z + (int64_t)i * a.dz + base;
    const uint32_t* __restrict__ mbits = a.Bbar + base / 32;
    uint32_t* __restrict__ obits = a.B + (int64_t)i * a.Wp + base / 32;
    const float s_old = a.s[(int64_t)i * a.Cp + c];
    const float Sbar = a.Sbar[c];
    double acc = 0.0;
    if (L == kFineSub) {
        float4 gv[kFineU], zv[kFineU];
#pragma unroll
        for (int u = 0; u < kFineU; ++u) {
            gv[u] = Grad<GT>::ld4(g, u * kGroup + lane * 4);
            zv[u] = ld_stream4(z + u * kGroup + lane * 4);
        }
        const uint32_t mine = (!SENDG && lane < 4 * kFineU) ? mbits[lane] : 0u;
        uint32_t outw = 0;
#pragma unroll
        for (int u = 0; u < kFineU; ++u) {
            const uint32_t nib = __shfl_sync(0xffffffffu, mine, u * 4 + (lane >> 3)) >> (4 * (lane & 7));
            const float gg[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
            const float zo[4] = {zv[u].x, zv[u].y, zv[u].z, zv[u].w};
            float zn[4];
            uint32_t nibble = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float mm = bit_scale((nib >> e) & 1u, Sbar);                    // m = +-Sbar
                const float mi = SENDG ? gg[e] : __fmaf_rn(a.beta1, mm, __fmul_rn(a.omb1, gg[e]));    // local momentum
                zn[e] = __fadd_rn(mi, implied_error(zo[e], s_old));                   // compensated
                const double zd = (double)zn[e];
                acc = fma(zd, zd, acc);
                nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
            }
            st_stream4(z + u * kGroup + lane * 4, make_float4(zn[0], zn[1], zn[2], zn[3]));
            const uint32_t word = pack_group_words(nibble, lane);       // valid in lanes 0, 8, 16, 24
            const uint32_t got = __shfl_sync(0xffffffffu, word, (lane & 3) * 8);
            if ((lane >> 2) == u) outw = got;                               // lane 4u + j keeps word j of group u
        }
        if (lane < 4 * kFineU) __stcs(obits + lane, outw);
    } else {
        const int ngroups = (L + kGroup - 1) / kGroup;
        for (int grp = 0; grp < ngroups; ++grp) {
            const int k = grp * kGroup + lane * 4;
            const float4 gv = ld_grad4_checked<GT>(g, k, L);
            const float4 zv = ld4_checked(z, k, L, true);
            const uint32_t mw = (!SENDG && k < L) ? mbits[grp * 4 + (lane >> 3)] : 0u;
            worker_group<false, true>(a.beta1, a.omb1, z, obits, grp, lane, L, s_old, Sbar, gv, zv,
                                      make_float4(0, 0, 0, 0), mw, acc, false, SENDG);
        }
    }
    acc = warp_sum(acc);
    if (lane == 0) *slot = acc;
}

// Scales from the fine form's partial sums (one per 512 elements): one warp per (row, chunk) adds
// the chunk's slots in a fixed order (lane l takes slots l, l + 32, ..., then the shuffle tree)
// and takes sqrt(sum / L).
__global__ void __launch_bounds__(kThreads)
k_finalize_fine(const double* __restrict__ partial, int64_t Pp, float* __restrict__ scales, int64_t Cp,
                int rows, int64_t C, int64_t d, int64_t chunk)
{
    const int lane = threadIdx.x & 31;
    const int64_t idx = (int64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (idx >= (int64_t)rows * C) return;                        // whole warps
    const int r = (int)(idx / C);
    const int64_t c = idx % C;
    const int64_t cbeg = c * chunk;
    const int64_t Lc = (d - cbeg < chunk) ? d - cbeg : chunk;
    const int64_t q0 = cbeg / kFineSub, q1 = (cbeg + Lc + kFineSub - 1) / kFineSub;
    double total = 0.0;
    for (int64_t q = q0 + lane; q < q1; q += 32) total += partial[(int64_t)r * Pp + q];
    total = warp_sum(total);
    if (lane == 0) scales[(int64_t)r * Cp + c] = (float)sqrt(total / (double)Lc);
}

// Scales of split chunks: partial sums added in tile order, then sqrt(sum / L).
__global__ void k_finalize_scales(const double* __restrict__ partial, float* __restrict__ scales,
                                  int rows, int64_t C, int64_t Cp, Tiling t)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)rows * C) return;
    const int r = (int)(idx / C);
    const int64_t c = idx % C;
    const int64_t cbeg = c * t.chunk;
    const int64_t Lc = (t.d - cbeg < t.chunk) ? t.d - cbeg : t.chunk;
    double total = 0.0;
    for (int p = 0; p < t.P; ++p) total += partial[(int64_t)r * t.Pp + c * t.P + p];
    scales[(int64_t)r * Cp + c] = scale_from_sum(total, (double)Lc, t.l1 != 0);
}

// ------------------------------------------------------------------------------------------
// Server side: average the n decompressed messages, add the server error, recompress
// (Section 3.3 step 4).

struct ServerArgs {
    const uint32_t* B; int64_t Wp;
    const float* s; int64_t Cp;
    float* zbar; uint32_t* Bbar; float* Sbar;
    double* partial;
    Tiling t;
    int64_t item0, items;         // items [item0, items) of the C * P chunk tiles
    int n; float nf;
};

// U groups of one warp: the n sign words of every group are fetched worker by worker while
// the running sums (sequential in worker order, as the average is defined) are updated.
// +-s_i is formed by moving the complemented sign bit onto s_i's sign: no selects, no branches.
template <int U, bool CHECKED>
__device__ __forceinline__ void server_groups(const ServerArgs& a, const float* s_sh, const uint32_t* __restrict__ wb,
                                              float* __restrict__ zb, uint32_t* __restrict__ ob,
                                              int g0, int gstride, int lane, int L, float S_old, double& acc)
{
    const int sh = 4 * (lane & 7);
    const int wl = lane >> 3;
    float sum[U][4];
    float4 zo4[U];
    bool live[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int k = (g0 + gstride * u) * kGroup + lane * 4;
        live[u] = !CHECKED || (k < L);
        zo4[u] = CHECKED ? ld4_checked(zb, k, L, true) : ld_stream4(zb + k);
#pragma unroll
        for (int e = 0; e < 4; ++e) sum[u][e] = 0.0f;
    }
#pragma unroll 4
    for (int i = 0; i < a.n; ++i) {
        const uint32_t sbits = __float_as_uint(s_sh[i]);
        uint32_t w[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            w[u] = live[u] ? wb[(int64_t)i * a.Wp + (g0 + gstride * u) * 4 + wl] : 0u;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t neg = ~w[u] >> sh;            // bit e set: element e of this lane is negative
#pragma unroll
            for (int e = 0; e < 4; ++e)
                sum[u][e] = __fadd_rn(sum[u][e], __uint_as_float(sbits ^ ((neg << (31 - e)) & 0x80000000u)));
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int grp = g0 + gstride * u;
        const int k = grp * kGroup + lane * 4;
        const float zo[4] = {zo4[u].x, zo4[u].y, zo4[u].z, zo4[u].w};
        float zn[4];
        uint32_t nibble = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float avg = __fdiv_rn(sum[u][e], a.nf);
            zn[e] = __fadd_rn(avg, implied_error(zo[e], S_old));
            const bool valid = !CHECKED || (k + e < L);
            if (valid) {
                scale_accumulate(acc, zn[e], a.t.l1 != 0);
                nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
            }
        }
        const float4 out = make_float4(zn[0], zn[1], zn[2], zn[3]);
        if (CHECKED) st4_checked(zb, k, L, out); else st_stream4(zb + k, out);
        const uint32_t word = pack_group_words(nibble, lane);
        const int wk = grp * 4 + wl;
        if ((lane & 7) == 0 && (!CHECKED || wk * 32 < L)) ob[wk] = word;
    }
}

template <int U, int WPC>
__global__ void __launch_bounds__(kThreads, APMS_SERVER_CTAS)
k_server(const ServerArgs a)
{
    __shared__ double red[kWarps];
    __shared__ float s_all[kWarps / WPC][APMS_MAX_WORKERS];
    constexpr int TEAMS = kWarps / WPC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int team = (WPC == 1) ? warp : 0;
    const int64_t item = a.item0 + (int64_t)blockIdx.x * TEAMS + team;
    if (item >= a.items) return;
    const Item it = decode_item(a.t, item);
    const int L = it.L;
    float* s_sh = s_all[team];
    const int tid_in_team = (WPC == 1) ? lane : (int)threadIdx.x;
    for (int i = tid_in_team; i < a.n; i += WPC * 32) s_sh[i] = a.s[(int64_t)i * a.Cp + it.c];
    const float S_old = a.Sbar[it.c];
    if (WPC == 1) __syncwarp(); else __syncthreads();
    const uint32_t* __restrict__ wb = a.B + it.base / 32;
    float* __restrict__ zb = a.zbar + it.base;
    uint32_t* __restrict__ ob = a.Bbar + it.base / 32;
    const int full = L / kGroup;
    const int ngroups = (L + kGroup - 1) / kGroup;
    double acc = 0.0;
    // Each warp takes a contiguous run of groups, so that the 128-byte line of sign words it
    // fetches for a worker serves its next seven groups from L1.
    const int per_warp = (WPC == 1) ? ngroups : (ngroups + WPC - 1) / WPC;
    int g0 = (WPC == 1) ? 0 : warp * per_warp;
    const int g_end = (g0 + per_warp < ngroups) ? g0 + per_warp : ngroups;
    const int g_full = (full < g_end) ? full : g_end;
    for (; g0 + (U - 1) < g_full; g0 += U)
        server_groups<U, false>(a, s_sh, wb, zb, ob, g0, 1, lane, L, S_old, acc);
    for (; g0 < g_end; ++g0)
        server_groups<1, true>(a, s_sh, wb, zb, ob, g0, 1, lane, L, S_old, acc);
    const double total = team_sum<WPC>(acc, red);
    if ((WPC == 1) ? (lane == 0) : (threadIdx.x == 0)) {
        if (a.t.P == 1) a.Sbar[it.c] = scale_from_sum(total, (double)it.Lc, a.t.l1 != 0);
        else a.partial[it.c * a.t.P + it.p] = total;
    }
}

// ------------------------------------------------------------------------------------------
// Server side, staged form.  One CTA per chunk tile: a producer warp streams the tile through a
// ring of shared-memory stages with bulk asynchronous copies (an mbarrier per stage counts the
// arriving bytes, a second one collects the eight consumer warps' releases), so the bytes in
// flight depend neither on registers nor on occupancy, and no CTA-wide barrier sits in the loop.
// When the tile is the whole chunk, the CTA goes on to steps 5-6 for the same chunk (its new
// scale is known once the eight consumer warps have met): v and x travel through the same ring
// while other CTAs of the SM are still in their arithmetic-bound averaging phase.
// Needs every slab of kSlab elements to start on a 16-byte boundary in all streams, i.e.
// chunks that are multiples of kSlab; other shapes use k_server and k_apply.

constexpr int kSlab = 2048;                      // elements per ring stage
constexpr int kSlabGroups = kSlab / kGroup;      // 16 groups, two per consumer warp
constexpr int kSlabWords = kSlab / 32;           // 64 sign words per worker and slab
constexpr int kStages = 4;
constexpr int64_t kStagedSpanElems = 32768;   // a CTA of the fused form walks enough chunks to stream about this many elements
constexpr int kStagedThreads = kThreads + 32;    // eight consumer warps + one producer warp
constexpr long long kWaitCycles = 2000000000ll;  // bound of every wait: about a second of SM clocks

enum { DEVICE_OK = 0, DEVICE_WAIT_TIMEOUT = 1 };

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}
// Bounded wait: false when the phase did not complete within `limit` SM clocks.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long limit = kWaitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int k = 0; k < 32; ++k)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit) return false;
    }
}

// Self-test of the give-up path: a barrier that nothing ever completes, waited for with a short bound.
// No copy is in flight and nothing else is touched, so the CTA simply reports and ends.
__global__ void k_selftest_wait(int* status, long long limit)
{
    __shared__ uint64_t never;
    if (threadIdx.x == 0) { mbar_init(&never, 1); mbar_fence_init(); }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(&never, 0, limit)) atomicExch(status, DEVICE_WAIT_TIMEOUT);
}
// Global -> this CTA's shared memory; 16-byte aligned addresses, size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Barrier among the 256 consumer threads only (the producer warp never joins it).
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

struct ServerStagedArgs {
    ServerArgs a;
    int* status;          // device status word: set when a bounded wait gave up
    float inv_n;          // 1/n when n is a power of two (then avg = sum * inv_n is the exact quotient), else 0
    const float* v; float* x; float lr, eps;     // steps 5-6, used by the fused form only
    int span;             // chunks per CTA of the fused form
};

// Bytes of one ring stage: a slab of zbar plus n rows of sign words, or (fused form) a slab of v and of x.
__host__ __device__ __forceinline__ size_t staged_stage_bytes(int n, bool fused)
{
    const size_t server = (size_t)kSlab * 4 + (size_t)n * kSlabWords * 4;
    const size_t apply = (size_t)kSlab * 8;
    return (fused && apply > server) ? apply : server;
}

// Sum over the workers, in worker order, of +-s_i for the lane's 2 x 4 elements of one slab.
// NT > 0: the number of workers is the compile-time constant NT (fully unrolled).
template <int NT>
__device__ __forceinline__ void signed_scale_sums(const uint32_t* __restrict__ r0, const uint32_t* __restrict__ r1,
                                                  const uint32_t* __restrict__ neg_s, int n, int sh,
                                                  float2& s01, float2& s23, float2& t01, float2& t23)
{
    const int nn = NT > 0 ? NT : n;
#pragma unroll(NT > 0 ? NT : 4)
    for (int i = 0; i < nn; ++i) {
        const uint32_t ns = neg_s[i];
        // the lane's four sign bits moved to bits 28..31; a set bit turns -s_i into +s_i
        const uint32_t y0 = r0[i * kSlabWords] << (28 - sh);
        const uint32_t y1 = r1[i * kSlabWords] << (28 - sh);
        float2 q;
        q.x = __uint_as_float(((y0 << 3) & 0x80000000u) ^ ns); q.y = __uint_as_float(((y0 << 2) & 0x80000000u) ^ ns);
        s01 = __fadd2_rn(s01, q);
        q.x = __uint_as_float(((y0 << 1) & 0x80000000u) ^ ns); q.y = __uint_as_float((y0 & 0x80000000u) ^ ns);
        s23 = __fadd2_rn(s23, q);
        q.x = __uint_as_float(((y1 << 3) & 0x80000000u) ^ ns); q.y = __uint_as_float(((y1 << 2) & 0x80000000u) ^ ns);
        t01 = __fadd2_rn(t01, q);
        q.x = __uint_as_float(((y1 << 1) & 0x80000000u) ^ ns); q.y = __uint_as_float((y1 & 0x80000000u) ^ ns);
        t23 = __fadd2_rn(t23, q);
    }
}

// A CTA of the fused form walks `span` consecutive chunks (short chunks are grouped so that a CTA
// still streams about 32768 elements and the ring never drains between chunks); the unfused form
// (chunks cut into tiles) handles one tile.  Jobs are numbered across the CTA's whole walk: per
// chunk first its server slabs, then (fused) its slabs of v and x; job q uses stage q % kStages.
template <int NT, bool FUSED, bool MULTI>
__global__ void __launch_bounds__(kStagedThreads, 3)
k_server_staged(const ServerStagedArgs sa)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const ServerArgs& a = sa.a;
    __shared__ double red[kWarps];
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ uint32_t neg_s[2][APMS_MAX_WORKERS];   // bit patterns of -s_i, double-buffered over the walk
    __shared__ uint32_t nb[kTileMax / 32];            // the current tile's new sign words
    __shared__ int failed;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = NT > 0 ? NT : a.n;
    const size_t stage_bytes = staged_stage_bytes(n, FUSED);
    const int span = MULTI ? sa.span : 1;                  // MULTI = false: one item, the walk's loops fold away
    const int64_t item0 = a.item0 + (int64_t)blockIdx.x * span;
    const int nitems = MULTI ? (int)(a.items - item0 < span ? a.items - item0 : span) : 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWarps); }
        failed = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kWarps) {
        // ---- producer warp: one lane feeds the ring (only whole 16-byte pieces that hold live elements)
        if (lane == 0) {
            int q = 0;
            bool stop = false;
            for (int w = 0; w < nitems && !stop; ++w) {
                const Item it = decode_item(a.t, item0 + w);
                const int L = it.L;
                const int nslabs = (L + kSlab - 1) / kSlab;
                const int njobs = FUSED ? 2 * nslabs : nslabs;
                const float* __restrict__ zb_g = a.zbar + it.base;
                const uint32_t* __restrict__ wb_g = a.B + it.base / 32;
                for (int r = 0; r < njobs; ++r, ++q) {
                    const int st = q % kStages;
                    if (q >= kStages && !mbar_wait(&empty[st], (uint32_t)(q / kStages - 1) & 1u)) { failed = 1; stop = true; break; }
                    unsigned char* base = smem + (size_t)st * stage_bytes;
                    const int j = r < nslabs ? r : r - nslabs;
                    const int left = L - j * kSlab;
                    const int live = left < kSlab ? left : kSlab;
                    const uint32_t zbytes = (uint32_t)((live + 3) / 4) * 16u;
                    if (r < nslabs) {
                        const uint32_t wbytes = (uint32_t)(((live + 31) / 32 + 3) / 4) * 16u;
                        mbar_arrive_expect_tx(&full[st], zbytes + (uint32_t)n * wbytes);
                        bulk_load(base, zb_g + (size_t)j * kSlab, zbytes, &full[st]);
                        uint32_t* rows = reinterpret_cast<uint32_t*>(base + (size_t)kSlab * 4);
                        for (int i = 0; i < n; ++i)
                            bulk_load(rows + i * kSlabWords, wb_g + (int64_t)i * a.Wp + (size_t)j * kSlabWords, wbytes, &full[st]);
                    } else {
                        mbar_arrive_expect_tx(&full[st], 2 * zbytes);
                        bulk_load(base, sa.v + it.base + (size_t)j * kSlab, zbytes, &full[st]);
                        bulk_load(base + (size_t)kSlab * 4, sa.x + it.base + (size_t)j * kSlab, zbytes, &full[st]);
                    }
                }
            }
            if (failed) {
                // give the copies still in flight a bounded chance to land before shared memory is released
                const int first = q > kStages ? q - kStages : 0;
                for (int p = first; p < q; ++p) mbar_wait(&full[p % kStages], (uint32_t)(p / kStages) & 1u);
            }
        }
    } else {
        // ---- consumer warps: two 128-element groups of every slab each
        const int sh = 4 * (lane & 7);
        const int wl = lane >> 3;
        const int g0 = warp, g1 = warp + kWarps;
        // A warp whose wait gives up sets `failed`, skips the rest of its phase and still arrives at the next
        // consumer barrier; after every barrier all consumers read `failed` and leave together.
        int q = 0;
        for (int w = 0; w < nitems; ++w) {
            const Item it = decode_item(a.t, item0 + w);
            const int L = it.L;
            const int nslabs = (L + kSlab - 1) / kSlab;
            uint32_t* negs = neg_s[w & 1];
            for (int i = threadIdx.x; i < n; i += kThreads)
                negs[i] = __float_as_uint(a.s[(int64_t)i * a.Cp + it.c]) | 0x80000000u;
            const float S_old = a.Sbar[it.c];
            consumer_barrier();                        // -s_i in place; everybody is done with the previous chunk
            if (failed) break;
            bool ok = true;
            double acc = 0.0;
            for (int j = 0; j < nslabs; ++j, ++q) {
                const int st = q % kStages;
                if (!mbar_wait(&full[st], (uint32_t)(q / kStages) & 1u)) { failed = 1; ok = false; break; }
                const unsigned char* base = smem + (size_t)st * stage_bytes;
                const float* zs = reinterpret_cast<const float*>(base);
                const uint32_t* rows = reinterpret_cast<const uint32_t*>(base + (size_t)kSlab * 4);
                const float4 zo0 = *reinterpret_cast<const float4*>(zs + g0 * kGroup + lane * 4);
                const float4 zo1 = *reinterpret_cast<const float4*>(zs + g1 * kGroup + lane * 4);
                float2 s01 = make_float2(0.f, 0.f), s23 = s01, t01 = s01, t23 = s01;   // running sums, worker order
                signed_scale_sums<NT>(rows + g0 * 4 + wl, rows + g1 * 4 + wl, negs, n, sh, s01, s23, t01, t23);
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[st]);                  // this warp is done with the stage
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int grp = j * kSlabGroups + (u ? g1 : g0);
                    const int k = grp * kGroup + lane * 4;
                    const float4 zo4 = u ? zo1 : zo0;
                    const float zo[4] = {zo4.x, zo4.y, zo4.z, zo4.w};
                    const float sum[4] = {u ? t01.x : s01.x, u ? t01.y : s01.y, u ? t23.x : s23.x, u ? t23.y : s23.y};
                    float zn[4];
                    uint32_t nibble = 0;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float avg = (sa.inv_n != 0.0f) ? __fmul_rn(sum[e], sa.inv_n) : __fdiv_rn(sum[e], a.nf);
                        zn[e] = __fadd_rn(avg, implied_error(zo[e], S_old));
                        if (k + e < L) {
                            const double zd = (double)zn[e];
                            acc = fma(zd, zd, acc);
                            nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
                        }
                    }
                    st4_checked(a.zbar + it.base, k, L, make_float4(zn[0], zn[1], zn[2], zn[3]));
                    const uint32_t word = pack_group_words(nibble, lane);
                    if ((lane & 7) == 0) nb[grp * 4 + wl] = word;        // words past L hold zeros and are never stored
                }
            }
            acc = warp_sum(acc);
            if (lane == 0) red[warp] = acc;
            consumer_barrier();                        // partial sums and sign words of the tile are in shared memory
            double total = 0.0;
#pragma unroll
            for (int r = 0; r < kWarps; ++r) total += red[r];
            if (failed) break;
            if (FUSED) {
                // Section 3.3 steps 5-6 for this chunk: m <- +-Sbar, x <- x - lr m / (sqrt(v) + eps)
                const float S_new = (float)sqrt(total / (double)it.Lc);
                if (ok && threadIdx.x == 0) a.Sbar[it.c] = S_new;
                for (int j = 0; ok && j < nslabs; ++j, ++q) {
                    const int st = q % kStages;
                    if (!mbar_wait(&full[st], (uint32_t)(q / kStages) & 1u)) { failed = 1; ok = false; break; }
                    const float* vs = reinterpret_cast<const float*>(smem + (size_t)st * stage_bytes);
                    const float* xs = vs + kSlab;
                    float4 vv[2], xx[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        vv[u] = *reinterpret_cast<const float4*>(vs + (u ? g1 : g0) * kGroup + lane * 4);
                        xx[u] = *reinterpret_cast<const float4*>(xs + (u ? g1 : g0) * kGroup + lane * 4);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&empty[st]);
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int grp = j * kSlabGroups + (u ? g1 : g0);
                        const int k = grp * kGroup + lane * 4;
                        const uint32_t nib = nb[grp * 4 + wl] >> sh;
                        xx[u].x = apply_elem(xx[u].x, vv[u].x, bit_scale(nib & 1u, S_new), sa.lr, sa.eps);
                        xx[u].y = apply_elem(xx[u].y, vv[u].y, bit_scale(nib & 2u, S_new), sa.lr, sa.eps);
                        xx[u].z = apply_elem(xx[u].z, vv[u].z, bit_scale(nib & 4u, S_new), sa.lr, sa.eps);
                        xx[u].w = apply_elem(xx[u].w, vv[u].w, bit_scale(nib & 8u, S_new), sa.lr, sa.eps);
                        st4_checked(sa.x + it.base, k, L, xx[u]);
                    }
                }
            } else if (ok && threadIdx.x == 0) {
                if (a.t.P == 1) a.Sbar[it.c] = (float)sqrt(total / (double)it.Lc);
                else a.partial[it.c * a.t.P + it.p] = total;
            }
            // the tile's sign words leave in whole 16-byte pieces (full lines for full tiles)
            if (ok) {
                uint32_t* __restrict__ ob = a.Bbar + it.base / 32;
                const int nwords = (L + 31) / 32;
                for (int w4 = threadIdx.x * 4; w4 < nwords; w4 += kThreads * 4) {
                    if (w4 + 3 < nwords) __stcs(reinterpret_cast<uint4*>(ob + w4), *reinterpret_cast<const uint4*>(nb + w4));
                    else for (int r = w4; r < nwords; ++r) ob[r] = nb[r];
                }
            }
        }
    }
    __syncthreads();                                   // every warp has left its loops; shared memory may go
    if (threadIdx.x == 0 && failed) atomicExch(sa.status, DEVICE_WAIT_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// Worker side again: the received chunk replaces the momentum (it stays in its compressed
// form) and the model moves with the frozen variance (Section 3.3 steps 5-6).
// One CTA per 8192 consecutive elements, whatever the chunk length.

constexpr int kApplyTile = 4096;
constexpr int kApplyU = kApplyTile / (kThreads * 4);

struct ApplyArgs {
    const uint32_t* Bbar; const float* Sbar; const float* v; float* x;
    int64_t d; int64_t chunk; float lr, eps;
};

__global__ void __launch_bounds__(kThreads)
k_apply(const ApplyArgs a)
{
    const int64_t base = (int64_t)blockIdx.x * kApplyTile;
    const int64_t left = a.d - base;
    const int L = (int)(left < kApplyTile ? left : kApplyTile);
    const int64_t c0 = base / a.chunk;
    const uint32_t off0 = (uint32_t)(base - c0 * a.chunk);
    const uint32_t chunk32 = (uint32_t)a.chunk;
    const uint32_t* __restrict__ bits = a.Bbar + base / 32;
    const float* __restrict__ v = a.v + base;
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
            S[u] = Sb[rel < chunk32 ? 0u : rel / chunk32];
        }
#pragma unroll
        for (int u = 0; u < kApplyU; ++u) {
            const int k = (u * kThreads + threadIdx.x) * 4;
            xx[u].x = apply_elem(xx[u].x, vv[u].x, bit_scale(nib[u] & 1u, S[u]), a.lr, a.eps);
            xx[u].y = apply_elem(xx[u].y, vv[u].y, bit_scale(nib[u] & 2u, S[u]), a.lr, a.eps);
            xx[u].z = apply_elem(xx[u].z, vv[u].z, bit_scale(nib[u] & 4u, S[u]), a.lr, a.eps);
            xx[u].w = apply_elem(xx[u].w, vv[u].w, bit_scale(nib[u] & 8u, S[u]), a.lr, a.eps);
            st_stream4(x + k, xx[u]);
        }
        return;
    }
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        const uint32_t rel = off0 + (uint32_t)k;
        const float S = Sb[rel < chunk32 ? 0u : rel / chunk32];
        const uint32_t nib = bits[k >> 5] >> (k & 31);
        if (k + 3 < L) {
            const float4 vv = ld_stream4(v + k);
            float4 xx = ld_stream4(x + k);
            xx.x = apply_elem(xx.x, vv.x, bit_scale(nib & 1u, S), a.lr, a.eps);
            xx.y = apply_elem(xx.y, vv.y, bit_scale(nib & 2u, S), a.lr, a.eps);
            xx.z = apply_elem(xx.z, vv.z, bit_scale(nib & 4u, S), a.lr, a.eps);
            xx.w = apply_elem(xx.w, vv.w, bit_scale(nib & 8u, S), a.lr, a.eps);
            st_stream4(x + k, xx);
        } else {
            for (int e = 0; e < 4 && k + e < L; ++e)
                x[k + e] = apply_elem(x[k + e], v[k + e], bit_scale((nib >> e) & 1u, S), a.lr, a.eps);
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
                a.m[j + e] = mn;
                a.x[j + e] = apply_elem(a.x[j + e], a.v[j + e], mn, a.lr, a.eps);
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
            a.m[e] = m; a.x[e] = x;
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

// ------------------------------------------------------------------------------------------
// Top-k compressor (Section 5.1, second item): per chunk the K = ceil(k L) elements of largest |z| are
// sent, the others decompress to 0; equal magnitudes go to the lower index.  State in this mode: the
// compensated vectors z as before, and in place of the sign words a SELECTION MASK (bit j = element j
// was sent), from which  C[z] = mask ? z : 0  and  delta = z - C[z]  follow exactly; the momentum is
// kept in binary32.  One CTA per (chunk, worker) / per chunk; a chunk's z is written once and re-read
// from L2 by the selection passes.
//
// Selection: the K-th largest magnitude is found by a three-level radix select over the bit pattern of
// |z| (11 + 11 + 9 bits, shared-memory histograms), giving the threshold key tau and the number of
// elements equal to tau that are still to be kept; a last pass in index order marks  key > tau, and the
// first `ties` elements with key == tau.

constexpr int kTopkBins = 2048;

__device__ __forceinline__ uint32_t mag_key(float z) { return __float_as_uint(z) & 0x7fffffffu; }

// C[z] and the error it leaves, from a stored compensated value and its selection bit (the subtraction is
// the one the method performs, so that non-finite values behave as they do there).
__device__ __forceinline__ float topk_error(float z, uint32_t selected) { return __fsub_rn(z, selected ? z : 0.0f); }

// hist[0..nbins) are counts; K >= 1 is the rank wanted, counted from the top bin.  Returns (to all threads)
// the bin that holds the K-th key and reduces K to the rank inside that bin.  Ends with a barrier.
__device__ __forceinline__ int topk_find_bin(const uint32_t* hist, int nbins, uint32_t& K, uint32_t* sh)
{
    __syncthreads();                                   // the histogram is complete
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x, per = nbins / 32;
        const int hi = nbins - lane * per, lo = hi - per;             // lane 0 owns the top bins
        uint32_t mine = 0;
        for (int b = lo; b < hi; ++b) mine += hist[b];
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        const uint32_t excl = incl - mine;
        if (excl < K && K <= incl) {                   // exactly one lane
            uint32_t k = K - excl;
            int b = hi - 1;
            for (; b > lo; --b) { if (k <= hist[b]) break; k -= hist[b]; }
            sh[0] = (uint32_t)b; sh[1] = k;
        }
    }
    __syncthreads();
    K = sh[1];
    return (int)sh[0];
}

// Threshold of the K largest magnitudes of zc[0..L) (global memory, written by this CTA).  hist must hold
// the level-0 histogram (key >> 20) already.  Out: tau and the number of elements equal to tau to keep.
__device__ __forceinline__ void topk_threshold(const float* zc, int L, uint32_t K, uint32_t* hist, uint32_t* sh,
                                               uint32_t& tau, uint32_t& ties)
{
    const uint32_t b0 = (uint32_t)topk_find_bin(hist, kTopkBins, K, sh);
    for (int b = threadIdx.x; b < kTopkBins; b += kThreads) hist[b] = 0;
    __syncthreads();
    // the lower levels spread over many bins: plain atomics (combining equal bins costs more than it saves there)
#pragma unroll 4
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        const float4 zv = ld4_checked(zc, k, L, false);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (k + e < L && (key[e] >> 20) == b0) atomicAdd(&hist[(key[e] >> 9) & 0x7ffu], 1u);
    }
    const uint32_t b1 = (uint32_t)topk_find_bin(hist, kTopkBins, K, sh);
    for (int b = threadIdx.x; b < 512; b += kThreads) hist[b] = 0;
    __syncthreads();
    const uint32_t top = (b0 << 11) | b1;
#pragma unroll 4
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        const float4 zv = ld4_checked(zc, k, L, false);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (k + e < L && (key[e] >> 9) == top) atomicAdd(&hist[key[e] & 0x1ffu], 1u);
    }
    const uint32_t b2 = (uint32_t)topk_find_bin(hist, 512, K, sh);
    tau = (top << 9) | b2;
    ties = K;
}

// Last step's threshold of the same (worker, chunk) predicts this step's: only the keys at or above a
// floor a little below it (key lowered by 2^20, an eighth of an exponent step: 0.92 of the threshold) are
// looked at for the selection, which is exact either way - a chunk whose window turns out to hold fewer
// than K keys, or more than the list below can take, goes the general route (histograms over the whole
// chunk, re-read from L2).  Error feedback piles the unsent elements up just under the threshold, and while
// the errors still build up the threshold rises by 5 to 10 % a step, so the window holds several times K
// keys (about 4 K on the benchmark's gradients at k = 1 %).  Hence a window only for K <= kTopkList / 6;
// for larger K the first pass builds the top-level histogram of all keys itself.  A stored threshold of 0
// (first step) also means no window.  The list is kept small on purpose: shared memory comes out of the L1
// cache, which the first pass, the general route and the server's sparse sum live on (a list of 4096 entries
// made the worker 45 % and the server 30 % slower).
constexpr int kTopkList = 2048;
constexpr uint32_t kTopkFloorDrop = 1u << 20;
__device__ __forceinline__ uint32_t topk_floor(float last_threshold, uint32_t K)
{
    const uint32_t key = mag_key(last_threshold);
    return (6 * K <= (uint32_t)kTopkList && key > kTopkFloorDrop) ? key - kTopkFloorDrop : 0u;
}

// The keys inside the window are appended, with their positions in the chunk (16 bits: the list is used
// for chunks of up to 65536 elements), to a list in shared memory, and threshold and mask are then taken
// from the list alone - no further pass over the chunk.
// From this kept fraction on the server sums the workers' messages in registers (see k_topk_server): measured
// on 16 workers, 335 M elements, the scattered form takes 2.7 / 3.7 / 5.9 / 12.4 ms at k = 0.1 / 1 / 3 / 10 %,
// the register form 3.8 / 4.6 / 5.2 / 5.9 ms.
constexpr double kTopkDenseSum = 0.02;
// Resident CTAs per SM the top-k kernels are compiled for.  Their passes are latency-bound, so residency
// matters more than registers, but at eight (32 registers) the spills cost more than the two CTAs give:
// six measured fastest (worker 16.5 ms against 23.2 at eight and 17.9 at four, 16 workers, 335 M elements).
constexpr int kTopkResident = 6;

struct TopkList { uint32_t key[kTopkList]; uint16_t idx[kTopkList]; uint32_t count; };

__device__ __forceinline__ void topk_list_add(TopkList& l, uint32_t key, uint32_t idx)
{
    const uint32_t pos = atomicAdd(&l.count, 1u);
    if (pos < (uint32_t)kTopkList) { l.key[pos] = key; l.idx[pos] = (uint16_t)idx; }
}

// Threshold of the K largest keys of the list (n >= K entries, all >= floor_key).  The keys lie in a
// narrow band above the floor, so the select runs on rel = key - floor_key in three 8-bit levels (bits
// 23..16, clipped at 255; 15..8; 7..0) with 256-bin histograms: one bin per thread to clear, eight per lane
// to scan.  Returns false, with nothing decided, when the K-th key lies in the clipped bin (it is then
// more than four times the floor).  Also returns how many keys equal tau in all (ties_total); ties <=
// ties_total of them are to be kept.
static_assert(kThreads == 256, "one histogram bin per thread");
__device__ __forceinline__ bool topk_threshold_list(const TopkList& l, int n, uint32_t floor_key, uint32_t K,
                                                    uint32_t* hist /* 256 bins */, uint32_t* sh,
                                                    uint32_t& tau, uint32_t& ties, uint32_t& ties_total)
{
    hist[threadIdx.x] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < n; p += kThreads) {
        const uint32_t rel = l.key[p] - floor_key;
        atomicAdd(&hist[rel >> 16 < 255u ? rel >> 16 : 255u], 1u);
    }
    const uint32_t b0 = (uint32_t)topk_find_bin(hist, 256, K, sh);
    if (b0 == 255u) return false;                      // the same value in every thread
    hist[threadIdx.x] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < n; p += kThreads) {
        const uint32_t rel = l.key[p] - floor_key;
        if (rel >> 16 == b0) atomicAdd(&hist[(rel >> 8) & 0xffu], 1u);
    }
    const uint32_t b1 = (uint32_t)topk_find_bin(hist, 256, K, sh);
    hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t top = (b0 << 8) | b1;
    for (int p = threadIdx.x; p < n; p += kThreads) {
        const uint32_t rel = l.key[p] - floor_key;
        if (rel >> 8 == top) atomicAdd(&hist[rel & 0xffu], 1u);
    }
    const uint32_t b2 = (uint32_t)topk_find_bin(hist, 256, K, sh);
    tau = floor_key + ((top << 8) | b2);
    ties = K;
    ties_total = hist[b2];
    __syncthreads();                                   // the bins are reused by the caller
    return true;
}

// Is list entry p among the kept?  Keys above tau are; of the ties_total keys equal to tau the `ties` with
// the lowest positions are (the ranking scans the list: only when not every tie is kept).
__device__ __forceinline__ bool topk_list_selected(const TopkList& l, int n, int p, uint32_t tau, uint32_t ties, uint32_t ties_total)
{
    const uint32_t key = l.key[p];
    if (key != tau) return key > tau;
    if (ties == ties_total) return true;
    const uint32_t idx = l.idx[p];
    uint32_t before = 0;
    for (int q = 0; q < n; ++q) before += (l.key[q] == tau && l.idx[q] < idx) ? 1u : 0u;
    return before < ties;
}

// Without a window the first pass counts every key in 2048 bins of half the usual width (key >> 19: a
// sixteenth of an exponent step), laid around the last threshold (64 exponent steps either way; around 1
// when there is none yet), keys outside going to the end bins.  The bin of the K-th key then holds few
// enough keys for the list (about 1000 of 32768 at k = 10 % on the benchmark's gradients), so that a second
// pass settles the selection: keys in higher bins are kept, those of the bin itself go to the list, which
// decides them.  Chunks of more than 65536 elements count key >> 20 from 0 (every key has its own bin) and
// take the general route.
__device__ __forceinline__ int topk_fine_base(float last_threshold)
{
    const int t = (int)(mag_key(last_threshold) >> 19);
    if (t == 0) return 1024;
    return t < 1024 ? 0 : (t > 3072 ? 2048 : t - 1024);
}
__device__ __forceinline__ int topk_bin(uint32_t key, int shift, int base)
{
    const int b = (int)(key >> shift) - base;
    return b < 0 ? 0 : (b > kTopkBins - 1 ? kTopkBins - 1 : b);
}

// Top-level histogram over the whole chunk (general route).
__device__ __forceinline__ void topk_full_hist(const float* zc, int L, uint32_t* hist)
{
    for (int b = threadIdx.x; b < kTopkBins; b += kThreads) hist[b] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < L; j += kThreads) atomicAdd(&hist[mag_key(zc[j]) >> 20], 1u);
}

// One wave (1024 elements) of the ordered pass: the thread holds the keys of 4 consecutive elements
// (validmask: which of them exist) and gets back the nibble of its selected elements.  `seen` counts the
// elements equal to tau in earlier positions (same value in every thread).
__device__ __forceinline__ uint32_t topk_select_wave(const uint32_t key[4], uint32_t validmask, uint32_t tau, uint32_t ties,
                                                     uint32_t& seen, uint32_t* warp_ties)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t cnt = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) cnt += ((validmask >> e) & 1u) && key[e] == tau;
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_ties[warp] = incl;
    __syncthreads();
    uint32_t before = seen, total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { const uint32_t c = warp_ties[w]; if (w < warp) before += c; total += c; }
    before += incl - cnt;
    seen += total;
    __syncthreads();                                   // warp_ties may be rewritten by the next wave
    uint32_t nibble = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        if ((validmask >> e) & 1u) {
            const bool tie = key[e] == tau;
            if (key[e] > tau || (tie && before < ties)) nibble |= 1u << e;
            before += tie;
        }
    }
    return nibble;
}

struct TopkWorkerArgs {
    float* z; int64_t dz;
    uint32_t* B; int64_t Wp;          // selection masks
    const float* m32;
    float* thr; int64_t Cp;           // per (worker, chunk): the magnitude of the K-th element of the last step
    int64_t d, chunk, C;
    int i0, ni;
    float beta1, omb1;
    double frac;
};

__device__ __forceinline__ uint32_t topk_count(double frac, int L)
{
    long long K = (long long)ceil(frac * (double)L);
    if (K < 1) K = 1;
    if (K > L) K = L;
    return (uint32_t)K;
}

template <int GT>
__global__ void __launch_bounds__(kThreads, kTopkResident)
k_topk_worker(const __grid_constant__ GradPtrs G, const TopkWorkerArgs a)
{
    __shared__ uint32_t hist[kTopkBins];
    __shared__ uint32_t bins8[256];
    __shared__ uint32_t sh[2];
    __shared__ uint32_t warp_ties[kWarps];
    __shared__ TopkList list;
    const int ii = (int)(blockIdx.x % a.ni);
    const int64_t c = blockIdx.x / a.ni;
    const int i = a.i0 + ii;
    const int64_t base = c * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], base);
    float* zc = a.z + (int64_t)i * a.dz + base;
    uint32_t* maskw = a.B + (int64_t)i * a.Wp + base / 32;
    const float* __restrict__ m = a.m32 + base;
    float* thr = a.thr + (int64_t)i * a.Cp + c;
    const uint32_t K = topk_count(a.frac, L);
    const int nwords = (L + 31) / 32;
    const bool small = nwords <= kTopkBins;            // the mask fits the shared-memory words: list routes possible
    const uint32_t floor_key = small ? topk_floor(*thr, K) : 0u;
    const int shift = small ? 19 : 20, bin0 = small ? topk_fine_base(*thr) : 0;

    for (int b = threadIdx.x; b < kTopkBins; b += kThreads) hist[b] = 0;
    if (threadIdx.x == 0) list.count = 0;
    __syncthreads();
    // pass A: z = (b1 m + (1-b1) g) + delta_old, with delta_old from the stored z and last step's mask;
    // whole 1024-element sweeps without bounds checks, two sweeps' loads in flight, then the ragged rest
    const int Lfull = L & ~(kThreads * 4 - 1);
    auto sweep = [&](int k, float4 gv, float4 zv, float4 mv, uint32_t nib, bool checked) {
        const float gg[4] = {gv.x, gv.y, gv.z, gv.w}, zo[4] = {zv.x, zv.y, zv.z, zv.w}, mm[4] = {mv.x, mv.y, mv.z, mv.w};
        float zn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float mi = __fmaf_rn(a.beta1, mm[e], __fmul_rn(a.omb1, gg[e]));
            zn[e] = __fadd_rn(mi, topk_error(zo[e], (nib >> e) & 1u));
            if (!checked || k + e < L) {
                const uint32_t key = mag_key(zn[e]);
                if (floor_key == 0) atomicAdd(&hist[topk_bin(key, shift, bin0)], 1u);     // no window: every key counts
                else if (key >= floor_key) topk_list_add(list, key, (uint32_t)(k + e));
            }
        }
        if (!checked || k + 3 < L) *reinterpret_cast<float4*>(zc + k) = make_float4(zn[0], zn[1], zn[2], zn[3]);
        else for (int e = 0; e < 4 && k + e < L; ++e) zc[k + e] = zn[e];
    };
    int k = threadIdx.x * 4;
    for (; k + kThreads * 4 < Lfull; k += 2 * kThreads * 4) {
        const int k2 = k + kThreads * 4;
        const float4 g0 = Grad<GT>::ld4(g, k), g1 = Grad<GT>::ld4(g, k2);
        const float4 z0 = *reinterpret_cast<const float4*>(zc + k), z1 = *reinterpret_cast<const float4*>(zc + k2);
        const float4 m0 = *reinterpret_cast<const float4*>(m + k), m1 = *reinterpret_cast<const float4*>(m + k2);
        const uint32_t n0 = maskw[k >> 5] >> (k & 31), n1 = maskw[k2 >> 5] >> (k2 & 31);
        sweep(k, g0, z0, m0, n0, false);
        sweep(k2, g1, z1, m1, n1, false);
    }
    for (; k < Lfull; k += kThreads * 4)
        sweep(k, Grad<GT>::ld4(g, k), *reinterpret_cast<const float4*>(zc + k), *reinterpret_cast<const float4*>(m + k),
              maskw[k >> 5] >> (k & 31), false);
    for (; k < L; k += kThreads * 4)
        sweep(k, ld_grad4_checked<GT>(g, k, L), ld4_checked(zc, k, L, false), ld4_checked(m, k, L, false),
              maskw[k >> 5] >> (k & 31), true);
    __syncthreads();                                   // z stores, histogram and list are complete
    const int lane = threadIdx.x & 31;
    int n_list = 0;                                    // > 0: the list decides, hist[0..nwords) holds the mask so far
    uint32_t K_list = K, floor_list = floor_key;
    if (floor_key != 0) {                              // window route: the mask words are still all zero
        const uint32_t listed = list.count;
        if (listed >= K && listed <= (uint32_t)kTopkList) n_list = (int)listed;
    } else if (small) {                                // two-pass route
        uint32_t Kb = K;
        const int b0 = topk_find_bin(hist, kTopkBins, Kb, sh);
        const uint32_t inbin = hist[b0];
        __syncthreads();                               // everybody has read the histogram: its words become the mask
        if (b0 > 0 && b0 < kTopkBins - 1 && inbin <= (uint32_t)kTopkList) {
            for (int w0 = 0; w0 < L; w0 += kThreads * 4) {
                const int k = w0 + threadIdx.x * 4;
                const float4 zv = ld4_checked(zc, k, L, false);
                const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
                uint32_t nibble = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (k + e < L) {
                        const int b = topk_bin(key[e], 19, bin0);
                        if (b > b0) nibble |= 1u << e;
                        else if (b == b0) topk_list_add(list, key[e], (uint32_t)(k + e));
                    }
                }
                const uint32_t word = pack_group_words(nibble, lane);   // valid in lanes 0, 8, 16, 24
                if ((lane & 7) == 0 && k < L) hist[k >> 5] = word;
            }
            __syncthreads();
            n_list = (int)inbin; K_list = Kb; floor_list = (uint32_t)(b0 + bin0) << 19;
        }
    }
    uint32_t tau, ties;
    bool have_tau = false;
    if (n_list > 0) {
        uint32_t ties_total;
        have_tau = topk_threshold_list(list, n_list, floor_list, K_list, bins8, sh, tau, ties, ties_total);
        if (have_tau) {
            for (int p = threadIdx.x; p < n_list; p += kThreads)
                if (topk_list_selected(list, n_list, p, tau, ties, ties_total))
                    atomicOr(&hist[list.idx[p] >> 5], 1u << (list.idx[p] & 31u));
            __syncthreads();
            for (int w = threadIdx.x; w < nwords; w += kThreads) maskw[w] = hist[w];
            if (threadIdx.x == 0) *thr = __uint_as_float(tau);
            return;
        }
    }
    // general route: histograms over the whole chunk
    if (small) topk_full_hist(zc, L, hist);
    topk_threshold(zc, L, K, hist, sh, tau, ties);
    if (threadIdx.x == 0) *thr = __uint_as_float(tau);
    // ordered pass over the chunk: the selection mask with the tie rule
    uint32_t seen = 0;
    for (int w0 = 0; w0 < L; w0 += kThreads * 4) {
        const int k = w0 + threadIdx.x * 4;
        const float4 zv = ld4_checked(zc, k, L, false);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
        const uint32_t validmask = k + 3 < L ? 0xfu : (k < L ? (1u << (L - k)) - 1u : 0u);
        const uint32_t nibble = topk_select_wave(key, validmask, tau, ties, seen, warp_ties);
        const uint32_t word = pack_group_words(nibble, lane);       // valid in lanes 0, 8, 16, 24
        if ((lane & 7) == 0 && k < L) maskw[k >> 5] = word;
    }
}

struct TopkServerArgs {
    const float* z; int64_t dz;       // the workers' compensated vectors
    const uint32_t* B; int64_t Wp;    // and their masks
    float* zbar; uint32_t* Bbar;      // the server's compensated vector and mask
    float* m32;                       // accumulator during the step, the new momentum after it
    float* thr;                       // per chunk: the magnitude of the K-th element of the last step
    const float* v; float* x;
    int64_t d, chunk;
    int n; float nf, lr, eps;
    double frac;
};

__global__ void __launch_bounds__(kThreads, kTopkResident)
k_topk_server(const TopkServerArgs a)
{
    __shared__ uint32_t hist[kTopkBins];
    __shared__ uint32_t bins8[256];
    __shared__ uint32_t sh[2];
    __shared__ uint32_t warp_ties[kWarps];
    __shared__ TopkList list;
    const int64_t c = blockIdx.x;
    const int64_t base = c * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const int nwords = (L + 31) / 32;
    float* acc = a.m32 + base;
    float* zb = a.zbar + base;
    uint32_t* maskbar = a.Bbar + base / 32;

    for (int b = threadIdx.x; b < kTopkBins; b += kThreads) hist[b] = 0;
    if (threadIdx.x == 0) list.count = 0;
    // The sum of the n sparse messages, in worker order, has two forms.  Few kept elements (k below
    // kTopkDenseSum): scattered, through the momentum buffer - a thread owns the same mask words for every
    // worker, so an element is only ever updated by one thread and its program order is the worker order;
    // the mask words of eight workers are fetched together.  Many: in registers inside pass A (below).
    const bool dense = a.frac >= kTopkDenseSum;
    if (!dense) {
        for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
            if (k + 3 < L) *reinterpret_cast<float4*>(acc + k) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            else for (int e = 0; k + e < L; ++e) acc[k + e] = 0.0f;
        }
        __syncthreads();
        for (int w = threadIdx.x; w < nwords; w += kThreads) {
            for (int i0 = 0; i0 < a.n; i0 += 8) {
                uint32_t mw[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) mw[u] = i0 + u < a.n ? a.B[(int64_t)(i0 + u) * a.Wp + base / 32 + w] : 0u;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    uint32_t word = mw[u];
                    const float* zi = a.z + (int64_t)(i0 + u) * a.dz + base;
                    while (word) {
                        const int j = w * 32 + (__ffs(word) - 1);
                        word &= word - 1;
                        if (j < L) acc[j] = __fadd_rn(acc[j], zi[j]);
                    }
                }
            }
        }
    }
    __syncthreads();
    // pass A: zbar = sum / n + dbar_old.  In the dense form a thread sums its four elements here: it reads
    // the four mask bits of every worker (four workers at a time) and loads a worker's values only where one
    // of them is set.
    const uint32_t K = topk_count(a.frac, L);
    const bool small = nwords <= kTopkBins;            // the mask fits the shared-memory words: list routes possible
    const uint32_t floor_key = small ? topk_floor(a.thr[c], K) : 0u;
    const int shift = small ? 19 : 20, bin0 = small ? topk_fine_base(a.thr[c]) : 0;
    for (int k = threadIdx.x * 4; k < L; k += kThreads * 4) {
        float aa[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const uint32_t* mrow = a.B + base / 32 + (k >> 5);
        const float* zrow = a.z + base;
        if (!dense) {
            const float4 av = ld4_checked(acc, k, L, false);
            aa[0] = av.x; aa[1] = av.y; aa[2] = av.z; aa[3] = av.w;
        }
        for (int i0 = 0; dense && i0 < a.n; i0 += 4) {
            uint32_t nb[4];
            float4 zi[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) nb[u] = i0 + u < a.n ? (mrow[(int64_t)(i0 + u) * a.Wp] >> (k & 31)) & 0xfu : 0u;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                zi[u] = nb[u] ? ld4_checked(zrow + (int64_t)(i0 + u) * a.dz, k, L, false) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (nb[u] & 1u) aa[0] = __fadd_rn(aa[0], zi[u].x);
                if (nb[u] & 2u) aa[1] = __fadd_rn(aa[1], zi[u].y);
                if (nb[u] & 4u) aa[2] = __fadd_rn(aa[2], zi[u].z);
                if (nb[u] & 8u) aa[3] = __fadd_rn(aa[3], zi[u].w);
            }
        }
        const float4 zv = ld4_checked(zb, k, L, false);
        const uint32_t nib = maskbar[k >> 5] >> (k & 31);
        const float zo[4] = {zv.x, zv.y, zv.z, zv.w};
        float zn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            zn[e] = __fadd_rn(__fdiv_rn(aa[e], a.nf), topk_error(zo[e], (nib >> e) & 1u));
            if (k + e < L) {
                const uint32_t key = mag_key(zn[e]);
                if (floor_key == 0) atomicAdd(&hist[topk_bin(key, shift, bin0)], 1u);
                else if (key >= floor_key) topk_list_add(list, key, (uint32_t)(k + e));
            }
        }
        if (k + 3 < L) *reinterpret_cast<float4*>(zb + k) = make_float4(zn[0], zn[1], zn[2], zn[3]);
        else for (int e = 0; k + e < L; ++e) zb[k + e] = zn[e];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const float* __restrict__ v = a.v + base;
    float* __restrict__ x = a.x + base;
    uint32_t tau, ties;
    bool have_tau = false;
    bool keep_all_ties = false;                        // then "selected" is simply key >= tau
    if (floor_key != 0) {                              // window route: threshold from the list, then one ordered pass
        const uint32_t listed = list.count;
        if (listed >= K && listed <= (uint32_t)kTopkList) {
            uint32_t ties_total;
            have_tau = topk_threshold_list(list, (int)listed, floor_key, K, bins8, sh, tau, ties, ties_total);
            keep_all_ties = have_tau && ties_total == ties;
        }
    } else if (small) {                                // two-pass route
        uint32_t Kb = K;
        const int b0 = topk_find_bin(hist, kTopkBins, Kb, sh);
        const uint32_t inbin = hist[b0];
        __syncthreads();                               // everybody has read the histogram: its words become the mask
        if (b0 > 0 && b0 < kTopkBins - 1 && inbin <= (uint32_t)kTopkList) {
            // second pass: momentum and model update for every element outside the bin of the K-th key (kept
            // above it, dropped below); the elements of that bin go to the list, their x untouched
            for (int w0 = 0; w0 < L; w0 += kThreads * 4) {
                const int k = w0 + threadIdx.x * 4;
                const float4 zv = ld4_checked(zb, k, L, false);
                const float4 vv = ld4_checked(v, k, L, true);
                const float4 xv = ld4_checked(x, k, L, true);
                const float zz[4] = {zv.x, zv.y, zv.z, zv.w}, vs[4] = {vv.x, vv.y, vv.z, vv.w}, xs[4] = {xv.x, xv.y, xv.z, xv.w};
                float mn[4], xn[4];
                uint32_t nibble = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t key = mag_key(zz[e]);
                    const int b = topk_bin(key, 19, bin0);
                    const bool in_chunk = k + e < L;
                    if (in_chunk && b > b0) nibble |= 1u << e;
                    if (in_chunk && b == b0) topk_list_add(list, key, (uint32_t)(k + e));
                    mn[e] = ((nibble >> e) & 1u) ? zz[e] : 0.0f;
                    xn[e] = b == b0 ? xs[e] : apply_elem(xs[e], vs[e], mn[e], a.lr, a.eps);
                }
                const uint32_t word = pack_group_words(nibble, lane);   // valid in lanes 0, 8, 16, 24
                if ((lane & 7) == 0 && k < L) hist[k >> 5] = word;
                if (k + 3 < L) {
                    *reinterpret_cast<float4*>(acc + k) = make_float4(mn[0], mn[1], mn[2], mn[3]);
                    st_stream4(x + k, make_float4(xn[0], xn[1], xn[2], xn[3]));
                } else {
                    for (int e = 0; e < 4 && k + e < L; ++e) { acc[k + e] = mn[e]; x[k + e] = xn[e]; }
                }
            }
            __syncthreads();
            uint32_t ties_total;
            topk_threshold_list(list, (int)inbin, (uint32_t)(b0 + bin0) << 19, Kb, bins8, sh, tau, ties, ties_total);
            for (int p = threadIdx.x; p < (int)inbin; p += kThreads) {          // the listed elements, one by one
                const int j = (int)list.idx[p];
                const bool kept = topk_list_selected(list, (int)inbin, p, tau, ties, ties_total);
                const float mj = kept ? zb[j] : 0.0f;
                acc[j] = mj;
                x[j] = apply_elem(x[j], v[j], mj, a.lr, a.eps);
                if (kept) atomicOr(&hist[j >> 5], 1u << (j & 31));
            }
            __syncthreads();
            for (int w = threadIdx.x; w < nwords; w += kThreads) maskbar[w] = hist[w];
            if (threadIdx.x == 0) a.thr[c] = __uint_as_float(tau);
            return;
        }
    }
    if (!have_tau) {                                   // general route: histograms over the whole chunk
        if (small) topk_full_hist(zb, L, hist);
        topk_threshold(zb, L, K, hist, sh, tau, ties);
    }
    if (threadIdx.x == 0) a.thr[c] = __uint_as_float(tau);
    // ordered pass: mask, momentum m = C[zbar], model update (Section 3.3 steps 5-6)
    uint32_t seen = 0;
    for (int w0 = 0; w0 < L; w0 += kThreads * 4) {
        const int k = w0 + threadIdx.x * 4;
        const float4 zv = ld4_checked(zb, k, L, false);
        const float4 vv = ld4_checked(v, k, L, true);
        const float4 xv = ld4_checked(x, k, L, true);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
        const uint32_t validmask = k + 3 < L ? 0xfu : (k < L ? (1u << (L - k)) - 1u : 0u);
        uint32_t nibble;
        if (keep_all_ties) {                           // uniform: no ranking, no barriers
            nibble = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) nibble |= (((validmask >> e) & 1u) && key[e] >= tau) ? 1u << e : 0u;
        } else {
            nibble = topk_select_wave(key, validmask, tau, ties, seen, warp_ties);
        }
        const uint32_t word = pack_group_words(nibble, lane);       // valid in lanes 0, 8, 16, 24
        if ((lane & 7) == 0 && k < L) maskbar[k >> 5] = word;
        const float4 mn = make_float4((nibble & 1u) ? zv.x : 0.0f, (nibble & 2u) ? zv.y : 0.0f,
                                      (nibble & 4u) ? zv.z : 0.0f, (nibble & 8u) ? zv.w : 0.0f);
        const float4 xn = make_float4(apply_elem(xv.x, vv.x, mn.x, a.lr, a.eps), apply_elem(xv.y, vv.y, mn.y, a.lr, a.eps),
                                      apply_elem(xv.z, vv.z, mn.z, a.lr, a.eps), apply_elem(xv.w, vv.w, mn.w, a.lr, a.eps));
        if (k + 3 < L) {
            *reinterpret_cast<float4*>(acc + k) = mn;
            st_stream4(x + k, xn);
        } else {
            const float mm[4] = {mn.x, mn.y, mn.z, mn.w}, xx[4] = {xn.x, xn.y, xn.z, xn.w};
            for (int e = 0; e < 4 && k + e < L; ++e) { acc[k + e] = mm[e]; x[k + e] = xx[e]; }
        }
    }
}

__global__ void k_materialise_error_topk(const float* __restrict__ z, const uint32_t* __restrict__ mask,
                                         float* __restrict__ out, int64_t first, int64_t count)
{
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = first + j;
        out[j] = topk_error(z[e], (mask[e >> 5] >> (e & 31)) & 1u);
    }
}

// ------------------------------------------------------------------------------------------
// Error monitor: squared l2 norms of the compression errors (the quantities Assumption 1 bounds).
// Row r < n is worker r (delta = z_r - (+-s_r)), row n the server.  One CTA per (row, 4096-element
// tile) writes a binary64 partial sum; k_error_norm_rows adds a row's tiles in order.

struct ErrNormArgs {
    const float* z; int64_t dz; const float* s; int64_t Cp;      // worker rows
    const float* zbar; const float* Sbar;                         // server row
    double* partial; int64_t tiles; int n; int64_t d, chunk;
};

__global__ void __launch_bounds__(kThreads)
k_error_norm_tiles(const ErrNormArgs a)
{
    __shared__ double red[kWarps];
    const int row = (int)(blockIdx.x / a.tiles);
    const int64_t t = blockIdx.x % a.tiles;
    const float* __restrict__ z = row < a.n ? a.z + (int64_t)row * a.dz : a.zbar;
    const float* __restrict__ s = row < a.n ? a.s + (int64_t)row * a.Cp : a.Sbar;
    const int64_t base = t * 4096;
    double acc = 0.0;
    for (int k = threadIdx.x; k < 4096; k += kThreads) {
        const int64_t j = base + k;
        if (j < a.d) {
            const double e = (double)implied_error(z[j], s[j / a.chunk]);
            acc = fma(e, e, acc);
        }
    }
    const double total = block_sum(acc, red);
    if (threadIdx.x == 0) a.partial[(int64_t)row * a.tiles + t] = total;
}

__global__ void k_error_norm_rows(const double* __restrict__ partial, int64_t tiles, int rows, double* __restrict__ out)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    double total = 0.0;
    for (int64_t t = 0; t < tiles; ++t) total += partial[(int64_t)r * tiles + t];
    out[r] = total;
}

// ------------------------------------------------------------------------------------------
// host side

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    int64_t d, chunk, C, W, dz, Wp, Cp;
    int64_t fine_tiles, fine_Pp;   // 4096-element tiles of the fine worker form (0 when the chunk length does not allow it)
    int n;
    Tiling t;
    size_t off_x, off_v, off_m, off_zbar, off_z, off_B, off_Bbar, off_s, off_Sbar, off_part, off_fine, off_stage, off_mon, off_status, total;
};

bool make_layout(int64_t d, int n, int64_t chunk, Layout* L)
{
    if (d < 1 || n < 1 || n > APMS_MAX_WORKERS || chunk < 32 || chunk % 32 != 0) return false;
    if (chunk > (int64_t)1 << 30) return false;
    L->d = d; L->n = n; L->chunk = chunk;
    L->C = (d + chunk - 1) / chunk;
    L->W = (d + 31) / 32;
    L->dz = (int64_t)round_up((size_t)d, 64);
    L->Wp = (int64_t)round_up((size_t)L->W, 64);
    L->Cp = (int64_t)round_up((size_t)L->C, 64);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += round_up(bytes, 256); return at; };
    L->off_x = take((size_t)L->dz * 4);
    L->off_v = take((size_t)L->dz * 4);
    L->off_m = take((size_t)L->dz * 4);
    L->off_zbar = take((size_t)L->dz * 4);
    L->off_z = take((size_t)L->dz * 4 * (size_t)n);
    L->off_B = take((size_t)L->Wp * 4 * (size_t)n);
    L->off_Bbar = take((size_t)L->Wp * 4);
    L->off_s = take((size_t)L->Cp * 4 * (size_t)n);
    L->off_Sbar = take((size_t)L->Cp * 4);
    L->t.d = d; L->t.chunk = chunk;
    if (chunk <= kTileMax) { L->t.tile = chunk; L->t.P = 1; }
    else { L->t.tile = kTileSplit; L->t.P = (int)((chunk + kTileSplit - 1) / kTileSplit); }
    L->t.Pp = (int64_t)round_up((size_t)(L->C * L->t.P), 64);
    L->off_part = take(L->t.P > 1 ? (size_t)L->t.Pp * 8 * (size_t)(n + 1) : 0);   // n worker rows + 1 server row
    L->fine_tiles = (chunk % kFineSub == 0) ? (d + kFineTile - 1) / kFineTile : 0;
    L->fine_Pp = (int64_t)round_up((size_t)L->fine_tiles * kWarps, 64);
    L->off_fine = take((size_t)L->fine_Pp * 8 * (size_t)n);
    L->off_stage = take((size_t)L->dz * 4 * 2);
    L->off_mon = take(((size_t)(n + 1) * (size_t)((d + 4095) / 4096) + (size_t)(n + 1)) * 8);   // error monitor: tile sums + row sums
    L->off_status = take(256);
    L->total = o;
    return true;
}

thread_local char g_create_error[256] = "";

struct EventPair { cudaEvent_t a, b; };

}  // namespace

struct apms_ctx {
    Layout L;
    float beta1, beta2, eps, lr;
    int t;
    int64_t steps;           // steps taken through apms_step (warmup and compressed)
    int compressor;          // APMS_COMPRESSOR_*
    double topk_frac;        // top-k: fraction of a chunk that is sent
    int variant;             // APMS_VARIANT_*: what the workers compress
    int64_t csteps;          // compression-phase steps taken (the variant is fixed once one has run)
    int substep;             // phase-wise step: 0 = between steps, 1 = worker phase done, 2 = a server phase done
    apms_schedule sched; bool has_sched;
    apms_phase phase;
    bool m_is_fp32;          // momentum lives in the binary32 buffer (else in Bbar/Sbar)
    char* ws; size_t ws_bytes; bool owns_ws;
    cudaStream_t stream;
    cudaStream_t copy_stream; cudaEvent_t ev_copied[2], ev_used[2]; bool host_path_ready;
    int device;
    int sms;
    bool timing;
    apms_team_mode team_mode;
    int fine_run;            // tiles of one worker launched back to back in the fine worker form
    std::vector<EventPair> events[APMS_KERNEL_COUNT];
    std::vector<EventPair> pool;
    int64_t launches;
    char err[512];

    float* x() { return (float*)(ws + L.off_x); }
    float* v() { return (float*)(ws + L.off_v); }
    float* m() { return (float*)(ws + L.off_m); }
    float* zbar() { return (float*)(ws + L.off_zbar); }
    float* z(int i) { return (float*)(ws + L.off_z) + (int64_t)i * L.dz; }
    uint32_t* B(int i) { return (uint32_t*)(ws + L.off_B) + (int64_t)i * L.Wp; }
    uint32_t* Bbar() { return (uint32_t*)(ws + L.off_Bbar); }
    float* s(int i) { return (float*)(ws + L.off_s) + (int64_t)i * L.Cp; }
    float* Sbar() { return (float*)(ws + L.off_Sbar); }
    float* stage(int b) { return (float*)(ws + L.off_stage) + (int64_t)b * L.dz; }
    int* status() { return (int*)(ws + L.off_status); }
    double* fine_partial(int row) { return (double*)(ws + L.off_fine) + (int64_t)row * L.fine_Pp; }
    double* partial(int row) { return (double*)(ws + L.off_part) + (int64_t)row * L.t.Pp; }   // row n = server
};

namespace {

apms_status fail(apms_ctx* c, apms_status st, const char* fmt, const char* detail = "")
{
    if (c) snprintf(c->err, sizeof c->err, fmt, detail);
    return st;
}

#define APMS_CUDA(c, call)                                                                   \
    do {                                                                                     \
        cudaError_t e__ = (call);                                                            \
        if (e__ != cudaSuccess) {                                                            \
            snprintf((c)->err, sizeof (c)->err, "%s failed: %s", #call, cudaGetErrorString(e__)); \
            return APMS_ERR_CUDA;                                                            \
        }                                                                                    \
    } while (0)

apms_status ensure_workspace(apms_ctx* c)
{
    if (c->ws) return APMS_OK;
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, c->L.total);
    if (e != cudaSuccess) {
        snprintf(c->err, sizeof c->err, "cudaMalloc of %zu workspace bytes failed: %s", c->L.total,
                 cudaGetErrorString(e));
        return e == cudaErrorMemoryAllocation ? APMS_ERR_OOM : APMS_ERR_CUDA;
    }
    c->ws = (char*)p; c->ws_bytes = c->L.total; c->owns_ws = true;
    return APMS_OK;
}

// Event bracket around one kernel launch when timing is on.
struct Timed {
    apms_ctx* c; int k; EventPair ev; bool on;
    Timed(apms_ctx* ctx, int kernel) : c(ctx), k(kernel), on(ctx->timing) {
        if (!on) return;
        if (!c->pool.empty()) { ev = c->pool.back(); c->pool.pop_back(); }
        else if (cudaEventCreate(&ev.a) != cudaSuccess || cudaEventCreate(&ev.b) != cudaSuccess) { on = false; return; }
        cudaEventRecord(ev.a, c->stream);
    }
    ~Timed() {
        if (!on) return;
        cudaEventRecord(ev.b, c->stream);
        c->events[k].push_back(ev);
    }
};

bool valid_grad_type(int t) { return t == APMS_GRAD_F32 || t == APMS_GRAD_BF16 || t == APMS_GRAD_F16; }
size_t grad_elem_bytes(int t) { return t == APMS_GRAD_F32 ? 4 : 2; }

// Runs `call` with GT bound to the compile-time constant that equals the run-time gradient type.
#define APMS_DISPATCH_GRAD(type, ...)                                              \
    do {                                                                           \
        if ((type) == APMS_GRAD_BF16)     { constexpr int GT = APMS_GRAD_BF16; __VA_ARGS__; } \
        else if ((type) == APMS_GRAD_F16) { constexpr int GT = APMS_GRAD_F16;  __VA_ARGS__; } \
        else                              { constexpr int GT = APMS_GRAD_F32;  __VA_ARGS__; } \
    } while (0)

apms_status check_grads(apms_ctx* c, const void* const* g, int type, GradPtrs* out, int count)
{
    if (!valid_grad_type(type)) return fail(c, APMS_ERR_INVALID_ARG, "unknown gradient type");
    if (!g) return fail(c, APMS_ERR_INVALID_ARG, "gradient pointer array is NULL");
    const uintptr_t mask = type == APMS_GRAD_F32 ? 15u : 7u;          // one lane's four elements per access
    for (int i = 0; i < count; ++i) {
        if (!g[i]) return fail(c, APMS_ERR_INVALID_ARG, "a gradient pointer is NULL");
        if (((uintptr_t)g[i] & mask) != 0)
            return fail(c, APMS_ERR_INVALID_ARG, "a gradient pointer is not aligned (16 bytes for binary32, 8 bytes for 16-bit gradients)");
        out->p[i] = g[i];
    }
    return APMS_OK;
}

apms_status launch_check(apms_ctx* c, const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(c->err, sizeof c->err, "launch of %s failed: %s", what, cudaGetErrorString(e));
        return APMS_ERR_CUDA;
    }
    c->launches += 1;
    return APMS_OK;
}

// After a stream synchronisation: has a kernel recorded that one of its bounded waits gave up?
apms_status device_status_check(apms_ctx* c)
{
    int st = 0;
    APMS_CUDA(c, cudaMemcpy(&st, c->status(), sizeof st, cudaMemcpyDeviceToHost));
    if (st != 0) return fail(c, APMS_ERR_TIMEOUT, "a kernel gave up waiting for its own asynchronous copies; the state of this context is undefined");
    return APMS_OK;
}

// The staged server kernel needs every 2048-element slab of a tile to start on a 16-byte boundary
// in zbar and in the sign words, i.e. chunks that are multiples of 2048 elements.
bool use_staged_server(const apms_ctx* c)
{
    if (c->team_mode == APMS_TEAM_CTA || c->team_mode == APMS_TEAM_WARP) return false;
    if (c->L.t.l1) return false;             // the mean-|z| scale exists in the register-staged kernels only
    return c->L.chunk % kSlab == 0;
}

bool use_warp_teams(const apms_ctx* c, int64_t items)
{
    if (c->team_mode == APMS_TEAM_CTA) return false;
    if (c->team_mode == APMS_TEAM_WARP) return true;
    return items / kWarps >= (int64_t)kWarpTeamMinCtasPerSm * c->sms;
}

apms_status launch_finalize(apms_ctx* c, int first_row, int rows, float* scales)
{
    const int64_t total = (int64_t)rows * c->L.C;
    k_finalize_scales<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(c->partial(first_row), scales, rows,
                                                                            c->L.C, c->L.Cp, c->L.t);
    return launch_check(c, "k_finalize_scales");
}

bool use_fine_worker(const apms_ctx* c)
{
    if (c->team_mode == APMS_TEAM_CTA || c->team_mode == APMS_TEAM_WARP) return false;
    if (c->L.t.l1) return false;             // see use_staged_server
    return (!c->m_is_fp32 || c->variant == APMS_VARIANT_GRADIENT) && c->L.fine_tiles > 0;
}

apms_status launch_worker_fine(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni)
{
    WorkerFineArgs a;
    a.z = c->z(0); a.dz = c->L.dz;
    a.B = c->B(0); a.Wp = c->L.Wp;
    a.s = c->s(0); a.Cp = c->L.Cp;
    a.partial = c->fine_partial(i0); a.Pp = c->L.fine_Pp;
    a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.d = c->L.d; a.chunk = c->L.chunk; a.tiles = c->L.fine_tiles;
    a.i0 = i0; a.ni = ni;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1;
    a.run = c->fine_run;
    const int64_t stretches = (a.tiles + a.run - 1) / a.run;
    const int64_t blocks = stretches * a.run * ni;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (tile, worker) items for one launch");
    {
        Timed t(c, APMS_KERNEL_WORKER);
        if (c->variant == APMS_VARIANT_GRADIENT) APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, true><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
        else                                     APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, false><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
        apms_status st = launch_check(c, "k_worker_fine");
        if (st != APMS_OK) return st;
        const int64_t total = (int64_t)ni * c->L.C;
        k_finalize_fine<<<(unsigned)((total + kWarps - 1) / kWarps), kThreads, 0, c->stream>>>(c->fine_partial(i0), c->L.fine_Pp, c->s(i0),
                                                                             c->L.Cp, ni, c->L.C, c->L.d, c->L.chunk);
        st = launch_check(c, "k_finalize_fine");
        if (st != APMS_OK) return st;
    }
    return APMS_OK;
}

apms_status launch_worker_topk(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni)
{
    TopkWorkerArgs a;
    a.z = c->z(0); a.dz = c->L.dz; a.B = c->B(0); a.Wp = c->L.Wp; a.m32 = c->m();
    a.thr = c->s(0); a.Cp = c->L.Cp;
    a.d = c->L.d; a.chunk = c->L.chunk; a.C = c->L.C; a.i0 = i0; a.ni = ni;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1; a.frac = c->topk_frac;
    const int64_t blocks = c->L.C * ni;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (chunk, worker) items for one launch");
    Timed t(c, APMS_KERNEL_WORKER);
    APMS_DISPATCH_GRAD(gtype, k_topk_worker<GT><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
    return launch_check(c, "k_topk_worker");
}

apms_status launch_worker(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni)
{
    if (c->compressor == APMS_COMPRESSOR_TOPK) return launch_worker_topk(c, G, gtype, i0, ni);
    if (use_fine_worker(c)) return launch_worker_fine(c, G, gtype, i0, ni);
    WorkerArgs a;
    a.z = c->z(0); a.dz = c->L.dz;
    a.B = c->B(0); a.Wp = c->L.Wp;
    a.s = c->s(0); a.Cp = c->L.Cp;
    a.partial = c->partial(0);
    a.m32 = c->m(); a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.t = c->L.t; a.i0 = i0; a.ni = ni;
    a.items = c->L.C * c->L.t.P * ni;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1;
    a.send_gradient = c->variant == APMS_VARIANT_GRADIENT;
    const bool warp_teams = use_warp_teams(c, a.items);
    const int64_t blocks = warp_teams ? (a.items + kWarps - 1) / kWarps : a.items;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (chunk, worker) items for one launch");
    {
        Timed t(c, APMS_KERNEL_WORKER);
        const unsigned gridx = (unsigned)blocks;
        if (c->m_is_fp32 && !a.send_gradient) {
            if (warp_teams) APMS_DISPATCH_GRAD(gtype, k_worker<GT, true, 2, 1><<<gridx, kThreads, 0, c->stream>>>(G, a));
            else            APMS_DISPATCH_GRAD(gtype, k_worker<GT, true, 4, kWarps><<<gridx, kThreads, 0, c->stream>>>(G, a));
        } else {
            if (warp_teams) APMS_DISPATCH_GRAD(gtype, k_worker<GT, false, APMS_WORKER_U, 1><<<gridx, kThreads, 0, c->stream>>>(G, a));
            else            APMS_DISPATCH_GRAD(gtype, k_worker<GT, false, APMS_WORKER_U, kWarps><<<gridx, kThreads, 0, c->stream>>>(G, a));
        }
        apms_status st = launch_check(c, "k_worker");
        if (st != APMS_OK) return st;
    }
    if (c->L.t.P > 1) return launch_finalize(c, i0, ni, c->s(i0));
    return APMS_OK;
}

// Launch of one instantiation of the staged server kernel (its shared-memory limit is raised first).
template <int NT, bool FUSED>
cudaError_t launch_staged(const ServerStagedArgs& sa, unsigned blocks, size_t smem, cudaStream_t stream)
{
    if (FUSED && sa.span > 1) {
        cudaError_t e = cudaFuncSetAttribute(k_server_staged<NT, FUSED, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_server_staged<NT, FUSED, FUSED><<<blocks, kStagedThreads, smem, stream>>>(sa);
    } else {
        cudaError_t e = cudaFuncSetAttribute(k_server_staged<NT, FUSED, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_server_staged<NT, FUSED, false><<<blocks, kStagedThreads, smem, stream>>>(sa);
    }
    return cudaSuccess;
}

template <bool FUSED>
cudaError_t launch_staged_n(const ServerStagedArgs& sa, unsigned blocks, size_t smem, cudaStream_t stream)
{
    switch (sa.a.n) {        // the usual worker counts get a fully unrolled sum; any other count the generic loop
    case 2:  return launch_staged<2, FUSED>(sa, blocks, smem, stream);
    case 4:  return launch_staged<4, FUSED>(sa, blocks, smem, stream);
    case 8:  return launch_staged<8, FUSED>(sa, blocks, smem, stream);
    case 16: return launch_staged<16, FUSED>(sa, blocks, smem, stream);
    case 32: return launch_staged<32, FUSED>(sa, blocks, smem, stream);
    default: return launch_staged<0, FUSED>(sa, blocks, smem, stream);
    }
}

// Where the server finds the workers' messages: `rows` senders, row j holding sign words and scales
// addressed by ABSOLUTE word / chunk index (a pointer into a shard is shifted back by the caller).
struct ServerSource { const uint32_t* B; int64_t Wp; const float* s; int64_t Cp; int rows; };

// Section 3.3 step 4 for chunks [cb, ce).  With may_fuse and a shape that allows it, steps 5-6 for
// the same chunks run in the same kernel (*applied = true).
apms_status launch_server(apms_ctx* c, const ServerSource& src, int64_t cb, int64_t ce, bool may_fuse, bool* applied)
{
    *applied = false;
    ServerArgs a;
    a.B = src.B; a.Wp = src.Wp; a.s = src.s; a.Cp = src.Cp;
    a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.partial = c->partial(c->L.n);
    a.t = c->L.t; a.item0 = cb * c->L.t.P; a.items = ce * c->L.t.P; a.n = src.rows; a.nf = (float)src.rows;
    const int64_t count = a.items - a.item0;
    if (count <= 0) return APMS_OK;
    const bool staged = use_staged_server(c);
    const bool warp_teams = !staged && use_warp_teams(c, count);
    const int64_t blocks = warp_teams ? (count + kWarps - 1) / kWarps : count;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunk tiles for one launch");
    {
        Timed t(c, APMS_KERNEL_SERVER);
        if (staged) {
            const bool fused = may_fuse && c->L.t.P == 1;   // the CTA sees the whole chunk, so it knows the new scale
            ServerStagedArgs sa;
            sa.a = a; sa.status = c->status();
            sa.inv_n = ((a.n & (a.n - 1)) == 0) ? 1.0f / (float)a.n : 0.0f;
            sa.v = c->v(); sa.x = c->x(); sa.lr = c->lr; sa.eps = c->eps;
            const size_t smem = (size_t)kStages * staged_stage_bytes(a.n, fused);
            sa.span = fused ? (int)((kStagedSpanElems + c->L.chunk - 1) / c->L.chunk) : 1;
            const int64_t fill = count / (2 * (int64_t)c->sms);       // small problems: keep at least two CTAs per SM
            if (sa.span > 1 && fill < sa.span) sa.span = fill < 1 ? 1 : (int)fill;
            const int64_t ctas = (count + sa.span - 1) / sa.span;
            cudaError_t e = fused ? launch_staged_n<true>(sa, (unsigned)ctas, smem, c->stream)
                                  : launch_staged_n<false>(sa, (unsigned)ctas, smem, c->stream);
            if (e != cudaSuccess) {
                snprintf(c->err, sizeof c->err, "setting up k_server_staged failed: %s", cudaGetErrorString(e));
                return APMS_ERR_CUDA;
            }
            *applied = fused;
        }
        else if (warp_teams) k_server<APMS_SERVER_U, 1><<<(unsigned)blocks, kThreads, 0, c->stream>>>(a);
        else            k_server<APMS_SERVER_U, kWarps><<<(unsigned)blocks, kThreads, 0, c->stream>>>(a);
        apms_status st = launch_check(c, "k_server");
        if (st != APMS_OK) return st;
    }
    if (c->L.t.P > 1) {
        // scales of the range's split chunks: the same kernel on the range as a vector of its own
        Tiling t = c->L.t;
        t.d = c->L.d - cb * c->L.chunk;
        const int64_t nchunks = ce - cb;
        k_finalize_scales<<<(unsigned)((nchunks + 255) / 256), 256, 0, c->stream>>>(c->partial(c->L.n) + cb * c->L.t.P, c->Sbar() + cb,
                                                                                 1, nchunks, c->L.Cp, t);
        return launch_check(c, "k_finalize_scales");
    }
    return APMS_OK;
}

// Section 3.3 steps 5-6 over the whole vector, from the server message held in Bbar / Sbar.
apms_status launch_apply(apms_ctx* c)
{
    if (c->variant == APMS_VARIANT_GRADIENT) {
        ApplyGradArgs g;
        g.Bbar = c->Bbar(); g.Sbar = c->Sbar(); g.v = c->v(); g.x = c->x(); g.m = c->m();
        g.d = c->L.d; g.chunk = c->L.chunk; g.lr = c->lr; g.eps = c->eps; g.beta1 = c->beta1; g.omb1 = 1.0f - c->beta1;
        Timed t(c, APMS_KERNEL_APPLY);
        k_apply_gradient<<<(unsigned)((c->L.d + kApplyTile - 1) / kApplyTile), kThreads, 0, c->stream>>>(g);
        return launch_check(c, "k_apply_gradient");
    }
    ApplyArgs a;
    a.Bbar = c->Bbar(); a.Sbar = c->Sbar(); a.v = c->v(); a.x = c->x();
    a.d = c->L.d; a.chunk = c->L.chunk; a.lr = c->lr; a.eps = c->eps;
    Timed t(c, APMS_KERNEL_APPLY);
    k_apply<<<(unsigned)((c->L.d + kApplyTile - 1) / kApplyTile), kThreads, 0, c->stream>>>(a);
    return launch_check(c, "k_apply");
}

apms_status launch_server_and_apply(apms_ctx* c)
{
    if (c->compressor == APMS_COMPRESSOR_TOPK) {       // one kernel: sparse average, recompression, momentum, model update
        TopkServerArgs a;
        a.z = c->z(0); a.dz = c->L.dz; a.B = c->B(0); a.Wp = c->L.Wp;
        a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.m32 = c->m(); a.thr = c->Sbar(); a.v = c->v(); a.x = c->x();
        a.d = c->L.d; a.chunk = c->L.chunk; a.n = c->L.n; a.nf = (float)c->L.n; a.lr = c->lr; a.eps = c->eps;
        a.frac = c->topk_frac;
        if (c->L.C > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunks for one launch");
        Timed t(c, APMS_KERNEL_SERVER);
        k_topk_server<<<(unsigned)c->L.C, kThreads, 0, c->stream>>>(a);
        apms_status st = launch_check(c, "k_topk_server");
        if (st != APMS_OK) return st;
        c->m_is_fp32 = true;
        c->csteps += 1;
        return APMS_OK;
    }
    const ServerSource own = {c->B(0), c->L.Wp, c->s(0), c->L.Cp, c->L.n};
    bool applied = false;      // steps 5-6 already done by the fused server kernel
    const bool gradient = c->variant == APMS_VARIANT_GRADIENT;      // its apply differs: never fused
    apms_status st = launch_server(c, own, 0, c->L.C, !gradient, &applied);
    if (st != APMS_OK) return st;
    if (!applied) {
        st = launch_apply(c);
        if (st != APMS_OK) return st;
    }
    c->m_is_fp32 = gradient;   // momentum variant: from now on the momentum is the server's message
    c->csteps += 1;
    return APMS_OK;
}

int grid_for(const apms_ctx* c, int64_t items, int per_sm)
{
    int64_t blocks = (items + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)c->sms * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// C ABI

extern "C" {

size_t apms_workspace_bytes(int64_t d, int n, int64_t chunk)
{
    Layout L;
    return make_layout(d, n, chunk, &L) ? L.total : 0;
}

apms_status apms_create(apms_ctx** out, int64_t d, int n, float beta1, float beta2, float eps,
                        float lr, int64_t chunk)
{
    if (!out) { snprintf(g_create_error, sizeof g_create_error, "out is NULL"); return APMS_ERR_INVALID_ARG; }
    *out = nullptr;
    Layout L;
    if (!make_layout(d, n, chunk, &L)) {
        snprintf(g_create_error, sizeof g_create_error,
                 "invalid shape: need d >= 1, 1 <= n <= %d, chunk a positive multiple of 32 (got d=%lld n=%d chunk=%lld)",
                 APMS_MAX_WORKERS, (long long)d, n, (long long)chunk);
        return APMS_ERR_INVALID_ARG;
    }
    if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !isfinite(lr)) {
        snprintf(g_create_error, sizeof g_create_error, "invalid hyper-parameters: need 0 <= beta < 1, eps >= 0, finite lr");
        return APMS_ERR_INVALID_ARG;
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) {
        snprintf(g_create_error, sizeof g_create_error, "no usable CUDA device: %s", cudaGetErrorString(e));
        return APMS_ERR_CUDA;
    }
    apms_ctx* c = new (std::nothrow) apms_ctx();
    if (!c) { snprintf(g_create_error, sizeof g_create_error, "host allocation failed"); return APMS_ERR_OOM; }
    c->L = L; c->beta1 = beta1; c->beta2 = beta2; c->eps = eps; c->lr = lr;
    c->t = 0; c->phase = APMS_PHASE_CREATED; c->m_is_fp32 = true;
    c->ws = nullptr; c->ws_bytes = 0; c->owns_ws = false;
    c->stream = nullptr; c->copy_stream = nullptr; c->host_path_ready = false;
    c->device = dev; c->sms = sms; c->timing = false; c->launches = 0; c->err[0] = 0;
    c->team_mode = APMS_TEAM_AUTO;
    c->steps = 0; c->has_sched = false; c->substep = 0; c->variant = APMS_VARIANT_MOMENTUM; c->csteps = 0;
    c->compressor = APMS_COMPRESSOR_ONEBIT; c->topk_frac = 0.01;
    c->fine_run = kFineRunDefault;
    if (const char* e = getenv("APMS_FINE_RUN")) { const int r = atoi(e); if (r >= 1 && r <= (1 << 24)) c->fine_run = r; }   // tuning knob
    if ((int64_t)c->fine_run > L.fine_tiles && L.fine_tiles > 0) c->fine_run = (int)L.fine_tiles;
    *out = c;
    return APMS_OK;
}

apms_status apms_bind(apms_ctx* c, void* workspace_dev, size_t bytes, void* cuda_stream)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "apms_bind must precede apms_set_params");
    if (c->ws) return fail(c, APMS_ERR_BAD_STATE, "a workspace is already attached");
    if (!workspace_dev || ((uintptr_t)workspace_dev & 255u)) return fail(c, APMS_ERR_INVALID_ARG, "workspace must be non-NULL and 256-byte aligned");
    if (bytes < c->L.total) return fail(c, APMS_ERR_OOM, "workspace smaller than apms_workspace_bytes()");
    c->ws = (char*)workspace_dev; c->ws_bytes = bytes; c->owns_ws = false;
    c->stream = (cudaStream_t)cuda_stream;
    return APMS_OK;
}

apms_status apms_set_params(apms_ctx* c, const float* x0, int src_is_device)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!x0) return fail(c, APMS_ERR_INVALID_ARG, "x0 is NULL");
    apms_status st = ensure_workspace(c);
    if (st != APMS_OK) return st;
    const size_t bytes = (size_t)c->L.d * 4;
    APMS_CUDA(c, cudaMemcpyAsync(c->x(), x0, bytes, src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->m(), 0, (size_t)c->L.dz * 4, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->v(), 0, (size_t)c->L.dz * 4, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->status(), 0, 256, c->stream));
    if (!src_is_device) APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    c->t = 0; c->steps = 0; c->csteps = 0; c->substep = 0; c->phase = APMS_PHASE_WARMUP; c->m_is_fp32 = true;
    return APMS_OK;
}

apms_status apms_set_lr(apms_ctx* c, float lr)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!isfinite(lr)) return fail(c, APMS_ERR_INVALID_ARG, "lr must be finite");
    c->lr = lr;
    return APMS_OK;
}

apms_status apms_warmup_step(apms_ctx* c, const float* const* grads_dev)
{
    return apms_warmup_step_typed(c, (const void* const*)grads_dev, APMS_GRAD_F32);
}

apms_status apms_warmup_step_typed(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_WARMUP) return fail(c, APMS_ERR_BAD_STATE, "apms_warmup_step needs the WARMUP phase (after apms_set_params, before apms_freeze_v)");
    GradPtrs G;
    apms_status st = check_grads(c, grads_dev, (int)type, &G, c->L.n);
    if (st != APMS_OK) return st;
    c->t += 1;
    AdamArgs a;
    a.x = c->x(); a.m = c->m(); a.v = c->v(); a.d = c->L.d; a.n = c->L.n;
    a.beta1 = c->beta1; a.beta2 = c->beta2; a.omb1 = 1.0f - c->beta1; a.omb2 = 1.0f - c->beta2;
    a.bc1 = (float)(1.0 - pow((double)c->beta1, (double)c->t));
    a.bc2 = (float)(1.0 - pow((double)c->beta2, (double)c->t));
    a.lr = c->lr; a.eps = c->eps; a.nf = (float)c->L.n;
    Timed t(c, APMS_KERNEL_WARMUP_ADAM);
    const int64_t adam_blocks = (c->L.d + (int64_t)kThreads * 4 - 1) / ((int64_t)kThreads * 4);
    if (adam_blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "d too large for one launch");
    APMS_DISPATCH_GRAD((int)type, k_warmup_adam<GT><<<(unsigned)adam_blocks, kThreads, 0, c->stream>>>(G, a));
    return launch_check(c, "k_warmup_adam");
}

apms_status apms_freeze_v(apms_ctx* c)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_WARMUP) return fail(c, APMS_ERR_BAD_STATE, "apms_freeze_v needs the WARMUP phase");
    // errors start at zero: z = 0 with scale 0 implies delta = 0 - (+0) = 0
    APMS_CUDA(c, cudaMemsetAsync(c->ws + c->L.off_zbar, 0, c->L.off_part - c->L.off_zbar, c->stream));
    c->phase = APMS_PHASE_COMPRESSED;
    c->m_is_fp32 = true;
    return APMS_OK;
}

apms_status apms_compressed_step(apms_ctx* c, const float* const* grads_dev)
{
    return apms_compressed_step_typed(c, (const void* const*)grads_dev, APMS_GRAD_F32);
}

apms_status apms_compressed_step_typed(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_compressed_step needs the COMPRESSED phase (call apms_freeze_v first)");
    if (c->substep != 0) return fail(c, APMS_ERR_BAD_STATE, "a phase-wise step is in progress (finish it with apms_apply_phase)");
    GradPtrs G;
    apms_status st = check_grads(c, grads_dev, (int)type, &G, c->L.n);
    if (st != APMS_OK) return st;
    st = launch_worker(c, G, (int)type, 0, c->L.n);
    if (st != APMS_OK) return st;
    return launch_server_and_apply(c);
}

apms_status apms_worker_phase(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_worker_phase needs the COMPRESSED phase (call apms_freeze_v first)");
    if (c->substep != 0) return fail(c, APMS_ERR_BAD_STATE, "the previous phase-wise step is not finished (apms_apply_phase)");
    if (c->compressor != APMS_COMPRESSOR_ONEBIT) return fail(c, APMS_ERR_BAD_STATE, "the phase-wise step exists for the 1-bit compressor only");
    GradPtrs G;
    apms_status st = check_grads(c, grads_dev, (int)type, &G, c->L.n);
    if (st != APMS_OK) return st;
    st = launch_worker(c, G, (int)type, 0, c->L.n);
    if (st == APMS_OK) c->substep = 1;
    return st;
}

apms_status apms_get_message(apms_ctx* c, int worker, uint32_t** bits_dev, float** scales_dev)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (worker < -1 || worker >= c->L.n) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range (-1 = the server's message)");
    apms_status st = ensure_workspace(c);
    if (st != APMS_OK) return st;
    if (bits_dev) *bits_dev = worker < 0 ? c->Bbar() : c->B(worker);
    if (scales_dev) *scales_dev = worker < 0 ? c->Sbar() : c->s(worker);
    return APMS_OK;
}

apms_status apms_server_phase(apms_ctx* c, const uint32_t* bits_rows_dev, int64_t row_words, const float* scale_rows_dev,
                              int64_t row_scales, int rows, int64_t chunk_begin, int64_t chunk_end)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_server_phase needs the COMPRESSED phase");
    if (c->substep < 1) return fail(c, APMS_ERR_BAD_STATE, "apms_server_phase follows apms_worker_phase");
    if (!bits_rows_dev || !scale_rows_dev) return fail(c, APMS_ERR_INVALID_ARG, "a message pointer is NULL");
    if (rows < 1 || rows > APMS_MAX_WORKERS) return fail(c, APMS_ERR_INVALID_ARG, "rows must be between 1 and APMS_MAX_WORKERS");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    const int64_t first_elem = chunk_begin * c->L.chunk;
    const int64_t last_elem = chunk_end * c->L.chunk < c->L.d ? chunk_end * c->L.chunk : c->L.d;
    const int64_t need_words = (last_elem - first_elem + 31) / 32;
    // the staged kernel copies sign words in 16-byte pieces: rows must hold the range rounded up to 4 words
    if (row_words < (need_words + 3) / 4 * 4 || row_words % 4 != 0 || row_scales < chunk_end - chunk_begin)
        return fail(c, APMS_ERR_INVALID_ARG, "rows too short: row_words must be a multiple of 4 that covers the range's sign words rounded up to 4, row_scales its chunks");
    if (((uintptr_t)bits_rows_dev & 15u) != 0) return fail(c, APMS_ERR_INVALID_ARG, "bits_rows_dev is not 16-byte aligned");
    // kernels index by absolute word / chunk: shift the shard's pointers back to where index 0 would be
    const ServerSource src = {bits_rows_dev - first_elem / 32, row_words, scale_rows_dev - chunk_begin, row_scales, rows};
    bool applied = false;
    apms_status st = launch_server(c, src, chunk_begin, chunk_end, false, &applied);
    if (st == APMS_OK) c->substep = 2;
    return st;
}

apms_status apms_apply_phase(apms_ctx* c)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_apply_phase needs the COMPRESSED phase");
    if (c->substep != 2) return fail(c, APMS_ERR_BAD_STATE, "apms_apply_phase follows apms_server_phase");
    apms_status st = launch_apply(c);
    if (st != APMS_OK) return st;
    c->m_is_fp32 = c->variant == APMS_VARIANT_GRADIENT;
    c->csteps += 1;
    c->substep = 0;
    return APMS_OK;
}

apms_status apms_compressed_step_host(apms_ctx* c, const float* const* grads_host, float* x_out_host)
{
    return apms_compressed_step_host_typed(c, (const void* const*)grads_host, APMS_GRAD_F32, x_out_host);
}

apms_status apms_compressed_step_host_typed(apms_ctx* c, const void* const* grads_host, apms_grad_type type, float* x_out_host)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_compressed_step_host needs the COMPRESSED phase (call apms_freeze_v first)");
    if (c->substep != 0) return fail(c, APMS_ERR_BAD_STATE, "a phase-wise step is in progress (finish it with apms_apply_phase)");
    if (!valid_grad_type((int)type)) return fail(c, APMS_ERR_INVALID_ARG, "unknown gradient type");
    if (!grads_host) return fail(c, APMS_ERR_INVALID_ARG, "gradient pointer array is NULL");
    for (int i = 0; i < c->L.n; ++i)
        if (!grads_host[i]) return fail(c, APMS_ERR_INVALID_ARG, "a gradient pointer is NULL");
    if (!c->host_path_ready) {
        APMS_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            APMS_CUDA(c, cudaEventCreateWithFlags(&c->ev_copied[b], cudaEventDisableTiming));
            APMS_CUDA(c, cudaEventCreateWithFlags(&c->ev_used[b], cudaEventDisableTiming));
        }
        c->host_path_ready = true;
    }
    const size_t bytes = (size_t)c->L.d * 4;
    const size_t gbytes = (size_t)c->L.d * grad_elem_bytes((int)type);
    // the staging buffers may still be read by work queued earlier on the compute stream
    APMS_CUDA(c, cudaEventRecord(c->ev_used[0], c->stream));
    APMS_CUDA(c, cudaEventRecord(c->ev_used[1], c->stream));
    for (int i = 0; i < c->L.n; ++i) {
        const int b = i & 1;
        APMS_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_used[b], 0));
        APMS_CUDA(c, cudaMemcpyAsync(c->stage(b), grads_host[i], gbytes, cudaMemcpyHostToDevice, c->copy_stream));
        APMS_CUDA(c, cudaEventRecord(c->ev_copied[b], c->copy_stream));
        APMS_CUDA(c, cudaStreamWaitEvent(c->stream, c->ev_copied[b], 0));
        GradPtrs G;
        G.p[0] = c->stage(b);
        apms_status st = launch_worker(c, G, (int)type, i, 1);
        if (st != APMS_OK) return st;
        APMS_CUDA(c, cudaEventRecord(c->ev_used[b], c->stream));
    }
    apms_status st = launch_server_and_apply(c);
    if (st != APMS_OK) return st;
    if (x_out_host) APMS_CUDA(c, cudaMemcpyAsync(x_out_host, c->x(), bytes, cudaMemcpyDeviceToHost, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    return device_status_check(c);
}

apms_status apms_get_params(apms_ctx* c, float* dst, int dst_is_device)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!dst) return fail(c, APMS_ERR_INVALID_ARG, "dst is NULL");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "no parameters set yet");
    APMS_CUDA(c, cudaMemcpyAsync(dst, c->x(), (size_t)c->L.d * 4, dst_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, c->stream));
    if (!dst_is_device) {
        APMS_CUDA(c, cudaStreamSynchronize(c->stream));
        return device_status_check(c);
    }
    return APMS_OK;
}

apms_status apms_get_state_slice(apms_ctx* c, apms_state_id which, int worker, int64_t first,
                                 int64_t count, void* dst)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!dst) return fail(c, APMS_ERR_INVALID_ARG, "dst is NULL");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "no state yet");
    const bool per_worker = which == APMS_STATE_WORKER_ERR || which == APMS_STATE_WORKER_BITS || which == APMS_STATE_WORKER_SCALES;
    if (per_worker && (worker < 0 || worker >= c->L.n)) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range");
    int64_t extent = c->L.d;
    if (which == APMS_STATE_WORKER_BITS || which == APMS_STATE_SERVER_BITS) extent = c->L.W;
    if (which == APMS_STATE_WORKER_SCALES || which == APMS_STATE_SERVER_SCALES) extent = c->L.C;
    if (first < 0 || count < 0 || first > extent || count > extent - first) return fail(c, APMS_ERR_INVALID_ARG, "slice out of range");
    if (count == 0) return APMS_OK;
    const char* src = nullptr;
    const int grid = grid_for(c, count, 8);
    bool staged = false;
    switch (which) {
    case APMS_STATE_X: src = (const char*)c->x(); break;
    case APMS_STATE_V: src = (const char*)c->v(); break;
    case APMS_STATE_M:
        if (c->m_is_fp32) src = (const char*)c->m();
        else {
            k_materialise_momentum<<<grid, kThreads, 0, c->stream>>>(c->Bbar(), c->Sbar(), c->stage(0), first, count, c->L.chunk);
            staged = true;
        }
        break;
    case APMS_STATE_WORKER_ERR:
        if (c->compressor == APMS_COMPRESSOR_TOPK)
            k_materialise_error_topk<<<grid, kThreads, 0, c->stream>>>(c->z(worker), c->B(worker), c->stage(0), first, count);
        else
            k_materialise_error<<<grid, kThreads, 0, c->stream>>>(c->z(worker), c->s(worker), c->stage(0), first, count, c->L.chunk);
        staged = true;
        break;
    case APMS_STATE_SERVER_ERR:
        if (c->compressor == APMS_COMPRESSOR_TOPK)
            k_materialise_error_topk<<<grid, kThreads, 0, c->stream>>>(c->zbar(), c->Bbar(), c->stage(0), first, count);
        else
            k_materialise_error<<<grid, kThreads, 0, c->stream>>>(c->zbar(), c->Sbar(), c->stage(0), first, count, c->L.chunk);
        staged = true;
        break;
    case APMS_STATE_WORKER_BITS: src = (const char*)c->B(worker); break;
    case APMS_STATE_SERVER_BITS: src = (const char*)c->Bbar(); break;
    case APMS_STATE_WORKER_SCALES: src = (const char*)c->s(worker); break;
    case APMS_STATE_SERVER_SCALES: src = (const char*)c->Sbar(); break;
    default: return fail(c, APMS_ERR_INVALID_ARG, "unknown state id");
    }
    APMS_CUDA(c, cudaGetLastError());
    const char* from = staged ? (const char*)c->stage(0) : src + (size_t)first * 4;
    APMS_CUDA(c, cudaMemcpyAsync(dst, from, (size_t)count * 4, cudaMemcpyDeviceToHost, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    return device_status_check(c);
}

apms_status apms_get_state(apms_ctx* c, apms_state_id which, int worker, void* dst)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    int64_t extent = c->L.d;
    if (which == APMS_STATE_WORKER_BITS || which == APMS_STATE_SERVER_BITS) extent = c->L.W;
    if (which == APMS_STATE_WORKER_SCALES || which == APMS_STATE_SERVER_SCALES) extent = c->L.C;
    return apms_get_state_slice(c, which, worker, 0, extent, dst);
}

apms_status apms_set_state(apms_ctx* c, apms_state_id which, int worker, const void* src)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!src) return fail(c, APMS_ERR_INVALID_ARG, "src is NULL");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    const size_t bytes = (size_t)c->L.d * 4;
    float* dst = nullptr;
    switch (which) {
    case APMS_STATE_X: dst = c->x(); break;
    case APMS_STATE_V: dst = c->v(); break;
    case APMS_STATE_M: dst = c->m(); c->m_is_fp32 = true; break;
    case APMS_STATE_WORKER_ERR:
        if (worker < 0 || worker >= c->L.n) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range");
        if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "errors exist only in the COMPRESSED phase");
        // delta = z - (+-0) = z: store the error as z with all scales of this worker zero
        APMS_CUDA(c, cudaMemsetAsync(c->s(worker), 0, (size_t)c->L.Cp * 4, c->stream));
        if (c->compressor == APMS_COMPRESSOR_TOPK)      // top-k: delta = z - (mask ? z : 0) = z with an empty mask
            APMS_CUDA(c, cudaMemsetAsync(c->B(worker), 0, (size_t)c->L.Wp * 4, c->stream));
        dst = c->z(worker);
        break;
    case APMS_STATE_SERVER_ERR:
        if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "errors exist only in the COMPRESSED phase");
        if (!c->m_is_fp32) {   // Sbar is about to be zeroed: move the momentum it encodes to binary32 first
            k_materialise_momentum<<<grid_for(c, c->L.d, 8), kThreads, 0, c->stream>>>(c->Bbar(), c->Sbar(), c->m(), 0, c->L.d, c->L.chunk);
            APMS_CUDA(c, cudaGetLastError());
            c->m_is_fp32 = true;
        }
        APMS_CUDA(c, cudaMemsetAsync(c->Sbar(), 0, (size_t)c->L.Cp * 4, c->stream));
        if (c->compressor == APMS_COMPRESSOR_TOPK)
            APMS_CUDA(c, cudaMemsetAsync(c->Bbar(), 0, (size_t)c->L.Wp * 4, c->stream));
        dst = c->zbar();
        break;
    default: return fail(c, APMS_ERR_INVALID_ARG, "this state array cannot be set");
    }
    APMS_CUDA(c, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    return APMS_OK;
}

apms_status apms_restore(apms_ctx* c, int t, apms_phase phase)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    if (t < 0 || (phase != APMS_PHASE_WARMUP && phase != APMS_PHASE_COMPRESSED)) return fail(c, APMS_ERR_INVALID_ARG, "invalid t or phase");
    if (phase == APMS_PHASE_COMPRESSED && c->phase == APMS_PHASE_WARMUP) {
        apms_status st = apms_freeze_v(c);
        if (st != APMS_OK) return st;
    }
    c->t = t; c->phase = phase;
    return APMS_OK;
}

float apms_schedule_lr(const apms_schedule* sc, int64_t step)
{
    if (!sc || step < 0) return 0.0f;
    if (sc->lr_ramp_steps > 0 && step < sc->lr_ramp_steps)
        return (float)((double)sc->peak_lr * (double)(step + 1) / (double)sc->lr_ramp_steps);
    if (sc->lr_decay_every <= 0) return sc->peak_lr;
    const int64_t past = step - (sc->lr_ramp_steps > 0 ? sc->lr_ramp_steps : 0);
    return (float)((double)sc->peak_lr * pow((double)sc->lr_decay, (double)(past / sc->lr_decay_every)));
}

apms_status apms_set_schedule(apms_ctx* c, const apms_schedule* sc)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!sc) { c->has_sched = false; return APMS_OK; }
    if (sc->warmup_steps < 0 || !isfinite(sc->peak_lr) || sc->lr_ramp_steps < 0 || sc->lr_decay_every < 0 ||
        !(sc->lr_decay > 0.0f) || !isfinite(sc->lr_decay))
        return fail(c, APMS_ERR_INVALID_ARG, "invalid schedule: need warmup_steps >= 0, finite peak_lr, lr_ramp_steps >= 0, lr_decay > 0, lr_decay_every >= 0");
    c->sched = *sc; c->has_sched = true;
    return APMS_OK;
}

apms_status apms_step(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!c->has_sched) return fail(c, APMS_ERR_BAD_STATE, "apms_step needs a schedule (apms_set_schedule)");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    const float lr = apms_schedule_lr(&c->sched, c->steps);
    apms_status st = apms_set_lr(c, lr);
    if (st != APMS_OK) return st;
    if (c->phase == APMS_PHASE_WARMUP && c->steps >= c->sched.warmup_steps) {       // T_w Adam steps are done
        st = apms_freeze_v(c);
        if (st != APMS_OK) return st;
    }
    st = (c->phase == APMS_PHASE_WARMUP) ? apms_warmup_step_typed(c, grads_dev, type)
                                         : apms_compressed_step_typed(c, grads_dev, type);
    if (st == APMS_OK) c->steps += 1;
    return st;
}

int64_t apms_get_step(const apms_ctx* c) { return c ? c->steps : -1; }

apms_status apms_error_norms(apms_ctx* c, double* worker_sq_host, double* server_sq_host)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "errors exist only in the COMPRESSED phase");
    if (!worker_sq_host && !server_sq_host) return fail(c, APMS_ERR_INVALID_ARG, "both outputs are NULL");
    const int rows = c->L.n + 1;
    ErrNormArgs a;
    a.z = c->z(0); a.dz = c->L.dz; a.s = c->s(0); a.Cp = c->L.Cp; a.zbar = c->zbar(); a.Sbar = c->Sbar();
    a.tiles = (c->L.d + 4095) / 4096; a.n = c->L.n; a.d = c->L.d; a.chunk = c->L.chunk;
    a.partial = reinterpret_cast<double*>(c->ws + c->L.off_mon);
    double* out = a.partial + (size_t)rows * (size_t)a.tiles;
    const int64_t blocks = (int64_t)rows * a.tiles;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many tiles for one launch");
    k_error_norm_tiles<<<(unsigned)blocks, kThreads, 0, c->stream>>>(a);
    apms_status st = launch_check(c, "k_error_norm_tiles");
    if (st != APMS_OK) return st;
    k_error_norm_rows<<<(rows + 63) / 64, 64, 0, c->stream>>>(a.partial, a.tiles, rows, out);
    st = launch_check(c, "k_error_norm_rows");
    if (st != APMS_OK) return st;
    double host[APMS_MAX_WORKERS + 1];
    APMS_CUDA(c, cudaMemcpyAsync(host, out, (size_t)rows * sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    if (worker_sq_host) for (int i = 0; i < c->L.n; ++i) worker_sq_host[i] = host[i];
    if (server_sq_host) *server_sq_host = host[c->L.n];
    return device_status_check(c);
}

apms_phase apms_get_phase(const apms_ctx* c) { return c ? c->phase : APMS_PHASE_CREATED; }
int apms_get_t(const apms_ctx* c) { return c ? c->t : -1; }

apms_status apms_selftest_wait_report(apms_ctx* c, int leave_reported)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    k_selftest_wait<<<1, 32, 0, c->stream>>>(c->status(), 2000000ll);          // about a millisecond
    apms_status st = launch_check(c, "k_selftest_wait");
    if (st != APMS_OK) return st;
    int seen = 0;
    APMS_CUDA(c, cudaMemcpyAsync(&seen, c->status(), sizeof seen, cudaMemcpyDeviceToHost, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    if (!leave_reported) APMS_CUDA(c, cudaMemsetAsync(c->status(), 0, sizeof(int), c->stream));
    if (seen != DEVICE_WAIT_TIMEOUT) return fail(c, APMS_ERR_BAD_STATE, "the bounded wait did not report that it gave up");
    return APMS_OK;
}

apms_status apms_set_compressor(apms_ctx* c, apms_compressor kind, double topk_fraction)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (kind != APMS_COMPRESSOR_ONEBIT && kind != APMS_COMPRESSOR_TOPK) return fail(c, APMS_ERR_INVALID_ARG, "unknown compressor");
    if (c->csteps > 0 && (int)kind != c->compressor)
        return fail(c, APMS_ERR_BAD_STATE, "the compressor cannot change once a compression-phase step has run");
    if (kind == APMS_COMPRESSOR_TOPK) {
        if (!(topk_fraction > 0.0 && topk_fraction <= 1.0)) return fail(c, APMS_ERR_INVALID_ARG, "the top-k fraction must lie in (0, 1]");
        if (c->variant != APMS_VARIANT_MOMENTUM || c->L.t.l1) return fail(c, APMS_ERR_BAD_STATE, "top-k runs with the momentum variant and has no scale");
        c->topk_frac = topk_fraction;
    }
    c->compressor = (int)kind;
    return APMS_OK;
}

apms_status apms_set_variant(apms_ctx* c, apms_variant variant)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (variant != APMS_VARIANT_MOMENTUM && variant != APMS_VARIANT_GRADIENT) return fail(c, APMS_ERR_INVALID_ARG, "unknown variant");
    if (variant == APMS_VARIANT_GRADIENT && c->compressor == APMS_COMPRESSOR_TOPK)
        return fail(c, APMS_ERR_BAD_STATE, "the gradient variant exists for the 1-bit compressor only");
    if (c->csteps > 0 && (int)variant != c->variant)
        return fail(c, APMS_ERR_BAD_STATE, "the variant cannot change once a compression-phase step has run");
    c->variant = (int)variant;
    return APMS_OK;
}

apms_status apms_uncompressed_step_typed(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_uncompressed_step needs v frozen (call apms_freeze_v first)");
    if (c->substep != 0) return fail(c, APMS_ERR_BAD_STATE, "a phase-wise step is in progress (finish it with apms_apply_phase)");
    GradPtrs G;
    apms_status st = check_grads(c, grads_dev, (int)type, &G, c->L.n);
    if (st != APMS_OK) return st;
    if (!c->m_is_fp32) {       // the momentum lives in the server's message: spell it out in binary32 first
        k_materialise_momentum<<<grid_for(c, c->L.d, 8), kThreads, 0, c->stream>>>(c->Bbar(), c->Sbar(), c->m(), 0, c->L.d, c->L.chunk);
        st = launch_check(c, "k_materialise_momentum");
        if (st != APMS_OK) return st;
        c->m_is_fp32 = true;
    }
    UncompressedArgs a;
    a.x = c->x(); a.m = c->m(); a.v = c->v(); a.d = c->L.d; a.n = c->L.n;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1; a.lr = c->lr; a.eps = c->eps; a.nf = (float)c->L.n;
    const int64_t blocks = (c->L.d + (int64_t)kThreads * 4 - 1) / ((int64_t)kThreads * 4);
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "d too large for one launch");
    Timed t(c, APMS_KERNEL_WARMUP_ADAM);
    APMS_DISPATCH_GRAD((int)type, k_uncompressed<GT><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
    return launch_check(c, "k_uncompressed");
}

apms_status apms_set_scale_kind(apms_ctx* c, apms_scale_kind kind)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (kind != APMS_SCALE_L2 && kind != APMS_SCALE_L1_MEAN) return fail(c, APMS_ERR_INVALID_ARG, "unknown scale kind");
    c->L.t.l1 = kind == APMS_SCALE_L1_MEAN ? 1 : 0;
    return APMS_OK;
}

apms_status apms_set_team_mode(apms_ctx* c, apms_team_mode mode)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (mode != APMS_TEAM_AUTO && mode != APMS_TEAM_CTA && mode != APMS_TEAM_WARP && mode != APMS_TEAM_STAGED) return fail(c, APMS_ERR_INVALID_ARG, "unknown team mode");
    c->team_mode = mode;
    return APMS_OK;
}

apms_status apms_set_timing(apms_ctx* c, int enabled)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    c->timing = enabled != 0;
    return APMS_OK;
}

apms_status apms_kernel_time(apms_ctx* c, apms_kernel_id which, double* total_ms, int64_t* launches)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if ((int)which < 0 || which >= APMS_KERNEL_COUNT) return fail(c, APMS_ERR_INVALID_ARG, "unknown kernel id");
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    double sum = 0.0;
    for (EventPair& ev : c->events[which]) {
        float ms = 0.f;
        APMS_CUDA(c, cudaEventElapsedTime(&ms, ev.a, ev.b));
        sum += ms;
        c->pool.push_back(ev);
    }
    if (total_ms) *total_ms = sum;
    if (launches) *launches = (int64_t)c->events[which].size();
    c->events[which].clear();
    return APMS_OK;
}

int64_t apms_launch_count(const apms_ctx* c) { return c ? c->launches : 0; }

const char* apms_last_error(const apms_ctx* c) { return c ? c->err : g_create_error; }

void apms_destroy(apms_ctx* c)
{
    if (!c) return;
    if (c->stream || c->ws) cudaStreamSynchronize(c->stream);
    for (int k = 0; k < APMS_KERNEL_COUNT; ++k)
        for (EventPair& ev : c->events[k]) { cudaEventDestroy(ev.a); cudaEventDestroy(ev.b); }
    for (EventPair& ev : c->pool) { cudaEventDestroy(ev.a); cudaEventDestroy(ev.b); }
    if (c->host_path_ready) {
        for (int b = 0; b < 2; ++b) { cudaEventDestroy(c->ev_copied[b]); cudaEventDestroy(c->ev_used[b]); }
        cudaStreamDestroy(c->copy_stream);
    }
    if (c->owns_ws && c->ws) cudaFree(c->ws);
    delete c;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Allocation-free compression of a flat vector (apms_compress_noalloc).  Callers that may not
// allocate device memory (allocator-free regions of a framework, plugins given fixed buffers,
// loops that cannot afford cudaMalloc's device-wide synchronisation) get the Section 5.1
// compressor with its one piece of scratch - a binary64 partial sum per tile - in a fixed
// array of the library's device image instead of a workspace.

namespace {

constexpr int64_t kNoallocTile = 32768;

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) double g_noalloc_partial[APMS_NOALLOC_MAX_TILES];

constexpr int kNoallocMaxDevices = 64;
struct NoallocDevice { bool ready; double* partial; };
NoallocDevice g_noalloc_dev[kNoallocMaxDevices];
std::mutex g_noalloc_mutex;

// One CTA per tile: sign words of the tile, and the tile's sum of squares into its slot.
__global__ void __launch_bounds__(kThreads)
k_noalloc_compress(const float* __restrict__ z, uint32_t* __restrict__ bits, double* __restrict__ partial,
                   const Tiling t)
{
    __shared__ double red[kWarps];
    const Item it = decode_item(t, (int64_t)blockIdx.x);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int L = it.L;
    const float* __restrict__ zt = z + it.base;
    uint32_t* __restrict__ ob = bits + it.base / 32;
    const int ngroups = (L + kGroup - 1) / kGroup;
    double acc = 0.0;
    for (int grp = warp; grp < ngroups; grp += kWarps) {
        const int k = grp * kGroup + lane * 4;
        const float4 v4 = ld4_checked(zt, k, L, true);
        const float zv[4] = {v4.x, v4.y, v4.z, v4.w};
        uint32_t nibble = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (k + e < L) {
                const double zd = (double)zv[e];
                acc = fma(zd, zd, acc);
                nibble |= (zv[e] >= 0.0f ? 1u : 0u) << e;
            }
        }
        const uint32_t word = pack_group_words(nibble, lane);
        const int wk = grp * 4 + (lane >> 3);
        if ((lane & 7) == 0 && wk * 32 < L) ob[wk] = word;
    }
    const double total = block_sum(acc, red);
    if (threadIdx.x == 0) partial[blockIdx.x] = total;      // every slot is written before it is read
}

apms_status noalloc_fail(apms_status st, const char* msg)
{
    snprintf(g_create_error, sizeof g_create_error, "apms_compress_noalloc: %s", msg);
    return st;
}

}  // namespace

extern "C" apms_status apms_compress_noalloc(const float* z_dev, int64_t d, int64_t chunk,
                                             uint32_t* bits_dev, float* scales_dev, void* cuda_stream)
{
    if (!z_dev || !bits_dev || !scales_dev) return noalloc_fail(APMS_ERR_INVALID_ARG, "a buffer pointer is NULL");
    if (((uintptr_t)z_dev & 15u) != 0) return noalloc_fail(APMS_ERR_INVALID_ARG, "z_dev is not 16-byte aligned");
    if (d < 1 || chunk < 32 || chunk % 32 != 0 || chunk > ((int64_t)1 << 30))
        return noalloc_fail(APMS_ERR_INVALID_ARG, "need d >= 1 and chunk a positive multiple of 32 (at most 2^30)");
    Tiling t;
    t.d = d; t.chunk = chunk;
    if (chunk <= kNoallocTile) { t.tile = chunk; t.P = 1; }
    else { t.tile = kNoallocTile; t.P = (int)((chunk + kNoallocTile - 1) / kNoallocTile); }
    const int64_t C = (d + chunk - 1) / chunk;
    if (C > APMS_NOALLOC_MAX_TILES || C * t.P > APMS_NOALLOC_MAX_TILES) {
        char msg[200];
        snprintf(msg, sizeof msg, "shape needs %lld tiles of the fixed scratch array, the maximum is %d "
                 "(ceil(d/chunk) * ceil(chunk/32768) <= %d)", (long long)(C * t.P), APMS_NOALLOC_MAX_TILES,
                 APMS_NOALLOC_MAX_TILES);
        return noalloc_fail(APMS_ERR_INVALID_ARG, msg);
    }
    const int64_t tiles = C * t.P;
    t.Pp = tiles;

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(APMS_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= kNoallocMaxDevices) return noalloc_fail(APMS_ERR_INVALID_ARG, "device ordinal out of range");
    double* partial = nullptr;
    {
        // set-up, once per device, with that device current: the device address of the fixed array
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_dev[dev].ready) {
            double* p = nullptr;
            e = cudaGetSymbolAddress((void**)&p, g_noalloc_partial);
            if (e != cudaSuccess || !p) return noalloc_fail(APMS_ERR_CUDA, cudaGetErrorString(e));
            g_noalloc_dev[dev].partial = p;
            g_noalloc_dev[dev].ready = true;
        }
        partial = g_noalloc_dev[dev].partial;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    k_noalloc_compress<<<(unsigned)tiles, kThreads, 0, stream>>>(z_dev, bits_dev, partial, t);
    e = cudaGetLastError();
    if (e != cudaSuccess) return noalloc_fail(APMS_ERR_CUDA, cudaGetErrorString(e));
    k_finalize_scales<<<(unsigned)((C + 255) / 256), 256, 0, stream>>>(partial, scales_dev, 1, C, C, t);
    e = cudaGetLastError();
    if (e != cudaSuccess) return noalloc_fail(APMS_ERR_CUDA, cudaGetErrorString(e));
    return APMS_OK;
}
