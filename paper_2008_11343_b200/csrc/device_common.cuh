// Constants, tunables and the small device helpers every kernel uses (loads and stores,
// the per-element arithmetic with its roundings pinned, sign-word packing, block sums).
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

constexpr int kThreads = 256;            // threads per CTA in every kernel
constexpr int kWarps = kThreads / 32;
constexpr int kGroup = 128;              // elements one warp covers per 128-bit access (4 sign words)

// Tunables (defaults chosen by measurement on B200; override with -D to re-tune).
#ifndef APMS_WORKER_U
#define APMS_WORKER_U 4                  // 128-element groups in flight per warp, worker kernel
#endif
#ifndef APMS_SERVER_U
#define APMS_SERVER_U 4                  // the same for the server kernel (chunk 1024, n = 2: 0.84 ms at 2, 0.72 ms at 4)
#endif
#ifndef APMS_WORKER_CTAS
#define APMS_WORKER_CTAS 3               // resident CTAs per SM the worker kernel is compiled for
#endif
#ifndef APMS_SERVER_CTAS
#define APMS_SERVER_CTAS 3
#endif

struct GradPtrs { const void* p[APMS_MAX_WORKERS]; };     // element type given by the kernel's GT template argument

// ------------------------------------------------------------------------------------------
// Checked build (-DAPMS_BOUNDS_CHECK; stands in for a memory checker): every global store of the step's
// kernels, their streaming loads and the sources of their bulk copies first look the address up in a table
// of the live contexts' workspaces and guard regions (the guard layout of apms_set_guard_bytes).  An access
// that is not wholly inside an array - a store outside every workspace, or any access that touches guard
// bytes (loads may run up to 16 bytes into them: bulk copies are whole 16-byte pieces) - is NOT performed;
// the first such access is recorded in the owning context's status words and the next synchronising call
// returns APMS_ERR_BOUNDS.  Nothing traps.  In the ordinary build the macros below cost nothing.

enum { DEVICE_OK = 0, DEVICE_WAIT_TIMEOUT = 1, DEVICE_BOUNDS = 2 };

#ifdef APMS_BOUNDS_CHECK
struct CheckedWorkspace {
    unsigned long long lo, hi;                   // [lo, hi): the workspace
    const unsigned long long* guards;            // pairs (offset, bytes), ascending by offset
    int nguards;
    int* status;                                 // [0] code, [2..3] address, [4] bytes, [5] 1 = store
};
constexpr int kMaxCheckedWorkspaces = 64;
__device__ CheckedWorkspace g_checked[kMaxCheckedWorkspaces];
__device__ int g_checked_count;

__device__ __noinline__ bool checked_access(const void* p, unsigned bytes, bool store)
{
    const unsigned long long a0 = (unsigned long long)p, a1 = a0 + bytes;
    const int count = g_checked_count;
    int* report = count > 0 ? g_checked[0].status : nullptr;
    bool bad = store;                            // a store must land inside some workspace; a load may read the caller's memory
    for (int w = 0; w < count; ++w) {
        const CheckedWorkspace& ws = g_checked[w];
        if (a1 <= ws.lo || a0 >= ws.hi) continue;
        report = ws.status;
        bad = a0 < ws.lo || a1 > ws.hi;
        // the last guard region that begins below the end of the access
        int lo = 0, hi = ws.nguards;
        while (lo < hi) {
            const int mid = (lo + hi) / 2;
            if (ws.lo + ws.guards[2 * mid] < a1) lo = mid + 1; else hi = mid;
        }
        if (lo > 0) {
            const unsigned long long g0 = ws.lo + ws.guards[2 * (lo - 1)], g1 = g0 + ws.guards[2 * (lo - 1) + 1];
            const unsigned long long slack = store ? 0ull : 16ull;
            if (a1 > g0 + slack && a0 < g1) bad = true;
        }
        break;
    }
    if (bad && report && atomicCAS(report, DEVICE_OK, DEVICE_BOUNDS) == DEVICE_OK) {
        report[2] = (int)(a0 & 0xffffffffull); report[3] = (int)(a0 >> 32);
        report[4] = (int)bytes; report[5] = store ? 1 : 0;
    }
    return !bad;
}
// where a skipped bulk copy reads instead (its byte count is already promised to the mbarrier)
__device__ __forceinline__ const void* checked_safe_source() { return (const void*)g_checked[0].lo; }
#define APMS_CAN_LOAD(p, bytes) checked_access((p), (unsigned)(bytes), false)
#define APMS_CAN_STORE(p, bytes) checked_access((p), (unsigned)(bytes), true)
#else
#define APMS_CAN_LOAD(p, bytes) true
#define APMS_CAN_STORE(p, bytes) true
#endif
// a scalar (or vector) store to global memory, skipped when the checked build finds it out of bounds
#define APMS_STORE(lvalue, value) do { if (APMS_CAN_STORE(&(lvalue), sizeof(lvalue))) (lvalue) = (value); } while (0)

// ------------------------------------------------------------------------------------------
// small device helpers

__device__ __forceinline__ float4 ld_stream4(const float* p)
{
    if (!APMS_CAN_LOAD(p, 16)) return make_float4(0.f, 0.f, 0.f, 0.f);
    return __ldcs(reinterpret_cast<const float4*>(p));
}
// Hint that a line will be wanted soon: no register, no wait, no fault (the address is a valid element's).
__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" :: "l"(p)); }
__device__ __forceinline__ void st_stream4(float* p, float4 v) { if (APMS_CAN_STORE(p, 16)) __stcs(reinterpret_cast<float4*>(p), v); }
__device__ __forceinline__ void st_stream_word(uint32_t* p, uint32_t v) { if (APMS_CAN_STORE(p, 4)) __stcs(p, v); }
__device__ __forceinline__ void st_stream_words4(uint32_t* p, uint4 v) { if (APMS_CAN_STORE(p, 16)) __stcs(reinterpret_cast<uint4*>(p), v); }

// Up to four consecutive floats starting at p[k]; elements at or past `len` read as 0.
__device__ __forceinline__ float4 ld4_checked(const float* p, int k, int len, bool streaming) {
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k + 3 < len) {
        r = streaming ? ld_stream4(p + k) : (APMS_CAN_LOAD(p + k, 16) ? *reinterpret_cast<const float4*>(p + k) : r);
    } else if (k < len && APMS_CAN_LOAD(p + k, 4 * (len - k))) {
        if (k + 0 < len) r.x = p[k + 0];
        if (k + 1 < len) r.y = p[k + 1];
        if (k + 2 < len) r.z = p[k + 2];
    }
    return r;
}
__device__ __forceinline__ void st4_checked(float* p, int k, int len, float4 v) {
    if (k + 3 < len) {
        st_stream4(p + k, v);
    } else if (k < len && APMS_CAN_STORE(p + k, 4 * (len - k))) {
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
        if (!APMS_CAN_LOAD((const uint16_t*)p + k, 8)) return make_float4(0.f, 0.f, 0.f, 0.f);
        const uint2 r = __ldcs(reinterpret_cast<const uint2*>((const uint16_t*)p + k));
        return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                           __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
    }
};
template <> struct Grad<APMS_GRAD_F16> {
    static __device__ __forceinline__ const void* at(const void* p, int64_t e) { return (const __half*)p + e; }
    static __device__ __forceinline__ float ld1(const void* p, int64_t e) { return __half2float(((const __half*)p)[e]); }
    static __device__ __forceinline__ float4 ld4(const void* p, int k) {
        if (!APMS_CAN_LOAD((const __half*)p + k, 8)) return make_float4(0.f, 0.f, 0.f, 0.f);
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

// floor(a / b) for 0 <= a < 2^40, 0 < b, quotient below 2^21 (checked by the host, which passes 1 / b rounded to
// binary32): the product of the two binary32 values is within one of the quotient, two multiplications settle it.
// A general 64-bit division is a subroutine of about seventy instructions - per warp and 512 elements that is a
// sizeable share of the worker kernel's instructions.
__device__ __forceinline__ int64_t div_small_quotient(int64_t a, int64_t b, float inv_b)
{
    int64_t q = (int64_t)(__ll2float_rz(a) * inv_b);
    while (q * b > a) --q;                       // at most once for quotients below 2^21
    while ((q + 1) * b <= a) ++q;
    return q;
}

// floor(x / d) for 32-bit operands from an estimate (x times 1 / d in binary32) and exact corrections: the loops
// run zero times or once for the quotients that occur (block index over tiles per run and the like).
__device__ __forceinline__ uint32_t div_u32(uint32_t x, uint32_t d, float inv_d)
{
    uint32_t q = (uint32_t)(__uint2float_rz(x) * inv_d);
    while ((uint64_t)q * d > x) --q;
    while ((uint64_t)(q + 1) * d <= x) ++q;
    return q;
}

// +-s with the sign of the compressor: z >= 0 gives +s (so do +0 and -0), NaN gives -s.
__device__ __forceinline__ float signed_scale(float z, float s) { return (z >= 0.0f) ? s : -s; }
__device__ __forceinline__ float bit_scale(uint32_t bit, float s) { return bit ? s : -s; }

// The same update from its stored pieces: den = sqrt(v) + eps (formed once while v is frozen) and
// c = lr * S (once per chunk); lr * (+-S) = +-(lr * S) exactly, so this is apply_elem(x, v, +-S, lr, eps) bit for bit.
__device__ __forceinline__ float apply_stored(float x, float den, uint32_t bit, float c) {
    return __fsub_rn(x, __fdiv_rn(bit ? c : -c, den));
}

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

}  // namespace
