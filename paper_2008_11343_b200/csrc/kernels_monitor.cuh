// Error-norm monitor and the bounded-wait self-test kernel.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Error monitor: squared l2 norms of the compression errors (the quantities Assumption 1 bounds).
// Row r < n is worker r (delta = z_r - (+-s_r)), row n the server.  One CTA per (row, 4096-element
// tile) writes a binary64 partial sum; k_error_norm_rows adds a row's tiles in order.
// Top-k mode: the stored words are selection masks and the error of an element is z where it was
// not sent and +0 where it was (delta = z - C[z]).

struct ErrNormArgs {
    const float* z; int64_t dz; const float* s; int64_t Cp;      // worker rows
    const float* zbar; const float* Sbar;                         // server row
    const uint32_t* B; int64_t Wp; const uint32_t* Bbar; int topk; // top-k: masks in place of scales
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
    const uint32_t* __restrict__ mask = row < a.n ? a.B + (int64_t)row * a.Wp : a.Bbar;
    const int64_t base = t * 4096;
    double acc = 0.0;
    for (int k = threadIdx.x; k < 4096; k += kThreads) {
        const int64_t j = base + k;
        if (j < a.d) {
            const double e = a.topk ? (((mask[j >> 5] >> (j & 31)) & 1u) ? 0.0 : (double)z[j])
                                    : (double)implied_error(z[j], s[j / a.chunk]);
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

#ifdef APMS_BOUNDS_CHECK
// Self-test of the checked build: one checked store to an address the host chose inside guard bytes.
__global__ void k_selftest_bounds(float* target)
{
    if (threadIdx.x == 0) st_stream4(target, make_float4(1.f, 2.f, 3.f, 4.f));
}
#endif

}  // namespace
