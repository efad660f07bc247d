// The allocation-free compressor entry point (apms_compress_noalloc) and its kernel.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

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
