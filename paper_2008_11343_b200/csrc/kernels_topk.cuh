// Top-k compressor (Section 5.1, second item): worker and server kernels.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Top-k compressor (Section 5.1, second item): per chunk the K = ceil(k L) elements of largest |z| are
// sent, the others decompress to 0; equal magnitudes go to the lower index.  State in this mode: the
// compensated vectors z as before, and in place of the sign words a SELECTION MASK (bit j = element j
// was sent), from which  C[z] = mask ? z : 0  and  delta = z - C[z]  follow exactly; in place of the
// scales the chunk's last threshold.  The momentum C[zbar] is read as (server mask ? zbar : 0) unless it
// was written out in binary32.  One CTA per (chunk, worker) / per chunk.
//
// Selection.  Keys are the bit patterns of |z|; the K-th largest key tau and the number of elements
// equal to tau that are to be kept (`ties`, lowest positions first) define the mask.  Three routes, all
// exact, in the order of their cost:
//   window     small K: the first pass lists the keys at or above a floor a little below the chunk's last
//              threshold; tau and the mask come from that list alone (topk_threshold_list);
//   two passes the first pass counts all keys in fine bins around the last threshold; a second pass keeps
//              what lies above the K-th key's bin and lists that bin, which the list settles;
//   general    three-level radix select over the whole chunk (11 + 11 + 9 bits, topk_threshold) and a pass
//              in index order that ranks equal keys across the block (topk_select_wave).

constexpr int kTopkBins = 2048;

// CTA shape of the top-k kernels.  Their passes are latency-bound, so resident threads matter more than registers:
// 1536 threads per SM at 40 registers measured fastest (at 2048 threads and 32 registers the spills cost more than
// the extra warps give).  As 3 CTAs of 512 threads rather than 6 of 256: a chunk is then finished in half the
// time, half as many chunks are in flight (444 x 128 KB of compensated values), and the later passes over a chunk
// find it in L2 - with 888 chunks in flight they came from DRAM again (ncu, two-pass route, 8 workers x 116 M
// elements: 11.5 GB read against 8.1 GB).
constexpr int kTopkResident = 3;
constexpr int kTopkThreads = 512, kTopkWarps = kTopkThreads / 32;


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
    for (int b = threadIdx.x; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
    __syncthreads();
    // the lower levels spread over many bins: plain atomics (combining equal bins costs more than it saves there)
#pragma unroll 4
    for (int k = threadIdx.x * 4; k < L; k += kTopkThreads * 4) {
        const float4 zv = ld4_checked(zc, k, L, false);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (k + e < L && (key[e] >> 20) == b0) atomicAdd(&hist[(key[e] >> 9) & 0x7ffu], 1u);
    }
    const uint32_t b1 = (uint32_t)topk_find_bin(hist, kTopkBins, K, sh);
    for (int b = threadIdx.x; b < 512; b += kTopkThreads) hist[b] = 0;
    __syncthreads();
    const uint32_t top = (b0 << 11) | b1;
#pragma unroll 4
    for (int k = threadIdx.x * 4; k < L; k += kTopkThreads * 4) {
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
// floor a little below it (key lowered by up to 2^20, an eighth of an exponent step: 0.92 of the threshold) are
// looked at for the selection, which is exact either way - a chunk whose window turns out to hold fewer
// than K keys, or more than the list below can take, is counted in a further pass and goes the two-pass
// route.  Error feedback piles the unsent elements up just under the threshold, and while
// the errors still build up the threshold rises by 5 to 10 % a step, so the window holds several times K
// keys (about 4 K on the benchmark's gradients at k = 1 %).  Hence a window only for K <= kTopkList / 6
// (larger K: the two-sided band below), and every (worker, chunk) adapts how far below the threshold its window
// reaches to how many keys it listed last step (topk_window_learn).  A stored threshold of 0
// (first step) also means no window.  The list is kept small on purpose: shared memory comes out of the L1
// cache, which the first pass, the general route and the server's sparse sum live on (a list of 4096 entries
// made the worker 45 % and the server 30 % slower).
constexpr int kTopkList = 2048;
constexpr uint32_t kTopkFloorDrop = 1u << 20, kTopkFloorDropMin = 1u << 16;
__device__ __forceinline__ uint32_t topk_floor(float last_threshold, uint32_t K, uint32_t drop)
{
    const uint32_t key = mag_key(last_threshold);
    return (6 * K <= (uint32_t)kTopkList && key > drop) ? key - drop : 0u;
}
__device__ __forceinline__ uint32_t topk_window_drop(float learned)
{
    const uint32_t drop = __float_as_uint(learned);
    return (drop >= kTopkFloorDropMin && drop <= kTopkFloorDrop) ? drop : kTopkFloorDrop;
}
__device__ __forceinline__ uint32_t topk_window_learn(uint32_t drop, uint32_t listed, uint32_t K)
{
    if (listed > 3u * kTopkList / 4) return drop / 2 >= kTopkFloorDropMin ? drop / 2 : kTopkFloorDropMin;
    if (listed < K || listed < (uint32_t)kTopkList / 4) return drop * 2 <= kTopkFloorDrop ? drop * 2 : kTopkFloorDrop;
    return drop;
}

// Larger K: the window would hold more keys than the list takes, so the prediction has to be two-sided: keys at
// or above a band around the predicted threshold are kept at once, keys inside the band go to the list, which
// settles them, and the chunk is read once.  How wide the band may be depends on how densely the keys lie around
// the threshold, and error feedback piles them up there as the steps go on (measured on the benchmark's
// gradients: from 330 to more than 700 keys per 4 % of the value, of a chunk of 32768 at k = 10 %), so every
// (worker, chunk) learns its own band from its last step (topk_learn): the half-width that would have listed
// about kTopkBandTarget keys, and which of three simple predictions (topk_predict) came closest (keys are close
// to a logarithmic scale: a linear step in the key is a ratio in the value).  The
// band is only used if that prediction would have hit a band 0.7 times as wide last step; otherwise, and when
// the band misses after all (the K-th key outside it, or more keys inside than the list takes: the chunk is then
// counted in a further pass), the two-pass route runs and learns again.  Exact on every route.
constexpr uint32_t kTopkBandTarget = 1000;
constexpr uint32_t kTopkBandMaxHalf = 3u << 18;      // one and a half bins of a sixteenth of an exponent step: -6 % .. +7 %
constexpr uint32_t kTopkBandMinHalf = 1u << 12;
constexpr int64_t kTopkBandMaxStep = 4 << 19;
__device__ __forceinline__ int64_t topk_trend(uint32_t last_key, uint32_t prev_key)
{
    if (prev_key == 0) return 0;
    const int64_t step = (int64_t)last_key - (int64_t)prev_key;
    return step > kTopkBandMaxStep ? kTopkBandMaxStep : (step < -kTopkBandMaxStep ? -kTopkBandMaxStep : step);
}
// The candidates for this step's threshold key: 0 the last step's, 1 its extrapolation by the step before, 2 the
// key of the step before (a threshold that alternates, as it does when the same few batches come round).
__device__ __forceinline__ int64_t topk_predict(int which, uint32_t last_key, uint32_t prev_key)
{
    if (which == 1) return (int64_t)last_key + topk_trend(last_key, prev_key);
    if (which == 2 && prev_key != 0) return (int64_t)prev_key;
    return (int64_t)last_key;
}
// learned: the half-width (a multiple of 4) + the candidate to use; 0 = no band.
__device__ __forceinline__ void topk_band(uint32_t last_key, uint32_t prev_key, uint32_t learned, uint32_t& lo, uint32_t& hi)
{
    lo = hi = 0;
    const uint32_t half = learned & ~3u;
    if (half == 0 || last_key == 0) return;
    const int64_t pred = topk_predict((int)(learned & 3u), last_key, prev_key);
    if (pred <= (int64_t)(1u << 23) || pred >= (int64_t)0x7f000000) return;
    lo = (uint32_t)pred - half;
    hi = (uint32_t)pred + half;
}
// After a step: `count` keys were seen in `width` key units around the new threshold tau (the band's list, or the
// K-th key's bin of the two-pass route; width 0: nothing learned).  Returns what topk_band takes next step.
__device__ __forceinline__ uint32_t topk_learn(uint32_t tau, uint32_t last_key, uint32_t prev_key, uint32_t count, uint32_t width)
{
    if (width == 0 || last_key == 0) return 0;
    uint64_t half = count ? (uint64_t)width * (kTopkBandTarget / 2) / count : kTopkBandMaxHalf;
    if (half > kTopkBandMaxHalf) half = kTopkBandMaxHalf;
    if (half < kTopkBandMinHalf) return 0;
    int best = 0;
    int64_t err = llabs((int64_t)tau - topk_predict(0, last_key, prev_key));
#pragma unroll
    for (int which = 1; which < 3; ++which) {
        const int64_t e = llabs((int64_t)tau - topk_predict(which, last_key, prev_key));
        if (e < err) { err = e; best = which; }
    }
    if (err * 10 > (int64_t)half * 7) return 0;
    return ((uint32_t)half & ~3u) | (uint32_t)best;
}

// The keys inside the window are appended, with their positions in the chunk (16 bits: the list is used
// for chunks of up to 65536 elements), to a list in shared memory, and threshold and mask are then taken
// from the list alone - no further pass over the chunk.
// From this kept fraction on the server sums the workers' messages in registers (see k_topk_server): measured
// on 16 workers, 335 M elements, the scattered form takes 2.7 / 3.7 / 5.9 / 12.4 ms at k = 0.1 / 1 / 3 / 10 %,
// the register form 3.8 / 4.6 / 5.2 / 5.9 ms.
constexpr double kTopkDenseSum = 0.02;
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
static_assert(kTopkThreads >= 256, "one histogram bin per thread");
__device__ __forceinline__ bool topk_threshold_list(const TopkList& l, int n, uint32_t floor_key, uint32_t K,
                                                    uint32_t* hist /* 256 bins */, uint32_t* sh,
                                                    uint32_t& tau, uint32_t& ties, uint32_t& ties_total)
{
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < n; p += kTopkThreads) {
        const uint32_t rel = l.key[p] - floor_key;
        atomicAdd(&hist[rel >> 16 < 255u ? rel >> 16 : 255u], 1u);
    }
    const uint32_t b0 = (uint32_t)topk_find_bin(hist, 256, K, sh);
    if (b0 == 255u) return false;                      // the same value in every thread
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < n; p += kTopkThreads) {
        const uint32_t rel = l.key[p] - floor_key;
        if (rel >> 16 == b0) atomicAdd(&hist[(rel >> 8) & 0xffu], 1u);
    }
    const uint32_t b1 = (uint32_t)topk_find_bin(hist, 256, K, sh);
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t top = (b0 << 8) | b1;
    for (int p = threadIdx.x; p < n; p += kTopkThreads) {
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
    for (int b = threadIdx.x; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < L; j += kTopkThreads) atomicAdd(&hist[mag_key(zc[j]) >> 20], 1u);
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
    for (int w = 0; w < kTopkWarps; ++w) { const uint32_t c = warp_ties[w]; if (w < warp) before += c; total += c; }
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
    const float* m32;                 // the momentum in binary32 (M32 form of the kernel) ...
    const float* zbar; const uint32_t* Bbar;   // ... or as the server left it: m = C[zbar] = mask ? zbar : 0
    float* thr; int64_t Cp;           // per (worker, chunk): the magnitude of the K-th element of the last step
    float* hint; float* learned;      // ... of the step before, and what topk_learn made of it (same stride): only ever prediction aids
    int* route;                       // 6 counters: chunks settled by the predicted list / by two passes / by the general route;
                                      // predictions missed because the K-th key lay above / below the listed keys / the list overflowed
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

// M32: the momentum is read from the binary32 buffer (first step of the phase, after a state upload, or
// when the server applies densely); otherwise it is taken from the server's compensated vector where the
// server's mask has a bit, so that the server need not write a momentum vector at all.
// BAND: K is too large for the one-sided window (chosen by the host from the full chunk's K); the first pass
// then uses the two-sided band where both earlier thresholds are known.
template <int GT, bool M32, bool BAND>
__global__ void __launch_bounds__(kTopkThreads, kTopkResident)
k_topk_worker(const __grid_constant__ GradPtrs G, const TopkWorkerArgs a)
{
    __shared__ uint32_t hist[kTopkBins];
    __shared__ uint32_t bins8[256];
    __shared__ uint32_t sh[2];
    __shared__ uint32_t above_total;
    __shared__ uint32_t warp_ties[kTopkWarps];
    __shared__ TopkList list;
    const int ii = (int)(blockIdx.x % a.ni);
    const int64_t c = blockIdx.x / a.ni;
    const int i = a.i0 + ii;
    const int64_t base = c * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], base);
    float* zc = a.z + (int64_t)i * a.dz + base;
    uint32_t* maskw = a.B + (int64_t)i * a.Wp + base / 32;
    const float* __restrict__ m = (M32 ? a.m32 : a.zbar) + base;
    const uint32_t* __restrict__ mbar = a.Bbar + base / 32;
    float* thr = a.thr + (int64_t)i * a.Cp + c;
    float* hint = a.hint + (int64_t)i * a.Cp + c;
    const float last_thr = *thr;
    const uint32_t K = topk_count(a.frac, L);
    const int nwords = (L + 31) / 32;
    const bool small = nwords <= kTopkBins;            // the mask fits the shared-memory words: list routes possible
    float* learned = a.learned + (int64_t)i * a.Cp + c;
    const uint32_t drop = topk_window_drop(*learned);
    const uint32_t floor_key = (small && !BAND) ? topk_floor(last_thr, K, drop) : 0u;
    const uint32_t last_key = mag_key(last_thr), prev_key = mag_key(*hint);
    uint32_t band_lo = 0, band_hi = 0;
    if (BAND && small) topk_band(last_key, prev_key, __float_as_uint(*learned), band_lo, band_hi);
    const bool band = BAND && band_lo != 0;
    uint32_t learn_count = 0, learn_width = 0;
    const int shift = small ? 19 : 20, bin0 = small ? topk_fine_base(last_thr) : 0;
    const int lane = threadIdx.x & 31;
    uint32_t above = 0;                                // band: this thread's keys at or above it

    for (int b = threadIdx.x; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
    if (threadIdx.x == 0) { list.count = 0; above_total = 0; }
    __syncthreads();
    // pass A: z = (b1 m + (1-b1) g) + delta_old, with delta_old from the stored z and last step's mask;
    // whole 1024-element sweeps without bounds checks, two sweeps' loads in flight, then the ragged rest
    const int Lfull = L & ~(kTopkThreads * 4 - 1);
    auto sweep = [&](int k, float4 gv, float4 zv, float4 mv, uint32_t nib, bool checked) {
        const float gg[4] = {gv.x, gv.y, gv.z, gv.w}, zo[4] = {zv.x, zv.y, zv.z, zv.w}, mm[4] = {mv.x, mv.y, mv.z, mv.w};
        float zn[4];
        uint32_t kept = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float mi = __fmaf_rn(a.beta1, mm[e], __fmul_rn(a.omb1, gg[e]));
            zn[e] = __fadd_rn(mi, topk_error(zo[e], (nib >> e) & 1u));
            if (!checked || k + e < L) {
                const uint32_t key = mag_key(zn[e]);
                if (BAND && band) {
                    if (key >= band_hi) kept |= 1u << e;
                    else if (key >= band_lo) topk_list_add(list, key, (uint32_t)(k + e));
                } else if (floor_key == 0) atomicAdd(&hist[topk_bin(key, shift, bin0)], 1u);     // no prediction: every key counts
                else if (key >= floor_key) topk_list_add(list, key, (uint32_t)(k + e));
            }
        }
        if (BAND && band) {                            // every sweep is taken by whole warps
            above += __popc(kept);
            const uint32_t word = pack_group_words(kept, lane);     // valid in lanes 0, 8, 16, 24
            if ((lane & 7) == 0 && (!checked || k < L)) hist[k >> 5] = word;
        }
        if (!checked || k + 3 < L) *reinterpret_cast<float4*>(zc + k) = make_float4(zn[0], zn[1], zn[2], zn[3]);
        else for (int e = 0; e < 4 && k + e < L; ++e) zc[k + e] = zn[e];
    };
    // the momentum of elements k..k+3
    auto momentum = [&](int k, bool checked) -> float4 {
        if (M32) return checked ? ld4_checked(m, k, L, false) : *reinterpret_cast<const float4*>(m + k);
        const uint32_t nb = (!checked || k < L) ? (mbar[k >> 5] >> (k & 31)) & 0xfu : 0u;
        // loaded whether or not a bit is set: a load that waits for the mask word costs more than it saves
        const float4 zb = checked ? ld4_checked(m, k, L, false) : *reinterpret_cast<const float4*>(m + k);
        return make_float4((nb & 1u) ? zb.x : 0.0f, (nb & 2u) ? zb.y : 0.0f, (nb & 4u) ? zb.z : 0.0f, (nb & 8u) ? zb.w : 0.0f);
    };
    int k = threadIdx.x * 4;
    for (; k + kTopkThreads * 4 < Lfull; k += 2 * kTopkThreads * 4) {
        const int k2 = k + kTopkThreads * 4;
        const float4 g0 = Grad<GT>::ld4(g, k), g1 = Grad<GT>::ld4(g, k2);
        const float4 z0 = *reinterpret_cast<const float4*>(zc + k), z1 = *reinterpret_cast<const float4*>(zc + k2);
        const float4 m0 = momentum(k, false), m1 = momentum(k2, false);
        const uint32_t n0 = maskw[k >> 5] >> (k & 31), n1 = maskw[k2 >> 5] >> (k2 & 31);
        sweep(k, g0, z0, m0, n0, false);
        sweep(k2, g1, z1, m1, n1, false);
    }
    for (; k < Lfull; k += kTopkThreads * 4)
        sweep(k, Grad<GT>::ld4(g, k), *reinterpret_cast<const float4*>(zc + k), momentum(k, false),
              maskw[k >> 5] >> (k & 31), false);
    for (int w0 = k - threadIdx.x * 4; w0 < L; w0 += kTopkThreads * 4) {          // the ragged rest, by whole warps
        k = w0 + threadIdx.x * 4;
        sweep(k, ld_grad4_checked<GT>(g, k, L), ld4_checked(zc, k, L, false), momentum(k, true),
              k < L ? maskw[k >> 5] >> (k & 31) : 0u, true);
    }
    if (BAND && band) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) above += __shfl_xor_sync(0xffffffffu, above, o);
        if (lane == 0) atomicAdd(&above_total, above);
    }
    __syncthreads();                                   // z stores, histogram (or mask so far) and list are complete
    int n_list = 0;                                    // > 0: the list decides, hist[0..nwords) holds the mask so far
    uint32_t K_list = K, floor_list = floor_key;
    bool counted = !band && floor_key == 0;            // hist holds the fine counts of all keys
    bool two_pass = false, missed = false;
    uint32_t learned_next = BAND ? 0u : drop;
    if (BAND && band) {
        const uint32_t listed = list.count, over = above_total;
        if (over < K && K <= over + listed && listed <= (uint32_t)kTopkList) {
            n_list = (int)listed; K_list = K - over; floor_list = band_lo;
            learn_count = listed; learn_width = band_hi - band_lo;
        } else {
            missed = true;
            if (threadIdx.x == 0) atomicAdd(a.route + (listed > (uint32_t)kTopkList ? 5 : (over >= K ? 3 : 4)), 1);
        }
    } else if (floor_key != 0) {                       // window route: the mask words are still all zero
        const uint32_t listed = list.count;
        learned_next = topk_window_learn(drop, listed, K);
        if (listed >= K && listed <= (uint32_t)kTopkList) n_list = (int)listed;
        else {
            missed = true;
            if (threadIdx.x == 0) atomicAdd(a.route + (listed < K ? 4 : 5), 1);
        }
    }
    if (missed) {                                      // the prediction missed: count every key after all
        __syncthreads();
        for (int b = threadIdx.x; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
        if (threadIdx.x == 0) list.count = 0;
        __syncthreads();
        for (int kk = threadIdx.x * 4; kk < L; kk += kTopkThreads * 4) {
            const float4 zv = ld4_checked(zc, kk, L, false);
            const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (kk + e < L) atomicAdd(&hist[topk_bin(key[e], shift, bin0)], 1u);
        }
        counted = true;
    }
    if (n_list > 0) {
        // settled by the list below
    } else if (small && counted) {                     // two-pass route
        uint32_t Kb = K;
        const int b0 = topk_find_bin(hist, kTopkBins, Kb, sh);
        const uint32_t inbin = hist[b0];
        __syncthreads();                               // everybody has read the histogram: its words become the mask
        if (b0 > 0 && b0 < kTopkBins - 1 && inbin <= (uint32_t)kTopkList) {
            two_pass = true;
            learn_count = inbin; learn_width = 1u << 19;
            auto settle = [&](int k, float4 zv, bool checked) {
                const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
                uint32_t nibble = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (!checked || k + e < L) {
                        const int b = topk_bin(key[e], 19, bin0);
                        if (b > b0) nibble |= 1u << e;
                        else if (b == b0) topk_list_add(list, key[e], (uint32_t)(k + e));
                    }
                }
                const uint32_t word = pack_group_words(nibble, lane);   // valid in lanes 0, 8, 16, 24
                if ((lane & 7) == 0 && (!checked || k < L)) hist[k >> 5] = word;
            };
            int w0 = 0;
            for (; w0 + 4 * kTopkThreads * 4 <= L; w0 += 4 * kTopkThreads * 4) {      // four sweeps' loads in flight
                const int k = w0 + threadIdx.x * 4;
                float4 zv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) zv[u] = *reinterpret_cast<const float4*>(zc + k + u * kTopkThreads * 4);
#pragma unroll
                for (int u = 0; u < 4; ++u) settle(k + u * kTopkThreads * 4, zv[u], false);
            }
            for (; w0 < L; w0 += kTopkThreads * 4) {
                const int k = w0 + threadIdx.x * 4;
                settle(k, ld4_checked(zc, k, L, false), true);
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
            for (int p = threadIdx.x; p < n_list; p += kTopkThreads)
                if (topk_list_selected(list, n_list, p, tau, ties, ties_total))
                    atomicOr(&hist[list.idx[p] >> 5], 1u << (list.idx[p] & 31u));
            __syncthreads();
            for (int w = threadIdx.x; w < nwords; w += kTopkThreads) maskw[w] = hist[w];
            if (threadIdx.x == 0) {
                *thr = __uint_as_float(tau); *hint = last_thr;
                *learned = __uint_as_float(BAND ? topk_learn(tau, last_key, prev_key, learn_count, learn_width) : learned_next);
                atomicAdd(a.route + (two_pass ? 1 : 0), 1);
            }
            return;
        }
    }
    // general route: histograms over the whole chunk
    if (small) topk_full_hist(zc, L, hist);
    topk_threshold(zc, L, K, hist, sh, tau, ties);
    if (threadIdx.x == 0) { *thr = __uint_as_float(tau); *hint = last_thr; *learned = __uint_as_float(learned_next); atomicAdd(a.route + 2, 1); }
    // ordered pass over the chunk: the selection mask with the tie rule
    uint32_t seen = 0;
    for (int w0 = 0; w0 < L; w0 += kTopkThreads * 4) {
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
    float* m32;                       // accumulator during the step; the new momentum after it where the chunk was applied densely
    float* thr;                       // per chunk: the magnitude of the K-th element of the last step
    float* hint; float* learned;      // ... of the step before, and what topk_learn made of it
    int* route;                       // as in TopkWorkerArgs
    const float* v; float* x;
    int64_t d, chunk;
    int n; float nf, lr, eps;
    double frac;
    int64_t c0;                       // first chunk of this launch (a launch may serve a range of chunks from received rows)
    // An element that is not kept has m = +0, and x - (lr * 0) / (sqrt(v) + eps) is x itself whenever
    // lr >= +0, eps > 0 and v is neither negative nor NaN (the host checks all three).  Then only the
    // kept elements are touched (sparse != 0): the momentum stays implicit in (zbar, mask), v and x are read
    // and x written for K elements per chunk instead of all.  Otherwise every chunk takes the general
    // route, whose ordered pass updates every element and writes the momentum out.
    int sparse;
};

__global__ void __launch_bounds__(kTopkThreads, kTopkResident)
k_topk_server(const TopkServerArgs a)
{
    __shared__ uint32_t hist[kTopkBins];
    __shared__ uint32_t bins8[256];
    __shared__ uint32_t sh[2];
    __shared__ uint32_t warp_ties[kTopkWarps];
    __shared__ TopkList list;
    const int64_t c = a.c0 + blockIdx.x;
    const int64_t base = c * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const int nwords = (L + 31) / 32;
    float* acc = a.m32 + base;
    float* zb = a.zbar + base;
    uint32_t* maskbar = a.Bbar + base / 32;

    for (int b = threadIdx.x; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
    if (threadIdx.x == 0) list.count = 0;
    // The sum of the n sparse messages, in worker order, has two forms.  Few kept elements (k below
    // kTopkDenseSum): scattered, through the momentum buffer - a thread owns the same mask words for every
    // worker, so an element is only ever updated by one thread and its program order is the worker order;
    // the mask words of eight workers are fetched together.  Many: in registers inside pass A (below).
    const bool dense = a.frac >= kTopkDenseSum;
    if (!dense) {
        for (int k = threadIdx.x * 4; k < L; k += kTopkThreads * 4) {
            if (k + 3 < L) *reinterpret_cast<float4*>(acc + k) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            else for (int e = 0; k + e < L; ++e) acc[k + e] = 0.0f;
        }
        __syncthreads();
        for (int w = threadIdx.x; w < nwords; w += kTopkThreads) {
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
    const bool small = nwords <= kTopkBins && a.sparse != 0;      // list routes: the mask fits the shared-memory words, sparse update allowed
    const uint32_t drop = topk_window_drop(a.learned[c]);
    const uint32_t floor_key = small ? topk_floor(a.thr[c], K, drop) : 0u;
    const int shift = small ? 19 : 20, bin0 = small ? topk_fine_base(a.thr[c]) : 0;
    // The dense form waits on memory twice per four workers (mask words, then the values under them), so it asks
    // for the mask lines of the sweep after next ahead of time.
    auto ask_masks = [&](int k0) {                     // k0: first element of a sweep (64 mask words a worker: two lines, three when not aligned)
        if (dense && (int)threadIdx.x < 4 * a.n && (threadIdx.x & 3) != 3 && k0 < L) {
            const int w = (k0 >> 5) + ((threadIdx.x & 3) == 2 ? 63 : 32 * (int)(threadIdx.x & 3));
            if (w < nwords) prefetch_l1(a.B + (int64_t)(threadIdx.x >> 2) * a.Wp + base / 32 + w);
        }
    };
    ask_masks(0); ask_masks(kTopkThreads * 4);
    for (int k = threadIdx.x * 4; k < L; k += kTopkThreads * 4) {
        float aa[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const uint32_t* mrow = a.B + base / 32 + (k >> 5);
        const float* zrow = a.z + base;
        ask_masks(k - (int)threadIdx.x * 4 + 2 * kTopkThreads * 4);
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
    int n_list = 0;                                    // > 0: the list decides, hist[0..nwords) holds the mask so far
    uint32_t K_list = K, floor_list = floor_key;
    bool two_pass = false, counted = small && floor_key == 0;
    uint32_t learned_next = drop;
    if (floor_key != 0) {                              // window route: the mask words are still all zero
        const uint32_t listed = list.count;
        learned_next = topk_window_learn(drop, listed, K);
        if (listed >= K && listed <= (uint32_t)kTopkList) n_list = (int)listed;
        else {                                         // the window missed: count every key after all
            if (threadIdx.x == 0) atomicAdd(a.route + (listed < K ? 4 : 5), 1);
            __syncthreads();
            if (threadIdx.x == 0) list.count = 0;
            for (int kk = threadIdx.x * 4; kk < L; kk += kTopkThreads * 4) {       // (the bins are still all zero)
                const float4 zv = ld4_checked(zb, kk, L, false);
                const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (kk + e < L) atomicAdd(&hist[topk_bin(key[e], shift, bin0)], 1u);
            }
            counted = true;
        }
    }
    if (n_list > 0) {
        // settled by the list below
    } else if (counted) {                              // two-pass route
        uint32_t Kb = K;
        const int b0 = topk_find_bin(hist, kTopkBins, Kb, sh);
        const uint32_t inbin = hist[b0];
        __syncthreads();                               // everybody has read the histogram: its words become the mask
        if (b0 > 0 && b0 < kTopkBins - 1 && inbin <= (uint32_t)kTopkList) {
            two_pass = true;
            // second pass: the elements above the bin of the K-th key are kept - mask bit, model update
            // (Section 3.3 steps 5-6) - and those of that bin go to the list
            auto settle = [&](int k, float4 zv, bool checked) {
                const float zz[4] = {zv.x, zv.y, zv.z, zv.w};
                uint32_t nibble = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (!checked || k + e < L) {
                        const uint32_t key = mag_key(zz[e]);
                        const int b = topk_bin(key, 19, bin0);
                        if (b > b0) {
                            nibble |= 1u << e;
                            x[k + e] = apply_elem(x[k + e], v[k + e], zz[e], a.lr, a.eps);
                        } else if (b == b0) {
                            topk_list_add(list, key, (uint32_t)(k + e));
                        }
                    }
                }
                const uint32_t word = pack_group_words(nibble, lane);   // valid in lanes 0, 8, 16, 24
                if ((lane & 7) == 0 && (!checked || k < L)) hist[k >> 5] = word;
            };
            int w0 = 0;
            for (; w0 + 4 * kTopkThreads * 4 <= L; w0 += 4 * kTopkThreads * 4) {      // four sweeps' loads in flight
                const int k = w0 + threadIdx.x * 4;
                float4 zv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) zv[u] = *reinterpret_cast<const float4*>(zb + k + u * kTopkThreads * 4);
#pragma unroll
                for (int u = 0; u < 4; ++u) settle(k + u * kTopkThreads * 4, zv[u], false);
            }
            for (; w0 < L; w0 += kTopkThreads * 4) {
                const int k = w0 + threadIdx.x * 4;
                settle(k, ld4_checked(zb, k, L, false), true);
            }
            __syncthreads();
            n_list = (int)inbin; K_list = Kb; floor_list = (uint32_t)(b0 + bin0) << 19;
        }
    }
    bool have_tau = false;
    if (n_list > 0) {
        uint32_t ties_total;
        have_tau = topk_threshold_list(list, n_list, floor_list, K_list, bins8, sh, tau, ties, ties_total);
        if (have_tau) {
            for (int p = threadIdx.x; p < n_list; p += kTopkThreads) {              // the listed elements, one by one
                if (!topk_list_selected(list, n_list, p, tau, ties, ties_total)) continue;
                const int j = (int)list.idx[p];
                x[j] = apply_elem(x[j], v[j], zb[j], a.lr, a.eps);
                atomicOr(&hist[j >> 5], 1u << (j & 31));
            }
            __syncthreads();
            for (int w = threadIdx.x; w < nwords; w += kTopkThreads) maskbar[w] = hist[w];
            if (threadIdx.x == 0) {
                a.thr[c] = __uint_as_float(tau); a.learned[c] = __uint_as_float(learned_next);
                atomicAdd(a.route + (two_pass ? 1 : 0), 1);
            }
            return;
        }
    }
    // general route: histograms over the whole chunk
    if (small) topk_full_hist(zb, L, hist);
    topk_threshold(zb, L, K, hist, sh, tau, ties);
    if (threadIdx.x == 0) { a.thr[c] = __uint_as_float(tau); a.learned[c] = __uint_as_float(learned_next); atomicAdd(a.route + 2, 1); }
    // ordered pass: mask, momentum m = C[zbar] written out, model update (Section 3.3 steps 5-6) of every element
    uint32_t seen = 0;
    for (int w0 = 0; w0 < L; w0 += kTopkThreads * 4) {
        const int k = w0 + threadIdx.x * 4;
        const float4 zv = ld4_checked(zb, k, L, false);
        const float4 vv = ld4_checked(v, k, L, true);
        const float4 xv = ld4_checked(x, k, L, true);
        const uint32_t key[4] = {mag_key(zv.x), mag_key(zv.y), mag_key(zv.z), mag_key(zv.w)};
        const uint32_t validmask = k + 3 < L ? 0xfu : (k < L ? (1u << (L - k)) - 1u : 0u);
        const uint32_t nibble = topk_select_wave(key, validmask, tau, ties, seen, warp_ties);
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

// ------------------------------------------------------------------------------------------
// The top-k message on the wire (phase-wise step, one process per GPU): a selection mask plus the kept values in
// index order, K per chunk.  The kernels below turn the library's in-place form (mask + the compensated vector)
// into that message and back.  One CTA per (row, chunk); thread t owns a contiguous run of the chunk's mask words,
// a block-wide exclusive scan of the runs' popcounts gives every kept element its position in the message.

// Calls fn(j, rank) for every set bit j (element index in the chunk, ascending per thread) of words[0..nwords).
template <typename F>
__device__ __forceinline__ void topk_for_each_kept(const uint32_t* __restrict__ words, int nwords, uint32_t* scan /* kThreads + 1 words of shared memory */, F fn)
{
    const int per = (nwords + kThreads - 1) / kThreads;
    const int w0 = threadIdx.x * per, w1 = (w0 + per < nwords) ? w0 + per : nwords;
    uint32_t mine = 0;
    for (int w = w0; w < w1; ++w) mine += __popc(words[w]);
    scan[threadIdx.x + 1] = mine;
    if (threadIdx.x == 0) scan[0] = 0;
    __syncthreads();
    if (threadIdx.x == 0) for (int t = 1; t <= kThreads; ++t) scan[t] += scan[t - 1];      // 256 additions: not worth a tree
    __syncthreads();
    uint32_t rank = scan[threadIdx.x];
    for (int w = w0; w < w1; ++w) {
        uint32_t word = words[w];
        while (word) {
            const int j = w * 32 + (__ffs(word) - 1);
            word &= word - 1;
            fn(j, rank);
            ++rank;
        }
    }
}

struct TopkPackArgs {
    const float* z; int64_t dz;            // rows of compensated vectors (row stride dz)
    const uint32_t* mask; int64_t Wp;      // rows of selection masks
    float* vals; int64_t vstride;          // out: rows of packed values, (chunk - c0) * kmax + rank within a row
    int64_t d, chunk, c0, nchunks;
    int kmax;
};

// grid: rows * nchunks.  vals[row][(c - c0) * kmax + rank] = z[row][element of that rank in chunk c].
__global__ void __launch_bounds__(kThreads)
k_topk_pack(const TopkPackArgs a)
{
    __shared__ uint32_t scan[kThreads + 1];
    const int row = (int)(blockIdx.x / a.nchunks);
    const int64_t c = a.c0 + blockIdx.x % a.nchunks;
    const int64_t base = c * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const float* __restrict__ z = a.z + (int64_t)row * a.dz + base;
    float* __restrict__ out = a.vals + (int64_t)row * a.vstride + (c - a.c0) * a.kmax;
    const int kmax = a.kmax;
    topk_for_each_kept(a.mask + (int64_t)row * a.Wp + base / 32, (L + 31) / 32, scan,
                       [&](int j, uint32_t rank) { if (j < L && rank < (uint32_t)kmax) out[rank] = z[j]; });
}

struct TopkUnpackArgs {
    const uint32_t* mask; int64_t row_words;     // received rows: word 0 = first word of chunk c0
    const float* vals; int64_t row_vals;         // received rows of packed values
    float* dense; int64_t dstride;               // out: rows of compensated values, element 0 = first element of chunk c0
    int64_t d, chunk, c0, nchunks;
    int kmax;
};

// grid: rows * nchunks.  The kept values of every received row go back to their positions in a dense row.
__global__ void __launch_bounds__(kThreads)
k_topk_unpack(const TopkUnpackArgs a)
{
    __shared__ uint32_t scan[kThreads + 1];
    const int row = (int)(blockIdx.x / a.nchunks);
    const int64_t cr = blockIdx.x % a.nchunks;                  // chunk within the range
    const int64_t base = (a.c0 + cr) * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const float* __restrict__ in = a.vals + (int64_t)row * a.row_vals + cr * a.kmax;
    float* __restrict__ out = a.dense + (int64_t)row * a.dstride + cr * a.chunk;
    const int kmax = a.kmax;
    topk_for_each_kept(a.mask + (int64_t)row * a.row_words + cr * (a.chunk / 32), (L + 31) / 32, scan,
                       [&](int j, uint32_t rank) { if (j < L && rank < (uint32_t)kmax) out[j] = in[rank]; });
}

struct TopkPutArgs {
    const uint32_t* mask;                        // the range's server mask words, word 0 = first word of chunk c0
    const float* vals;                           // its kept values, cr * kmax + rank
    float* zbar; uint32_t* Bbar; const float* v; float* x;
    int64_t d, chunk, c0;
    int kmax; float lr, eps;
};

// grid: chunks of the range.  A server range computed elsewhere becomes this context's: mask words, the kept
// values at their places in zbar (where the workers read the momentum C[zbar] under the mask), and Section 3.3
// step 6 for the kept elements (the others have momentum +0 and do not move: see TopkServerArgs::sparse).
__global__ void __launch_bounds__(kThreads)
k_topk_put(const TopkPutArgs a)
{
    __shared__ uint32_t scan[kThreads + 1];
    const int64_t cr = blockIdx.x;
    const int64_t base = (a.c0 + cr) * a.chunk;
    const int L = (int)((a.d - base < a.chunk) ? a.d - base : a.chunk);
    const int nwords = (L + 31) / 32;
    const uint32_t* __restrict__ words = a.mask + cr * (a.chunk / 32);
    const float* __restrict__ in = a.vals + cr * a.kmax;
    float* __restrict__ zb = a.zbar + base;
    const float* __restrict__ v = a.v + base;
    float* __restrict__ x = a.x + base;
    const int kmax = a.kmax;
    topk_for_each_kept(words, nwords, scan, [&](int j, uint32_t rank) {
        if (j < L && rank < (uint32_t)kmax) {
            const float m = in[rank];
            zb[j] = m;
            x[j] = apply_elem(x[j], v[j], m, a.lr, a.eps);
        }
    });
    for (int w = threadIdx.x; w < nwords; w += kThreads) a.Bbar[base / 32 + w] = words[w];
}

// Sets *flag if any v[j] is negative or NaN (v >= 0 fails); -0 and +inf pass.
__global__ void k_any_negative_or_nan(const float* __restrict__ v, int64_t d, int* flag)
{
    bool found = false;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x)
        found |= !(v[j] >= 0.0f);
    if (found) *flag = 1;
}

__global__ void k_materialise_momentum_topk(const float* __restrict__ zbar, const uint32_t* __restrict__ mask,
                                            float* __restrict__ out, int64_t first, int64_t count)
{
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = first + j;
        out[j] = ((mask[e >> 5] >> (e & 31)) & 1u) ? zbar[e] : 0.0f;
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

}  // namespace
