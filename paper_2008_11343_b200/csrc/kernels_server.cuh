// Server side (Section 3.3 step 4): the register-staged kernel and the kernel that streams its
// tiles through a shared-memory ring, optionally fused with the model update.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

// ------------------------------------------------------------------------------------------
// Server side: average the n decompressed messages, add the server error, recompress
// (Section 3.3 step 4).

// The messages the server averages: row j (one sender) is addressed by ABSOLUTE word / chunk index through
// its own pair of pointers, so that the rows may lie anywhere - this context's workers, a buffer of received
// rows, or the mapped workspaces of other processes' GPUs (plain and bulk loads only).
struct ServerArgs {
    const uint32_t* Brow[APMS_MAX_WORKERS];
    const float* srow[APMS_MAX_WORKERS];
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
__device__ __forceinline__ void server_groups(const ServerArgs& a, const float* s_sh, int64_t wofs,
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
            w[u] = live[u] ? a.Brow[i][wofs + (g0 + gstride * u) * 4 + wl] : 0u;
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
        if ((lane & 7) == 0 && (!CHECKED || wk * 32 < L)) APMS_STORE(ob[wk], word);
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
    for (int i = tid_in_team; i < a.n; i += WPC * 32) s_sh[i] = a.srow[i][it.c];
    const float S_old = a.Sbar[it.c];
    if (WPC == 1) __syncwarp(); else __syncthreads();
    const int64_t wofs = it.base / 32;
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
        server_groups<U, false>(a, s_sh, wofs, zb, ob, g0, 1, lane, L, S_old, acc);
    for (; g0 < g_end; ++g0)
        server_groups<1, true>(a, s_sh, wofs, zb, ob, g0, 1, lane, L, S_old, acc);
    const double total = team_sum<WPC>(acc, red);
    if ((WPC == 1) ? (lane == 0) : (threadIdx.x == 0)) {
        if (a.t.P == 1) APMS_STORE(a.Sbar[it.c], scale_from_sum(total, (double)it.Lc, a.t.l1 != 0));
        else APMS_STORE(a.partial[it.c * a.t.P + it.p], total);
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
// Bulk copies start on 16-byte boundaries.  Every slab of zbar, v and x does (chunks are multiples of
// 32 elements); a chunk's first sign word need not.  The rows of sign words are therefore copied from
// the 16-byte boundary at or below the slab's first word - up to three words early - and everything
// held in shared memory as sign words (the rows and the tile's new words) is indexed by the distance
// from that boundary, so that whole 16-byte pieces in shared memory are whole 16-byte pieces in global
// memory.  All rows of a launch must share one alignment (`row_align`); chunks shorter than a slab use
// k_server and k_apply.

constexpr int kSlab = 2048;                      // elements per ring stage
constexpr int kSlabGroups = kSlab / kGroup;      // 16 groups, two per consumer warp
constexpr int kSlabWords = kSlab / 32;           // 64 sign words per worker and slab
constexpr int kRowWords = kSlabWords + 4;        // a row in shared memory: up to three words before the slab's first, rounded to 16 bytes
constexpr int kStages = 4;
constexpr int64_t kStagedSpanElems = 32768;   // a CTA of the fused form walks enough chunks to stream about this many elements
constexpr int kStagedThreads = kThreads + 32;    // eight consumer warps + one producer warp
constexpr long long kWaitCycles = 2000000000ll;  // bound of every wait: about a second of SM clocks

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
#ifdef APMS_BOUNDS_CHECK
    if (!APMS_CAN_LOAD(gmem_src, bytes)) gmem_src = checked_safe_source();     // reported; the bytes are owed to the barrier
#endif
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Barrier among the 256 consumer threads only (the producer warp never joins it).
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// The same barrier that also ORs a flag
// over them: every consumer gets the same answer, so a decision to leave taken on it is uniform even
// when the flag it is fed from changes while the threads arrive.
__device__ __forceinline__ bool consumer_barrier_any(bool flag)
{
    uint32_t any;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(any) : "r"(flag ? 1u : 0u) : "memory");
    return any != 0;
}

struct ServerStagedArgs {
    ServerArgs a;
    int* status;          // device status word: set when a bounded wait gave up
    float inv_n;          // 1/n when n is a power of two (then avg = sum * inv_n is the exact quotient), else 0
    const float* den; float* x; float lr;        // steps 5-6 (fused form only): den = sqrt(v) + eps, see k_make_den
    int span;             // chunks per CTA of the fused form
    int row_align;        // (address of every row's word 0 / 4) mod 4: the rows' common distance from a 16-byte boundary, in words
    // Lagged form (chunks cut into several tiles, whole step): see k_server_staged.  lag = 0: off.
    int64_t lag;          // a CTA applies the model update of the tile `lag` tickets before its own
    unsigned int* ticket; // the next tile to hand out
    unsigned int* done;   // per chunk: tiles finished so far in this launch
    unsigned int* ready;  // per chunk: `epoch` once the chunk's new scale is stored
    unsigned int epoch;   // differs from launch to launch, never 0
};

// Bytes of one ring stage: a slab of zbar plus n rows of sign words, or (fused form) a slab of v and of x.
__host__ __device__ __forceinline__ size_t staged_stage_bytes(int n, bool fused)
{
    const size_t server = (size_t)kSlab * 4 + (size_t)n * kRowWords * 4;
    const size_t apply = (size_t)kSlab * 8;
    return (fused && apply > server) ? apply : server;
}

// Bytes of the buffer of new sign words behind the ring: the words of all slabs of a tile - every consumer warp
// writes its words of the last slab too, live or not - plus up to three words before the first.
__host__ __device__ __forceinline__ size_t staged_nb_bytes(int64_t tile_elems)
{
    const int64_t nslabs = (tile_elems + kSlab - 1) / kSlab;
    return (size_t)(nslabs * kSlabWords + 4) * 4;
}

// Sum over the workers, in worker order, of +-s_i for the lane's 2 x 4 elements of one slab.
// NT > 0: the number of workers is the compile-time constant NT (fully unrolled).
// NT >= 8: the running sum starts at zero, so after the first eight workers it is a function of their
// eight sign bits alone; `prefix8` holds it for all 256 patterns (built once per chunk with the same
// eight additions in the same order, see build_prefix8).  The lane gathers, per group, its four elements'
// bits of the eight workers into the four bytes of one word - the nibble times 0x00204081 spreads bits
// 0..3 to bits 0, 8, 16, 24 (all partial products fall on distinct bits, so nothing carries), shifted
// left by the worker's index - and looks the four sums up; the other workers are added one by one.
constexpr int kPrefixWorkers = 8;

template <int NT>
__device__ __forceinline__ void signed_scale_sums(const uint32_t* __restrict__ r0, const uint32_t* __restrict__ r1,
                                                  const uint32_t* __restrict__ neg_s, const float* __restrict__ prefix8, int n, int sh,
                                                  float2& s01, float2& s23, float2& t01, float2& t23)
{
    const int nn = NT > 0 ? NT : n;
    constexpr int kFirst = NT >= kPrefixWorkers ? kPrefixWorkers : 0;
    if (NT >= kPrefixWorkers) {
        uint32_t i0 = 0u, i1 = 0u;
#pragma unroll
        for (int i = 0; i < kPrefixWorkers; ++i) {
            const uint32_t n0 = (r0[i * kRowWords] >> sh) & 0xFu;
            const uint32_t n1 = (r1[i * kRowWords] >> sh) & 0xFu;
            i0 |= (n0 * (0x00204081u << i)) & (0x01010101u << i);
            i1 |= (n1 * (0x00204081u << i)) & (0x01010101u << i);
        }
        s01.x = prefix8[i0 & 0xFFu]; s01.y = prefix8[(i0 >> 8) & 0xFFu]; s23.x = prefix8[(i0 >> 16) & 0xFFu]; s23.y = prefix8[i0 >> 24];
        t01.x = prefix8[i1 & 0xFFu]; t01.y = prefix8[(i1 >> 8) & 0xFFu]; t23.x = prefix8[(i1 >> 16) & 0xFFu]; t23.y = prefix8[i1 >> 24];
    }
#pragma unroll(NT > 0 ? NT : 4)
    for (int i = kFirst; i < nn; ++i) {
        const uint32_t ns = neg_s[i];
        // the lane's four sign bits moved to bits 28..31; a set bit turns -s_i into +s_i
        const uint32_t y0 = r0[i * kRowWords] << (28 - sh);
        const uint32_t y1 = r1[i * kRowWords] << (28 - sh);
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

// Entry t of the table: 0 + (+-s_0) + (+-s_1) + ... + (+-s_7) in this order, bit i of t set meaning +s_i.
// `mine` is, in lanes 0..7 of every warp, the bit pattern of -s_lane; one entry per consumer thread.
__device__ __forceinline__ float prefix8_entry(uint32_t mine, uint32_t t)
{
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < kPrefixWorkers; ++i) {
        const uint32_t ns = __shfl_sync(0xffffffffu, mine, i);
        acc = __fadd_rn(acc, __uint_as_float(ns ^ (((t >> i) & 1u) << 31)));
    }
    return acc;
}

// One lane's four elements of a group after the sums over the workers: average, plus the implied old error,
// stored as the new compensated values; returns the four sign bits and adds the squares to acc.
// CHECKED = false: the whole slab lies inside the tile (no element needs a bounds test).
template <bool CHECKED>
__device__ __forceinline__ uint32_t server_finish_group(float4 zo4, float sum0, float sum1, float sum2, float sum3, float S_old,
                                                        float inv_n, float nf, float* __restrict__ zdst, int k, int L, double& acc)
{
    const float zo[4] = {zo4.x, zo4.y, zo4.z, zo4.w};
    const float sum[4] = {sum0, sum1, sum2, sum3};
    float zn[4];
    uint32_t nibble = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float avg = (inv_n != 0.0f) ? __fmul_rn(sum[e], inv_n) : __fdiv_rn(sum[e], nf);
        zn[e] = __fadd_rn(avg, implied_error(zo[e], S_old));
        if (!CHECKED || k + e < L) {
            const double zd = (double)zn[e];
            acc = fma(zd, zd, acc);
            nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
        }
    }
    if (CHECKED) st4_checked(zdst, k, L, make_float4(zn[0], zn[1], zn[2], zn[3]));
    else st_stream4(zdst + k, make_float4(zn[0], zn[1], zn[2], zn[3]));
    return nibble;
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
    __shared__ uint32_t neg_s[APMS_MAX_WORKERS];      // bit patterns of -s_i of the current chunk
    __shared__ float prefix8[NT >= kPrefixWorkers ? 256 : 1];         // see signed_scale_sums
    __shared__ int failed;

    __shared__ unsigned int my_ticket;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = NT > 0 ? NT : a.n;
    const size_t stage_bytes = staged_stage_bytes(n, FUSED);
    // behind the ring: the current tile's new sign words, from the 16-byte boundary below the first (staged_nb_bytes)
    uint32_t* const nb = reinterpret_cast<uint32_t*>(smem + (size_t)kStages * stage_bytes);
    const int span = MULTI ? sa.span : 1;                  // MULTI = false: one item, the walk's loops fold away
    // Lagged form.  A chunk cut into P tiles knows its new scale only when its last tile is done, so steps 5-6
    // cannot follow step 4 inside the tile's CTA; run as a kernel of their own they cost the step 3 % (the
    // server part is bound by instruction issue, the update by memory: one after the other neither unit is busy).
    // Here the CTAs take their tiles from a ticket counter, in order; a CTA does step 4 for tile t, counts it in
    // (the chunk's last tile adds the P partial sums in tile order, stores the scale and raises the chunk's flag),
    // and then does steps 5-6 for tile t - lag, whose chunk is complete or about to be: with lag >= P all of its
    // tiles hold lower tickets, so they belong to CTAs that are already running and that wait for nobody
    // before they have counted their tile in - the wait (bounded like every other) cannot deadlock.  `lag` more
    // CTAs than tiles do the last updates.
    const bool lagged = !FUSED && !MULTI && sa.lag > 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWarps); }
        failed = 0;
        if (lagged) my_ticket = atomicAdd(sa.ticket, 1u);
        mbar_fence_init();
    }
    __syncthreads();
    const int64_t item0 = lagged ? a.item0 + (int64_t)my_ticket : a.item0 + (int64_t)blockIdx.x * span;
    const int nitems = lagged ? (item0 < a.items ? 1 : 0) : (MULTI ? (int)(a.items - item0 < span ? a.items - item0 : span) : 1);

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
                const int64_t wofs = it.base / 32;
                for (int r = 0; r < njobs; ++r, ++q) {
                    const int st = q % kStages;
                    if (q >= kStages && !mbar_wait(&empty[st], (uint32_t)(q / kStages - 1) & 1u)) { failed = 1; stop = true; break; }
                    unsigned char* base = smem + (size_t)st * stage_bytes;
                    const int j = r < nslabs ? r : r - nslabs;
                    const int left = L - j * kSlab;
                    const int live = left < kSlab ? left : kSlab;
                    const uint32_t zbytes = (uint32_t)((live + 3) / 4) * 16u;
                    if (r < nslabs) {
                        const int off_in = (int)((wofs + sa.row_align) & 3);       // words between the 16-byte boundary and the slab's first word
                        const uint32_t wbytes = (uint32_t)((off_in + (live + 31) / 32 + 3) / 4) * 16u;
                        mbar_arrive_expect_tx(&full[st], zbytes + (uint32_t)n * wbytes);
                        bulk_load(base, zb_g + (size_t)j * kSlab, zbytes, &full[st]);
                        uint32_t* rows = reinterpret_cast<uint32_t*>(base + (size_t)kSlab * 4);
                        for (int i = 0; i < n; ++i)
                            bulk_load(rows + i * kRowWords, a.Brow[i] + (wofs - off_in) + (size_t)j * kSlabWords, wbytes, &full[st]);
                    } else {
                        mbar_arrive_expect_tx(&full[st], 2 * zbytes);
                        bulk_load(base, sa.den + it.base + (size_t)j * kSlab, zbytes, &full[st]);
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
        // consumer barrier.  Each thread hands its own reading of `failed` to that barrier, which ORs them:
        // all consumers see the same result and leave together, whenever the producer may have set the flag.
        const volatile int* vfailed = &failed;
        int q = 0;
        // The scales of a chunk are fetched from global memory while the chunk before it is being worked on:
        // lane i of every warp (and lane i of warps 0, 1 for i + 32 when there are more than 32 workers) holds
        // -s_i, every thread the server's old scale.
        static_assert(APMS_MAX_WORKERS <= 64, "two scales per lane of the first two warps at most");
        uint32_t pre_neg = 0u;
        float pre_S = 0.0f;
        const int my_worker = (warp < 2 && n > 32) ? warp * 32 + lane : lane;     // n <= 32: every warp fetches workers 0..n-1
        if (nitems > 0) {
            const Item it0 = decode_item(a.t, item0);
            if (my_worker < n) pre_neg = __float_as_uint(a.srow[my_worker][it0.c]) | 0x80000000u;
            pre_S = a.Sbar[it0.c];
        }
        bool tile_done = false;
        for (int w = 0; w < nitems; ++w) {
            const Item it = decode_item(a.t, item0 + w);
            const int L = it.L;
            const int nslabs = (L + kSlab - 1) / kSlab;
            const int64_t wofs = it.base / 32;
            const int off_in = (int)((wofs + sa.row_align) & 3), off_out = (int)(wofs & 3);
            const uint32_t* negs = neg_s;
            if ((warp == 0 || (warp == 1 && n > 32)) && my_worker < n) neg_s[my_worker] = pre_neg;
            if (NT >= kPrefixWorkers) prefix8[threadIdx.x] = prefix8_entry(pre_neg, threadIdx.x);
            const float S_old = pre_S;
            if (MULTI && w + 1 < nitems) {
                const Item nx = decode_item(a.t, item0 + w + 1);
                if (my_worker < n) pre_neg = __float_as_uint(a.srow[my_worker][nx.c]) | 0x80000000u;
                pre_S = a.Sbar[nx.c];
            }
            if (consumer_barrier_any(*vfailed != 0)) break;      // -s_i in place; everybody is done with the previous chunk
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
                signed_scale_sums<NT>(rows + off_in + g0 * 4 + wl, rows + off_in + g1 * 4 + wl, negs, prefix8, n, sh, s01, s23, t01, t23);
                const bool whole = (j + 1) * kSlab <= L;                 // no element of this slab needs a bounds test (warp-uniform)
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int grp = j * kSlabGroups + (u ? g1 : g0);
                    const int k = grp * kGroup + lane * 4;
                    const float4 zo4 = u ? zo1 : zo0;
                    const float2 lo = u ? t01 : s01, hi = u ? t23 : s23;
                    const uint32_t nibble = whole
                        ? server_finish_group<false>(zo4, lo.x, lo.y, hi.x, hi.y, S_old, sa.inv_n, a.nf, a.zbar + it.base, k, L, acc)
                        : server_finish_group<true>(zo4, lo.x, lo.y, hi.x, hi.y, S_old, sa.inv_n, a.nf, a.zbar + it.base, k, L, acc);
                    const uint32_t word = pack_group_words(nibble, lane);
                    if ((lane & 7) == 0) nb[off_out + grp * 4 + wl] = word;   // words past L hold zeros and are never stored
                }
                // The stage is handed back only now: the stores above needed every value this warp loaded from it, so
                // the loads have returned.  (Handed back right after the loads were issued, the stage was now and then
                // refilled before a load had read it, when the SM's load/store path was backed up.)
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[st]);
            }
            acc = warp_sum(acc);
            if (lane == 0) red[warp] = acc;
            const bool leave = consumer_barrier_any(!ok || *vfailed != 0);   // partial sums and sign words of the tile are in shared memory
            double total = 0.0;
#pragma unroll
            for (int r = 0; r < kWarps; ++r) total += red[r];
            if (leave) break;
            if (FUSED) {
                // Section 3.3 steps 5-6 for this chunk: m <- +-Sbar, x <- x - lr m / (sqrt(v) + eps)
                const float S_new = (float)sqrt(total / (double)it.Lc);
                if (ok && threadIdx.x == 0) APMS_STORE(a.Sbar[it.c], S_new);
                const float c_new = __fmul_rn(sa.lr, S_new);        // lr * (+-S) = +-(lr * S)
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
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int grp = j * kSlabGroups + (u ? g1 : g0);
                        const int k = grp * kGroup + lane * 4;
                        const uint32_t nib = nb[off_out + grp * 4 + wl] >> sh;
                        xx[u].x = apply_stored(xx[u].x, vv[u].x, nib & 1u, c_new);
                        xx[u].y = apply_stored(xx[u].y, vv[u].y, nib & 2u, c_new);
                        xx[u].z = apply_stored(xx[u].z, vv[u].z, nib & 4u, c_new);
                        xx[u].w = apply_stored(xx[u].w, vv[u].w, nib & 8u, c_new);
                        if ((j + 1) * kSlab <= L) st_stream4(sa.x + it.base + k, xx[u]);
                        else st4_checked(sa.x + it.base, k, L, xx[u]);
                    }
                    __syncwarp();                                        // after the stores: see above
                    if (lane == 0) mbar_arrive(&empty[st]);
                }
            } else if (ok && threadIdx.x == 0) {
                if (a.t.P == 1) APMS_STORE(a.Sbar[it.c], (float)sqrt(total / (double)it.Lc));
                else APMS_STORE(a.partial[it.c * a.t.P + it.p], total);
            }
            // the tile's sign words leave in whole 16-byte pieces (full lines for full tiles)
            if (ok) {
                uint32_t* __restrict__ ob = a.Bbar + (wofs - off_out);          // 16-byte aligned; the tile's words are [off_out, wend)
                const int wend = off_out + (L + 31) / 32;
                for (int w4 = threadIdx.x * 4; w4 < wend; w4 += kThreads * 4) {
                    if (w4 >= off_out && w4 + 3 < wend) st_stream_words4(ob + w4, *reinterpret_cast<const uint4*>(nb + w4));
                    else for (int r = (w4 < off_out ? off_out : w4); r < w4 + 4 && r < wend; ++r) APMS_STORE(ob[r], nb[r]);
                }
            }
            tile_done = ok;
        }
        if (lagged) {
            if (nitems > 0 && tile_done) {
                __threadfence();                       // this thread's sign words, thread 0's partial sum: visible before the count
                consumer_barrier();
                if (threadIdx.x == 0) {
                    const Item it = decode_item(a.t, item0);
                    if (atomicAdd(sa.done + it.c, 1u) + 1u == (unsigned int)a.t.P) {
                        __threadfence();
                        double total = 0.0;            // as k_finalize_scales: the tiles' sums in tile order
                        for (int p = 0; p < a.t.P; ++p) total += __ldcg(a.partial + it.c * a.t.P + p);
                        APMS_STORE(a.Sbar[it.c], scale_from_sum(total, (double)it.Lc, a.t.l1 != 0));
                        sa.done[it.c] = 0u;            // for the next launch
                        __threadfence();
                        atomicExch(sa.ready + it.c, sa.epoch);
                    }
                }
            }
            const int64_t u = item0 - sa.lag;
            if (u >= a.item0 && u < a.items) {
                const Item iu = decode_item(a.t, u);
                if (threadIdx.x == 0 && *vfailed == 0) {
                    const volatile unsigned int* flag = sa.ready + iu.c;
                    const volatile int* status = sa.status;
                    const long long t0 = clock64();
                    while (*flag != sa.epoch) {
                        if (*status != DEVICE_OK || clock64() - t0 > kWaitCycles) { failed = 1; break; }
                        __nanosleep(200);
                    }
                    __threadfence();
                }
                if (!consumer_barrier_any(*vfailed != 0)) {
                    const float c_new = __fmul_rn(sa.lr, __ldcg(a.Sbar + iu.c));
                    const uint32_t* __restrict__ bw = a.Bbar + iu.base / 32;
                    const float* __restrict__ dn = sa.den + iu.base;
                    float* __restrict__ xo = sa.x + iu.base;
                    constexpr int kAhead = 4;                                 // sweeps whose loads are in flight together
                    const int Lfull = iu.L - iu.L % (kAhead * kThreads * 4);
                    int k = threadIdx.x * 4;
                    for (; k < Lfull; k += kAhead * kThreads * 4) {
                        float4 dd[kAhead], xx[kAhead];
                        uint32_t nn[kAhead];
#pragma unroll
                        for (int u2 = 0; u2 < kAhead; ++u2) {
                            const int kk = k + u2 * kThreads * 4;
                            dd[u2] = ld_stream4(dn + kk);
                            xx[u2] = ld_stream4(xo + kk);
                            nn[u2] = __ldcg(bw + (kk >> 5)) >> (kk & 31);
                        }
#pragma unroll
                        for (int u2 = 0; u2 < kAhead; ++u2) {
                            xx[u2].x = apply_stored(xx[u2].x, dd[u2].x, nn[u2] & 1u, c_new);
                            xx[u2].y = apply_stored(xx[u2].y, dd[u2].y, nn[u2] & 2u, c_new);
                            xx[u2].z = apply_stored(xx[u2].z, dd[u2].z, nn[u2] & 4u, c_new);
                            xx[u2].w = apply_stored(xx[u2].w, dd[u2].w, nn[u2] & 8u, c_new);
                            st_stream4(xo + k + u2 * kThreads * 4, xx[u2]);
                        }
                    }
                    for (; k < iu.L; k += kThreads * 4) {
                        const float4 d0 = ld4_checked(dn, k, iu.L, true);
                        float4 x0 = ld4_checked(xo, k, iu.L, true);
                        const uint32_t n0 = __ldcg(bw + (k >> 5)) >> (k & 31);
                        x0.x = apply_stored(x0.x, d0.x, n0 & 1u, c_new); x0.y = apply_stored(x0.y, d0.y, n0 & 2u, c_new);
                        x0.z = apply_stored(x0.z, d0.z, n0 & 4u, c_new); x0.w = apply_stored(x0.w, d0.w, n0 & 8u, c_new);
                        st4_checked(xo, k, iu.L, x0);
                    }
                }
            }
            if (threadIdx.x == 0 && my_ticket + 1u == gridDim.x) *sa.ticket = 0u;    // every ticket has been handed out
        }
    }
    __syncthreads();                                   // every warp has left its loops; shared memory may go
    if (threadIdx.x == 0 && failed) atomicExch(sa.status, DEVICE_WAIT_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// Server side, staged and fused, for short chunks: 128, 256, 512 or 1024 elements, so that a slab of
// kSlab elements holds K = kSlab / chunk whole chunks.  The ring, the producer and the split of a slab
// over the consumer warps are those of k_server_staged (a slab is contiguous in every stream whatever
// the chunk length); what differs is that a warp's two groups lie in two different chunks: each group
// has its own set of -s_i, its own old and new server scale, and the sums of squares are kept per group
// and added per chunk in group order.  A CTA walks `span` slabs; per slab one job for the server step and
// one for steps 5-6.  Slabs start at multiples of kSlab elements, so the new sign words of a slab are
// whole 16-byte pieces; the rows may still lie `row_align` words off a 16-byte boundary.

constexpr int kPackedMaxChunks = kSlab / kGroup;         // 16 chunks of 128 elements

template <int NT>
__device__ __forceinline__ void signed_scale_sums2(const uint32_t* __restrict__ r0, const uint32_t* __restrict__ r1,
                                                   const uint32_t* __restrict__ neg_s0, const uint32_t* __restrict__ neg_s1,
                                                   int n, int sh, float2& s01, float2& s23, float2& t01, float2& t23)
{
    const int nn = NT > 0 ? NT : n;
#pragma unroll(NT > 0 ? NT : 4)
    for (int i = 0; i < nn; ++i) {
        const uint32_t ns0 = neg_s0[i], ns1 = neg_s1[i];
        const uint32_t y0 = r0[i * kRowWords] << (28 - sh);
        const uint32_t y1 = r1[i * kRowWords] << (28 - sh);
        float2 q;
        q.x = __uint_as_float(((y0 << 3) & 0x80000000u) ^ ns0); q.y = __uint_as_float(((y0 << 2) & 0x80000000u) ^ ns0);
        s01 = __fadd2_rn(s01, q);
        q.x = __uint_as_float(((y0 << 1) & 0x80000000u) ^ ns0); q.y = __uint_as_float((y0 & 0x80000000u) ^ ns0);
        s23 = __fadd2_rn(s23, q);
        q.x = __uint_as_float(((y1 << 3) & 0x80000000u) ^ ns1); q.y = __uint_as_float(((y1 << 2) & 0x80000000u) ^ ns1);
        t01 = __fadd2_rn(t01, q);
        q.x = __uint_as_float(((y1 << 1) & 0x80000000u) ^ ns1); q.y = __uint_as_float((y1 & 0x80000000u) ^ ns1);
        t23 = __fadd2_rn(t23, q);
    }
}

template <int NT>
__global__ void __launch_bounds__(kStagedThreads, 3)
k_server_packed(const ServerStagedArgs sa)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const ServerArgs& a = sa.a;
    // The model update of a slab lags one slab behind its server step: jobs run in the order
    //   S(0), S(1), U(0), S(2), U(1), ..., U(last)          (S = steps 4, U = steps 5-6 of Section 3.3)
    // with ONE barrier per slab, after S(w).  One warp (they take turns) then forms the slab's new scales -
    // the binary64 division and square root - while the others already update slab w-1, whose scales were
    // formed a slab earlier: no warp waits for that arithmetic.  Everything the consumers hand to each other is
    // double-buffered over the walk: what slab w+2 writes, slab w was the last to read, and barrier w+1 lies in between.
    __shared__ double red[2][kPackedMaxChunks];                          // one sum of squares per group of the slab
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ uint32_t neg_s[2][kPackedMaxChunks * APMS_MAX_WORKERS];   // -s_i per chunk of the slab
    __shared__ float S_old_sh[2][kPackedMaxChunks], S_new_sh[2][kPackedMaxChunks];
    __shared__ int failed;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = NT > 0 ? NT : a.n;
    const size_t stage_bytes = staged_stage_bytes(n, true);
    const int chunk = (int)a.t.chunk;                                  // 128, 256, 512 or 1024: a power of two that divides kSlab
    const int cshift = 31 - __clz(chunk);                              // divisions by the chunk length are shifts
    const int gpc = chunk >> 7;                                        // groups per chunk (kGroup = 128)
    const int gshift = cshift - 7;
    const int64_t slab_first = a.item0 + (int64_t)blockIdx.x * sa.span;       // items are slabs here
    const int nmine = (int)(a.items - slab_first < sa.span ? a.items - slab_first : sa.span);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWarps); }
        failed = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kWarps) {
        if (lane == 0) {
            int q = 0;
            bool stop = false;
            // step t issues S(t) (t < nmine) and then U(t-1) (t >= 1): the order the consumers take them in
            for (int t = 0; t <= nmine && !stop; ++t) {
                for (int r = 0; r < 2 && !stop; ++r) {
                    const int w = r == 0 ? t : t - 1;
                    if (r == 0 ? t >= nmine : t < 1) continue;
                    const int64_t base_e = (slab_first + w) * kSlab;
                    const int64_t left = a.t.d - base_e;
                    const int live = (int)(left < kSlab ? left : kSlab);
                    const uint32_t zbytes = (uint32_t)((live + 3) / 4) * 16u;
                    const int st = q % kStages;
                    if (q >= kStages && !mbar_wait(&empty[st], (uint32_t)(q / kStages - 1) & 1u)) { failed = 1; stop = true; break; }
                    unsigned char* base = smem + (size_t)st * stage_bytes;
                    if (r == 0) {
                        const int64_t wofs = base_e / 32;
                        const int off_in = sa.row_align;                 // slabs start at multiples of 64 words
                        const uint32_t wbytes = (uint32_t)((off_in + (live + 31) / 32 + 3) / 4) * 16u;
                        mbar_arrive_expect_tx(&full[st], zbytes + (uint32_t)n * wbytes);
                        bulk_load(base, a.zbar + base_e, zbytes, &full[st]);
                        uint32_t* rows = reinterpret_cast<uint32_t*>(base + (size_t)kSlab * 4);
                        for (int i = 0; i < n; ++i)
                            bulk_load(rows + i * kRowWords, a.Brow[i] + (wofs - off_in), wbytes, &full[st]);
                    } else {
                        mbar_arrive_expect_tx(&full[st], 2 * zbytes);
                        bulk_load(base, sa.den + base_e, zbytes, &full[st]);
                        bulk_load(base + (size_t)kSlab * 4, sa.x + base_e, zbytes, &full[st]);
                    }
                    ++q;
                }
            }
            if (failed) {
                const int first = q > kStages ? q - kStages : 0;
                for (int p = first; p < q; ++p) mbar_wait(&full[p % kStages], (uint32_t)(p / kStages) & 1u);
            }
        }
    } else {
        const int sh = 4 * (lane & 7);
        const int wl = lane >> 3;
        const int g0 = warp, g1 = warp + kWarps;
        const int k0 = g0 >> gshift, k1 = g1 >> gshift;                          // the chunks (within the slab) of this warp's two groups
        const int kmax = kSlab >> cshift;                                  // chunks per whole slab
        const volatile int* vfailed = &failed;
        const int off_in = sa.row_align;
        // this thread's share of a slab's scales: entry idx = kk * n + i for idx = threadIdx.x + 256 r
        constexpr int kPre = kPackedMaxChunks * APMS_MAX_WORKERS / kThreads;
        uint32_t pre[kPre];
        float pre_S = 0.0f;
        auto fetch_scales = [&](int w) {                                  // global loads only: issued long before they are stored
            const int64_t base_e = (slab_first + w) * kSlab;
            const int64_t left = a.t.d - base_e;
            const int L = (int)(left < kSlab ? left : kSlab);
            const int64_t c0 = base_e >> cshift;
            const int nchunks = (L + chunk - 1) >> cshift;
#pragma unroll
            for (int r = 0; r < kPre; ++r) {
                const int idx = (int)threadIdx.x + r * kThreads;
                pre[r] = 0u;
                if (warp * 32 + r * kThreads < nchunks * n && idx < nchunks * n) {      // first test: warp-uniform, skips whole warps
                    const int kk = idx / n, i = idx - kk * n;
                    pre[r] = __float_as_uint(a.srow[i][c0 + kk]) | 0x80000000u;
                }
            }
            pre_S = ((int)threadIdx.x < nchunks) ? a.Sbar[c0 + threadIdx.x] : 0.0f;
        };
        auto store_scales = [&](int buf) {
#pragma unroll
            for (int r = 0; r < kPre; ++r) {
                const int idx = (int)threadIdx.x + r * kThreads;
                if (warp * 32 + r * kThreads < kmax * n && idx < kmax * n) {
                    const int kk = idx / n, i = idx - kk * n;
                    neg_s[buf][kk * APMS_MAX_WORKERS + i] = pre[r];
                }
            }
            if ((int)threadIdx.x < kmax) S_old_sh[buf][threadIdx.x] = pre_S;
        };
        int q = 0;
        bool ok = true;
        // Steps 5-6 for slab w from its job in the ring, the scales in S_new_sh[w & 1] and this lane's own sign bits.
        auto update_slab = [&](int w, uint32_t bits0, uint32_t bits1) {
            const int64_t base_e = (slab_first + w) * kSlab;
            const int64_t left = a.t.d - base_e;
            const int L = (int)(left < kSlab ? left : kSlab);
            const int nchunks = (L + chunk - 1) >> cshift;
            const float c0n = __fmul_rn(sa.lr, k0 < nchunks ? S_new_sh[w & 1][k0] : 0.0f);      // lr * (+-S) = +-(lr * S)
            const float c1n = __fmul_rn(sa.lr, k1 < nchunks ? S_new_sh[w & 1][k1] : 0.0f);
            const int st = q % kStages;
            if (!mbar_wait(&full[st], (uint32_t)(q / kStages) & 1u)) { failed = 1; ok = false; }
            if (ok) {
                const float* vs = reinterpret_cast<const float*>(smem + (size_t)st * stage_bytes);
                const float* xs = vs + kSlab;
                float4 vv[2], xx[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    vv[u] = *reinterpret_cast<const float4*>(vs + (u ? g1 : g0) * kGroup + lane * 4);
                    xx[u] = *reinterpret_cast<const float4*>(xs + (u ? g1 : g0) * kGroup + lane * 4);
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int k = (u ? g1 : g0) * kGroup + lane * 4;
                    const uint32_t nib = u ? bits1 : bits0;
                    const float cn = u ? c1n : c0n;
                    xx[u].x = apply_stored(xx[u].x, vv[u].x, nib & 1u, cn);
                    xx[u].y = apply_stored(xx[u].y, vv[u].y, nib & 2u, cn);
                    xx[u].z = apply_stored(xx[u].z, vv[u].z, nib & 4u, cn);
                    xx[u].w = apply_stored(xx[u].w, vv[u].w, nib & 8u, cn);
                    st4_checked(sa.x + base_e, k, L, xx[u]);
                }
                __syncwarp();                                            // the stage goes back after the stores that needed its values
                if (lane == 0) mbar_arrive(&empty[st]);
            }
            ++q;
        };
        if (nmine > 0) {
            fetch_scales(0);
            store_scales(0);
        }
        bool leave = consumer_barrier_any(*vfailed != 0);                 // the first slab's scales are in place
        uint32_t prev0 = 0u, prev1 = 0u;                                  // this lane's sign bits of the slab before
        int w = 0;
        for (; w < nmine && !leave; ++w) {
            const int buf = w & 1;
            const int64_t base_e = (slab_first + w) * kSlab;
            const int64_t left = a.t.d - base_e;
            const int L = (int)(left < kSlab ? left : kSlab);
            const int64_t c0 = base_e >> cshift;
            const int nchunks = (L + chunk - 1) >> cshift;
            const uint32_t* negs = neg_s[buf];
            if (w + 1 < nmine) fetch_scales(w + 1);                       // in flight during this slab's arithmetic
            double acc0 = 0.0, acc1 = 0.0;
            uint32_t mine0 = 0u, mine1 = 0u;
            {
                const int st = q % kStages;
                if (!mbar_wait(&full[st], (uint32_t)(q / kStages) & 1u)) { failed = 1; ok = false; }
                if (ok) {
                    const unsigned char* base = smem + (size_t)st * stage_bytes;
                    const float* zs = reinterpret_cast<const float*>(base);
                    const uint32_t* rows = reinterpret_cast<const uint32_t*>(base + (size_t)kSlab * 4);
                    const float4 zo0 = *reinterpret_cast<const float4*>(zs + g0 * kGroup + lane * 4);
                    const float4 zo1 = *reinterpret_cast<const float4*>(zs + g1 * kGroup + lane * 4);
                    float2 s01 = make_float2(0.f, 0.f), s23 = s01, t01 = s01, t23 = s01;   // running sums, worker order
                    // a group past the end of the vector has no chunk: it reads the first chunk's values and is masked below
                    const int kk0 = k0 < nchunks ? k0 : 0, kk1 = k1 < nchunks ? k1 : 0;
                    signed_scale_sums2<NT>(rows + off_in + g0 * 4 + wl, rows + off_in + g1 * 4 + wl,
                                           negs + kk0 * APMS_MAX_WORKERS, negs + kk1 * APMS_MAX_WORKERS, n, sh, s01, s23, t01, t23);
                    const float So0 = S_old_sh[buf][kk0], So1 = S_old_sh[buf][kk1];
                    uint32_t* __restrict__ ob = a.Bbar + base_e / 32;
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int grp = u ? g1 : g0;
                        const int k = grp * kGroup + lane * 4;
                        const float4 zo4 = u ? zo1 : zo0;
                        const float zo[4] = {zo4.x, zo4.y, zo4.z, zo4.w};
                        const float sum[4] = {u ? t01.x : s01.x, u ? t01.y : s01.y, u ? t23.x : s23.x, u ? t23.y : s23.y};
                        const float S_old = u ? So1 : So0;
                        float zn[4];
                        uint32_t nibble = 0;
                        double acc = 0.0;
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
                        if (u) { acc1 = acc; mine1 = nibble; } else { acc0 = acc; mine0 = nibble; }
                        st4_checked(a.zbar + base_e, k, L, make_float4(zn[0], zn[1], zn[2], zn[3]));
                        // the group's four new sign words: lanes 0, 8, 16, 24 hold one each - one 16-byte piece per group
                        const uint32_t word = pack_group_words(nibble, lane);
                        const int wk = grp * 4 + wl;
                        if ((lane & 7) == 0 && wk * 32 < L) st_stream_word(ob + wk, word);
                    }
                    __syncwarp();                                            // the stage goes back after the stores that needed its values
                    if (lane == 0) mbar_arrive(&empty[st]);
                }
                ++q;
            }
            acc0 = warp_sum(acc0);
            acc1 = warp_sum(acc1);
            if (lane == 0) { red[buf][g0] = acc0; red[buf][g1] = acc1; }
            if (w + 1 < nmine) store_scales(buf ^ 1);                     // the next slab's scales, fetched above
            leave = consumer_barrier_any(!ok || *vfailed != 0);           // the groups' sums of this slab are in shared memory
            if (leave) break;
            // The new scale of every chunk of the slab, one chunk per lane of one warp (the warps take turns).
            if (warp == (w & (kWarps - 1)) && lane < nchunks) {
                double total = 0.0;
                for (int r = 0; r < gpc; ++r) total += red[buf][lane * gpc + r];           // group order
                const int64_t cbeg = (c0 + lane) * (int64_t)chunk;
                const int64_t Lc = (a.t.d - cbeg < chunk) ? a.t.d - cbeg : chunk;
                const float S_lane = (float)sqrt(total / (double)Lc);
                S_new_sh[buf][lane] = S_lane;
                APMS_STORE(a.Sbar[c0 + lane], S_lane);
            }
            if (w >= 1) update_slab(w - 1, prev0, prev1);                 // its scales were formed a slab ago, before this slab's barrier
            prev0 = mine0; prev1 = mine1;
        }
        if (!leave && nmine > 0) {
            leave = consumer_barrier_any(!ok || *vfailed != 0);           // the last slab's scales are in shared memory
            if (!leave) update_slab(nmine - 1, prev0, prev1);
        }
    }
    __syncthreads();                                   // every warp has left its loops; shared memory may go
    if (threadIdx.x == 0 && failed) atomicExch(sa.status, DEVICE_WAIT_TIMEOUT);
}

}  // namespace
