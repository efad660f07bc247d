// Worker side of a compression-phase step (Section 3.3 steps 1-2): general and fine-tiled kernels,
// and the kernels that finish the per-chunk scales.
// Part of libapms.so: included by apms.cu, which is the only translation unit.
#pragma once

namespace {

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
    int64_t items;                // chunk tiles of this launch * ni
    int64_t tile0;                // first chunk tile of this launch (a launch may cover a range of chunks)
    int i0, ni;                   // this launch covers workers i0 .. i0+ni-1
    float beta1, omb1;
    int send_gradient;            // gradient-compressing variant: z = g_i + delta_i, the momentum is not read
};

template <bool M32, bool CHECKED>
__device__ __forceinline__ void worker_group(float beta1, float omb1, float* __restrict__ z, uint32_t* __restrict__ obits,
                                             int grp, int lane, int L, float s_old, float Sbar,
                                             float4 gv, float4 zv, float4 mv, uint32_t mw, double& acc, bool l1,
                                             bool send_gradient = false, bool keep = true)      // keep = false: this lane's elements are not this launch's
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
    if (keep) { if (CHECKED) st4_checked(z, k, L, out); else st_stream4(z + k, out); }
    const uint32_t word = pack_group_words(nibble, lane);
    if ((lane & 7) == 0 && keep) {
        const int wk = grp * 4 + (lane >> 3);
        if (!CHECKED || wk * 32 < L) st_stream_word(obits + wk, word);     // streaming: a plain store here costs ~4 % of the kernel
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
    const Item it = decode_item(a.t, a.tile0 + item / a.ni);
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
        if (a.t.P == 1) APMS_STORE(*sptr, scale_from_sum(total, (double)it.Lc, a.t.l1 != 0));    // ||z||_2 / sqrt(L)
        else APMS_STORE(a.partial[(int64_t)i * a.t.Pp + it.c * a.t.P + it.p], total);
    }
}

// Worker side, fine-tiled form (steady state, chunks of at least kFineSub elements): one CTA per
// (worker, 4096-element tile), every load of the tile issued before the first use.  Short-lived
// CTAs that each touch 16 KiB of every stream once keep DRAM pages and the memory pipeline busier
// than long-running warps that each follow their own stream.
// Warp w owns the tile's groups 4w..4w+3 (kFineSub = 512 consecutive elements), so its 16 momentum
// words are one 64-byte load handed round by shuffles, its 16 new sign words one 64-byte store, and
// its binary64 sum of squares one slot of a partial-sum array that k_finalize_fine adds up per chunk
// in element order: the kernel has no barrier at all.
// Chunks are multiples of 32 elements, so a chunk boundary inside a warp's 512 elements falls
// between two sign words, i.e. between two 8-lane groups of one 128-element access, and there is at
// most one of them (chunk >= 512).  With SPLIT (chunks that are not multiples of 512) a warp that
// sees a boundary reads the scales of both chunks and keeps two sums; a piece then has two slots:
// [0] = its elements of the chunk its first element belongs to, [1] = those of the next chunk (written
// and read only where there is one).  A warp without a boundary runs the same code as without SPLIT.
// Launch order: runs of `run` consecutive tiles of one worker, then the same tiles of the next
// worker: every stream is read in long sequential pieces (measured: the longer the better for
// DRAM), while the momentum bits of a run (run * 512 bytes) stay in L2 for the other workers.

constexpr int kFineTile = 4096;           // 256 threads x 4 x (4 floats)
constexpr int kFineU = kFineTile / (kThreads * 4);
constexpr int kFineSub = kFineTile / kWarps;      // elements per warp = per partial sum
constexpr int kFineSubWords = kFineSub / 32;
constexpr int kFineRunDefault = 4096;
constexpr int64_t kFineLongSlots = 1024;  // chunks with more 512-element pieces than this get a whole CTA in the finalize

struct WorkerFineArgs {
    float* z; int64_t dz;
    uint32_t* B; int64_t Wp;
    const float* s; int64_t Cp;       // the scales of the previous step (read only here)
    double* partial; int64_t Pp;      // ni rows of tiles * kWarps (* 2 with SPLIT) partial sums, row stride Pp
    const uint32_t* Bbar; const float* Sbar;
    int64_t d, chunk, tiles;          // tiles: 4096-element tiles of this launch, the first one being tile0
    int64_t tile0, e0, e1;            // a launch may cover the elements [e0, e1) of whole chunks only (multiples of 512 without SPLIT)
    int i0, ni, run;
    float beta1, omb1;
    float inv_chunk;                  // 1 / chunk in binary32 when there are fewer than 2^20 chunks (see div_small_quotient), else 0
    float inv_run, inv_per_stretch;   // 1 / run and 1 / (ni * run) in binary32 (see div_u32)
};

// One warp's 512 elements (L of them live).  TWO: a chunk boundary lies inside, at sign word `bw`: the lanes whose
// word lies past it use the next chunk's scales (s_hi, S_hi) and add their squares to acc_hi.  `keep`: bit 0 - the
// elements before the boundary belong to this launch, bit 1 - those past it do (a launch over a range of chunks
// ends at a chunk boundary, which may be this one; what does not belong is neither stored nor summed).
template <int GT, bool SENDG, bool TWO>
__device__ __forceinline__ void fine_piece(const WorkerFineArgs& a, const void* __restrict__ g, float* __restrict__ z,
                                           const uint32_t* __restrict__ mbits, uint32_t* __restrict__ obits, int lane, int L,
                                           int bw, float s_lo, float S_lo, float s_hi, float S_hi, double& acc, double& acc_hi,
                                           int keep = 3)
{
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
            const bool hi = TWO && (u * 4 + (lane >> 3) >= bw);      // this lane's word lies in the next chunk
            const float s_old = hi ? s_hi : s_lo, Sbar = hi ? S_hi : S_lo;
            const float gg[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
            const float zo[4] = {zv[u].x, zv[u].y, zv[u].z, zv[u].w};
            float zn[4];
            uint32_t nibble = 0;
            double part = TWO ? 0.0 : acc;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float mm = bit_scale((nib >> e) & 1u, Sbar);                    // m = +-Sbar
                const float mi = SENDG ? gg[e] : __fmaf_rn(a.beta1, mm, __fmul_rn(a.omb1, gg[e]));    // local momentum
                zn[e] = __fadd_rn(mi, implied_error(zo[e], s_old));                   // compensated
                const double zd = (double)zn[e];
                part = fma(zd, zd, part);
                nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
            }
            if (TWO) { acc += hi ? 0.0 : part; acc_hi += hi ? part : 0.0; }
            else acc = part;
            if (!TWO || (keep & (hi ? 2 : 1))) st_stream4(z + u * kGroup + lane * 4, make_float4(zn[0], zn[1], zn[2], zn[3]));
            const uint32_t word = pack_group_words(nibble, lane);       // valid in lanes 0, 8, 16, 24
            const uint32_t got = __shfl_sync(0xffffffffu, word, (lane & 3) * 8);
            if ((lane >> 2) == u) outw = got;                               // lane 4u + j keeps word j of group u
        }
        if (lane < 4 * kFineU && (!TWO || (keep & (lane >= bw ? 2 : 1)))) st_stream_word(obits + lane, outw);
    } else {
        const int ngroups = (L + kGroup - 1) / kGroup;
        for (int grp = 0; grp < ngroups; ++grp) {
            const int k = grp * kGroup + lane * 4;
            const float4 gv = ld_grad4_checked<GT>(g, k, L);
            const float4 zv = ld4_checked(z, k, L, true);
            const uint32_t mw = (!SENDG && k < L) ? mbits[grp * 4 + (lane >> 3)] : 0u;
            if (TWO) {
                const bool hi = grp * 4 + (lane >> 3) >= bw;
                double part = 0.0;
                worker_group<false, true>(a.beta1, a.omb1, z, obits, grp, lane, L, hi ? s_hi : s_lo, hi ? S_hi : S_lo, gv, zv,
                                          make_float4(0, 0, 0, 0), mw, part, false, SENDG, (keep & (hi ? 2 : 1)) != 0);
                acc += hi ? 0.0 : part; acc_hi += hi ? part : 0.0;
            } else {
                worker_group<false, true>(a.beta1, a.omb1, z, obits, grp, lane, L, s_lo, S_lo, gv, zv,
                                          make_float4(0, 0, 0, 0), mw, acc, false, SENDG);
            }
        }
    }
}

template <int GT, bool SENDG, bool SPLIT>          // SENDG: the gradient-compressing variant (no momentum is read)
__global__ void __launch_bounds__(kThreads, 4)
k_worker_fine(const __grid_constant__ GradPtrs G, const WorkerFineArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t per_stretch = (uint32_t)a.ni * (uint32_t)a.run;        // the grid has fewer than 2^31 blocks
    const uint32_t stretch = div_u32(blockIdx.x, per_stretch, a.inv_per_stretch);
    const uint32_t rem = blockIdx.x - stretch * per_stretch;
    const int ii = (int)div_u32(rem, (uint32_t)a.run, a.inv_run);
    const int64_t tl = (int64_t)stretch * a.run + (rem - (uint32_t)ii * (uint32_t)a.run);
    if (tl >= a.tiles) return;                                 // whole CTA: the last stretch may be short
    const int64_t t = a.tile0 + tl;
    const int i = a.i0 + ii;
    const int64_t base = t * kFineTile + (int64_t)warp * kFineSub;     // this warp's 512 elements
    if (base + kFineSub <= a.e0 || base >= a.e1) return;       // a launch over a range of chunks: the tiles at its ends are shared
    double* __restrict__ slot = a.partial + (int64_t)ii * a.Pp + (t * kWarps + warp) * (SPLIT ? 2 : 1);
    const int64_t left = a.d - base;
    if (left <= 0) {                                           // past the end of the vector
        if (lane == 0) APMS_STORE(*slot, 0.0);
        return;
    }
    const int L = (int)(left < kFineSub ? left : kFineSub);
    const int64_t c = a.inv_chunk != 0.0f ? div_small_quotient(base, a.chunk, a.inv_chunk) : base / a.chunk;
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], base);
    float* __restrict__ z = a.z + (int64_t)i * a.dz + base;
    const uint32_t* __restrict__ mbits = a.Bbar + base / 32;
    uint32_t* __restrict__ obits = a.B + (int64_t)i * a.Wp + base / 32;
    const float* __restrict__ srow = a.s + (int64_t)i * a.Cp;
    const float s_lo = srow[c], S_lo = a.Sbar[c];
    double acc = 0.0, acc_hi = 0.0;
    // elements of this warp that belong to chunk c + 1 begin at its sign word bw (SPLIT only; rare for long chunks)
    const int64_t next = (c + 1) * a.chunk - base;
    if (SPLIT && next < L) {
        // the boundary may be the start or the end of the launch's range: then only one side is this launch's
        const int keep = (base + next <= a.e0) ? 2 : ((base + next >= a.e1) ? 1 : 3);
        fine_piece<GT, SENDG, true>(a, g, z, mbits, obits, lane, L, (int)(next >> 5), s_lo, S_lo, srow[c + 1], a.Sbar[c + 1], acc, acc_hi, keep);
        acc = warp_sum(acc);
        acc_hi = warp_sum(acc_hi);
        if (lane == 0) { if (keep & 1) APMS_STORE(slot[0], acc); if (keep & 2) APMS_STORE(slot[1], acc_hi); }
    } else {
        if (base < a.e0) return;                               // (only with SPLIT: a piece before the range that holds no boundary)
        fine_piece<GT, SENDG, false>(a, g, z, mbits, obits, lane, L, 0, s_lo, S_lo, s_lo, S_lo, acc, acc_hi);
        acc = warp_sum(acc);
        if (lane == 0) APMS_STORE(slot[0], acc);                          // slot [1] of a piece without a boundary is never read
    }
}

// The same tiling for chunks below 512 elements: a warp's 512 elements then hold several chunks, but a sign word
// (32 elements = the 8 lanes of one access) still lies in one chunk.  Every lane looks up the scales of its word's
// chunk, the squares are summed per word (three shuffle steps inside the 8 lanes) into one slot per word, and
// k_finalize_words adds a chunk's words in order.  A launch over a range of chunks skips the words outside it.
template <int GT, bool SENDG>
__global__ void __launch_bounds__(kThreads, 4)
k_worker_fine_words(const __grid_constant__ GradPtrs G, const WorkerFineArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t per_stretch = (uint32_t)a.ni * (uint32_t)a.run;
    const uint32_t stretch = div_u32(blockIdx.x, per_stretch, a.inv_per_stretch);
    const uint32_t rem = blockIdx.x - stretch * per_stretch;
    const int ii = (int)div_u32(rem, (uint32_t)a.run, a.inv_run);
    const int64_t tl = (int64_t)stretch * a.run + (rem - (uint32_t)ii * (uint32_t)a.run);
    if (tl >= a.tiles) return;
    const int64_t t = a.tile0 + tl;
    const int i = a.i0 + ii;
    const int64_t base = t * kFineTile + (int64_t)warp * kFineSub;
    if (base + kFineSub <= a.e0 || base >= a.e1 || base >= a.d) return;
    const int64_t left = a.d - base;
    const int L = (int)(left < kFineSub ? left : kFineSub);
    const void* __restrict__ g = Grad<GT>::at(G.p[ii], base);
    float* __restrict__ z = a.z + (int64_t)i * a.dz + base;
    const uint32_t* __restrict__ mbits = a.Bbar + base / 32;
    uint32_t* __restrict__ obits = a.B + (int64_t)i * a.Wp + base / 32;
    const float* __restrict__ srow = a.s + (int64_t)i * a.Cp;
    double* __restrict__ slots = a.partial + (int64_t)ii * a.Pp + base / 32;      // one slot per sign word
    // the chunk of this lane's word in each of the four accesses: first chunk of the piece plus a small quotient
    const int64_t c_first = base / a.chunk;
    const uint32_t rel0 = (uint32_t)(base - c_first * a.chunk), chunk32 = (uint32_t)a.chunk;
    const float inv_c = 1.0f / (float)chunk32;
    const int wl = lane >> 3;
    float s_old[kFineU], Sb[kFineU];
    bool mine[kFineU];                                          // the word exists and belongs to this launch's range
#pragma unroll
    for (int u = 0; u < kFineU; ++u) {
        const int wi = u * 4 + wl;
        const int64_t e = base + 32 * wi;
        mine[u] = 32 * wi < L && e >= a.e0 && e < a.e1;
        const int64_t cw = c_first + div_u32(rel0 + 32u * (uint32_t)wi, chunk32, inv_c);
        s_old[u] = 32 * wi < L ? srow[cw] : 0.0f;
        Sb[u] = 32 * wi < L ? a.Sbar[cw] : 0.0f;
    }
    if (L == kFineSub) {
        float4 gv[kFineU], zv[kFineU];
#pragma unroll
        for (int u = 0; u < kFineU; ++u) {
            gv[u] = Grad<GT>::ld4(g, u * kGroup + lane * 4);
            zv[u] = ld_stream4(z + u * kGroup + lane * 4);
        }
        const uint32_t mw = (!SENDG && lane < 4 * kFineU) ? mbits[lane] : 0u;
        uint32_t outw = 0;
#pragma unroll
        for (int u = 0; u < kFineU; ++u) {
            const uint32_t nib = __shfl_sync(0xffffffffu, mw, u * 4 + wl) >> (4 * (lane & 7));
            const float gg[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
            const float zo[4] = {zv[u].x, zv[u].y, zv[u].z, zv[u].w};
            float zn[4];
            uint32_t nibble = 0;
            double part = 0.0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float mm = bit_scale((nib >> e) & 1u, Sb[u]);
                const float mi = SENDG ? gg[e] : __fmaf_rn(a.beta1, mm, __fmul_rn(a.omb1, gg[e]));
                zn[e] = __fadd_rn(mi, implied_error(zo[e], s_old[u]));
                const double zd = (double)zn[e];
                part = fma(zd, zd, part);
                nibble |= (zn[e] >= 0.0f ? 1u : 0u) << e;
            }
            if (mine[u]) st_stream4(z + u * kGroup + lane * 4, make_float4(zn[0], zn[1], zn[2], zn[3]));
            part += __shfl_xor_sync(0xffffffffu, part, 1);      // the word's 32 squares: lanes 8k .. 8k+7
            part += __shfl_xor_sync(0xffffffffu, part, 2);
            part += __shfl_xor_sync(0xffffffffu, part, 4);
            if ((lane & 7) == 0 && mine[u]) APMS_STORE(slots[u * 4 + wl], part);
            const uint32_t word = pack_group_words(nibble, lane);
            const uint32_t got = __shfl_sync(0xffffffffu, word, (lane & 3) * 8);
            if ((lane >> 2) == u) outw = got;
        }
        if (lane < 4 * kFineU) {                                // lane j keeps word j: stored if it belongs to the range
            const int64_t e = base + 32 * lane;
            if (e >= a.e0 && e < a.e1) st_stream_word(obits + lane, outw);
        }
    } else {
        const int ngroups = (L + kGroup - 1) / kGroup;
#pragma unroll
        for (int u = 0; u < kFineU; ++u) {
            if (u >= ngroups) break;
            const int k = u * kGroup + lane * 4;
            const float4 gv = ld_grad4_checked<GT>(g, k, L);
            const float4 zv = ld4_checked(z, k, L, true);
            const uint32_t mw = (!SENDG && k < L) ? mbits[u * 4 + wl] : 0u;
            double part = 0.0;
            worker_group<false, true>(a.beta1, a.omb1, z, obits, u, lane, L, s_old[u], Sb[u], gv, zv,
                                      make_float4(0, 0, 0, 0), mw, part, false, SENDG, mine[u]);
            part += __shfl_xor_sync(0xffffffffu, part, 1);
            part += __shfl_xor_sync(0xffffffffu, part, 2);
            part += __shfl_xor_sync(0xffffffffu, part, 4);
            if ((lane & 7) == 0 && mine[u]) APMS_STORE(slots[u * 4 + wl], part);
        }
    }
}

// Scales from one sum of squares per sign word: a thread per (row, chunk) adds the chunk's words in order.
__global__ void __launch_bounds__(kThreads)
k_finalize_words(const double* __restrict__ partial, int64_t Pp, float* __restrict__ scales, int64_t Cp,
                 int rows, int64_t c_first, int64_t C, int64_t d, int64_t chunk)
{
    const int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (idx >= (int64_t)rows * C) return;
    const int r = (int)(idx / C);
    const int64_t c = c_first + idx % C;
    const int64_t cbeg = c * chunk;
    const int64_t Lc = (d - cbeg < chunk) ? d - cbeg : chunk;
    const double* __restrict__ p = partial + (int64_t)r * Pp + cbeg / 32;
    double total = 0.0;
    for (int w = 0; w < (int)((Lc + 31) / 32); ++w) total += p[w];
    APMS_STORE(scales[(int64_t)r * Cp + c], (float)sqrt(total / (double)Lc));
}

// Scales from the fine form's partial sums (one - or, with chunks that are not multiples of 512, two -
// per 512 elements): a team of T lanes per (row, chunk) adds the chunk's slots in a fixed order (lane l
// of the team takes the 512-element pieces l, l + T, ..., then the shuffle tree) and takes sqrt(sum / L).
// With two slots per piece (`per` = 2) a chunk takes slot [1] of the piece it begins inside of and slot
// [0] of all later ones.  T is the number of pieces a chunk can touch rounded up to a power of two, at
// most a warp; the sums are not negative, so a team's tree gives bit for bit what a whole warp's tree
// with zeros in the other lanes gives, and short chunks do not leave most of a warp idle (chunk = 1024:
// 16 chunks per warp; one warp per chunk took 1.2 ms longer at n = 16).
template <int T>
__global__ void __launch_bounds__(kThreads)
k_finalize_fine(const double* __restrict__ partial, int64_t Pp, float* __restrict__ scales, int64_t Cp,
                int rows, int64_t c_first, int64_t C, int64_t d, int64_t chunk, int per)
{
    const int lane = threadIdx.x & 31, sub = lane % T;
    const int64_t idx = ((int64_t)blockIdx.x * kWarps + (threadIdx.x >> 5)) * (32 / T) + lane / T;
    const bool live = idx < (int64_t)rows * C;                   // every lane stays for the shuffles; C chunks from c_first on
    const int r = live ? (int)(idx / C) : 0;
    const int64_t c = c_first + (live ? idx % C : 0);
    const int64_t cbeg = c * chunk;
    const int64_t Lc = (d - cbeg < chunk) ? d - cbeg : chunk;
    const int64_t q0 = cbeg / kFineSub, q1 = (cbeg + Lc + kFineSub - 1) / kFineSub;
    double total = 0.0;
    if (live) for (int64_t q = q0 + sub; q < q1; q += T)
        total += partial[(int64_t)r * Pp + q * per + ((per == 2 && q * kFineSub < cbeg) ? 1 : 0)];
#pragma unroll
    for (int o = T / 2; o > 0; o >>= 1) total += __shfl_down_sync(0xffffffffu, total, o, T);
    if (live && sub == 0) APMS_STORE(scales[(int64_t)r * Cp + c], (float)sqrt(total / (double)Lc));
}

// The same for long chunks (thousands of pieces each, few chunks): one CTA per (row, chunk); thread t adds the
// pieces t, t + 256, ... and the block sum adds the threads in a fixed order.
__global__ void __launch_bounds__(kThreads)
k_finalize_fine_cta(const double* __restrict__ partial, int64_t Pp, float* __restrict__ scales, int64_t Cp,
                    int rows, int64_t c_first, int64_t C, int64_t d, int64_t chunk, int per)
{
    __shared__ double red[kWarps];
    const int r = (int)(blockIdx.x / C);
    const int64_t c = c_first + blockIdx.x % C;
    const int64_t cbeg = c * chunk;
    const int64_t Lc = (d - cbeg < chunk) ? d - cbeg : chunk;
    const int64_t q0 = cbeg / kFineSub, q1 = (cbeg + Lc + kFineSub - 1) / kFineSub;
    const double* __restrict__ row = partial + (int64_t)r * Pp;
    double total = 0.0;
#pragma unroll 4
    for (int64_t q = q0 + threadIdx.x; q < q1; q += kThreads)
        total += row[q * per + ((per == 2 && q * kFineSub < cbeg) ? 1 : 0)];
    total = block_sum(total, red);
    if (threadIdx.x == 0) APMS_STORE(scales[(int64_t)r * Cp + c], (float)sqrt(total / (double)Lc));
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
    APMS_STORE(scales[(int64_t)r * Cp + c], scale_from_sum(total, (double)Lc, t.l1 != 0));
}

}  // namespace
