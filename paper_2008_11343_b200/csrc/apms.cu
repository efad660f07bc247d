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


#include "device_common.cuh"
#include "kernels_adam.cuh"
#include "tiling.cuh"
#include "kernels_worker.cuh"
#include "kernels_server.cuh"
#include "kernels_apply.cuh"
#include "kernels_topk.cuh"
#include "kernels_monitor.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// host side

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// A guard region: bytes of the workspace that no kernel may write (see apms_set_guard_bytes).
struct GuardRegion { size_t off, bytes; const char* what; };

struct Layout {
    int64_t d, chunk, C, W, dz, Wp, Cp;
    int64_t fine_tiles, fine_Pp;   // 4096-element tiles of the fine worker form (0 when the chunk length does not allow it)
    int fine_split, fine_words;
    int n;
    Tiling t;
    size_t off_x, off_v, off_m, off_zbar, off_z, off_B, off_Bbar, off_s, off_Sbar, off_hint, off_tiles, off_part, off_fine, off_stage, off_mon, off_den, off_status, total;
    size_t guard;                  // guard bytes behind every row of every array (0 = the ordinary layout)
};

size_t g_guard_bytes = 0;          // process-wide, read when a context is created

// guard > 0: every row of every array is followed by at least `guard` bytes that belong to no array, and
// so is the start of the workspace; `regions` (if given) receives them.
bool make_layout(int64_t d, int n, int64_t chunk, Layout* L, size_t guard = 0, std::vector<GuardRegion>* regions = nullptr)
{
    if (d < 1 || n < 1 || n > APMS_MAX_WORKERS || chunk < 32 || chunk % 32 != 0) return false;
    if (chunk > (int64_t)1 << 30) return false;
    L->d = d; L->n = n; L->chunk = chunk; L->guard = guard;
    L->C = (d + chunk - 1) / chunk;
    L->W = (d + 31) / 32;
    L->dz = (int64_t)round_up((size_t)d, 64) + (int64_t)(guard / 4);
    L->Wp = (int64_t)round_up((size_t)L->W, 64) + (int64_t)(guard / 4);
    L->Cp = (int64_t)round_up((size_t)L->C, 64) + (int64_t)(guard / 4);
    size_t o = 0;
    // `rows` rows of `stride` elements of `es` bytes, of which the first `used` are the array's own
    auto take = [&](const char* what, size_t rows, size_t stride, size_t used, size_t es) {
        const size_t at = o;
        if (guard && regions)
            for (size_t r = 0; r < rows; ++r)
                if (stride > used) regions->push_back({at + (r * stride + used) * es, (stride - used) * es, what});
        o += round_up(rows * stride * es, 256);
        return at;
    };
    if (guard) {
        if (regions) regions->push_back({0, guard, "the start of the workspace"});
        o = guard;
    }
    const size_t ud = (size_t)d, un = (size_t)n;
    L->off_x = take("x", 1, L->dz, ud, 4);
    L->off_v = take("v", 1, L->dz, ud, 4);
    L->off_m = take("m", 1, L->dz, ud, 4);
    L->off_zbar = take("zbar", 1, L->dz, ud, 4);
    L->off_z = take("z_i", un, L->dz, ud, 4);
    L->off_B = take("B_i", un, L->Wp, L->W, 4);
    L->off_Bbar = take("Bbar", 1, L->Wp, L->W, 4);
    L->off_s = take("s_i", un, L->Cp, L->C, 4);
    L->off_Sbar = take("Sbar", 1, L->Cp, L->C, 4);
    // top-k: the thresholds of the step before last (n worker rows + 1 server row), then as many rows of learned bands
    L->off_hint = take("threshold hints", 2 * (un + 1), L->Cp, L->C, 4);
    L->t.d = d; L->t.chunk = chunk;
    if (chunk <= kTileMax) { L->t.tile = chunk; L->t.P = 1; }
    else { L->t.tile = kTileSplit; L->t.P = (int)((chunk + kTileSplit - 1) / kTileSplit); }
    // counters of the lagged server form (chunks cut into tiles): 64 words for the ticket, then per chunk the tiles done and the ready flag
    L->off_tiles = take("server tile counters", 1, 64 + 2 * (size_t)L->Cp, L->t.P > 1 ? 64 + 2 * (size_t)L->Cp - guard / 4 : 0, 4);
    L->t.Pp = (int64_t)round_up((size_t)(L->C * L->t.P), 64) + (int64_t)(guard / 8);
    L->off_part = take("partial sums of split chunks", L->t.P > 1 ? un + 1 : 0, L->t.Pp, (size_t)(L->C * L->t.P), 8);   // n worker rows + 1 server row
    L->fine_tiles = (d + kFineTile - 1) / kFineTile;
    L->fine_split = (chunk % kFineSub != 0) ? 1 : 0;     // a warp's 512 elements may lie in two chunks: two partial sums each
    L->fine_words = chunk < kFineSub ? 1 : 0;            // ... or in several: one partial sum per sign word
    const size_t fine_used = L->fine_words ? (size_t)L->W : (size_t)L->fine_tiles * kWarps * (size_t)(L->fine_split ? 2 : 1);
    L->fine_Pp = (int64_t)round_up(fine_used, 64) + (int64_t)(guard / 8);
    L->off_fine = take("partial sums of the fine worker form", un, L->fine_Pp, fine_used, 8);
    L->off_stage = take("staging buffers", 2, L->dz, ud, 4);
    const size_t mon_used = (un + 1) * (size_t)((d + 4095) / 4096) + (un + 1);
    L->off_mon = take("error monitor sums", 1, round_up(mon_used, 32) + guard / 8, mon_used, 8);   // tile sums + row sums
    L->off_den = take("den", 1, L->dz, ud, 4);              // sqrt(v) + eps of the frozen v
    L->off_status = take("status", 1, 64 + guard / 4, 64, 4);
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
    int substep;             // phase-wise step: 0 = between steps, 1 = in or past the worker phase, 2 = a server phase done
    int64_t worker_chunks;   // phase-wise step: chunks the worker phase has covered so far
    apms_schedule sched; bool has_sched;
    apms_phase phase;
    bool m_is_fp32;          // momentum lives in the binary32 buffer (else in Bbar/Sbar; top-k: in zbar under the mask Bbar)
    bool v_checked, v_plain; // top-k: has v been looked at since it last changed, and is every entry >= 0 (not NaN)
    bool den_valid;          // den holds sqrt(v) + eps of the current v
    char* ws; size_t ws_bytes; bool owns_ws;
    cudaStream_t stream;
    cudaStream_t copy_stream; cudaEvent_t ev_copied[2], ev_used[2]; bool host_path_ready;
    int device;
    int sms;
    bool timing;
    apms_team_mode team_mode;
    int fine_run;            // tiles of one worker launched back to back in the fine worker form
    unsigned int tile_epoch; // launches of the lagged server form so far (never 0 in a launch)
    std::vector<EventPair> events[APMS_KERNEL_COUNT];
    std::vector<EventPair> pool;
    int64_t launches;
    std::vector<GuardRegion> guards;   // empty in the ordinary layout
    unsigned long long* guard_table;   // checked build: the guard regions as (offset, bytes) pairs on the device
    bool registered;                   // checked build: this workspace is in the device's table of checked workspaces
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
    float* hint(int i) { return (float*)(ws + L.off_hint) + (int64_t)i * L.Cp; }   // i = n: the server's
    float* learned(int i) { return hint(L.n + 1 + i); }
    unsigned int* tile_ticket() { return (unsigned int*)(ws + L.off_tiles); }
    unsigned int* tiles_done() { return tile_ticket() + 64; }
    unsigned int* tiles_ready() { return tiles_done() + L.Cp; }
    float* stage(int b) { return (float*)(ws + L.off_stage) + (int64_t)b * L.dz; }
    int* status() { return (int*)(ws + L.off_status); }
    float* den() { return (float*)(ws + L.off_den); }
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
    return APMS_OK;            // guard regions are written by apms_set_params, the first call that touches the workspace
}

// Guard layout only: (re)writes the pattern into every guard region, on the context's stream.
constexpr int kGuardByte = 0xA5;
apms_status fill_guards(apms_ctx* c)
{
    for (const GuardRegion& g : c->guards)
        APMS_CUDA(c, cudaMemsetAsync(c->ws + g.off, kGuardByte, g.bytes, c->stream));
    return APMS_OK;
}

#ifdef APMS_BOUNDS_CHECK
// Checked build: the table of live workspaces the device-side accessors consult (see device_common.cuh).
std::mutex g_checked_mutex;
std::vector<CheckedWorkspace> g_checked_host;

apms_status upload_checked_table(apms_ctx* c)
{
    const int count = (int)g_checked_host.size();
    if (count > 0) APMS_CUDA(c, cudaMemcpyToSymbol(g_checked, g_checked_host.data(), sizeof(CheckedWorkspace) * (size_t)count));
    APMS_CUDA(c, cudaMemcpyToSymbol(g_checked_count, &count, sizeof count));
    return APMS_OK;
}

apms_status register_checked(apms_ctx* c)
{
    if (c->registered) return APMS_OK;
    std::lock_guard<std::mutex> lock(g_checked_mutex);
    if ((int)g_checked_host.size() >= kMaxCheckedWorkspaces) return fail(c, APMS_ERR_OOM, "too many live contexts for the checked build's table");
    std::vector<unsigned long long> pairs;
    for (const GuardRegion& g : c->guards) { pairs.push_back(g.off); pairs.push_back(g.bytes); }     // ascending by construction
    if (!pairs.empty()) {
        APMS_CUDA(c, cudaMalloc((void**)&c->guard_table, pairs.size() * sizeof(unsigned long long)));
        APMS_CUDA(c, cudaMemcpy(c->guard_table, pairs.data(), pairs.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice));
    }
    CheckedWorkspace w;
    w.lo = (unsigned long long)c->ws; w.hi = w.lo + c->L.total;
    w.guards = c->guard_table; w.nguards = (int)c->guards.size(); w.status = c->status();
    APMS_CUDA(c, cudaDeviceSynchronize());
    g_checked_host.push_back(w);
    c->registered = true;
    return upload_checked_table(c);
}

void unregister_checked(apms_ctx* c)
{
    if (!c->registered) return;
    std::lock_guard<std::mutex> lock(g_checked_mutex);
    cudaDeviceSynchronize();
    for (size_t k = 0; k < g_checked_host.size(); ++k)
        if (g_checked_host[k].lo == (unsigned long long)c->ws) { g_checked_host.erase(g_checked_host.begin() + (long)k); break; }
    (void)upload_checked_table(c);
    if (c->guard_table) cudaFree(c->guard_table);
    c->guard_table = nullptr; c->registered = false;
}
#else
apms_status register_checked(apms_ctx*) { return APMS_OK; }
void unregister_checked(apms_ctx*) {}
#endif

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
    if (st == DEVICE_BOUNDS) {
        int rec[6] = {0, 0, 0, 0, 0, 0};
        APMS_CUDA(c, cudaMemcpy(rec, c->status(), sizeof rec, cudaMemcpyDeviceToHost));
        const unsigned long long addr = ((unsigned long long)(unsigned)rec[3] << 32) | (unsigned)rec[2];
        const long long off = (long long)(addr - (unsigned long long)c->ws);
        const char* what = "outside this workspace";
        for (const GuardRegion& g : c->guards)
            if (off + rec[4] > (long long)g.off && off < (long long)(g.off + g.bytes)) { what = g.what; break; }
        snprintf(c->err, sizeof c->err, "a checked accessor refused a %s of %d bytes at workspace offset %lld (guard bytes behind: %s); the access was skipped",
                 rec[5] ? "store" : "load", rec[4], off, what);
        return APMS_ERR_BOUNDS;
    }
    if (st != 0) return fail(c, APMS_ERR_TIMEOUT, "a kernel gave up waiting for its own asynchronous copies; the state of this context is undefined");
    return APMS_OK;
}

// The staged server kernel streams slabs of 2048 elements: chunks of at least one slab.
bool use_staged_server(const apms_ctx* c)
{
    if (c->team_mode == APMS_TEAM_CTA || c->team_mode == APMS_TEAM_WARP) return false;
    if (c->L.t.l1) return false;             // the mean-|z| scale exists in the register-staged kernels only
    return c->L.chunk >= kSlab;
}

// Chunks of 128, 256, 512 or 1024 elements: whole chunks per slab, the fused kernel k_server_packed.
bool use_packed_server(const apms_ctx* c)
{
    if (c->team_mode == APMS_TEAM_CTA || c->team_mode == APMS_TEAM_WARP) return false;
    if (c->L.t.l1) return false;
    return c->L.chunk >= kGroup && c->L.chunk < kSlab && kSlab % c->L.chunk == 0;
}

bool use_warp_teams(const apms_ctx* c, int64_t items)
{
    if (c->team_mode == APMS_TEAM_CTA) return false;
    if (c->team_mode == APMS_TEAM_WARP) return true;
    return items / kWarps >= (int64_t)kWarpTeamMinCtasPerSm * c->sms;
}

// Scales of the split chunks [cb, ce) of `rows` workers from first_row on: the range as a vector of its own.
apms_status launch_finalize(apms_ctx* c, int first_row, int rows, int64_t cb, int64_t ce)
{
    const int64_t nchunks = ce - cb;
    const int64_t total = (int64_t)rows * nchunks;
    Tiling t = c->L.t;
    t.d = c->L.d - cb * c->L.chunk;
    k_finalize_scales<<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(c->partial(first_row) + cb * c->L.t.P, c->s(first_row) + cb, rows,
                                                                            nchunks, c->L.Cp, t);
    return launch_check(c, "k_finalize_scales");
}

bool use_fine_worker(const apms_ctx* c)
{
    if (c->team_mode == APMS_TEAM_CTA || c->team_mode == APMS_TEAM_WARP) return false;
    if (c->L.t.l1) return false;             // see use_staged_server
    return (!c->m_is_fp32 || c->variant == APMS_VARIANT_GRADIENT) && c->L.fine_tiles > 0;
}

// Workers i0 .. i0+ni-1 on chunks [cb, ce).
apms_status launch_worker_fine(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni, int64_t cb, int64_t ce)
{
    WorkerFineArgs a;
    a.z = c->z(0); a.dz = c->L.dz;
    a.B = c->B(0); a.Wp = c->L.Wp;
    a.s = c->s(0); a.Cp = c->L.Cp;
    a.partial = c->fine_partial(i0); a.Pp = c->L.fine_Pp;
    a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.d = c->L.d; a.chunk = c->L.chunk;
    a.e0 = cb * c->L.chunk; a.e1 = ce * c->L.chunk < c->L.d ? ce * c->L.chunk : c->L.d;
    a.tile0 = a.e0 / kFineTile; a.tiles = (a.e1 + kFineTile - 1) / kFineTile - a.tile0;
    a.i0 = i0; a.ni = ni;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1;
    a.inv_chunk = (c->L.C < ((int64_t)1 << 20) && c->L.d < ((int64_t)1 << 40)) ? 1.0f / (float)c->L.chunk : 0.0f;
    a.run = c->fine_run;
    if ((int64_t)a.run > a.tiles) a.run = a.tiles < 1 ? 1 : (int)a.tiles;
    const int64_t stretches = (a.tiles + a.run - 1) / a.run;
    const int64_t blocks = stretches * a.run * ni;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (tile, worker) items for one launch");
    a.inv_run = 1.0f / (float)a.run; a.inv_per_stretch = 1.0f / ((float)a.run * (float)ni);
    {
        Timed t(c, APMS_KERNEL_WORKER);
        const bool sendg = c->variant == APMS_VARIANT_GRADIENT;
        if (c->L.fine_words) {                     // chunks below 512 elements: per-word scales and sums
            if (sendg) APMS_DISPATCH_GRAD(gtype, k_worker_fine_words<GT, true><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
            else       APMS_DISPATCH_GRAD(gtype, k_worker_fine_words<GT, false><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
            apms_status st = launch_check(c, "k_worker_fine_words");
            if (st != APMS_OK) return st;
            const int64_t total = (int64_t)ni * (ce - cb);
            k_finalize_words<<<(unsigned)((total + kThreads - 1) / kThreads), kThreads, 0, c->stream>>>(c->fine_partial(i0), c->L.fine_Pp, c->s(i0), c->L.Cp,
                                                                                                    ni, cb, ce - cb, c->L.d, c->L.chunk);
            return launch_check(c, "k_finalize_words");
        }
        if (c->L.fine_split) {
            if (sendg) APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, true, true><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
            else       APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, false, true><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
        } else {
            if (sendg) APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, true, false><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
            else       APMS_DISPATCH_GRAD(gtype, k_worker_fine<GT, false, false><<<(unsigned)blocks, kThreads, 0, c->stream>>>(G, a));
        }
        apms_status st = launch_check(c, "k_worker_fine");
        if (st != APMS_OK) return st;
        const int64_t nchunks = ce - cb;
        const int64_t total = (int64_t)ni * nchunks;
        const int per = c->L.fine_split ? 2 : 1;
        // 512-element pieces a whole chunk can touch: its own, plus one at each end that it shares
        const int64_t slots = c->L.fine_split ? c->L.chunk / kFineSub + 2 : c->L.chunk / kFineSub;
        if (slots > kFineLongSlots) {                 // long chunks: a CTA per (worker, chunk)
            if (total > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (chunk, worker) pairs for one launch");
            k_finalize_fine_cta<<<(unsigned)total, kThreads, 0, c->stream>>>(c->fine_partial(i0), c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks,
                                                                           c->L.d, c->L.chunk, per);
            return launch_check(c, "k_finalize_fine_cta");
        }
        int team = 1;
        while (team < 32 && team < slots) team *= 2;
        const int64_t per_cta = (int64_t)kWarps * (32 / team);
        const unsigned grid = (unsigned)((total + per_cta - 1) / per_cta);
        const double* part = c->fine_partial(i0);
        switch (team) {
        case 1:  k_finalize_fine<1><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        case 2:  k_finalize_fine<2><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        case 4:  k_finalize_fine<4><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        case 8:  k_finalize_fine<8><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        case 16: k_finalize_fine<16><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        default: k_finalize_fine<32><<<grid, kThreads, 0, c->stream>>>(part, c->L.fine_Pp, c->s(i0), c->L.Cp, ni, cb, nchunks, c->L.d, c->L.chunk, per); break;
        }
        st = launch_check(c, "k_finalize_fine");
        if (st != APMS_OK) return st;
    }
    return APMS_OK;
}

// Where the top-k kernels count the routes their chunks took (ints of the status block).
constexpr int kRouteWorker = 16, kRouteServer = 24, kRoutes = 6;

apms_status launch_worker_topk(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni)
{
    TopkWorkerArgs a;
    a.z = c->z(0); a.dz = c->L.dz; a.B = c->B(0); a.Wp = c->L.Wp; a.m32 = c->m();
    a.zbar = c->zbar(); a.Bbar = c->Bbar();
    a.thr = c->s(0); a.hint = c->hint(0); a.learned = c->learned(0); a.route = c->status() + kRouteWorker; a.Cp = c->L.Cp;
    a.d = c->L.d; a.chunk = c->L.chunk; a.C = c->L.C; a.i0 = i0; a.ni = ni;
    a.beta1 = c->beta1; a.omb1 = 1.0f - c->beta1; a.frac = c->topk_frac;
    const int64_t blocks = c->L.C * ni;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (chunk, worker) items for one launch");
    const bool band = 6 * apms_topk_values_per_chunk(c) > kTopkList;       // too many for the one-sided window
    Timed t(c, APMS_KERNEL_WORKER);
    if (c->m_is_fp32) {
        if (band) APMS_DISPATCH_GRAD(gtype, k_topk_worker<GT, true, true><<<(unsigned)blocks, kTopkThreads, 0, c->stream>>>(G, a));
        else      APMS_DISPATCH_GRAD(gtype, k_topk_worker<GT, true, false><<<(unsigned)blocks, kTopkThreads, 0, c->stream>>>(G, a));
    } else {
        if (band) APMS_DISPATCH_GRAD(gtype, k_topk_worker<GT, false, true><<<(unsigned)blocks, kTopkThreads, 0, c->stream>>>(G, a));
        else      APMS_DISPATCH_GRAD(gtype, k_topk_worker<GT, false, false><<<(unsigned)blocks, kTopkThreads, 0, c->stream>>>(G, a));
    }
    return launch_check(c, "k_topk_worker");
}

// Section 3.3 steps 1-2 for workers i0 .. i0+ni-1 on chunks [cb, ce).
apms_status launch_worker(apms_ctx* c, const GradPtrs& G, int gtype, int i0, int ni, int64_t cb, int64_t ce)
{
    if (c->compressor == APMS_COMPRESSOR_TOPK) return launch_worker_topk(c, G, gtype, i0, ni);      // whole vector only (checked by the callers)
    if (ce <= cb) return APMS_OK;
    if (use_fine_worker(c)) return launch_worker_fine(c, G, gtype, i0, ni, cb, ce);
    WorkerArgs a;
    a.z = c->z(0); a.dz = c->L.dz;
    a.B = c->B(0); a.Wp = c->L.Wp;
    a.s = c->s(0); a.Cp = c->L.Cp;
    a.partial = c->partial(0);
    a.m32 = c->m(); a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.t = c->L.t; a.i0 = i0; a.ni = ni;
    a.tile0 = cb * c->L.t.P;
    a.items = (ce - cb) * c->L.t.P * ni;
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
    if (c->L.t.P > 1) return launch_finalize(c, i0, ni, cb, ce);
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

template <int NT>
cudaError_t launch_packed(const ServerStagedArgs& sa, unsigned blocks, size_t smem, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(k_server_packed<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_server_packed<NT><<<blocks, kStagedThreads, smem, stream>>>(sa);
    return cudaSuccess;
}

cudaError_t launch_packed_n(const ServerStagedArgs& sa, unsigned blocks, size_t smem, cudaStream_t stream)
{
    switch (sa.a.n) {
    case 2:  return launch_packed<2>(sa, blocks, smem, stream);
    case 4:  return launch_packed<4>(sa, blocks, smem, stream);
    case 8:  return launch_packed<8>(sa, blocks, smem, stream);
    case 16: return launch_packed<16>(sa, blocks, smem, stream);
    case 32: return launch_packed<32>(sa, blocks, smem, stream);
    default: return launch_packed<0>(sa, blocks, smem, stream);
    }
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

int grid_for(const apms_ctx* c, int64_t items, int per_sm);

// The denominator of the model update, sqrt(v) + eps, is the same in every step of the compression phase
// (v is frozen): it is formed once - the same two rounded operations - and the update kernels of the 1-bit
// path read it in place of v.
apms_status ensure_den(apms_ctx* c)
{
    if (c->den_valid) return APMS_OK;
    k_make_den<<<grid_for(c, c->L.d, 8), kThreads, 0, c->stream>>>(c->v(), c->den(), c->L.d, c->eps);
    apms_status st = launch_check(c, "k_make_den");
    if (st == APMS_OK) c->den_valid = true;
    return st;
}

// Where the server finds the workers' messages: `rows` senders, row j holding sign words and scales
// addressed by ABSOLUTE word / chunk index (a pointer into a shard is shifted back by the caller).
struct ServerSource {
    const uint32_t* B[APMS_MAX_WORKERS];
    const float* s[APMS_MAX_WORKERS];
    int rows;
    // Distance of every row's word 0 from a 16-byte boundary, in words, if all rows share it (what the staged
    // kernel's bulk copies need); -1 otherwise.
    int common_alignment() const
    {
        const int first = (int)(((uintptr_t)B[0] >> 2) & 3u);
        for (int j = 1; j < rows; ++j)
            if ((int)(((uintptr_t)B[j] >> 2) & 3u) != first) return -1;
        return first;
    }
    // rows at a fixed stride from a base
    static ServerSource strided(const uint32_t* B0, int64_t Wp, const float* s0, int64_t Cp, int rows)
    {
        ServerSource src;
        for (int j = 0; j < APMS_MAX_WORKERS; ++j) {
            src.B[j] = j < rows ? B0 + (int64_t)j * Wp : nullptr;
            src.s[j] = j < rows ? s0 + (int64_t)j * Cp : nullptr;
        }
        src.rows = rows;
        return src;
    }
};

// Section 3.3 step 4 for chunks [cb, ce).  With may_fuse and a shape that allows it, steps 5-6 for
// the same chunks run in the same kernel (*applied = true).
apms_status launch_server(apms_ctx* c, const ServerSource& src, int64_t cb, int64_t ce, bool may_fuse, bool* applied)
{
    *applied = false;
    ServerArgs a;
    for (int j = 0; j < APMS_MAX_WORKERS; ++j) { a.Brow[j] = src.B[j]; a.srow[j] = src.s[j]; }
    a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.Sbar = c->Sbar();
    a.partial = c->partial(c->L.n);
    a.t = c->L.t; a.item0 = cb * c->L.t.P; a.items = ce * c->L.t.P; a.n = src.rows; a.nf = (float)src.rows;
    const int64_t count = a.items - a.item0;
    if (count <= 0) return APMS_OK;
    const int row_align = src.common_alignment();
    if (may_fuse && use_packed_server(c) && row_align >= 0 && cb == 0 && ce == c->L.C) {
        // short chunks, several per slab: the fused kernel for them (items are slabs of the whole vector)
        apms_status dst = ensure_den(c);
        if (dst != APMS_OK) return dst;
        ServerStagedArgs sa;
        sa.a = a; sa.status = c->status();
        sa.a.item0 = 0; sa.a.items = (c->L.d + kSlab - 1) / kSlab;
        sa.inv_n = ((a.n & (a.n - 1)) == 0) ? 1.0f / (float)a.n : 0.0f;
        sa.den = c->den(); sa.x = c->x(); sa.lr = c->lr; sa.row_align = row_align;
        const size_t smem = (size_t)kStages * staged_stage_bytes(a.n, true);
        sa.span = (int)(kStagedSpanElems / kSlab);
        const int64_t fill = sa.a.items / (2 * (int64_t)c->sms);       // small problems: keep at least two CTAs per SM
        if (fill < sa.span) sa.span = fill < 1 ? 1 : (int)fill;
        const int64_t ctas = (sa.a.items + sa.span - 1) / sa.span;
        if (ctas > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many slabs for one launch");
        Timed t(c, APMS_KERNEL_SERVER);
        cudaError_t e = launch_packed_n(sa, (unsigned)ctas, smem, c->stream);
        if (e != cudaSuccess) {
            snprintf(c->err, sizeof c->err, "setting up k_server_packed failed: %s", cudaGetErrorString(e));
            return APMS_ERR_CUDA;
        }
        *applied = true;
        return launch_check(c, "k_server_packed");
    }
    const bool staged = use_staged_server(c) && row_align >= 0;
    const bool warp_teams = !staged && use_warp_teams(c, count);
    const int64_t blocks = warp_teams ? (count + kWarps - 1) / kWarps : count;
    if (blocks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunk tiles for one launch");
    {
        Timed t(c, APMS_KERNEL_SERVER);
        if (staged) {
            const bool fused = may_fuse && c->L.t.P == 1;   // the CTA sees the whole chunk, so it knows the new scale
            // chunks cut into tiles, whole vector: steps 5-6 follow `lag` tiles behind in the same kernel
            const bool lagged = may_fuse && c->L.t.P > 1 && cb == 0 && ce == c->L.C && c->team_mode == APMS_TEAM_AUTO;
            if (fused || lagged) {
                apms_status dst = ensure_den(c);
                if (dst != APMS_OK) return dst;
            }
            ServerStagedArgs sa;
            sa.lag = 0; sa.ticket = sa.done = sa.ready = nullptr; sa.epoch = 0;
            if (lagged) {
                // at least the tiles of a chunk (no deadlock, see the kernel); about the resident CTAs more, so that the wait is rare
                sa.lag = (int64_t)c->L.t.P + 3 * (int64_t)c->sms;
                sa.ticket = c->tile_ticket(); sa.done = c->tiles_done(); sa.ready = c->tiles_ready();
                if (++c->tile_epoch == 0) c->tile_epoch = 1;
                sa.epoch = c->tile_epoch;
            }
            sa.a = a; sa.status = c->status();
            sa.inv_n = ((a.n & (a.n - 1)) == 0) ? 1.0f / (float)a.n : 0.0f;
            sa.den = c->den(); sa.x = c->x(); sa.lr = c->lr; sa.row_align = row_align;
            const size_t smem = (size_t)kStages * staged_stage_bytes(a.n, fused) + staged_nb_bytes(c->L.t.tile);
            sa.span = fused ? (int)((kStagedSpanElems + c->L.chunk - 1) / c->L.chunk) : 1;
            const int64_t fill = count / (2 * (int64_t)c->sms);       // small problems: keep at least two CTAs per SM
            if (sa.span > 1 && fill < sa.span) sa.span = fill < 1 ? 1 : (int)fill;
            const int64_t ctas = (count + sa.span - 1) / sa.span + sa.lag;
            if (ctas > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunk tiles for one launch");
            cudaError_t e = fused ? launch_staged_n<true>(sa, (unsigned)ctas, smem, c->stream)
                                  : launch_staged_n<false>(sa, (unsigned)ctas, smem, c->stream);
            if (e != cudaSuccess) {
                snprintf(c->err, sizeof c->err, "setting up k_server_staged failed: %s", cudaGetErrorString(e));
                return APMS_ERR_CUDA;
            }
            *applied = fused || lagged;
            if (lagged) return launch_check(c, "k_server_staged");      // the chunks' scales are stored by their last tiles
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
    apms_status dst = ensure_den(c);
    if (dst != APMS_OK) return dst;
    ApplyArgs a;
    a.Bbar = c->Bbar(); a.Sbar = c->Sbar(); a.den = c->den(); a.x = c->x();
    a.d = c->L.d; a.chunk = c->L.chunk; a.lr = c->lr;
    a.inv_chunk = (c->L.C < ((int64_t)1 << 20) && c->L.d < ((int64_t)1 << 40)) ? 1.0f / (float)c->L.chunk : 0.0f;
    Timed t(c, APMS_KERNEL_APPLY);
    k_apply<<<(unsigned)((c->L.d + kApplyTile - 1) / kApplyTile), kThreads, 0, c->stream>>>(a);
    return launch_check(c, "k_apply");
}

// Top-k: may the server leave the elements it does not keep alone?  Their momentum is +0, and
// x - (lr * 0) / (sqrt(v) + eps) returns x itself iff lr is not negative (nor -0), eps > 0 and v is neither
// negative nor NaN.  v is looked at once after it last changed (one pass and a synchronisation).
apms_status topk_sparse_update_allowed(apms_ctx* c, bool* allowed)
{
    *allowed = false;
    if (!(c->eps > 0.0f) || signbit(c->lr)) return APMS_OK;
    if (!c->v_checked) {
        int* flag = c->status() + 1;
        int host_flag = 0;
        APMS_CUDA(c, cudaMemsetAsync(flag, 0, sizeof(int), c->stream));
        k_any_negative_or_nan<<<grid_for(c, c->L.d, 8), kThreads, 0, c->stream>>>(c->v(), c->L.d, flag);
        apms_status st = launch_check(c, "k_any_negative_or_nan");
        if (st != APMS_OK) return st;
        APMS_CUDA(c, cudaMemcpyAsync(&host_flag, flag, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
        APMS_CUDA(c, cudaStreamSynchronize(c->stream));
        c->v_plain = host_flag == 0;
        c->v_checked = true;
    }
    *allowed = c->v_plain;
    return APMS_OK;
}

// The momentum, spelled out in binary32 into out[0..count) from where it lives when !m_is_fp32.
apms_status launch_materialise_momentum(apms_ctx* c, float* out, int64_t first, int64_t count)
{
    const int grid = grid_for(c, count, 8);
    if (c->compressor == APMS_COMPRESSOR_TOPK)
        k_materialise_momentum_topk<<<grid, kThreads, 0, c->stream>>>(c->zbar(), c->Bbar(), out, first, count);
    else
        k_materialise_momentum<<<grid, kThreads, 0, c->stream>>>(c->Bbar(), c->Sbar(), out, first, count, c->L.chunk);
    return launch_check(c, "k_materialise_momentum");
}

apms_status launch_server_and_apply(apms_ctx* c)
{
    if (c->compressor == APMS_COMPRESSOR_TOPK) {       // one kernel: sparse average, recompression, momentum, model update
        bool sparse = false;
        apms_status sst = topk_sparse_update_allowed(c, &sparse);
        if (sst != APMS_OK) return sst;
        TopkServerArgs a;
        a.sparse = sparse ? 1 : 0;
        a.z = c->z(0); a.dz = c->L.dz; a.B = c->B(0); a.Wp = c->L.Wp;
        a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.m32 = c->m(); a.thr = c->Sbar(); a.hint = c->hint(c->L.n); a.learned = c->learned(c->L.n); a.route = c->status() + kRouteServer; a.v = c->v(); a.x = c->x();
        a.d = c->L.d; a.chunk = c->L.chunk; a.n = c->L.n; a.nf = (float)c->L.n; a.lr = c->lr; a.eps = c->eps;
        a.frac = c->topk_frac; a.c0 = 0;
        if (c->L.C > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunks for one launch");
        Timed t(c, APMS_KERNEL_SERVER);
        k_topk_server<<<(unsigned)c->L.C, kTopkThreads, 0, c->stream>>>(a);
        apms_status st = launch_check(c, "k_topk_server");
        if (st != APMS_OK) return st;
        c->m_is_fp32 = !sparse;    // sparse update: the momentum stays implicit in (zbar, Bbar)
        c->csteps += 1;
        return APMS_OK;
    }
    const ServerSource own = ServerSource::strided(c->B(0), c->L.Wp, c->s(0), c->L.Cp, c->L.n);
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
    return make_layout(d, n, chunk, &L, g_guard_bytes) ? L.total : 0;
}

apms_status apms_create(apms_ctx** out, int64_t d, int n, float beta1, float beta2, float eps,
                        float lr, int64_t chunk)
{
    if (!out) { snprintf(g_create_error, sizeof g_create_error, "out is NULL"); return APMS_ERR_INVALID_ARG; }
    *out = nullptr;
    Layout L;
    std::vector<GuardRegion> guards;
    if (!make_layout(d, n, chunk, &L, g_guard_bytes, &guards)) {
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
    c->L = L; c->guards.swap(guards); c->beta1 = beta1; c->beta2 = beta2; c->eps = eps; c->lr = lr;
    c->t = 0; c->phase = APMS_PHASE_CREATED; c->m_is_fp32 = true; c->v_checked = false; c->v_plain = false; c->den_valid = false;
    c->ws = nullptr; c->ws_bytes = 0; c->owns_ws = false;
    c->stream = nullptr; c->copy_stream = nullptr; c->host_path_ready = false;
    c->device = dev; c->sms = sms; c->timing = false; c->launches = 0; c->err[0] = 0;
    c->team_mode = APMS_TEAM_AUTO; c->guard_table = nullptr; c->registered = false;
    c->steps = 0; c->has_sched = false; c->substep = 0; c->worker_chunks = 0; c->variant = APMS_VARIANT_MOMENTUM; c->csteps = 0;
    c->compressor = APMS_COMPRESSOR_ONEBIT; c->topk_frac = 0.01;
    c->fine_run = kFineRunDefault;
    c->tile_epoch = 0;
    if ((int64_t)c->fine_run > L.fine_tiles && L.fine_tiles > 0) c->fine_run = (int)L.fine_tiles;
    *out = c;
    return APMS_OK;
}

apms_status apms_bind(apms_ctx* c, void* workspace_dev, size_t bytes, void* cuda_stream)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "apms_bind must precede apms_set_params");
    if (c->ws) return fail(c, APMS_ERR_BAD_STATE, "a workspace is already attached");
    if (!workspace_dev && bytes == 0) {                // the stream only: the library allocates the workspace itself
        c->stream = (cudaStream_t)cuda_stream;
        return APMS_OK;
    }
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
    APMS_CUDA(c, cudaMemsetAsync(c->m(), 0, (size_t)c->L.d * 4, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->v(), 0, (size_t)c->L.d * 4, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->status(), 0, 256, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->tile_ticket(), 0, (64 + 2 * (size_t)c->L.Cp) * 4, c->stream));
    st = fill_guards(c);
    if (st != APMS_OK) return st;
    st = register_checked(c);
    if (st != APMS_OK) return st;
    if (!src_is_device) APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    c->t = 0; c->steps = 0; c->csteps = 0; c->substep = 0; c->worker_chunks = 0; c->phase = APMS_PHASE_WARMUP; c->m_is_fp32 = true;
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
    if (!c->guards.empty()) {                      // the one memset above ran over the guard regions in between
        apms_status gst = fill_guards(c);
        if (gst != APMS_OK) return gst;
    }
    c->phase = APMS_PHASE_COMPRESSED;
    c->m_is_fp32 = true;
    c->v_checked = false;
    c->den_valid = false;
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
    st = launch_worker(c, G, (int)type, 0, c->L.n, 0, c->L.C);
    if (st != APMS_OK) return st;
    return launch_server_and_apply(c);
}

apms_status apms_worker_phase(apms_ctx* c, const void* const* grads_dev, apms_grad_type type)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    return apms_worker_phase_range(c, grads_dev, type, 0, c->L.C);
}

apms_status apms_worker_phase_range(apms_ctx* c, const void* const* grads_dev, apms_grad_type type, int64_t chunk_begin, int64_t chunk_end)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_worker_phase needs the COMPRESSED phase (call apms_freeze_v first)");
    if (c->substep > 1 || (c->substep == 1 && c->worker_chunks >= c->L.C))
        return fail(c, APMS_ERR_BAD_STATE, "the worker phase of this step is complete (continue with the server and apply phases)");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    if (c->compressor == APMS_COMPRESSOR_TOPK) {
        if (chunk_begin != 0 || chunk_end != c->L.C) return fail(c, APMS_ERR_INVALID_ARG, "with the top-k compressor the worker phase covers the whole vector in one call");
        if (c->variant != APMS_VARIANT_MOMENTUM) return fail(c, APMS_ERR_BAD_STATE, "top-k runs with the momentum variant");
        bool sparse = false;
        apms_status sst = topk_sparse_update_allowed(c, &sparse);
        if (sst != APMS_OK) return sst;
        if (!sparse) return fail(c, APMS_ERR_BAD_STATE, "the phase-wise top-k step needs lr >= +0, eps > 0 and a variance without negative or NaN entries");
    }
    if (c->worker_chunks + (chunk_end - chunk_begin) > c->L.C) return fail(c, APMS_ERR_INVALID_ARG, "the ranges of one step's worker phase cover more chunks than there are");
    GradPtrs G;
    apms_status st = check_grads(c, grads_dev, (int)type, &G, c->L.n);
    if (st != APMS_OK) return st;
    st = launch_worker(c, G, (int)type, 0, c->L.n, chunk_begin, chunk_end);
    if (st != APMS_OK) return st;
    c->worker_chunks += chunk_end - chunk_begin;
    c->substep = 1;
    return APMS_OK;
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
    if (c->substep < 1 || c->worker_chunks < c->L.C) return fail(c, APMS_ERR_BAD_STATE, "apms_server_phase follows a complete worker phase (every chunk once)");
    if (c->compressor != APMS_COMPRESSOR_ONEBIT) return fail(c, APMS_ERR_BAD_STATE, "top-k messages go through apms_topk_server_phase");
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
    const ServerSource src = ServerSource::strided(bits_rows_dev - first_elem / 32, row_words, scale_rows_dev - chunk_begin, row_scales, rows);
    bool applied = false;
    apms_status st = launch_server(c, src, chunk_begin, chunk_end, false, &applied);
    if (st == APMS_OK) c->substep = 2;
    return st;
}

apms_status apms_server_phase_rows(apms_ctx* c, const uint32_t* const* bits_rows, const float* const* scale_rows, int rows,
                                   int64_t chunk_begin, int64_t chunk_end)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_server_phase_rows needs the COMPRESSED phase");
    if (c->substep < 1 || c->worker_chunks < c->L.C) return fail(c, APMS_ERR_BAD_STATE, "apms_server_phase_rows follows a complete worker phase (every chunk once)");
    if (c->compressor != APMS_COMPRESSOR_ONEBIT) return fail(c, APMS_ERR_BAD_STATE, "top-k messages go through apms_topk_server_phase");
    if (!bits_rows || !scale_rows) return fail(c, APMS_ERR_INVALID_ARG, "a pointer array is NULL");
    if (rows < 1 || rows > APMS_MAX_WORKERS) return fail(c, APMS_ERR_INVALID_ARG, "rows must be between 1 and APMS_MAX_WORKERS");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    const int64_t first_elem = chunk_begin * c->L.chunk;
    ServerSource src;
    for (int j = 0; j < APMS_MAX_WORKERS; ++j) { src.B[j] = nullptr; src.s[j] = nullptr; }
    for (int j = 0; j < rows; ++j) {
        if (!bits_rows[j] || !scale_rows[j]) return fail(c, APMS_ERR_INVALID_ARG, "a message pointer is NULL");
        // kernels index by absolute word / chunk: shift the row's pointers back to where index 0 would be
        src.B[j] = bits_rows[j] - first_elem / 32;
        src.s[j] = scale_rows[j] - chunk_begin;
        if (((uintptr_t)src.B[j] & 3u) != 0) return fail(c, APMS_ERR_INVALID_ARG, "a sign-word row is not 4-byte aligned");
    }
    src.rows = rows;
    bool applied = false;
    apms_status st = launch_server(c, src, chunk_begin, chunk_end, false, &applied);
    if (st == APMS_OK) c->substep = 2;
    return st;
}

apms_status apms_put_server_range(apms_ctx* c, uint32_t* dst_bits_dev, float* dst_scales_dev, int64_t chunk_begin, int64_t chunk_end)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED || c->substep != 2) return fail(c, APMS_ERR_BAD_STATE, "apms_put_server_range follows the server phase of a phase-wise step");
    if (!dst_bits_dev || !dst_scales_dev) return fail(c, APMS_ERR_INVALID_ARG, "a destination pointer is NULL");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    if (chunk_begin == chunk_end) return APMS_OK;
    const int64_t first_elem = chunk_begin * c->L.chunk;
    const int64_t last_elem = chunk_end * c->L.chunk < c->L.d ? chunk_end * c->L.chunk : c->L.d;
    const int64_t w0 = first_elem / 32, w1 = (last_elem + 31) / 32;
    APMS_CUDA(c, cudaMemcpyAsync(dst_bits_dev + w0, c->Bbar() + w0, (size_t)(w1 - w0) * 4, cudaMemcpyDefault, c->stream));
    APMS_CUDA(c, cudaMemcpyAsync(dst_scales_dev + chunk_begin, c->Sbar() + chunk_begin, (size_t)(chunk_end - chunk_begin) * 4,
                                 cudaMemcpyDefault, c->stream));
    return APMS_OK;
}

apms_status apms_message_offsets(apms_ctx* c, int worker, size_t* bits_offset, size_t* scales_offset)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (worker < -1 || worker >= c->L.n) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range (-1 = the server's message)");
    apms_status st = ensure_workspace(c);
    if (st != APMS_OK) return st;
    if (bits_offset) *bits_offset = (size_t)((char*)(worker < 0 ? c->Bbar() : c->B(worker)) - c->ws);
    if (scales_offset) *scales_offset = (size_t)((char*)(worker < 0 ? c->Sbar() : c->s(worker)) - c->ws);
    return APMS_OK;
}

apms_status apms_topk_route_counts(apms_ctx* c, int64_t worker_routes[6], int64_t server_routes[6])
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!worker_routes || !server_routes) return fail(c, APMS_ERR_INVALID_ARG, "an output array is NULL");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "no workspace yet");
    int counts[16];
    static_assert(kRouteServer - kRouteWorker + kRoutes <= 16 && kRouteServer + kRoutes <= 64, "the counters lie inside the status block");
    APMS_CUDA(c, cudaMemcpyAsync(counts, c->status() + kRouteWorker, sizeof counts, cudaMemcpyDeviceToHost, c->stream));
    APMS_CUDA(c, cudaMemsetAsync(c->status() + kRouteWorker, 0, sizeof counts, c->stream));
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    for (int r = 0; r < kRoutes; ++r) { worker_routes[r] = counts[r]; server_routes[r] = counts[kRouteServer - kRouteWorker + r]; }
    return APMS_OK;
}

int64_t apms_topk_values_per_chunk(const apms_ctx* c)
{
    if (!c || c->compressor != APMS_COMPRESSOR_TOPK) return 0;
    long long K = (long long)ceil(c->topk_frac * (double)c->L.chunk);
    if (K < 1) K = 1;
    if (K > c->L.chunk) K = c->L.chunk;
    return (int64_t)K;
}

apms_status apms_topk_pack_values(apms_ctx* c, int worker, int64_t chunk_begin, int64_t chunk_end, float* vals_dev)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->compressor != APMS_COMPRESSOR_TOPK) return fail(c, APMS_ERR_BAD_STATE, "the context does not run the top-k compressor");
    if (c->phase != APMS_PHASE_COMPRESSED || c->substep < 1) return fail(c, APMS_ERR_BAD_STATE, "apms_topk_pack_values belongs to a phase-wise step (after apms_worker_phase)");
    if (worker < -1 || worker >= c->L.n) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range (-1 = the server's message)");
    if (worker < 0 && c->substep < 2) return fail(c, APMS_ERR_BAD_STATE, "the server's message exists after apms_topk_server_phase");
    if (!vals_dev) return fail(c, APMS_ERR_INVALID_ARG, "vals_dev is NULL");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    if (chunk_begin == chunk_end) return APMS_OK;
    TopkPackArgs a;
    a.z = worker < 0 ? c->zbar() : c->z(worker); a.dz = c->L.dz;
    a.mask = worker < 0 ? c->Bbar() : c->B(worker); a.Wp = c->L.Wp;
    a.vals = vals_dev; a.vstride = 0;
    a.d = c->L.d; a.chunk = c->L.chunk; a.c0 = chunk_begin; a.nchunks = chunk_end - chunk_begin;
    a.kmax = (int)apms_topk_values_per_chunk(c);
    if (a.nchunks > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunks for one launch");
    k_topk_pack<<<(unsigned)a.nchunks, kThreads, 0, c->stream>>>(a);
    return launch_check(c, "k_topk_pack");
}

size_t apms_topk_server_scratch_bytes(const apms_ctx* c, int rows, int64_t chunk_begin, int64_t chunk_end)
{
    if (!c || rows < 1 || chunk_begin < 0 || chunk_end > c->L.C || chunk_begin >= chunk_end) return 0;
    const int64_t elems = (chunk_end - chunk_begin) * c->L.chunk;
    return (size_t)rows * round_up((size_t)elems, 64) * 4;
}

apms_status apms_topk_server_phase(apms_ctx* c, const uint32_t* mask_rows_dev, int64_t row_words, const float* val_rows_dev,
                                   int64_t row_vals, int rows, int64_t chunk_begin, int64_t chunk_end, void* scratch_dev, size_t scratch_bytes)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->compressor != APMS_COMPRESSOR_TOPK) return fail(c, APMS_ERR_BAD_STATE, "the context does not run the top-k compressor");
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_topk_server_phase needs the COMPRESSED phase");
    if (c->substep < 1 || c->worker_chunks < c->L.C) return fail(c, APMS_ERR_BAD_STATE, "apms_topk_server_phase follows apms_worker_phase");
    if (!mask_rows_dev || !val_rows_dev || !scratch_dev) return fail(c, APMS_ERR_INVALID_ARG, "a buffer pointer is NULL");
    if (rows < 1 || rows > APMS_MAX_WORKERS) return fail(c, APMS_ERR_INVALID_ARG, "rows must be between 1 and APMS_MAX_WORKERS");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    if (chunk_begin == chunk_end) { c->substep = 2; return APMS_OK; }
    const int64_t nchunks = chunk_end - chunk_begin;
    const int kmax = (int)apms_topk_values_per_chunk(c);
    const int64_t first_elem = chunk_begin * c->L.chunk;
    const int64_t last_elem = chunk_end * c->L.chunk < c->L.d ? chunk_end * c->L.chunk : c->L.d;
    const int64_t need_words = (last_elem - first_elem + 31) / 32;
    if (row_words < need_words || row_vals < nchunks * kmax)
        return fail(c, APMS_ERR_INVALID_ARG, "rows too short: row_words must cover the range's mask words, row_vals its chunks times apms_topk_values_per_chunk");
    if (scratch_bytes < apms_topk_server_scratch_bytes(c, rows, chunk_begin, chunk_end) || ((uintptr_t)scratch_dev & 15u))
        return fail(c, APMS_ERR_INVALID_ARG, "scratch too small (apms_topk_server_scratch_bytes) or not 16-byte aligned");
    if (nchunks * rows > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many (row, chunk) pairs for one launch");
    bool sparse = false;
    apms_status st = topk_sparse_update_allowed(c, &sparse);
    if (st != APMS_OK) return st;
    if (!sparse) return fail(c, APMS_ERR_BAD_STATE, "the phase-wise top-k step needs lr >= +0, eps > 0 and a variance without negative or NaN entries");
    const int64_t dstride = (int64_t)round_up((size_t)(nchunks * c->L.chunk), 64);
    TopkUnpackArgs u;
    u.mask = mask_rows_dev; u.row_words = row_words; u.vals = val_rows_dev; u.row_vals = row_vals;
    u.dense = (float*)scratch_dev; u.dstride = dstride;
    u.d = c->L.d; u.chunk = c->L.chunk; u.c0 = chunk_begin; u.nchunks = nchunks; u.kmax = kmax;
    {
        Timed t(c, APMS_KERNEL_SERVER);
        k_topk_unpack<<<(unsigned)(nchunks * rows), kThreads, 0, c->stream>>>(u);
        st = launch_check(c, "k_topk_unpack");
        if (st != APMS_OK) return st;
        // the server kernel addresses rows by absolute element / word: shift the received rows back to where index 0 would be
        TopkServerArgs a;
        a.sparse = 1;
        a.z = (const float*)scratch_dev - first_elem; a.dz = dstride;
        a.B = mask_rows_dev - first_elem / 32; a.Wp = row_words;
        a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.m32 = c->m(); a.thr = c->Sbar(); a.hint = c->hint(c->L.n); a.learned = c->learned(c->L.n); a.route = c->status() + kRouteServer; a.v = c->v(); a.x = c->x();
        a.d = c->L.d; a.chunk = c->L.chunk; a.n = rows; a.nf = (float)rows; a.lr = c->lr; a.eps = c->eps;
        a.frac = c->topk_frac; a.c0 = chunk_begin;
        k_topk_server<<<(unsigned)nchunks, kTopkThreads, 0, c->stream>>>(a);
        st = launch_check(c, "k_topk_server");
        if (st != APMS_OK) return st;
    }
    c->substep = 2;
    return APMS_OK;
}

apms_status apms_topk_put_server_range(apms_ctx* c, const uint32_t* mask_words_dev, const float* vals_dev, int64_t chunk_begin, int64_t chunk_end)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->compressor != APMS_COMPRESSOR_TOPK) return fail(c, APMS_ERR_BAD_STATE, "the context does not run the top-k compressor");
    if (c->phase != APMS_PHASE_COMPRESSED || c->substep < 1 || c->worker_chunks < c->L.C)
        return fail(c, APMS_ERR_BAD_STATE, "apms_topk_put_server_range belongs to a phase-wise step (after apms_worker_phase)");
    if (!mask_words_dev || !vals_dev) return fail(c, APMS_ERR_INVALID_ARG, "a buffer pointer is NULL");
    if (chunk_begin < 0 || chunk_end > c->L.C || chunk_begin > chunk_end) return fail(c, APMS_ERR_INVALID_ARG, "chunk range out of bounds");
    if (chunk_begin == chunk_end) { c->substep = 2; return APMS_OK; }
    if (chunk_end - chunk_begin > 0x7fffffff) return fail(c, APMS_ERR_INVALID_ARG, "too many chunks for one launch");
    TopkPutArgs a;
    a.mask = mask_words_dev; a.vals = vals_dev;
    a.zbar = c->zbar(); a.Bbar = c->Bbar(); a.v = c->v(); a.x = c->x();
    a.d = c->L.d; a.chunk = c->L.chunk; a.c0 = chunk_begin;
    a.kmax = (int)apms_topk_values_per_chunk(c); a.lr = c->lr; a.eps = c->eps;
    Timed t(c, APMS_KERNEL_APPLY);
    k_topk_put<<<(unsigned)(chunk_end - chunk_begin), kThreads, 0, c->stream>>>(a);
    apms_status st = launch_check(c, "k_topk_put");
    if (st == APMS_OK) c->substep = 2;
    return st;
}

apms_status apms_ipc_export(apms_ctx* c, void* handle_out)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (!handle_out) return fail(c, APMS_ERR_INVALID_ARG, "handle_out is NULL");
    apms_status st = ensure_workspace(c);
    if (st != APMS_OK) return st;
    if (!c->owns_ws) return fail(c, APMS_ERR_BAD_STATE, "only a workspace the library allocated itself can be exported (do not call apms_bind)");
    static_assert(sizeof(cudaIpcMemHandle_t) == APMS_IPC_HANDLE_BYTES, "handle size");
    cudaIpcMemHandle_t h;
    APMS_CUDA(c, cudaIpcGetMemHandle(&h, c->ws));
    memcpy(handle_out, &h, sizeof h);
    return APMS_OK;
}

apms_status apms_ipc_open(const void* handle, void** base_dev)
{
    if (!handle || !base_dev) return APMS_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle, sizeof h);
    void* p = nullptr;
    const cudaError_t e = cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess);
    if (e != cudaSuccess) {
        snprintf(g_create_error, sizeof g_create_error, "cudaIpcOpenMemHandle failed: %s", cudaGetErrorString(e));
        (void)cudaGetLastError();
        return APMS_ERR_CUDA;
    }
    *base_dev = p;
    return APMS_OK;
}

apms_status apms_ipc_close(void* base_dev)
{
    if (!base_dev) return APMS_ERR_INVALID_ARG;
    const cudaError_t e = cudaIpcCloseMemHandle(base_dev);
    if (e != cudaSuccess) {
        snprintf(g_create_error, sizeof g_create_error, "cudaIpcCloseMemHandle failed: %s", cudaGetErrorString(e));
        (void)cudaGetLastError();
        return APMS_ERR_CUDA;
    }
    return APMS_OK;
}

apms_status apms_apply_phase(apms_ctx* c)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "apms_apply_phase needs the COMPRESSED phase");
    if (c->substep != 2) return fail(c, APMS_ERR_BAD_STATE, "apms_apply_phase follows apms_server_phase");
    if (c->compressor == APMS_COMPRESSOR_TOPK) {
        // the kept elements were updated where their server range was computed (apms_topk_server_phase) or taken
        // over (apms_topk_put_server_range); the momentum stays implicit in (zbar, mask)
        c->m_is_fp32 = false;
        c->csteps += 1;
        c->substep = 0; c->worker_chunks = 0;
        return APMS_OK;
    }
    apms_status st = launch_apply(c);
    if (st != APMS_OK) return st;
    c->m_is_fp32 = c->variant == APMS_VARIANT_GRADIENT;
    c->csteps += 1;
    c->substep = 0; c->worker_chunks = 0;
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
        apms_status st = launch_worker(c, G, (int)type, i, 1, 0, c->L.C);
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
            apms_status mst = launch_materialise_momentum(c, c->stage(0), first, count);
            if (mst != APMS_OK) return mst;
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
    case APMS_STATE_V: dst = c->v(); c->v_checked = false; c->den_valid = false; break;
    case APMS_STATE_M: dst = c->m(); c->m_is_fp32 = true; break;
    case APMS_STATE_WORKER_ERR:
        if (worker < 0 || worker >= c->L.n) return fail(c, APMS_ERR_INVALID_ARG, "worker index out of range");
        if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "errors exist only in the COMPRESSED phase");
        // delta = z - (+-0) = z: store the error as z with all scales of this worker zero
        APMS_CUDA(c, cudaMemsetAsync(c->s(worker), 0, (size_t)c->L.C * 4, c->stream));
        if (c->compressor == APMS_COMPRESSOR_TOPK)      // top-k: delta = z - (mask ? z : 0) = z with an empty mask
            APMS_CUDA(c, cudaMemsetAsync(c->B(worker), 0, (size_t)c->L.W * 4, c->stream));
        dst = c->z(worker);
        break;
    case APMS_STATE_SERVER_ERR:
        if (c->phase != APMS_PHASE_COMPRESSED) return fail(c, APMS_ERR_BAD_STATE, "errors exist only in the COMPRESSED phase");
        if (!c->m_is_fp32) {   // Sbar (top-k: the mask) is about to be zeroed: move the momentum it encodes to binary32 first
            apms_status mst = launch_materialise_momentum(c, c->m(), 0, c->L.d);
            if (mst != APMS_OK) return mst;
            c->m_is_fp32 = true;
        }
        APMS_CUDA(c, cudaMemsetAsync(c->Sbar(), 0, (size_t)c->L.C * 4, c->stream));
        if (c->compressor == APMS_COMPRESSOR_TOPK)
            APMS_CUDA(c, cudaMemsetAsync(c->Bbar(), 0, (size_t)c->L.W * 4, c->stream));
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
    if (phase == APMS_PHASE_WARMUP && !c->m_is_fp32) {
        // Adam reads the binary32 momentum: spell out the one held as a server message first
        apms_status st = launch_materialise_momentum(c, c->m(), 0, c->L.d);
        if (st != APMS_OK) return st;
        c->m_is_fp32 = true;
    }
    c->t = t; c->phase = phase; c->substep = 0; c->worker_chunks = 0;
    return APMS_OK;
}

apms_status apms_set_step(apms_ctx* c, int64_t steps)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    if (steps < 0) return fail(c, APMS_ERR_INVALID_ARG, "the step count cannot be negative");
    c->steps = steps;
    // compression-phase steps among them: what fixes the variant and the compressor
    c->csteps = (c->phase == APMS_PHASE_COMPRESSED && steps > (int64_t)c->t) ? steps - (int64_t)c->t : 0;
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
    a.B = c->B(0); a.Wp = c->L.Wp; a.Bbar = c->Bbar(); a.topk = c->compressor == APMS_COMPRESSOR_TOPK ? 1 : 0;
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
        st = launch_materialise_momentum(c, c->m(), 0, c->L.d);
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

apms_status apms_set_guard_bytes(size_t bytes)
{
    if (bytes % 256 != 0 || bytes > ((size_t)1 << 20)) {
        snprintf(g_create_error, sizeof g_create_error, "guard bytes must be a multiple of 256, at most 1 MiB");
        return APMS_ERR_INVALID_ARG;
    }
    g_guard_bytes = bytes;
    return APMS_OK;
}

apms_status apms_check_guards(apms_ctx* c, int64_t* bad_offset)
{
    if (!c) return APMS_ERR_INVALID_ARG;
    if (bad_offset) *bad_offset = -1;
    if (c->guards.empty()) return fail(c, APMS_ERR_BAD_STATE, "this context was created without guard bytes (apms_set_guard_bytes)");
    if (c->phase == APMS_PHASE_CREATED || !c->ws) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    std::vector<unsigned char> host;
    for (const GuardRegion& g : c->guards) {
        host.resize(g.bytes);
        APMS_CUDA(c, cudaMemcpy(host.data(), c->ws + g.off, g.bytes, cudaMemcpyDeviceToHost));
        for (size_t k = 0; k < g.bytes; ++k) {
            if (host[k] != (unsigned char)kGuardByte) {
                if (bad_offset) *bad_offset = (int64_t)(g.off + k);
                snprintf(c->err, sizeof c->err, "guard bytes behind %s were overwritten: workspace offset %zu (byte %zu of the %zu guard bytes there)",
                         g.what, g.off + k, k, g.bytes);
                return APMS_ERR_BOUNDS;
            }
        }
    }
    return device_status_check(c);
}

int apms_build_is_checked(void)
{
#ifdef APMS_BOUNDS_CHECK
    return 1;
#else
    return 0;
#endif
}

apms_status apms_selftest_bounds(apms_ctx* c)
{
    if (!c) return APMS_ERR_INVALID_ARG;
#ifdef APMS_BOUNDS_CHECK
    if (c->guards.empty()) return fail(c, APMS_ERR_BAD_STATE, "the self-test needs the guard layout (apms_set_guard_bytes before apms_create)");
    if (c->phase == APMS_PHASE_CREATED) return fail(c, APMS_ERR_BAD_STATE, "call apms_set_params first");
    // a checked 16-byte store to the first whole 16 bytes behind x's d elements: inside the guard bytes that follow x
    float* target = c->x() + (c->L.d + 3) / 4 * 4;
    k_selftest_bounds<<<1, 32, 0, c->stream>>>(target);
    apms_status st = launch_check(c, "k_selftest_bounds");
    if (st != APMS_OK) return st;
    APMS_CUDA(c, cudaStreamSynchronize(c->stream));
    st = device_status_check(c);
    APMS_CUDA(c, cudaMemsetAsync(c->status(), 0, 256, c->stream));
    if (st != APMS_ERR_BOUNDS) return fail(c, APMS_ERR_BAD_STATE, "the checked accessor did not refuse a store into guard bytes");
    int64_t bad = -1;
    st = apms_check_guards(c, &bad);           // the refused store must not have happened
    if (st != APMS_OK) return st;
    return APMS_OK;
#else
    return fail(c, APMS_ERR_BAD_STATE, "this library was built without checked accessors (-DAPMS_BOUNDS_CHECK)");
#endif
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
    unregister_checked(c);
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


#include "noalloc.cuh"
