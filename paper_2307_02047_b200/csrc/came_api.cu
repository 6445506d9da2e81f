// Host side of the C ABI declared in include/came_b200.h: argument validation,
// launch planning (tile list over all tensors), workspace layout, and the
// per-step kernel launches.  All arithmetic of Algorithm 2 is in came_kernels.cuh.
#include "../../include/came_b200.h"
#include "came_kernels.cuh"
#include "came_pipelined.cuh"
#include "came_stream.cuh"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using came::TensorDev;
using came::Tile;
using came::StepConsts;

namespace {

constexpr int kMaxPhases = 5;
constexpr int kProfSlots = 128;        // profiled steps kept for averaging
const char* const kPhaseNames[kMaxPhases] = {
    "p1_reduce_g2", "p2_sum_u2", "p3_momentum_instability", "p4_apply", "p34_adafactor_apply"};

thread_local std::string g_create_error;
// Tuning knobs (came_tune): process-wide, each one an atomic so that a knob set on one thread
// is read whole on another; a context reads them once, while it is being created.
std::atomic<long long> g_tile_elems_override{0};   // came_tune(CAME_TUNE_TILE_ELEMS)
std::atomic<bool> g_use_pdl{true};                 // came_tune(CAME_TUNE_PDL)
std::atomic<long long> g_sched_group_bytes{0};     // came_tune(CAME_TUNE_SCHED_GROUP_BYTES); 0 = one group
std::atomic<long long> g_host_group_bytes{1ll << 30};   // came_tune(CAME_TUNE_HOST_GROUP_BYTES)

std::atomic<int> g_schedule{0};                    // came_tune(CAME_TUNE_SCHEDULE): 0 auto, 1 phase grids, 2 pipelined
std::atomic<long long> g_pipe_tile_elems{0};       // came_tune(CAME_TUNE_PIPE_TILE_ELEMS); 0 = default
std::atomic<long long> g_pipe_group_bytes{0};      // came_tune(CAME_TUNE_PIPE_GROUP_BYTES); 0 = default
std::atomic<long long> g_pipe_wait_ns{0};          // came_tune(CAME_TUNE_PIPE_WAIT_NS); 0 = default (2 s)
std::atomic<long long> g_pipe_order{0};            // came_tune(CAME_TUNE_PIPE_ORDER)
constexpr long long kPipeTileElemsDefault = 32768;
constexpr long long kPipeGroupBytesDefault = 48ll << 20;
constexpr long long kPipeWaitNsDefault = 2000000000ll;

std::atomic<int> g_p1_stream{0};                   // came_tune(CAME_TUNE_P1_STREAM): 0 default (off), 1 off, 2 on
std::atomic<int> g_p1_stream_ring{0};              // came_tune(CAME_TUNE_P1_STREAM_RING): batches in the ring; 0 = default
constexpr int kP1StreamRingDefault = 2;

std::atomic<bool> g_f32_vec8{true};                // came_tune(CAME_TUNE_F32_VEC8)
inline bool g_f32_vec8_ok(bool bf) { return bf || g_f32_vec8; }

struct Plan {
    int vec = 1, tx = 256, tr = 0, n_rb = 0, n_cb = 0, n_seg = 0, n_parts = 0, kind = 0;
    int n_grp = 0;
    size_t counters() const { return static_cast<size_t>(n_rb) + n_cb + 2 + static_cast<size_t>(n_grp) * n_cb; }
};

inline long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }
inline long long round_up(long long a, long long b) { return ceil_div(a, b) * b; }

// Tile geometry of one tensor.  A tile is `tr` rows by `tx * vec` columns; a block of 256
// threads covers it with tx threads across the columns and 256/tx row groups.
Plan plan_tensor(long long rows, long long cols, int ndim, int dtype, bool aligned32,
                 long long target)
{
    Plan p;
    const bool bf = dtype == CAME_BF16;
    if (ndim == 1) {
        p.kind = bf ? came::kBF16x1 : came::kF32x1;
        p.n_parts = static_cast<int>(ceil_div(rows, came::kVecChunk));
        return p;
    }
    // 8 elements per thread (256-bit fp32 accesses) when rows start 32-byte aligned, else 4 for
    // fp32 gradients (128-bit), else one element at a time
    if (cols % 8 == 0 && aligned32 && g_f32_vec8_ok(bf)) {
        p.vec = 8;
        p.kind = bf ? came::kBF16x8 : came::kF32x8;
    } else if (!bf && cols % 4 == 0) {
        p.vec = 4;
        p.kind = came::kF32x4;
    } else {
        p.vec = 1;
        p.kind = bf ? came::kBF16x1 : came::kF32x1;
    }
    const long long lanes = ceil_div(cols, p.vec);
    // widest block row whose padding wastes at most 1/8 of the lanes; else the least padding
    int best = 32;
    long long best_pad = round_up(lanes, 32);
    bool chosen = false;
    for (int tx = 256; tx >= 32; tx >>= 1) {
        const long long padded = round_up(lanes, tx);
        if (!chosen && padded * 8 <= lanes * 9) { best = tx; chosen = true; }
        if (!chosen && padded < best_pad) { best = tx; best_pad = padded; }
    }
    p.tx = best;
    const long long sw = static_cast<long long>(p.tx) * p.vec;
    const int ty = came::kThreads / p.tx;
    p.n_cb = static_cast<int>(ceil_div(cols, sw));
    if (target <= 0) target = 32768;
    long long tr = std::max<long long>(1, target / sw);
    tr = round_up(tr, ty);
    tr = std::max(tr, round_up(ceil_div(rows, 256), ty));   // at most 256 row blocks per tensor
    tr = std::min(tr, round_up(rows, ty));
    p.tr = static_cast<int>(tr);
    p.n_rb = static_cast<int>(ceil_div(rows, tr));
    p.n_seg = p.n_cb * (p.tx / 32);
    p.n_parts = p.n_rb * p.n_cb;
    p.n_grp = (p.n_rb + came::kColGroup - 1) / came::kColGroup;   // <= kColGroup since n_rb <= 256
    return p;
}

}  // namespace

// A run of consecutive tensors handled together: [t0, t1) and their tiles.
struct Group { int t0, t1, tile0, tile1; };

struct came_ctx {
    int device = 0;
    int n = 0;
    std::vector<came_tensor> tensors;
    std::vector<TensorDev> host_table;
    TensorDev* d_table = nullptr;
    TensorDev* pinned_table[2] = {nullptr, nullptr};
    came::StreamTile* pinned_stream[2] = {nullptr, nullptr};
    cudaEvent_t pinned_free[2] = {nullptr, nullptr};
    bool pinned_used[2] = {false, false};
    int pinned_next = 0;
    Tile* d_tiles = nullptr;
    int n_tiles = 0;                            // matrix tiles and vector chunks
    std::vector<int> tile_begin;                // [n+1] first tile of each tensor
    std::vector<Group> sched_groups;            // device-resident step: launch order (empty = one grid)
    std::vector<Group> host_groups;             // host-buffer step: pipeline stages
    cudaStream_t s_up = nullptr, s_down = nullptr;   // copy streams of the host-buffer step
    std::vector<cudaEvent_t> ev_up, ev_done;         // per host group: gradients landed / step done
    cudaEvent_t ev_start = nullptr, ev_all_down = nullptr;
    char* d_ws = nullptr;
    size_t ws_bytes = 0, table_bytes = 0;
    long long numel = 0, matrix_numel = 0, state_bytes = 0, stream_bytes = 0, comp_bytes = 0;
    long long last_step = 0;
    came::StreamTile* d_stream = nullptr;      // streaming P1: the matrix tiles its ring can serve
    std::vector<came::StreamTile> h_stream;
    std::vector<long long> stream_goff;        // byte offset of every stream tile inside its gradient
    int n_stream = 0;
    Tile* d_others = nullptr;                  // streaming P1: all other tiles (scalar kinds, vector chunks)
    int n_others = 0;
    int p1_stream_grid = 0, p1_stream_ring = 0;
    bool pipelined = false;                    // one persistent grid per step instead of one grid per phase
    came::Item* d_items = nullptr;             // pipelined schedule: work items in ticket order
    int n_items = 0;
    came::PipeSync* d_sync = nullptr;
    int pipe_grid = 0;                         // blocks of the persistent grid
    int pipe_groups = 0;
    unsigned long long pipe_wait_ns = 0;
    bool adafactor = false;                    // Algorithm 1 instead of Algorithm 2
    bool profiling = false;
    std::vector<cudaEvent_t> prof_ev;          // [kProfSlots][kMaxPhases + 1], made on demand
    long long prof_count = 0;                  // profiled steps since profiling was switched on
    int n_intervals = 0;
    std::string err;
};

namespace {

came_status fail(came_ctx* ctx, came_status s, const std::string& msg)
{
    if (ctx) ctx->err = msg; else g_create_error = msg;
    return s;
}

came_status cuda_fail(came_ctx* ctx, cudaError_t e, const char* what)
{
    std::string msg = std::string(what) + ": " + cudaGetErrorString(e);
    const came_status s = (e == cudaErrorMemoryAllocation) ? CAME_ERR_OOM : CAME_ERR_CUDA;
    return fail(ctx, s, msg);
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Byte alignment a gradient pointer must have for a plan that reads `vec` elements per
// thread per load: 8 fp32 elements are one 256-bit load (32 bytes); every other plan reads at
// most 128 bits at a time, and 16 bytes is the contract for all tensor pointers.
size_t grad_alignment_for(int grad_dtype, int vec)
{
    return (grad_dtype == CAME_F32 && vec == 8) ? 32 : 16;
}

came_status validate_tensor(const came_tensor& t, int i, bool adafactor, std::string& msg)
{
    char buf[160];
    auto err = [&](came_status s, const char* what) {
        std::snprintf(buf, sizeof buf, "tensor %d: %s", i, what);
        msg = buf;
        return s;
    };
    if (t.ndim != 1 && t.ndim != 2) return err(CAME_ERR_SHAPE, "ndim must be 1 or 2");
    if (t.rows < 1 || t.cols < 1) return err(CAME_ERR_SHAPE, "rows and cols must be >= 1");
    if (t.ndim == 1 && t.cols != 1) return err(CAME_ERR_SHAPE, "a vector must have cols == 1");
    if (t.rows > (1ll << 40) / t.cols) return err(CAME_ERR_SHAPE, "tensor too large");
    if (t.grad_dtype != CAME_F32 && t.grad_dtype != CAME_BF16) return err(CAME_ERR_DTYPE, "unknown grad_dtype");
    if (t.reserved != 0) return err(CAME_ERR_SHAPE, "reserved must be 0");
    if (!t.param || !t.grad || !t.m || !t.r) return err(CAME_ERR_NULL, "param, grad, m, r are required");
    if (t.ndim == 2 && !t.c) return err(CAME_ERR_NULL, "a matrix needs c");
    if (!adafactor && !(t.ndim == 1 && (t.flags & CAME_T_VEC_NO_CONFIDENCE))) {
        if (!t.R) return err(CAME_ERR_NULL, "R is required");
        if (t.ndim == 2 && !t.C) return err(CAME_ERR_NULL, "a matrix needs C");
    }
    const void* ptrs[8] = {t.param, t.grad, t.m, t.r, t.c, t.R, t.C, t.param_bf16};
    for (const void* p : ptrs)
        if (p && !aligned(p, 16)) return err(CAME_ERR_ALIGN, "pointer not 16-byte aligned");
    if ((t.flags & CAME_T_VEC_NO_CONFIDENCE) && t.ndim != 1)
        return err(CAME_ERR_SHAPE, "CAME_T_VEC_NO_CONFIDENCE applies to vectors only");
    return CAME_OK;
}

// Every buffer of every tensor must be its own memory: the phases read one tensor's state
// while they write another's, and the tiles of one buffer are written by different blocks.
// Sorts all [address, address + bytes) ranges and compares neighbours.
came_status check_no_overlap(const came_tensor* t, int n, bool adafactor, std::string& msg)
{
    struct Range { uintptr_t lo, hi; int tensor; const char* what; };
    std::vector<Range> rs;
    rs.reserve(static_cast<size_t>(n) * 8);
    for (int i = 0; i < n; ++i) {
        const came_tensor& x = t[i];
        const unsigned long long numel = static_cast<unsigned long long>(x.rows) * x.cols;
        const unsigned long long sg = x.grad_dtype == CAME_BF16 ? 2 : 4;
        auto add = [&](const void* p, unsigned long long bytes, const char* what) {
            if (p && bytes) rs.push_back(Range{reinterpret_cast<uintptr_t>(p),
                                               reinterpret_cast<uintptr_t>(p) + bytes, i, what});
        };
        add(x.param, 4 * numel, "param");
        add(x.grad, sg * numel, "grad");
        add(x.m, 4 * numel, "m");
        add(x.r, 4ull * x.rows, "r");
        if (x.ndim == 2) add(x.c, 4ull * x.cols, "c");
        const bool conf = !adafactor && !(x.ndim == 1 && (x.flags & CAME_T_VEC_NO_CONFIDENCE));
        if (conf) {
            add(x.R, 4ull * x.rows, "R");
            if (x.ndim == 2) add(x.C, 4ull * x.cols, "C");
        }
        add(x.param_bf16, 2 * numel, "param_bf16");
    }
    std::sort(rs.begin(), rs.end(), [](const Range& a, const Range& b) { return a.lo < b.lo; });
    for (size_t k = 1; k < rs.size(); ++k) {
        if (rs[k].lo < rs[k - 1].hi) {
            char buf[200];
            std::snprintf(buf, sizeof buf, "buffers overlap: %s of tensor %d and %s of tensor %d",
                          rs[k - 1].what, rs[k - 1].tensor, rs[k].what, rs[k].tensor);
            msg = buf;
            return CAME_ERR_OVERLAP;
        }
    }
    return CAME_OK;
}

came_status validate_hparams(const came_hparams& h, long long last_step, std::string& msg)
{
    const double v[9] = {h.lr, h.beta1, h.beta2, h.beta3, h.eps1, h.eps2, h.clip_d, h.weight_decay,
                         h.grad_scale};
    for (double x : v)
        if (!std::isfinite(x)) { msg = "hyper-parameter not finite"; return CAME_ERR_HPARAM; }
    if (h.lr < 0) { msg = "lr must be >= 0"; return CAME_ERR_HPARAM; }
    const double betas[3] = {h.beta1, h.beta2, h.beta3};
    for (double b : betas)
        if (b < 0.0 || b >= 1.0) { msg = "betas must lie in [0,1)"; return CAME_ERR_HPARAM; }
    if (h.eps1 < 0 || h.eps2 < 0) { msg = "eps1, eps2 must be >= 0"; return CAME_ERR_HPARAM; }
    if (!(h.clip_d > 0)) { msg = "clip_d must be > 0"; return CAME_ERR_HPARAM; }
    if (h.weight_decay < 0) { msg = "weight_decay must be >= 0"; return CAME_ERR_HPARAM; }
    if (h.grad_scale < 0) { msg = "grad_scale must be > 0 (or 0 for 1)"; return CAME_ERR_HPARAM; }
    if (h.step < 1) { msg = "step must be >= 1"; return CAME_ERR_STEP_ORDER; }
    if (last_step > 0 && h.step != last_step + 1) {
        msg = "step must be the previous step + 1";
        return CAME_ERR_STEP_ORDER;
    }
    return CAME_OK;
}

StepConsts make_consts(const came_hparams& h)
{
    StepConsts c;
    c.beta1 = static_cast<float>(h.beta1);
    c.omb1 = static_cast<float>(1.0 - h.beta1);
    c.b1sq = static_cast<float>(h.beta1 * h.beta1);
    c.beta2 = static_cast<float>(h.beta2);
    c.omb2 = static_cast<float>(1.0 - h.beta2);
    c.beta3 = static_cast<float>(h.beta3);
    c.omb3 = static_cast<float>(1.0 - h.beta3);
    c.eps1 = static_cast<float>(h.eps1);
    c.eps2 = static_cast<float>(h.eps2);
    c.lr = static_cast<float>(h.lr);
    c.wd = static_cast<float>(h.weight_decay);
    const double gs = h.grad_scale == 0.0 ? 1.0 : h.grad_scale;
    c.gscale = static_cast<float>(gs);
    c.gscale2 = static_cast<float>(gs * gs);
    c.pad_ = 0.f;
    c.clip_d = h.clip_d;
    return c;
}

void free_ctx(came_ctx* ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    cudaFree(ctx->d_table);
    cudaFree(ctx->d_tiles);
    cudaFree(ctx->d_ws);
    cudaFree(ctx->d_items);
    cudaFree(ctx->d_sync);
    cudaFree(ctx->d_stream);
    cudaFree(ctx->d_others);
    for (int k = 0; k < 2; ++k) {
        if (ctx->pinned_table[k]) cudaFreeHost(ctx->pinned_table[k]);
        if (ctx->pinned_stream[k]) cudaFreeHost(ctx->pinned_stream[k]);
        if (ctx->pinned_free[k]) cudaEventDestroy(ctx->pinned_free[k]);
    }
    for (cudaEvent_t e : ctx->prof_ev)
        if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_up) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_done) if (e) cudaEventDestroy(e);
    if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
    if (ctx->ev_all_down) cudaEventDestroy(ctx->ev_all_down);
    if (ctx->s_up) cudaStreamDestroy(ctx->s_up);
    if (ctx->s_down) cudaStreamDestroy(ctx->s_down);
    delete ctx;
}

// Upload the host tensor table through a pinned staging slot (two slots, each guarded by an
// event, so that a copy still in flight from an earlier step is never overwritten).
came_status upload_table(came_ctx* ctx, cudaStream_t stream)
{
    const int k = ctx->pinned_next;
    ctx->pinned_next ^= 1;
    if (ctx->pinned_used[k]) {
        const cudaError_t e = cudaEventSynchronize(ctx->pinned_free[k]);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventSynchronize(table slot)");
    }
    std::memcpy(ctx->pinned_table[k], ctx->host_table.data(), ctx->table_bytes);
    cudaError_t e = cudaMemcpyAsync(ctx->d_table, ctx->pinned_table[k], ctx->table_bytes,
                                    cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemcpyAsync(table)");
    if (ctx->n_stream > 0 && ctx->pinned_stream[k]) {
        // the streaming P1 reads gradient addresses from its own tile records: rebuild them
        for (int j = 0; j < ctx->n_stream; ++j) {
            came::StreamTile r = ctx->h_stream[j];
            r.g = static_cast<const char*>(ctx->host_table[r.tensor].g) + ctx->stream_goff[j];
            ctx->h_stream[j] = r;
            ctx->pinned_stream[k][j] = r;
        }
        e = cudaMemcpyAsync(ctx->d_stream, ctx->pinned_stream[k], sizeof(came::StreamTile) * ctx->n_stream,
                            cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemcpyAsync(stream tiles)");
    }
    e = cudaEventRecord(ctx->pinned_free[k], stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventRecord(table slot)");
    ctx->pinned_used[k] = true;
    return CAME_OK;
}

// Launch one phase kernel with programmatic stream serialisation (see pdl_* in the kernels).
template <typename K>
void launch_phase(K kernel, int grid, cudaStream_t stream, const TensorDev* table, const Tile* tiles,
                  int ntiles, int reverse, const StepConsts& hc)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(came::kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, table, tiles, ntiles, reverse, hc);
}

// The streaming form of P1 over the whole tile list (persistent grid, dynamic shared memory
// for the copy ring), launched like the other phase kernels.
void launch_p1_stream(const came_ctx* ctx, const StepConsts& hc, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctx->p1_stream_grid));
    cfg.blockDim = dim3(came::kThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(ctx->p1_stream_ring) * came::kStreamSlots * came::kThreads * 16;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, came::k_p1_stream, static_cast<const TensorDev*>(ctx->d_table),
                       static_cast<const came::StreamTile*>(ctx->d_stream), ctx->n_stream,
                       static_cast<const Tile*>(ctx->d_others), ctx->n_others, ctx->p1_stream_ring, hc);
}

// Enqueue the kernels of one step for the tensors of `g` (all phases, in dependency order).
// `ev` (may be NULL) receives one event before the first kernel and one after each kernel.
int launch_range(const came_ctx* ctx, const StepConsts& hc, cudaStream_t stream, const Group& g,
                 cudaEvent_t* ev)
{
    int iv = 0;
    auto mark = [&](int slot) { if (ev) cudaEventRecord(ev[slot], stream); };
    const int nt = g.tile1 - g.tile0;
    const Tile* tiles = ctx->d_tiles + g.tile0;
    mark(0);
    if (nt > 0) {
        if (ctx->p1_stream_grid > 0 && g.tile0 == 0 && g.tile1 == ctx->n_tiles)
            launch_p1_stream(ctx, hc, stream);
        else
            launch_phase(came::k_p1_reduce_g2, nt, stream, ctx->d_table, tiles, nt, 0, hc);
        mark(++iv);
        launch_phase(came::k_p2_sum_u2, nt, stream, ctx->d_table, tiles, nt, 1, hc);
        mark(++iv);
        if (ctx->adafactor) {
            launch_phase(came::k_p34_adafactor_apply, nt, stream, ctx->d_table, tiles, nt, 0, hc);
            mark(++iv);
        } else {
            launch_phase(came::k_p3_momentum_instability, nt, stream, ctx->d_table, tiles, nt, 0, hc);
            mark(++iv);
            launch_phase(came::k_p4_apply, nt, stream, ctx->d_table, tiles, nt, 1, hc);
            mark(++iv);
        }
    }
    return iv;
}

came_status launch_step(came_ctx* ctx, const came_hparams* hp, cudaStream_t stream)
{
    const StepConsts hc = make_consts(*hp);
    if (ctx->pipelined) {
        const bool prof = ctx->profiling && !ctx->prof_ev.empty();
        cudaEvent_t* ev = prof ? &ctx->prof_ev[(ctx->prof_count % kProfSlots) * (kMaxPhases + 1)] : nullptr;
        if (ev) cudaEventRecord(ev[0], stream);
        came::k_step_pipelined<<<ctx->pipe_grid, came::kPipeThreads, 0, stream>>>(
            ctx->d_table, ctx->d_items, ctx->n_items, ctx->d_sync, hc, ctx->adafactor ? 1 : 0,
            ctx->pipe_wait_ns);
        if (ev) cudaEventRecord(ev[1], stream);
        ctx->n_intervals = 1;
        if (prof) ++ctx->prof_count;
    } else if (ctx->sched_groups.empty()) {
        const bool prof = ctx->profiling && !ctx->prof_ev.empty();
        cudaEvent_t* ev = prof ? &ctx->prof_ev[(ctx->prof_count % kProfSlots) * (kMaxPhases + 1)] : nullptr;
        const Group all{0, ctx->n, 0, ctx->n_tiles};
        ctx->n_intervals = launch_range(ctx, hc, stream, all, ev);
        if (prof) ++ctx->prof_count;
    } else {
        // grouped schedule: all phases of one group before the next group starts, so that a
        // group sized to the L2 re-reads its gradients and momentum from there
        for (const Group& g : ctx->sched_groups) launch_range(ctx, hc, stream, g, nullptr);
        ctx->n_intervals = 0;
    }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kernel launch");
    ctx->last_step = hp->step;
    return CAME_OK;
}

// Consecutive tensors are grouped until a group holds `limit` bytes (by `bytes_of`).
template <typename F>
std::vector<Group> make_groups(const came_ctx* ctx, long long limit, F bytes_of)
{
    std::vector<Group> out;
    int t0 = 0;
    long long acc = 0;
    for (int i = 0; i < ctx->n; ++i) {
        acc += bytes_of(ctx->tensors[i]);
        if (acc >= limit || i == ctx->n - 1) {
            out.push_back(Group{t0, i + 1, ctx->tile_begin[t0], ctx->tile_begin[i + 1]});
            t0 = i + 1;
            acc = 0;
        }
    }
    return out;
}

// Which schedule a new context gets: one grid per phase unless the pipelined grid is asked
// for.  (Measured on B200 the pipelined grid is the slower of the two on every workload
// tried: at 6.5 TB/s the 126 MB L2 turns over in under 20 us, less than the four dependent
// phases of a tensor group need to pass through it, so the groups either stall on their
// flags or fall out of the L2.)
bool choose_pipelined(const came_tensor*, int)
{
    return g_schedule == 2;
}

// Ticket order of the pipelined schedule.  Consecutive tensors form a group until the group's
// gradients and momenta reach the group size; stage s then holds, oldest first, P4 of group
// s-3, P3 of group s-2, P2 of group s-1 and P1 of group s.  Every item therefore comes after
// all items of the phase it depends on (they sit in the stage before), with two other
// sub-phases in between, which is what keeps the waits short.
std::vector<came::Item> build_pipeline_items(came_ctx* ctx, const std::vector<Tile>& tiles)
{
    const long long pipe_group = g_pipe_group_bytes.load();
    const long long group_bytes = pipe_group > 0 ? pipe_group : kPipeGroupBytesDefault;
    auto resident = [](const came_tensor& x) {
        return x.rows * x.cols * (4ll + (x.grad_dtype == CAME_BF16 ? 2 : 4)); };
    const std::vector<Group> groups = make_groups(ctx, group_bytes, resident);
    ctx->pipe_groups = static_cast<int>(groups.size());
    const int phases = ctx->adafactor ? 3 : 4;
    const int ng = static_cast<int>(groups.size());
    std::vector<came::Item> items;
    items.reserve(tiles.size() * phases);
    auto emit = [&](const Group& g, int phase) {
        for (int k = g.tile0; k < g.tile1; ++k) {
            const Tile& tl = tiles[k];
            const bool vec = ctx->tensors[tl.tensor].ndim == 1;
            if (vec && phase != 0 && phase != 2) continue;     // vectors: two halves only
            items.push_back(came::Item{tl.tensor, tl.rb, tl.cb, phase});
        }
    };
    if (g_pipe_order == 1) {
        // no skew: every group runs its phases back to back (dependent items are adjacent,
        // so the waits are real; kept for tests and measurements)
        for (int s = 0; s < ng; ++s)
            for (int ph = 0; ph < phases; ++ph) emit(groups[s], ph);
        return items;
    }
    for (int s = 0; s < ng + phases - 1; ++s)
        for (int ph = phases - 1; ph >= 0; --ph) {
            const int grp = s - ph;
            if (grp >= 0 && grp < ng) emit(groups[grp], ph);
        }
    return items;
}

// A step launched with another device current would run on that GPU with this context's
// pointers.  The comparison itself is came_device_status, so it can be exercised without a GPU.
came_status check_current_device(came_ctx* ctx)
{
    int cur = -1;
    const cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetDevice");
    if (came_device_status(ctx->device, cur) != CAME_OK) {
        char buf[120];
        std::snprintf(buf, sizeof buf, "the context lives on device %d but device %d is current",
                      ctx->device, cur);
        return fail(ctx, CAME_ERR_DEVICE, buf);
    }
    return CAME_OK;
}

}  // namespace

extern "C" {

came_status came_device_status(int32_t context_device, int32_t current_device)
{
    return (context_device >= 0 && context_device == current_device) ? CAME_OK : CAME_ERR_DEVICE;
}

int32_t came_required_grad_alignment(int32_t grad_dtype, int32_t vec)
{
    return static_cast<int32_t>(grad_alignment_for(grad_dtype, vec));
}

double came_lr_warmup(double lr_peak, double lr_start, int64_t step, int64_t warmup_steps)
{
    if (warmup_steps <= 0 || step >= warmup_steps) return lr_peak;
    if (step < 0) step = 0;
    return lr_start + (lr_peak - lr_start) * (static_cast<double>(step) / static_cast<double>(warmup_steps));
}

const char* came_status_string(came_status s)
{
    switch (s) {
        case CAME_OK: return "CAME_OK";
        case CAME_ERR_NULL: return "CAME_ERR_NULL";
        case CAME_ERR_SHAPE: return "CAME_ERR_SHAPE";
        case CAME_ERR_DTYPE: return "CAME_ERR_DTYPE";
        case CAME_ERR_ALIGN: return "CAME_ERR_ALIGN";
        case CAME_ERR_HPARAM: return "CAME_ERR_HPARAM";
        case CAME_ERR_STEP_ORDER: return "CAME_ERR_STEP_ORDER";
        case CAME_ERR_DEVICE: return "CAME_ERR_DEVICE";
        case CAME_ERR_OOM: return "CAME_ERR_OOM";
        case CAME_ERR_CUDA: return "CAME_ERR_CUDA";
        case CAME_ERR_INTERNAL: return "CAME_ERR_INTERNAL";
        case CAME_ERR_UNSUPPORTED: return "CAME_ERR_UNSUPPORTED";
        case CAME_ERR_OVERLAP: return "CAME_ERR_OVERLAP";
    }
    return "CAME_ERR_?";
}

const char* came_last_error(const came_ctx* ctx)
{
    return ctx ? ctx->err.c_str() : g_create_error.c_str();
}

came_status came_tune(int32_t key, int64_t value)
{
    if (value < 0) return CAME_ERR_UNSUPPORTED;
    switch (key) {
        case CAME_TUNE_TILE_ELEMS: g_tile_elems_override = value; break;
        case CAME_TUNE_SCHED_GROUP_BYTES: g_sched_group_bytes = value; break;
        case CAME_TUNE_PDL: g_use_pdl = value != 0; break;
        case CAME_TUNE_F32_VEC8: g_f32_vec8 = value != 0; break;
        case CAME_TUNE_HOST_GROUP_BYTES: g_host_group_bytes = value > 0 ? value : (1ll << 30); break;
        case CAME_TUNE_P1_STREAM: if (value > 2) return CAME_ERR_UNSUPPORTED; g_p1_stream = static_cast<int>(value); break;
        case CAME_TUNE_P1_STREAM_RING: if (value > came::kStreamMaxBatches) return CAME_ERR_UNSUPPORTED; g_p1_stream_ring = static_cast<int>(value); break;
        case CAME_TUNE_SCHEDULE: if (value > 2) return CAME_ERR_UNSUPPORTED; g_schedule = static_cast<int>(value); break;
        case CAME_TUNE_PIPE_TILE_ELEMS: g_pipe_tile_elems = value; break;
        case CAME_TUNE_PIPE_GROUP_BYTES: g_pipe_group_bytes = value; break;
        case CAME_TUNE_PIPE_WAIT_NS: g_pipe_wait_ns = value; break;
        case CAME_TUNE_PIPE_ORDER: if (value > 1) return CAME_ERR_UNSUPPORTED; g_pipe_order = value; break;
        default: return CAME_ERR_UNSUPPORTED;
    }
    return CAME_OK;
}

came_status came_plan_tensor(int64_t rows, int64_t cols, int32_t ndim, int32_t grad_dtype,
                             int32_t aligned32, int64_t tile_elems_target, int32_t* out_vec,
                             int32_t* out_threads_x, int32_t* out_tile_rows, int32_t* out_n_rb,
                             int32_t* out_n_cb)
{
    if (!out_vec || !out_threads_x || !out_tile_rows || !out_n_rb || !out_n_cb) return CAME_ERR_NULL;
    if (rows < 1 || cols < 1 || (ndim != 1 && ndim != 2) || (ndim == 1 && cols != 1)) return CAME_ERR_SHAPE;
    if (grad_dtype != CAME_F32 && grad_dtype != CAME_BF16) return CAME_ERR_DTYPE;
    const Plan p = plan_tensor(rows, cols, ndim, grad_dtype, aligned32 != 0, tile_elems_target);
    *out_vec = p.vec; *out_threads_x = p.tx; *out_tile_rows = p.tr; *out_n_rb = p.n_rb; *out_n_cb = p.n_cb;
    return CAME_OK;
}

came_status came_create(came_ctx** out, const came_tensor* t, int32_t n, int32_t device,
                        uint32_t flags)
{
    if (!out) return fail(nullptr, CAME_ERR_NULL, "out is NULL");
    *out = nullptr;
    if (!t) return fail(nullptr, CAME_ERR_NULL, "tensor array is NULL");
    if (n < 1) return fail(nullptr, CAME_ERR_SHAPE, "need at least one tensor");
    if (flags & ~static_cast<uint32_t>(CAME_CREATE_KEEP_STATE | CAME_CREATE_ADAFACTOR))
        return fail(nullptr, CAME_ERR_UNSUPPORTED, "unknown create flag");
    const bool adafactor = (flags & CAME_CREATE_ADAFACTOR) != 0;
    std::string msg;
    for (int i = 0; i < n; ++i) {
        const came_status s = validate_tensor(t[i], i, adafactor, msg);
        if (s != CAME_OK) return fail(nullptr, s, msg);
    }
    {
        const came_status s = check_no_overlap(t, n, adafactor, msg);
        if (s != CAME_OK) return fail(nullptr, s, msg);
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        cudaGetLastError();
        return fail(nullptr, CAME_ERR_DEVICE, "no usable CUDA device");
    }
    if (device < 0 || device >= ndev) return fail(nullptr, CAME_ERR_DEVICE, "device ordinal out of range");
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaSetDevice");

    came_ctx* ctx = new (std::nothrow) came_ctx;
    if (!ctx) return fail(nullptr, CAME_ERR_OOM, "host allocation failed");
    ctx->device = device;
    ctx->adafactor = adafactor;
    ctx->n = n;
    ctx->tensors.assign(t, t + n);
    ctx->host_table.resize(n);

    // ---- plan -----------------------------------------------------------------------------
    long long matrix_numel = 0;
    for (int i = 0; i < n; ++i)
        if (t[i].ndim == 2) matrix_numel += t[i].rows * t[i].cols;
    ctx->pipelined = choose_pipelined(t, n);
    long long target = g_tile_elems_override;
    if (target <= 0 && ctx->pipelined)
        target = g_pipe_tile_elems.load() > 0 ? g_pipe_tile_elems.load() : kPipeTileElemsDefault;
    if (target <= 0) {
        // aim for a few thousand tiles in all; between 4 Ki and 256 Ki elements per tile
        target = 4096;
        while (target < 262144 && target * 2 * 2400 <= matrix_numel) target *= 2;
    }
    std::vector<Plan> plans(n);
    ctx->tile_begin.assign(n + 1, 0);
    std::vector<Tile> tiles;
    size_t ws = 0;
    auto take = [&](size_t bytes) { const size_t off = ws; ws += (bytes + 255) / 256 * 256; return off; };
    struct Off { size_t colpart, colpart2, rowpart, blocksum, usq, cnt, scal, rowscale, colscale, done; };
    std::vector<Off> offs(n);
    for (int i = 0; i < n; ++i) {
        const came_tensor& x = t[i];
        const bool a32 = aligned(x.param, 32) && aligned(x.m, 32) &&
                         (x.grad_dtype == CAME_BF16 || aligned(x.grad, 32));
        // a contiguous n x 1 matrix is the same memory as 1 x n: planned (and run) in that
        // view, with the factor roles swapped, every lane has a column to work on
        const bool flat = x.ndim == 2 && x.cols == 1 && x.rows > 1;
        Plan p = flat ? plan_tensor(1, x.rows, 2, x.grad_dtype, a32, target)
                      : plan_tensor(x.rows, x.cols, x.ndim, x.grad_dtype, a32, target);
        if (p.n_grp > came::kColGroup) {      // the two-level column reduction covers 16 x 16 row blocks
            delete ctx;
            return fail(nullptr, CAME_ERR_INTERNAL, "tile plan exceeds the column-reduction fan-in");
        }
        plans[i] = p;
        const long long numel = x.rows * x.cols;
        const long long sg = x.grad_dtype == CAME_BF16 ? 2 : 4;
        ctx->numel += numel;
        if (x.param_bf16) { ctx->stream_bytes += 2 * numel; ctx->comp_bytes += 2 * numel; }
        if (x.ndim == 2) {
            ctx->matrix_numel += numel;
            if (adafactor) {
                ctx->state_bytes += 4 * (numel + (x.rows + x.cols));
                ctx->stream_bytes += numel * (3 * sg + 16) + 8 * (x.rows + x.cols);
                ctx->comp_bytes += numel * (sg + 16) + 8 * (x.rows + x.cols);
            } else {
                ctx->state_bytes += 4 * (numel + 2 * (x.rows + x.cols));
                ctx->stream_bytes += numel * (3 * sg + 20) + 16 * (x.rows + x.cols);
                ctx->comp_bytes += numel * (sg + 16) + 16 * (x.rows + x.cols);
            }
            for (int rb = 0; rb < p.n_rb; ++rb)
                for (int cb = 0; cb < p.n_cb; ++cb) tiles.push_back(Tile{i, rb, cb});
            const size_t vrows = flat ? 1 : static_cast<size_t>(x.rows);      // the view that runs
            const size_t vcols = flat ? static_cast<size_t>(x.rows) : static_cast<size_t>(x.cols);
            offs[i].colpart = take(sizeof(float) * static_cast<size_t>(p.n_rb) * vcols);
            offs[i].colpart2 = take(sizeof(float) * static_cast<size_t>(p.n_grp) * vcols);
            offs[i].rowpart = take(sizeof(float) * static_cast<size_t>(p.n_seg) * vrows);
            offs[i].blocksum = take(sizeof(float) * (static_cast<size_t>(p.n_rb) + (flat ? p.n_cb : 0)));
            offs[i].rowscale = take(sizeof(float) * vrows);
            offs[i].colscale = take(sizeof(float) * vcols);
        } else {
            const bool conf = !adafactor && !(x.flags & CAME_T_VEC_NO_CONFIDENCE);
            ctx->state_bytes += 4 * (conf ? 3 : 2) * numel;
            ctx->stream_bytes += numel * (sg + (conf ? 32 : 24));
            ctx->comp_bytes += numel * (sg + (conf ? 32 : 24));
            for (int c = 0; c < p.n_parts; ++c) tiles.push_back(Tile{i, c, 0});
            offs[i].colpart = offs[i].colpart2 = offs[i].rowpart = offs[i].blocksum = 0;
            offs[i].rowscale = offs[i].colscale = 0;
        }
        offs[i].usq = take(sizeof(float) * p.n_parts);
        offs[i].cnt = take(sizeof(unsigned) * p.counters());
        offs[i].scal = take(sizeof(float) * 4);
        offs[i].done = take(sizeof(unsigned) * 4);
        ctx->tile_begin[i + 1] = static_cast<int>(tiles.size());
        if (tiles.size() > (1u << 30)) {
            delete ctx;
            return fail(nullptr, CAME_ERR_SHAPE, "too many tiles");
        }
    }
    ctx->n_tiles = static_cast<int>(tiles.size());
    ctx->ws_bytes = ws;
    ctx->table_bytes = sizeof(TensorDev) * n;

    // ---- device memory --------------------------------------------------------------------
#define CAME_TRY(call, what)                                                     \
    do { e = (call); if (e != cudaSuccess) { const came_status s_ = cuda_fail(nullptr, e, what); \
         free_ctx(ctx); return s_; } } while (0)
    CAME_TRY(cudaMalloc(&ctx->d_ws, std::max<size_t>(ws, 256)), "cudaMalloc(workspace)");
    CAME_TRY(cudaMemset(ctx->d_ws, 0, std::max<size_t>(ws, 256)), "cudaMemset(workspace)");
    CAME_TRY(cudaMalloc(&ctx->d_table, ctx->table_bytes), "cudaMalloc(table)");
    if (ctx->n_tiles) {
        CAME_TRY(cudaMalloc(&ctx->d_tiles, sizeof(Tile) * tiles.size()), "cudaMalloc(tiles)");
        CAME_TRY(cudaMemcpy(ctx->d_tiles, tiles.data(), sizeof(Tile) * tiles.size(),
                            cudaMemcpyHostToDevice), "cudaMemcpy(tiles)");
    }
    if (ctx->pipelined) {
        if (tiles.size() > (1u << 28)) {
            free_ctx(ctx);
            return fail(nullptr, CAME_ERR_SHAPE, "too many tiles for the pipelined schedule");
        }
        const std::vector<came::Item> items = build_pipeline_items(ctx, tiles);
        ctx->n_items = static_cast<int>(items.size());
        CAME_TRY(cudaMalloc(&ctx->d_items, sizeof(came::Item) * std::max<size_t>(items.size(), 1)),
                 "cudaMalloc(items)");
        CAME_TRY(cudaMemcpy(ctx->d_items, items.data(), sizeof(came::Item) * items.size(),
                            cudaMemcpyHostToDevice), "cudaMemcpy(items)");
        CAME_TRY(cudaMalloc(&ctx->d_sync, sizeof(came::PipeSync)), "cudaMalloc(sync)");
        CAME_TRY(cudaMemset(ctx->d_sync, 0, sizeof(came::PipeSync)), "cudaMemset(sync)");
        int sms = 0, per_sm = 0;
        CAME_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device), "cudaDeviceGetAttribute");
        CAME_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, came::k_step_pipelined,
                                                               came::kPipeThreads, 0), "occupancy query");
        ctx->pipe_grid = std::max(1, std::min(ctx->n_items, sms * std::max(per_sm, 1)));
        ctx->pipe_wait_ns = static_cast<unsigned long long>(g_pipe_wait_ns.load() > 0 ? g_pipe_wait_ns.load()
                                                                                       : kPipeWaitNsDefault);
    }
    for (int k = 0; k < 2; ++k) {
        CAME_TRY(cudaMallocHost(&ctx->pinned_table[k], ctx->table_bytes), "cudaMallocHost(table)");
        CAME_TRY(cudaEventCreateWithFlags(&ctx->pinned_free[k], cudaEventDisableTiming), "cudaEventCreate");
    }

    {
        auto state_bytes = [](const came_tensor& x) {
            return x.rows * x.cols * (8ll + (x.grad_dtype == CAME_BF16 ? 2 : 4)); };
        auto xfer_bytes = [](const came_tensor& x) {
            return x.rows * x.cols * (4ll + (x.grad_dtype == CAME_BF16 ? 2 : 4)); };
        if (g_sched_group_bytes > 0) ctx->sched_groups = make_groups(ctx, g_sched_group_bytes, state_bytes);
        ctx->host_groups = make_groups(ctx, g_host_group_bytes, xfer_bytes);
        CAME_TRY(cudaStreamCreateWithFlags(&ctx->s_up, cudaStreamNonBlocking), "cudaStreamCreate");
        CAME_TRY(cudaStreamCreateWithFlags(&ctx->s_down, cudaStreamNonBlocking), "cudaStreamCreate");
        CAME_TRY(cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming), "cudaEventCreate");
        CAME_TRY(cudaEventCreateWithFlags(&ctx->ev_all_down, cudaEventDisableTiming), "cudaEventCreate");
        ctx->ev_up.assign(ctx->host_groups.size(), nullptr);
        ctx->ev_done.assign(ctx->host_groups.size(), nullptr);
        for (cudaEvent_t& ev : ctx->ev_up)
            CAME_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate");
        for (cudaEvent_t& ev : ctx->ev_done)
            CAME_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "cudaEventCreate");
    }
    for (int i = 0; i < n; ++i) {
        const came_tensor& x = t[i];
        const Plan& p = plans[i];
        TensorDev& d = ctx->host_table[i];
        std::memset(&d, 0, sizeof d);
        d.p = x.param; d.g = x.grad; d.m = x.m; d.r = x.r; d.c = x.c; d.R = x.R; d.C = x.C;
        d.p_bf16 = static_cast<uint16_t*>(x.param_bf16);
        d.rows = x.rows; d.cols = x.cols;
        d.ws_colpart = reinterpret_cast<float*>(ctx->d_ws + offs[i].colpart);
        d.ws_colpart2 = reinterpret_cast<float*>(ctx->d_ws + offs[i].colpart2);
        d.ws_rowpart = reinterpret_cast<float*>(ctx->d_ws + offs[i].rowpart);
        d.ws_blocksum = reinterpret_cast<float*>(ctx->d_ws + offs[i].blocksum);
        d.ws_usq = reinterpret_cast<float*>(ctx->d_ws + offs[i].usq);
        d.ws_rowscale = reinterpret_cast<float*>(ctx->d_ws + offs[i].rowscale);
        d.ws_colscale = reinterpret_cast<float*>(ctx->d_ws + offs[i].colscale);
        d.cnt = reinterpret_cast<unsigned*>(ctx->d_ws + offs[i].cnt);
        d.scal = reinterpret_cast<float*>(ctx->d_ws + offs[i].scal);
        d.done = reinterpret_cast<unsigned*>(ctx->d_ws + offs[i].done);
        d.kind = p.kind; d.vec = p.vec;
        int lg = 0; while ((1 << lg) < p.tx) ++lg;
        d.tx_log2 = lg; d.tr = p.tr; d.n_rb = p.n_rb; d.n_cb = p.n_cb; d.n_seg = p.n_seg;
        d.n_grp = p.n_grp;
        d.n_parts = p.n_parts; d.ndim = x.ndim; d.flags = x.flags;
        if (x.ndim == 2 && x.cols == 1 && x.rows > 1) {
            d.rows = 1; d.cols = x.rows;
            d.r = x.c; d.c = x.r; d.R = x.C; d.C = x.R;
            d.flags |= came::kFlagSumCols;
        }
        if (adafactor && x.ndim == 1) d.flags |= came::kFlagVecNoConf;   // Algorithm 1 has no S
        if (!(flags & CAME_CREATE_KEEP_STATE)) {
            const size_t numel = static_cast<size_t>(x.rows) * x.cols;
            CAME_TRY(cudaMemsetAsync(x.m, 0, 4 * numel, 0), "cudaMemset(m)");
            CAME_TRY(cudaMemsetAsync(x.r, 0, 4 * static_cast<size_t>(x.rows), 0), "cudaMemset(r)");
            if (x.R) CAME_TRY(cudaMemsetAsync(x.R, 0, 4 * static_cast<size_t>(x.rows), 0), "cudaMemset(R)");
            if (x.ndim == 2) {
                CAME_TRY(cudaMemsetAsync(x.c, 0, 4 * static_cast<size_t>(x.cols), 0), "cudaMemset(c)");
                if (x.C) CAME_TRY(cudaMemsetAsync(x.C, 0, 4 * static_cast<size_t>(x.cols), 0), "cudaMemset(C)");
            }
        }
    }
    // ---- streaming P1: tile records for the matrices whose rows load in 16-byte pieces ---------
    // (Off unless asked for: measured on B200 the ring hides the memory latency as intended --
    // long-scoreboard stalls drop from 7.9 to 1.4 cycles per issued instruction -- but P1 then
    // turns out to be bound by instruction issue, and the ring's extra copy, shared-memory read
    // and bookkeeping instructions, 1.5x the per-tile form's count, make it 1.5-2x slower.)
    if (g_p1_stream == 2) {
        std::vector<Tile> others;
        bool fits = true;
        for (const Tile& tl : tiles) {
            const TensorDev& d = ctx->host_table[tl.tensor];
            const bool ring_kind = d.ndim == 2 && (d.kind == came::kF32x4 || d.kind == came::kBF16x8 ||
                                                   d.kind == came::kF32x8);
            if (!ring_kind) { others.push_back(tl); continue; }
            if (d.cols >= (1ll << 31)) { fits = false; break; }
            const long long sw = (1ll << d.tx_log2) * d.vec;
            const long long row0 = static_cast<long long>(tl.rb) * d.tr, col0 = static_cast<long long>(tl.cb) * sw;
            const int esz = d.kind == came::kBF16x8 ? 2 : 4;
            came::StreamTile r;
            std::memset(&r, 0, sizeof r);
            const long long goff = (row0 * d.cols + col0) * esz;
            r.g = static_cast<const char*>(d.g) + goff;
            r.rowpart = d.ws_rowpart + static_cast<long long>(tl.cb) * ((1 << d.tx_log2) / 32) * d.rows + row0;
            r.rows = d.rows;
            r.tensor = tl.tensor; r.rb = tl.rb; r.cb = tl.cb;
            r.nrows = static_cast<int>(std::min<long long>(d.rows, row0 + d.tr) - row0);
            r.ncols = static_cast<int>(std::min<long long>(d.cols - col0, sw));
            r.cols = static_cast<int>(d.cols);
            r.kind_tx = d.kind | (d.tx_log2 << 8);
            ctx->h_stream.push_back(r);
            ctx->stream_goff.push_back(goff);
        }
        const long long n_st = static_cast<long long>(ctx->h_stream.size());
        const bool want = fits && n_st > 0;
        if (want) {
            ctx->n_stream = static_cast<int>(n_st);
            ctx->n_others = static_cast<int>(others.size());
            ctx->p1_stream_ring = std::min(came::kStreamMaxBatches,
                                           std::max(1, g_p1_stream_ring.load() > 0 ? g_p1_stream_ring.load() : kP1StreamRingDefault));
            const size_t ring_bytes = static_cast<size_t>(ctx->p1_stream_ring) * came::kStreamSlots * came::kThreads * 16;
            CAME_TRY(cudaFuncSetAttribute(came::k_p1_stream, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(ring_bytes)), "cudaFuncSetAttribute(ring)");
            int sms = 0, per_sm = 0;
            CAME_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device), "cudaDeviceGetAttribute");
            CAME_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, came::k_p1_stream, came::kThreads,
                                                                   ring_bytes), "occupancy query");
            ctx->p1_stream_grid = std::max(1, std::min(std::max(ctx->n_stream, ctx->n_others), sms * std::max(per_sm, 1)));
            CAME_TRY(cudaMalloc(&ctx->d_stream, sizeof(came::StreamTile) * ctx->n_stream), "cudaMalloc(stream tiles)");
            CAME_TRY(cudaMemcpy(ctx->d_stream, ctx->h_stream.data(), sizeof(came::StreamTile) * ctx->n_stream,
                                cudaMemcpyHostToDevice), "cudaMemcpy(stream tiles)");
            CAME_TRY(cudaMalloc(&ctx->d_others, sizeof(Tile) * std::max<size_t>(others.size(), 1)), "cudaMalloc(other tiles)");
            if (!others.empty())
                CAME_TRY(cudaMemcpy(ctx->d_others, others.data(), sizeof(Tile) * others.size(),
                                    cudaMemcpyHostToDevice), "cudaMemcpy(other tiles)");
            for (int k = 0; k < 2; ++k)
                CAME_TRY(cudaMallocHost(&ctx->pinned_stream[k], sizeof(came::StreamTile) * ctx->n_stream),
                         "cudaMallocHost(stream tiles)");
        } else {
            ctx->h_stream.clear();
            ctx->stream_goff.clear();
        }
    }
    CAME_TRY(cudaMemcpy(ctx->d_table, ctx->host_table.data(), ctx->table_bytes,
                        cudaMemcpyHostToDevice), "cudaMemcpy(table)");
    CAME_TRY(cudaDeviceSynchronize(), "cudaDeviceSynchronize");
#undef CAME_TRY
    *out = ctx;
    return CAME_OK;
}

came_status came_step(came_ctx* ctx, const came_hparams* hp, const void* const* grads,
                      void* cuda_stream)
{
    if (!ctx) return CAME_ERR_NULL;
    if (!hp) return fail(ctx, CAME_ERR_NULL, "hparams is NULL");
    std::string msg;
    came_status s = validate_hparams(*hp, ctx->last_step, msg);
    if (s != CAME_OK) return fail(ctx, s, msg);
    s = check_current_device(ctx);
    if (s != CAME_OK) return s;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (grads) {
        bool changed = false;
        for (int i = 0; i < ctx->n; ++i) {
            if (!grads[i]) return fail(ctx, CAME_ERR_NULL, "a gradient pointer is NULL");
            // the tile plan (and with it the width of the loads) was fixed at create
            const size_t need = grad_alignment_for(ctx->tensors[i].grad_dtype, ctx->host_table[i].vec);
            if (!aligned(grads[i], need)) {
                char buf[120];
                std::snprintf(buf, sizeof buf, "tensor %d: replacement gradient pointer not %zu-byte aligned",
                              i, need);
                return fail(ctx, CAME_ERR_ALIGN, buf);
            }
            changed |= (grads[i] != ctx->host_table[i].g);
        }
        if (changed) {
            for (int i = 0; i < ctx->n; ++i) { ctx->host_table[i].g = grads[i]; ctx->tensors[i].grad = grads[i]; }
            s = upload_table(ctx, stream);
            if (s != CAME_OK) return s;
        }
    }
    return launch_step(ctx, hp, stream);
}

came_status came_step_host(came_ctx* ctx, const came_hparams* hp, const void* const* host_grads,
                           void* const* host_params_out, void* cuda_stream)
{
    if (!ctx) return CAME_ERR_NULL;
    if (!hp || !host_grads) return fail(ctx, CAME_ERR_NULL, "hparams or host_grads is NULL");
    std::string msg;
    came_status s = validate_hparams(*hp, ctx->last_step, msg);
    if (s != CAME_OK) return fail(ctx, s, msg);
    for (int i = 0; i < ctx->n; ++i)
        if (!host_grads[i]) return fail(ctx, CAME_ERR_NULL, "a host gradient pointer is NULL");
    s = check_current_device(ctx);
    if (s != CAME_OK) return s;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const StepConsts hc = make_consts(*hp);
    cudaError_t e;
#define CAME_CK(call, what) do { e = (call); if (e != cudaSuccess) return cuda_fail(ctx, e, what); } while (0)
    // Three-stage pipeline over groups of consecutive tensors (tensors are independent):
    // upload gradients of group k+1 | step group k | download parameters of group k-1.
    // The copy streams start after everything already queued on the caller's stream, and the
    // caller's stream ends up waiting for the last download.
    CAME_CK(cudaEventRecord(ctx->ev_start, stream), "cudaEventRecord");
    CAME_CK(cudaStreamWaitEvent(ctx->s_up, ctx->ev_start, 0), "cudaStreamWaitEvent");
    CAME_CK(cudaStreamWaitEvent(ctx->s_down, ctx->ev_start, 0), "cudaStreamWaitEvent");
    const size_t ng = ctx->host_groups.size();
    for (size_t k = 0; k < ng; ++k) {
        const Group& g = ctx->host_groups[k];
        for (int i = g.t0; i < g.t1; ++i) {
            const came_tensor& x = ctx->tensors[i];
            const size_t bytes = static_cast<size_t>(x.rows) * x.cols * (x.grad_dtype == CAME_BF16 ? 2 : 4);
            CAME_CK(cudaMemcpyAsync(const_cast<void*>(x.grad), host_grads[i], bytes,
                                    cudaMemcpyHostToDevice, ctx->s_up), "cudaMemcpyAsync(grad H2D)");
        }
        CAME_CK(cudaEventRecord(ctx->ev_up[k], ctx->s_up), "cudaEventRecord");
    }
    for (size_t k = 0; k < ng; ++k) {
        const Group& g = ctx->host_groups[k];
        CAME_CK(cudaStreamWaitEvent(stream, ctx->ev_up[k], 0), "cudaStreamWaitEvent");
        launch_range(ctx, hc, stream, g, nullptr);
        CAME_CK(cudaGetLastError(), "kernel launch");
        if (host_params_out) {
            CAME_CK(cudaEventRecord(ctx->ev_done[k], stream), "cudaEventRecord");
            CAME_CK(cudaStreamWaitEvent(ctx->s_down, ctx->ev_done[k], 0), "cudaStreamWaitEvent");
            for (int i = g.t0; i < g.t1; ++i) {
                if (!host_params_out[i]) continue;
                const came_tensor& x = ctx->tensors[i];
                const size_t bytes = static_cast<size_t>(x.rows) * x.cols * 4;
                CAME_CK(cudaMemcpyAsync(host_params_out[i], x.param, bytes, cudaMemcpyDeviceToHost,
                                        ctx->s_down), "cudaMemcpyAsync(param D2H)");
            }
        }
    }
    CAME_CK(cudaEventRecord(ctx->ev_all_down, ctx->s_down), "cudaEventRecord");
    CAME_CK(cudaStreamWaitEvent(stream, ctx->ev_all_down, 0), "cudaStreamWaitEvent");
#undef CAME_CK
    ctx->n_intervals = 0;
    ctx->last_step = hp->step;
    return CAME_OK;
}

came_status came_destroy(came_ctx* ctx)
{
    if (!ctx) return CAME_ERR_NULL;
    free_ctx(ctx);
    return CAME_OK;
}

came_status came_query(const came_ctx* ctx, int32_t what, int64_t* out)
{
    if (!ctx || !out) return CAME_ERR_NULL;
    switch (what) {
        case CAME_Q_NUMEL: *out = ctx->numel; break;
        case CAME_Q_STATE_BYTES: *out = ctx->state_bytes; break;
        case CAME_Q_STREAM_BYTES: *out = ctx->stream_bytes; break;
        case CAME_Q_COMPULSORY_BYTES: *out = ctx->comp_bytes; break;
        case CAME_Q_WORKSPACE_BYTES:
            *out = static_cast<int64_t>(ctx->ws_bytes + ctx->table_bytes + sizeof(Tile) * ctx->n_tiles +
                                        sizeof(came::Item) * ctx->n_items +
                                        sizeof(came::StreamTile) * ctx->n_stream + sizeof(Tile) * ctx->n_others +
                                        (ctx->d_sync ? sizeof(came::PipeSync) : 0));
            break;
        case CAME_Q_NUM_TILES: *out = ctx->n_tiles; break;
        case CAME_Q_LAUNCHES_PER_STEP:
            *out = ctx->pipelined ? 1 : (ctx->adafactor ? 3 : 4); break;
        case CAME_Q_LAST_STEP: *out = ctx->last_step; break;
        case CAME_Q_NUM_PHASES:
            *out = ctx->pipelined ? 1 : (ctx->adafactor ? 3 : 4); break;
        case CAME_Q_MATRIX_NUMEL: *out = ctx->matrix_numel; break;
        case CAME_Q_SCHEDULE: *out = ctx->pipelined ? 1 : 0; break;
        case CAME_Q_P1_STREAM_GRID: *out = ctx->pipelined ? 0 : ctx->p1_stream_grid; break;
        case CAME_Q_PIPE_GROUPS: *out = ctx->pipe_groups; break;
        case CAME_Q_PIPE_GRID: *out = ctx->pipe_grid; break;
        case CAME_Q_DEVICE_ERROR: {
            *out = 0;
            if (ctx->pipelined) {
                came::PipeSync h;
                const cudaError_t e = cudaMemcpy(&h, ctx->d_sync, sizeof h, cudaMemcpyDeviceToHost);
                if (e != cudaSuccess) return CAME_ERR_CUDA;
                *out = h.error ? (static_cast<int64_t>(h.error) | (static_cast<int64_t>(h.err_item) << 8)) : 0;
            }
            break;
        }
        default: return CAME_ERR_UNSUPPORTED;
    }
    return CAME_OK;
}

came_status came_clear_device_error(came_ctx* ctx, void* cuda_stream)
{
    if (!ctx) return CAME_ERR_NULL;
    const came_status s = check_current_device(ctx);
    if (s != CAME_OK) return s;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // arrival counters, flags and partial sums all start from zero again
    cudaError_t e = cudaMemsetAsync(ctx->d_ws, 0, std::max<size_t>(ctx->ws_bytes, 256), stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemsetAsync(workspace)");
    if (ctx->d_sync) {
        e = cudaMemsetAsync(ctx->d_sync, 0, sizeof(came::PipeSync), stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemsetAsync(sync)");
    }
    return CAME_OK;
}

came_status came_selftest_wait_timeout(int32_t device, int64_t limit_ns, int32_t* out_timed_out,
                                       int32_t* out_error_word, float* out_elapsed_ms)
{
    if (!out_timed_out || !out_error_word || !out_elapsed_ms)
        return fail(nullptr, CAME_ERR_NULL, "output pointer is NULL");
    if (limit_ns < 1000 || limit_ns > 1000000000ll)
        return fail(nullptr, CAME_ERR_UNSUPPORTED, "limit_ns must lie in [1 us, 1 s]");
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(nullptr, CAME_ERR_DEVICE, "cudaSetDevice failed"); }
    unsigned* d = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    came_status st = CAME_OK;
    unsigned h[4] = {0, 0, 0, 0};
    float ms = 0.f;
    do {
        if ((e = cudaMalloc(&d, sizeof h)) != cudaSuccess) break;
        if ((e = cudaMemset(d, 0, sizeof h)) != cudaSuccess) break;
        if ((e = cudaEventCreate(&a)) != cudaSuccess) break;
        if ((e = cudaEventCreate(&b)) != cudaSuccess) break;
        cudaEventRecord(a, 0);
        came::k_wait_probe<<<1, 32>>>(d, static_cast<unsigned long long>(limit_ns));
        cudaEventRecord(b, 0);
        if ((e = cudaGetLastError()) != cudaSuccess) break;
        if ((e = cudaMemcpy(h, d, sizeof h, cudaMemcpyDeviceToHost)) != cudaSuccess) break;
        if ((e = cudaEventElapsedTime(&ms, a, b)) != cudaSuccess) break;
    } while (false);
    if (e != cudaSuccess) st = cuda_fail(nullptr, e, "wait self-test");
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    cudaFree(d);
    if (st != CAME_OK) return st;
    *out_timed_out = static_cast<int32_t>(h[3]);
    *out_error_word = static_cast<int32_t>(h[1]);
    *out_elapsed_ms = ms;
    return CAME_OK;
}

came_status came_debug_bounds(int32_t device, uint32_t* out6)
{
    if (!out6) return fail(nullptr, CAME_ERR_NULL, "output pointer is NULL");
#ifdef CAME_DEBUG_BOUNDS
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(nullptr, CAME_ERR_DEVICE, "cudaSetDevice failed"); }
    unsigned h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    e = cudaMemcpyFromSymbol(h, came::g_debug_bounds, sizeof h);        // synchronises
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaMemcpyFromSymbol(debug record)");
    for (int k = 0; k < 6; ++k) out6[k] = h[k];
    return CAME_OK;
#else
    (void)device;
    for (int k = 0; k < 6; ++k) out6[k] = 0u;
    return fail(nullptr, CAME_ERR_UNSUPPORTED, "this library was built without CAME_DEBUG_BOUNDS");
#endif
}

came_status came_set_profiling(came_ctx* ctx, int32_t enabled)
{
    if (!ctx) return CAME_ERR_NULL;
    if (enabled && ctx->prof_ev.empty()) {
        cudaSetDevice(ctx->device);
        ctx->prof_ev.assign(static_cast<size_t>(kProfSlots) * (kMaxPhases + 1), nullptr);
        for (cudaEvent_t& e : ctx->prof_ev) {
            const cudaError_t err = cudaEventCreate(&e);
            if (err != cudaSuccess) return cuda_fail(ctx, err, "cudaEventCreate");
        }
    }
    ctx->profiling = enabled != 0;
    ctx->prof_count = 0;
    return CAME_OK;
}

came_status came_get_phase_ms(came_ctx* ctx, float* out_ms, int32_t cap, int32_t* out_count)
{
    if (!ctx || !out_ms || !out_count) return CAME_ERR_NULL;
    *out_count = 0;
    if (ctx->prof_count == 0) return fail(ctx, CAME_ERR_UNSUPPORTED, "no profiled step recorded");
    const int slots = static_cast<int>(std::min<long long>(ctx->prof_count, kProfSlots));
    const int last = static_cast<int>((ctx->prof_count - 1) % kProfSlots);
    cudaError_t e = cudaEventSynchronize(ctx->prof_ev[last * (kMaxPhases + 1) + ctx->n_intervals]);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventSynchronize");
    const int k = std::min<int>(cap, ctx->n_intervals);
    for (int i = 0; i < k; ++i) {
        double sum = 0.0;
        for (int sl = 0; sl < slots; ++sl) {
            float ms = 0.f;
            const cudaEvent_t* ev = &ctx->prof_ev[sl * (kMaxPhases + 1)];
            e = cudaEventElapsedTime(&ms, ev[i], ev[i + 1]);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventElapsedTime");
            sum += ms;
        }
        out_ms[i] = static_cast<float>(sum / slots);
    }
    *out_count = k;
    return CAME_OK;
}

const char* came_phase_name(const came_ctx* ctx, int32_t phase)
{
    if (!ctx || phase < 0) return "";
    if (ctx->pipelined) return phase == 0 ? "step_pipelined" : "";
    // phases are reported in launch order
    const bool ada = ctx->adafactor;
    const bool has[kMaxPhases] = {true, true, !ada, !ada, ada};
    int idx = 0;
    for (int k = 0; k < kMaxPhases; ++k) {
        if (!has[k]) continue;
        if (idx == phase) return kPhaseNames[k];
        ++idx;
    }
    return "";
}

}  // extern "C"

// =============================================================================================
// Allocation-free factor update (came_factor_update_static).  Everything it needs on the
// device beyond the caller's buffers lives in g_static_scratch below.
// =============================================================================================
namespace {

// Partial sums, finished-factor scales, arrival counters and scalars of ONE matrix.
// Device memory owned by the library image; see the header for the sharing rules.
static __device__ __align__(256) unsigned char g_static_scratch[CAME_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// One block per tile of the single matrix described by `d` (passed by value): the tile
// indices come from the block index, so no device-resident table or tile list is needed.
__global__ void __launch_bounds__(came::kThreads, CAME_P1_MINB)
k_p1_reduce_g2_single(const TensorDev d, StepConsts hc)
{
    __shared__ came::Shared sm;
    const int rb = static_cast<int>(blockIdx.x) / d.n_cb;
    const int cb = static_cast<int>(blockIdx.x) % d.n_cb;
    using namespace came;
    CAME_DISPATCH(p1_tile, d, rb, cb, hc, sm)
}

}  // namespace

namespace {

struct StaticLayout {
    Plan p;
    size_t need = 0;
    size_t colpart = 0, colpart2 = 0, rowpart = 0, blocksum = 0, rowscale = 0, colscale = 0, cnt = 0,
           scal = 0;
};

// Host-only: validates the arguments of came_factor_update_static and lays its partial sums
// out in the built-in scratch array.  The tile grows (fewer, taller tiles) until they fit.
// The width of the gradient loads follows the pointer actually passed: 256-bit loads of fp32
// gradients only when it is 32-byte aligned, else 128-bit.
came_status plan_static(const void* grad, int32_t grad_dtype, int64_t rows, int64_t cols,
                        const float* r, const float* c, double beta2, double eps1, int32_t device,
                        StaticLayout& L)
{
    if (!grad || !r || !c) return fail(nullptr, CAME_ERR_NULL, "grad, r and c are required");
    if (rows < 1 || cols < 1 || rows > (1ll << 40) / cols)
        return fail(nullptr, CAME_ERR_SHAPE, "rows and cols must be >= 1 and rows*cols <= 2^40");
    if (grad_dtype != CAME_F32 && grad_dtype != CAME_BF16)
        return fail(nullptr, CAME_ERR_DTYPE, "unknown grad_dtype");
    if (!aligned(grad, 16) || !aligned(r, 16) || !aligned(c, 16))
        return fail(nullptr, CAME_ERR_ALIGN, "pointer not 16-byte aligned");
    if (!std::isfinite(beta2) || beta2 < 0.0 || beta2 >= 1.0 || !std::isfinite(eps1) || eps1 < 0.0)
        return fail(nullptr, CAME_ERR_HPARAM, "beta2 must lie in [0,1) and eps1 must be >= 0");
    if (device < 0 || device >= kMaxDevices)
        return fail(nullptr, CAME_ERR_DEVICE, "device ordinal out of range");

    const bool a32 = grad_dtype == CAME_BF16 || aligned(grad, 32);
    for (long long target = 32768; ; target *= 2) {
        Plan& p = L.p;
        p = plan_tensor(rows, cols, 2, grad_dtype, a32, target);
        size_t ws = 0;
        auto take = [&](size_t bytes) { const size_t o = ws; ws += (bytes + 255) / 256 * 256; return o; };
        L.cnt = take(sizeof(unsigned) * p.counters());
        L.scal = take(sizeof(float) * 4);
        L.blocksum = take(sizeof(float) * p.n_rb);
        L.colpart = take(sizeof(float) * static_cast<size_t>(p.n_rb) * cols);
        L.colpart2 = take(sizeof(float) * static_cast<size_t>(p.n_grp) * cols);
        L.rowpart = take(sizeof(float) * static_cast<size_t>(p.n_seg) * rows);
        L.rowscale = take(sizeof(float) * static_cast<size_t>(rows));
        L.colscale = take(sizeof(float) * static_cast<size_t>(cols));
        L.need = ws;
        if (L.need <= CAME_STATIC_SCRATCH_BYTES || p.n_rb == 1 || target >= (1ll << 40)) break;
    }
    if (L.need > CAME_STATIC_SCRATCH_BYTES) {
        char buf[200];
        std::snprintf(buf, sizeof buf,
                      "matrix %lld x %lld needs %zu bytes of partial sums; the built-in scratch holds %u",
                      static_cast<long long>(rows), static_cast<long long>(cols), L.need,
                      static_cast<unsigned>(CAME_STATIC_SCRATCH_BYTES));
        return fail(nullptr, CAME_ERR_UNSUPPORTED, buf);
    }
    if (static_cast<long long>(L.p.n_rb) * L.p.n_cb > (1ll << 30))
        return fail(nullptr, CAME_ERR_SHAPE, "too many tiles");
    if (grad_alignment_for(grad_dtype, L.p.vec) > 16 && !aligned(grad, 32))
        return fail(nullptr, CAME_ERR_INTERNAL, "plan wider than the gradient pointer's alignment");
    return CAME_OK;
}

}  // namespace

extern "C" came_status came_factor_update_static_plan(const void* grad, int32_t grad_dtype,
                                                      int64_t rows, int64_t cols, const float* r,
                                                      const float* c, double beta2, double eps1,
                                                      int32_t device, int32_t* out_vec,
                                                      int64_t* out_scratch_bytes)
{
    StaticLayout L;
    const came_status s = plan_static(grad, grad_dtype, rows, cols, r, c, beta2, eps1, device, L);
    if (s != CAME_OK) return s;
    if (out_vec) *out_vec = L.p.vec;
    if (out_scratch_bytes) *out_scratch_bytes = static_cast<int64_t>(L.need);
    return CAME_OK;
}

extern "C" came_status came_factor_update_static(const void* grad, int32_t grad_dtype, int64_t rows,
                                                 int64_t cols, float* r, float* c, double beta2,
                                                 double eps1, float* out_sqrt_sum_r, int32_t device,
                                                 void* cuda_stream)
{
    StaticLayout off;
    const came_status st = plan_static(grad, grad_dtype, rows, cols, r, c, beta2, eps1, device, off);
    if (st != CAME_OK) return st;
    if (out_sqrt_sum_r && !aligned(out_sqrt_sum_r, 4))
        return fail(nullptr, CAME_ERR_ALIGN, "out_sqrt_sum_r not 4-byte aligned");
    const Plan& p = off.p;

    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(nullptr, CAME_ERR_DEVICE, "cudaSetDevice failed"); }
    if (!g_static_scratch_addr[device]) {
        // The array's name is only a host-side handle; kernels need its device address.
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetSymbolAddress(scratch)");
        g_static_scratch_addr[device] = ptr;
    }
    char* base = static_cast<char*>(g_static_scratch_addr[device]);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // The arrival counters and scalars must start at zero whatever the last call left behind.
    e = cudaMemsetAsync(base, 0, off.blocksum, stream);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaMemsetAsync(scratch counters)");

    TensorDev d;
    std::memset(&d, 0, sizeof d);
    d.g = grad; d.r = r; d.c = c;
    d.rows = rows; d.cols = cols;
    d.cnt = reinterpret_cast<unsigned*>(base + off.cnt);
    d.scal = reinterpret_cast<float*>(base + off.scal);
    d.ws_blocksum = reinterpret_cast<float*>(base + off.blocksum);
    d.ws_colpart = reinterpret_cast<float*>(base + off.colpart);
    d.ws_colpart2 = reinterpret_cast<float*>(base + off.colpart2);
    d.ws_rowpart = reinterpret_cast<float*>(base + off.rowpart);
    d.ws_rowscale = reinterpret_cast<float*>(base + off.rowscale);
    d.ws_colscale = reinterpret_cast<float*>(base + off.colscale);
    d.ws_usq = d.scal;          // unused by this phase
    d.kind = p.kind; d.vec = p.vec;
    int lg = 0; while ((1 << lg) < p.tx) ++lg;
    d.tx_log2 = lg; d.tr = p.tr; d.n_rb = p.n_rb; d.n_cb = p.n_cb; d.n_seg = p.n_seg;
    d.n_grp = p.n_grp;
    d.n_parts = p.n_parts; d.ndim = 2; d.flags = 0;

    StepConsts hc;
    std::memset(&hc, 0, sizeof hc);
    hc.beta2 = static_cast<float>(beta2);
    hc.omb2 = static_cast<float>(1.0 - beta2);
    hc.eps1 = static_cast<float>(eps1);
    hc.gscale = 1.f;
    hc.gscale2 = 1.f;
    hc.clip_d = 1.0;
    k_p1_reduce_g2_single<<<p.n_rb * p.n_cb, came::kThreads, 0, stream>>>(d, hc);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "kernel launch");
    if (out_sqrt_sum_r) {
        e = cudaMemcpyAsync(out_sqrt_sum_r, d.scal, sizeof(float), cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaMemcpyAsync(sqrt sum r)");
    }
    return CAME_OK;
}
