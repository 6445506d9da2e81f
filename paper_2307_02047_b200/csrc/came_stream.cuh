// Streaming form of the first phase of the CAME step (r_t, c_t of Algorithm 2) for sm_100a:
// a persistent grid that stages the gradient through per-thread rings of asynchronous copies.
// Uses the tile routines and reductions of came_kernels.cuh.
#pragma once
#include "came_kernels.cuh"

namespace came {

// ---------------------------------------------------------------------------
// Streaming P1 (Algorithm 2: r_t, c_t): the same sums as p1_tile, bit for bit, with the
// gradient staged through a per-thread ring of asynchronous 16-byte copies into shared
// memory (cp.async) and a persistent grid.
//
// Why: p1_tile keeps the loads of one batch of rows in registers, so a block has nothing in
// flight while it runs its per-tile epilogue (store partials -> fence -> barrier -> arrival
// atomics -> barrier, about 3 us).  With tiles of 64-128 KB that epilogue is a fifth of the
// tile's time and P1 is limited by bytes in flight, not by DRAM.  Here every thread owns
// NB x 8 slots of 16 bytes in shared memory and keeps up to NB batches of its own loads in
// flight, across tile boundaries: while the block is in the epilogue of one tile the first
// batches of its next tile are already on their way.  A thread only ever reads the slots it
// filled itself, after cp.async.wait_group, so the ring needs no barrier and no waiting on
// anybody else.  Batches, row order and reduction trees are those of p1_tile, hence the
// identical results.
//
// Measured on B200 (BERT-large-shaped set, ncu): the ring does what it is for -- long-scoreboard
// stalls per issued instruction fall from 7.9 to 1.4 -- but the phase then proves to be bound by
// instruction issue (about 40 % of peak in both forms), and this form executes 96 M warp
// instructions where p1_tile executes 63 M (copy, shared-memory read, ring bookkeeping), so it
// takes 204 us against 132 us.  It is therefore an option (CAME_TUNE_P1_STREAM), not the default.
//
// The grid is persistent: block b takes stream tiles b, b + gridDim.x, ...; afterwards it
// runs the tiles the ring cannot serve (scalar kinds) and the vector chunks through the
// ordinary routines.
// ---------------------------------------------------------------------------
struct __align__(16) StreamTile {
    const char* g;        // first element of the tile: (first row, first column of the strip)
    float*      rowpart;  // ws_rowpart + (first segment of the strip) * rows + first row
    long long   rows;     // rows of the tensor (distance between two segments in rowpart)
    int         tensor, rb, cb;
    int         nrows;    // rows in the tile
    int         ncols;    // valid columns in the strip (<= threads across * vec)
    int         cols;     // row pitch in elements
    int         kind_tx;  // kind | tx_log2 << 8
    int         pad_[3];
};
static_assert(sizeof(StreamTile) == 64, "four 16-byte loads");

__device__ __forceinline__ StreamTile load_stream_tile(const StreamTile* p)
{
    StreamTile r;
    const uint4* src = reinterpret_cast<const uint4*>(p);
    uint4* dst = reinterpret_cast<uint4*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) dst[i] = __ldg(src + i);
    return r;
}

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src)
{
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most `pending` of this thread's most recent copy groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending)
{
    switch (pending) {
        case 0:  asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1:  asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2:  asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    }
}

constexpr int kStreamSlots = 8;          // 16-byte slots per thread per batch, whatever the kind
constexpr int kStreamMaxBatches = 4;     // ring depth the wait above can express

template <int KIND> struct StreamTraits;            // U thread-rows per batch, CH 16-byte chunks per row
template <> struct StreamTraits<kF32x4>  { static constexpr int U = 8, CH = 1; };
template <> struct StreamTraits<kBF16x8> { static constexpr int U = 8, CH = 1; };
template <> struct StreamTraits<kF32x8>  { static constexpr int U = 4, CH = 2; };
static_assert(CAME_P12_U == 8, "the streaming kernel reproduces p1_tile's batches of 8 (4) thread-rows");

__device__ __forceinline__ int stream_batches(const StreamTile& r)
{
    const int txl = r.kind_tx >> 8;
    const int TY = kThreads >> txl;
    const int U = ((r.kind_tx & 0xff) == kF32x8) ? 4 : 8;
    const int thread_rows = (r.nrows + TY - 1) / TY;
    return (thread_rows + U - 1) / U;
}

// Starts the copies of batch `b` of tile `r` into this thread's slots of one ring batch
// (`ring` points at [kStreamSlots][kThreads] uint4) and closes the copy group.
__device__ __forceinline__ void stream_issue(const StreamTile& r, int b, uint4* ring, int tid)
{
    const int kind = r.kind_tx & 0xff, txl = r.kind_tx >> 8;
    const int tx = tid & ((1 << txl) - 1), ty = tid >> txl, TY = kThreads >> txl;
    const int vec = (kind == kF32x4) ? 4 : 8;
    const int esz = (kind == kBF16x8) ? 2 : 4;
    const int chl = (kind == kF32x8) ? 1 : 0;                // log2 of chunks per row
    const int U = kStreamSlots >> chl;
    const int col = tx * vec;
    if (col < r.ncols) {
        const long long pitch = static_cast<long long>(r.cols) * esz;
        const char* src0 = r.g + static_cast<long long>(col) * esz;
#pragma unroll
        for (int j = 0; j < kStreamSlots; ++j) {
            const int k = j >> chl, c = j & ((1 << chl) - 1);
            const int row = ty + (b * U + k) * TY;
            if (row < r.nrows) cp_async_16(ring + j * kThreads + tid, src0 + row * pitch + 16 * c);
        }
    }
    cp_async_commit();
}

// Adds batch `b` of tile `r`, which has landed in `ring`, to the column accumulators and
// stores its row partial sums: the arithmetic of p1_tile's loop body.
template <int KIND>
__device__ __forceinline__ void stream_consume_p1(const StreamTile& r, int b, const uint4* ring,
                                                  float (&cacc)[Traits<KIND>::VEC], int tid)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = StreamTraits<KIND>::U, CH = StreamTraits<KIND>::CH;
    const int txl = r.kind_tx >> 8;
    const int tx = tid & ((1 << txl) - 1), ty = tid >> txl, TY = kThreads >> txl;
    const bool colok = tx * VEC < r.ncols;
    float rs[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int row = ty + (b * U + k) * TY;
        Raw<KIND> raw;
        if (colok && row < r.nrows) {
            if constexpr (KIND == kF32x8) {
                const uint4 a = ring[(k * CH) * kThreads + tid], bb = ring[(k * CH + 1) * kThreads + tid];
                raw.v[0] = __uint_as_float(a.x); raw.v[1] = __uint_as_float(a.y);
                raw.v[2] = __uint_as_float(a.z); raw.v[3] = __uint_as_float(a.w);
                raw.v[4] = __uint_as_float(bb.x); raw.v[5] = __uint_as_float(bb.y);
                raw.v[6] = __uint_as_float(bb.z); raw.v[7] = __uint_as_float(bb.w);
            } else if constexpr (KIND == kF32x4) {
                const uint4 a = ring[k * kThreads + tid];
                raw.v = make_float4(__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z),
                                    __uint_as_float(a.w));
            } else {
                raw.v = ring[k * kThreads + tid];
            }
        } else {
            zero_raw<KIND>(raw);
        }
        float x[VEC];
        unpack<KIND>(raw, x);
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            cacc[v] = fmaf(x[v], x[v], cacc[v]);
            s = fmaf(x[v], x[v], s);
        }
        rs[k] = s;
    }
    float* const rowpart_seg = r.rowpart + static_cast<long long>(tx >> 5) * r.rows;
    store_row_partials<U>(rs, rowpart_seg, ty + static_cast<long long>(b) * U * TY, TY, r.nrows, tid & 31);
}

// One tile of the streaming P1: consumes its batches (topping the ring up from this tile and
// the next one as slots free up), then the per-tile epilogue of p1_tile.
template <int KIND>
__device__ __forceinline__ void stream_tile_p1(const TensorDev* __restrict__ T, const StreamTile& cur,
                                               const StreamTile& nxt, bool has_nxt, int nb_ring,
                                               uint4* ring, unsigned& issued, unsigned& consumed,
                                               int& iq, int& ib, const StepConsts& hc, Shared& sm)
{
    constexpr int VEC = Traits<KIND>::VEC;
    const int tid = threadIdx.x;
    const int nb_cur = stream_batches(cur), nb_nxt = has_nxt ? stream_batches(nxt) : 0;
    float cacc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) cacc[v] = 0.f;
    for (int b = 0; b < nb_cur; ++b) {
        // top the ring up: next batch of this tile, else of the next tile
        while (static_cast<int>(issued - consumed) < nb_ring) {
            if (iq == 0 && ib == nb_cur) { iq = 1; ib = 0; }
            uint4* slot = ring + static_cast<size_t>(issued % nb_ring) * (kStreamSlots * kThreads);
            if (iq == 0) stream_issue(cur, ib, slot, tid);
            else if (ib < nb_nxt) stream_issue(nxt, ib, slot, tid);
            else break;
            ++ib;
            ++issued;
        }
        cp_async_wait_pending(static_cast<int>(issued - consumed) - 1);
        stream_consume_p1<KIND>(cur, b, ring + static_cast<size_t>(consumed % nb_ring) * (kStreamSlots * kThreads),
                                cacc, tid);
        ++consumed;
    }
    const TensorDev d = T[cur.tensor];
    const Geo q = make_geo<VEC>(d, cur.rb, cur.cb);
    CAME_DEBUG_SKIP_TILE(q);
    write_col_partials<VEC>(d, q, cur.rb, cacc, sm);
    finalize_factors(d, cur.rb, cur.cb, hc.beta2, hc.omb2, hc.eps1, hc.gscale2, d.r, d.c, d.scal + 0, sm);
    block_sync();          // the scratch is free again before the next tile's epilogue uses it
}

#ifndef CAME_P1_STREAM_MINB
#define CAME_P1_STREAM_MINB 3
#endif

__global__ void __launch_bounds__(kThreads, CAME_P1_STREAM_MINB)
k_p1_stream(const TensorDev* __restrict__ T, const StreamTile* __restrict__ st, int nstream,
            const Tile* __restrict__ others, int nothers, int nb_ring, StepConsts hc)
{
    extern __shared__ uint4 stream_ring[];      // [nb_ring][kStreamSlots][kThreads]
    __shared__ Shared sm;
    pdl_release_dependents();
    const int G = static_cast<int>(gridDim.x);
    int t = static_cast<int>(blockIdx.x);
    StreamTile cur, nxt;
    bool has_cur = t < nstream, has_nxt = t + G < nstream;
    if (has_cur) cur = load_stream_tile(st + t);
    if (has_nxt) nxt = load_stream_tile(st + t + G);
    pdl_wait_for_previous_grid();
    unsigned issued = 0u, consumed = 0u;
    int iq = 0, ib = 0;                         // where the next copy batch comes from: tile (0 cur, 1 nxt), batch
    while (has_cur) {
        switch (cur.kind_tx & 0xff) {
            case kF32x4:  stream_tile_p1<kF32x4>(T, cur, nxt, has_nxt, nb_ring, stream_ring, issued, consumed, iq, ib, hc, sm); break;
            case kF32x8:  stream_tile_p1<kF32x8>(T, cur, nxt, has_nxt, nb_ring, stream_ring, issued, consumed, iq, ib, hc, sm); break;
            default:      stream_tile_p1<kBF16x8>(T, cur, nxt, has_nxt, nb_ring, stream_ring, issued, consumed, iq, ib, hc, sm); break;
        }
        // advance: the next tile becomes the current one; copies already started for it stay valid
        if (iq == 1) { iq = 0; } else { ib = 0; }
        t += G;
        has_cur = has_nxt;
        cur = nxt;
        has_nxt = t + G < nstream;
        if (has_nxt) nxt = load_stream_tile(st + t + G);
    }
    // what the ring cannot serve: element-at-a-time matrices and the vector chunks
    for (int o = static_cast<int>(blockIdx.x); o < nothers; o += G) {
        const Tile tl = others[o];
        const TensorDev d = T[tl.tensor];
        if (d.ndim == 1) vec_second_moment_chunk(d, tl.rb, hc, sm);
        else if (d.kind == kF32x1) p1_tile<kF32x1>(d, tl.rb, tl.cb, hc, sm);
        else p1_tile<kBF16x1>(d, tl.rb, tl.cb, hc, sm);
        block_sync();
    }
}

}  // namespace came
