// CAME optimizer step, device code for sm_100a.
//
// One step of Algorithm 2 has three grid-wide data dependencies per tensor
// (r,c need all of g; the clip factor needs all of u; S needs all of U), so a
// matrix is streamed in four phases, each one kernel over a multi-tensor tile
// list (vectors ride along as extra tiles of P1 and P3):
//   P1  g            -> row/column sums of g^2        -> r_t, c_t, sqrt(1^T r_t)
//   P2  g, r, c      -> sum of u^2                    -> clip factor kappa (Eq. 1)
//   P3  g, m, r, c   -> m_t, row/column sums of (uhat - m_{t-1})^2 -> R_t, C_t, sqrt(1^T R_t)
//   P4  m, theta, R, C -> theta_t
// v_t and S_t (Eq. 2, rank one) are never formed: u = g * rsqrt(r_i) * sqrt(sum r) * rsqrt(c_j),
// which also keeps r_i * c_j out of fp32 (it underflows for zero-gradient rows).  The
// rsqrt of every finished row and column factor is stored once by the tile that finishes it.
//
// Reductions are deterministic: every tile writes its partial sums to a
// workspace and the LAST tile to arrive (per row block; per group of 16 row
// blocks of a column strip, then per strip; per tensor -- counted with atomics)
// adds them in a fixed order.  In the one-grid-per-phase schedule no thread ever
// waits on another block.
//
// Second schedule, k_step_pipelined: ONE persistent grid runs the whole step.  Its blocks
// draw tickets, in order, from a list of (tensor, tile, phase) items that the host has
// arranged so that groups of tensors small enough for the L2 move through P1..P4 one
// pipeline stage apart: a group's gradient is read from HBM once (P1) and from the L2 in P2
// and P3, and its momentum written by P3 is still in the L2 when P4 reads it.  An item that
// needs a tensor-wide result (r,c / kappa / R,C) of an earlier phase waits for that tensor's
// "phase done" flag.  Every flag an item waits for is set by items with LOWER ticket numbers,
// and a ticket is only ever held by a block that is running, so the lowest unfinished ticket
// can always proceed: the waits end without any assumption about how many blocks are
// resident.  Each wait is nevertheless bounded (time and iteration limit): when it runs out
// the block records an error word and every block leaves the grid.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace came {

// Occupancy and unroll choices (resident blocks per SM, thread-rows in flight per thread).
#ifndef CAME_P1_MINB
#define CAME_P1_MINB 4
#endif
#ifndef CAME_P2_MINB
#define CAME_P2_MINB 4
#endif
#ifndef CAME_P3_MINB
#define CAME_P3_MINB 2
#endif
#ifndef CAME_P4_MINB
#define CAME_P4_MINB 2
#endif
#ifndef CAME_P12_U
#define CAME_P12_U 8
#endif
#ifndef CAME_P34_U
#define CAME_P34_U 4
#endif

constexpr int kThreads = 256;          // threads that work on a tile
constexpr int kHelperThreads = 32;     // pipelined grid only: one more warp that runs ahead
constexpr int kVecPerThread = 4;
constexpr int kVecChunk = kThreads * kVecPerThread;   // vector elements per tile (one block)
constexpr int kColGroup = 16;         // row blocks per group in the two-level column reduction

enum Kind : int { kF32x4 = 0, kBF16x8 = 1, kF32x1 = 2, kBF16x1 = 3, kF32x8 = 4 };

struct TensorDev {
    float*       p;
    const void*  g;
    float*       m;
    float*       r;      // vectors: v
    float*       c;
    float*       R;      // vectors: S
    float*       C;
    long long    rows, cols;
    float*       ws_colpart;   // [n_rb][cols]   per-tile column partial sums
    float*       ws_colpart2;  // [n_grp][cols]  sums of kColGroup consecutive row blocks' partials
    float*       ws_rowpart;   // [n_seg][rows]  per-warp-segment row partial sums
    float*       ws_blocksum;  // [n_rb]         sum of the finished row factor over one row block
                               // (+ [n_cb] sums of the column factor per strip for kFlagSumCols)
    float*       ws_usq;       // [n_parts]      per-tile partial sums of u^2
    float*       ws_rowscale;  // [rows]  rsqrt of the row factor last finished (r_t, then R_t)
    float*       ws_colscale;  // [cols]  rsqrt of the column factor last finished (c_t, then C_t)
    unsigned*    cnt;          // [n_rb] row-block arrivals, [n_cb] finished groups per strip,
                               // [1] finished, [1] usq, [n_grp*n_cb] arrivals per (group, strip)
    float*       scal;         // [0] sqrt(sum r)  [1] kappa  [2] sqrt(sum R)
    unsigned*    done;         // pipelined schedule: [0] r,c final  [1] kappa final  [2] R,C final,
                               // each holding the number of the last step that finished it
    uint16_t*    p_bf16;       // optional bf16 copy of the updated parameters (NULL = none)
    int          kind;
    int          vec;          // elements per thread per load
    int          tx_log2;      // threads across columns = 1 << tx_log2 (32..256)
    int          tr;           // rows per tile
    int          n_rb, n_cb, n_seg;
    int          n_grp;        // ceil(n_rb / kColGroup)
    int          n_parts;      // matrices: n_rb*n_cb; vectors: number of chunks
    int          ndim;
    unsigned     flags;
};

struct Tile { int tensor, rb, cb; };   // vectors: rb = chunk of kVecChunk elements, cb = 0

// One unit of work of the pipelined schedule: a tile (or vector chunk) in one phase.
// phase 0 = P1 (vectors: second moment and kappa), 1 = P2, 2 = P3 (vectors: apply;
// Algorithm 1: the fused momentum + apply pass), 3 = P4.
struct Item { int tensor, rb, cb, phase; };

// Device-resident control block of the pipelined schedule (one per context).
struct PipeSync {
    unsigned ticket;      // next item to hand out; reset by the last block to leave
    unsigned exited;      // blocks that have left the current grid
    unsigned epoch;       // number of steps completed; a step publishes flags equal to epoch + 1
    unsigned error;       // 0 = fine; kPipeErr* once a wait has run out (sticky until cleared)
    unsigned err_item;    // ticket whose wait ran out
    unsigned pad_[3];
};
constexpr unsigned kPipeErrWaitTimeout = 1u;

struct StepConsts {
    float beta1, omb1, b1sq;
    float beta2, omb2;
    float beta3, omb3;
    float eps1, eps2;
    float lr, wd;
    float gscale, gscale2;   // gradient pre-scale s and s^2 (g_t = s * gradient buffer)
    float pad_;
    double clip_d;
};

constexpr unsigned kFlagNoWd = 1u << 0;
constexpr unsigned kFlagVecNoConf = 1u << 1;
// Internal: the tensor is an n x 1 matrix handled as its 1 x n view (same memory) with the
// row and column factors swapped, so that all lanes work; the normaliser 1_n^T r of
// Algorithm 2 is then the sum of the view's COLUMN factor.
constexpr unsigned kFlagSumCols = 1u << 8;

// ---------------------------------------------------------------------------
// loads / stores
// ---------------------------------------------------------------------------
template <int KIND> struct Traits;
template <> struct Traits<kF32x4>  { static constexpr int VEC = 4; };
template <> struct Traits<kBF16x8> { static constexpr int VEC = 8; };
template <> struct Traits<kF32x8>  { static constexpr int VEC = 8; };   // 256-bit gradient loads
template <> struct Traits<kF32x1>  { static constexpr int VEC = 1; };
template <> struct Traits<kBF16x1> { static constexpr int VEC = 1; };

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// fp32 state load/store: 1, 4 (128-bit) or 8 (256-bit, sm_100) floats per thread
template <int VEC>
__device__ __forceinline__ void load_f(const float* p, float (&x)[VEC])
{
    if constexpr (VEC == 8) {
        asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]),
                       "=f"(x[4]), "=f"(x[5]), "=f"(x[6]), "=f"(x[7]) : "l"(p));
    } else if constexpr (VEC == 4) {
        asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]) : "l"(p));
    } else {
        x[0] = __ldcg(p);
    }
}

template <int VEC>
__device__ __forceinline__ void store_f(float* p, const float (&x)[VEC])
{
    if constexpr (VEC == 8) {
        asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]),
                        "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7]) : "memory");
    } else if constexpr (VEC == 4) {
        asm volatile("st.global.v4.f32 [%0], {%1,%2,%3,%4};"
                     :: "l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]) : "memory");
    } else {
        *p = x[0];
    }
}

// two fp32 -> packed bf16x2, round to nearest even (lo in the low half)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// bf16 copy of VEC consecutive fp32 values (VEC = 8: one 128-bit store, 4: 64-bit, 1: 16-bit)
template <int VEC>
__device__ __forceinline__ void store_bf16(uint16_t* p, const float (&x)[VEC])
{
    if constexpr (VEC == 8) {
        uint4 v;
        v.x = pack_bf16x2(x[0], x[1]); v.y = pack_bf16x2(x[2], x[3]);
        v.z = pack_bf16x2(x[4], x[5]); v.w = pack_bf16x2(x[6], x[7]);
        *reinterpret_cast<uint4*>(p) = v;
    } else if constexpr (VEC == 4) {
        uint2 v;
        v.x = pack_bf16x2(x[0], x[1]); v.y = pack_bf16x2(x[2], x[3]);
        *reinterpret_cast<uint2*>(p) = v;
    } else {
        *p = static_cast<uint16_t>(pack_bf16x2(x[0], 0.f) & 0xffffu);
    }
}

// ---------------------------------------------------------------------------
// block-level helpers (deterministic: fixed shuffle tree, fixed warp order)
// ---------------------------------------------------------------------------
// Barrier over the kThreads threads that work on a tile (hardware barrier 1).  In the phase
// kernels these are all threads of the block; the pipelined grid has one more warp that must
// not take part.
__device__ __forceinline__ void block_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
static_assert(kThreads == 256, "block_sync names the thread count");
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct Shared {
    float  colred[kThreads * 8];   // cross-row-group column reduction
    double red[kThreads / 32];
    int    flag[4];
};

// Sum over the tile's threads; result valid in every one of them.  Two barriers.
template <typename T>
__device__ __forceinline__ T block_sum(T v, Shared& sm)
{
    v = warp_sum(v);
    block_sync();
    if ((threadIdx.x & 31) == 0) sm.red[threadIdx.x >> 5] = static_cast<double>(v);
    block_sync();
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) s += sm.red[w];
    return static_cast<T>(s);
}

// Sums U per-thread values across the 32 lanes of a warp with (U-1) + (5 - log2 U) shuffles.
// On return every lane holds the full sum of v[k] for k = lane >> (5 - log2 U).
template <int U>
__device__ __forceinline__ float multi_row_warp_sum(float (&v)[U], int lane)
{
    int o = 16;
#pragma unroll
    for (int n = U; n > 1; n >>= 1, o >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float keep = up ? v[i + n / 2] : v[i];
            const float send = up ? v[i] : v[i + n / 2];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    float r = v[0];
#pragma unroll
    for (; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    return r;
}

template <int U> struct Log2;
template <> struct Log2<1> { static constexpr int v = 0; };
template <> struct Log2<2> { static constexpr int v = 1; };
template <> struct Log2<4> { static constexpr int v = 2; };
template <> struct Log2<8> { static constexpr int v = 3; };

// Adds `count` (<= kColGroup) rows of partial sums, `stride` floats apart, for VW adjacent
// columns: eight rows are fetched per round trip to L2 before they are added, and the adds
// run in row order, so the result does not depend on timing.
template <int VW>
__device__ __forceinline__ void sum_partial_rows(const float* __restrict__ p, long long stride,
                                                 int count, float (&acc)[VW])
{
    constexpr int B = 8;                       // rows fetched per round trip
#pragma unroll
    for (int j = 0; j < VW; ++j) acc[j] = 0.f;
#pragma unroll
    for (int k0 = 0; k0 < kColGroup; k0 += B) {
        if (k0 >= count) break;
        float v[B][VW];
#pragma unroll
        for (int k = 0; k < B; ++k) {
            if (k0 + k < count) {
                if constexpr (VW == 4) {
                    const float4 t = __ldcg(reinterpret_cast<const float4*>(p + (k0 + k) * stride));
                    v[k][0] = t.x; v[k][1] = t.y; v[k][2] = t.z; v[k][3] = t.w;
                } else {
                    v[k][0] = __ldcg(p + (k0 + k) * stride);
                }
            } else {
#pragma unroll
                for (int j = 0; j < VW; ++j) v[k][j] = 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < B; ++k)
#pragma unroll
            for (int j = 0; j < VW; ++j) acc[j] += v[k][j];
    }
}

// ---------------------------------------------------------------------------
// "phase done" flags of the pipelined schedule.  The writer has made its results visible
// (fence, block barrier, counted arrival) before it publishes; the reader acquires the flag
// in one thread and the block barrier that follows orders every thread's later loads after it.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void publish_flag(unsigned* flag, unsigned epoch)
{
    __threadfence();
    asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(flag), "r"(epoch) : "memory");
}

__device__ __forceinline__ unsigned load_acquire(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Called by ONE thread.  Polls until *flag == epoch, another block has reported an error, or
// the limit runs out (limit_ns of wall time, and as a backstop limit_ns / 8 + 4096 polls, each
// of which takes well over 8 ns).  Returns true when the flag arrived.  On a timeout the
// error word is set (first reporter wins) and false is returned; the caller must then leave.
__device__ __forceinline__ bool wait_for_flag(const unsigned* flag, unsigned epoch,
                                              unsigned* error_word, unsigned* err_item,
                                              unsigned item, unsigned long long limit_ns)
{
    if (load_acquire(flag) == epoch) return true;
    const unsigned long long t0 = global_timer_ns();
    const unsigned long long max_polls = limit_ns / 8ull + 4096ull;
    unsigned ns = 32;
    for (unsigned long long it = 0; it < max_polls; ++it) {
        if (load_acquire(flag) == epoch) return true;
        if (load_acquire(error_word) != 0u) return false;
        if (global_timer_ns() - t0 > limit_ns) break;
        __nanosleep(ns);
        if (ns < 1024) ns <<= 1;
    }
    if (atomicCAS(error_word, 0u, kPipeErrWaitTimeout) == 0u) *err_item = item;
    __threadfence();
    return false;
}

// ---------------------------------------------------------------------------
// Last-arriver finalisation of one factored EMA (Algorithm 2: r_t, c_t from g^2
// with beta2/eps1; R_t, C_t from U_t with beta3/eps2):
//   row[i] = beta row[i] + (1-beta) (scale * sum_j X[i][j] + cols * eps)
//   col[j] = beta col[j] + (1-beta) (scale * sum_i X[i][j] + rows * eps)
// It also stores rsqrt(row[i]) and rsqrt(col[j]) for the phases that follow and,
// once every row block and strip of the tensor is finished, *sqrt_sum = sqrt(1_n^T row).
// Called by every tile of the tensor after it has written its partials.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void finalize_factors(const TensorDev& d, int rb, int cb, float beta,
                                                 float omb, float eps, float scale,
                                                 float* __restrict__ rowfac,
                                                 float* __restrict__ colfac,
                                                 float* __restrict__ sqrt_sum, Shared& sm,
                                                 unsigned* done_flag = nullptr, unsigned epoch = 0u)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grp = rb / kColGroup;
    const int grp_size = min(kColGroup, d.n_rb - grp * kColGroup);
    unsigned* const cnt_grp = d.cnt + d.n_rb + d.n_cb + 2;
    __threadfence();
    block_sync();
    if (tid == 0) {
        const unsigned a = atomicAdd(&d.cnt[rb], 1u);
        const unsigned b = atomicAdd(&cnt_grp[grp * d.n_cb + cb], 1u);
        sm.flag[0] = (a == static_cast<unsigned>(d.n_cb - 1));
        sm.flag[1] = (b == static_cast<unsigned>(grp_size - 1));
    }
    block_sync();
    const bool last_r = sm.flag[0] != 0, last_g = sm.flag[1] != 0;
    if (!last_r && !last_g) return;
    __threadfence();

    const long long rows = d.rows, cols = d.cols;
    if (last_r) {
        const long long row0 = static_cast<long long>(rb) * d.tr;
        const long long row1 = min(rows, row0 + d.tr);
        const float add = static_cast<float>(cols) * eps;
        float bs = 0.f;
        if (d.n_seg <= 32) {
            // few segments per row: one thread per row, segments added in order
            for (long long row = row0 + tid; row < row1; row += kThreads) {
                float s = 0.f;
#pragma unroll 8
                for (int sg = 0; sg < d.n_seg; ++sg) s += __ldcg(d.ws_rowpart + sg * rows + row);
                const float nv = fmaf(beta, __ldcg(rowfac + row), omb * fmaf(scale, s, add));
                rowfac[row] = nv;
                d.ws_rowscale[row] = __frsqrt_rn(nv);
                bs += nv;
            }
        } else {
            // many segments: one warp per row, lanes stride over the segments, fixed shuffle tree
            for (long long row = row0 + warp; row < row1; row += kThreads / 32) {
                float s = 0.f;
#pragma unroll 4
                for (int sg = lane; sg < d.n_seg; sg += 32) s += __ldcg(d.ws_rowpart + sg * rows + row);
                s = warp_sum(s);
                if (lane == 0) {
                    const float nv = fmaf(beta, __ldcg(rowfac + row), omb * fmaf(scale, s, add));
                    rowfac[row] = nv;
                    d.ws_rowscale[row] = __frsqrt_rn(nv);
                    bs += nv;
                }
            }
        }
        bs = block_sum(bs, sm);          // fixed order: warp tree, then warps 0..7
        if (tid == 0) { d.ws_blocksum[rb] = bs; d.cnt[rb] = 0u; }
    }
    bool last_c = false;
    if (last_g) {
        // level 1: this group's (<= kColGroup) row-block partials of the strip -> one group partial
        const int sw = (1 << d.tx_log2) * d.vec;
        const long long col0 = static_cast<long long>(cb) * sw;
        const long long col1 = min(cols, col0 + sw);
        const int rb0 = grp * kColGroup;
        const float* src = d.ws_colpart + static_cast<long long>(rb0) * cols;
        float* dst = d.ws_colpart2 + static_cast<long long>(grp) * cols;
        if (d.vec >= 4) {
            for (long long col = col0 + 4 * tid; col < col1; col += 4 * kThreads) {
                float acc[4];
                sum_partial_rows<4>(src + col, cols, grp_size, acc);
                *reinterpret_cast<float4*>(dst + col) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            }
        } else {
            for (long long col = col0 + tid; col < col1; col += kThreads) {
                float acc[1];
                sum_partial_rows<1>(src + col, cols, grp_size, acc);
                dst[col] = acc[0];
            }
        }
        __threadfence();
        block_sync();
        if (tid == 0) {
            cnt_grp[grp * d.n_cb + cb] = 0u;
            const unsigned c = atomicAdd(&d.cnt[d.n_rb + cb], 1u);
            sm.flag[1] = (c == static_cast<unsigned>(d.n_grp - 1));
        }
        block_sync();
        last_c = sm.flag[1] != 0;
        if (last_c) {
            // level 2: the strip's group partials -> EMA, factor and its rsqrt
            __threadfence();
            const float add = static_cast<float>(rows) * eps;
            if (d.vec >= 4) {
                for (long long col = col0 + 4 * tid; col < col1; col += 4 * kThreads) {
                    float acc[4];
                    sum_partial_rows<4>(d.ws_colpart2 + col, cols, d.n_grp, acc);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float nv = fmaf(beta, __ldcg(colfac + col + j), omb * fmaf(scale, acc[j], add));
                        colfac[col + j] = nv;
                        d.ws_colscale[col + j] = __frsqrt_rn(nv);
                    }
                }
            } else {
                for (long long col = col0 + tid; col < col1; col += kThreads) {
                    float acc[1];
                    sum_partial_rows<1>(d.ws_colpart2 + col, cols, d.n_grp, acc);
                    const float nv = fmaf(beta, __ldcg(colfac + col), omb * fmaf(scale, acc[0], add));
                    colfac[col] = nv;
                    d.ws_colscale[col] = __frsqrt_rn(nv);
                }
            }
            if (tid == 0) d.cnt[d.n_rb + cb] = 0u;
            if (d.flags & kFlagSumCols) {
                // this strip's share of the normaliser (the values just stored, by the threads
                // that stored them; fixed order: thread stride, warp tree, warps 0..7)
                float cs = 0.f;
                if (d.vec >= 4) {
                    for (long long col = col0 + 4 * tid; col < col1; col += 4 * kThreads)
                        cs += (colfac[col] + colfac[col + 1]) + (colfac[col + 2] + colfac[col + 3]);
                } else {
                    for (long long col = col0 + tid; col < col1; col += kThreads) cs += colfac[col];
                }
                cs = block_sum(cs, sm);
                if (tid == 0) d.ws_blocksum[d.n_rb + cb] = cs;
            }
        }
    }
    const unsigned done = (last_r ? 1u : 0u) + (last_c ? 1u : 0u);
    if (done == 0u) return;
    __threadfence();
    block_sync();
    if (tid == 0) {
        const unsigned a = atomicAdd(&d.cnt[d.n_rb + d.n_cb], done);
        sm.flag[2] = (a + done == static_cast<unsigned>(d.n_rb + d.n_cb));
    }
    block_sync();
    if (sm.flag[2]) {
        __threadfence();
        double s = 0.0;
        const int k0 = (d.flags & kFlagSumCols) ? d.n_rb : 0;
        const int k1 = (d.flags & kFlagSumCols) ? d.n_rb + d.n_cb : d.n_rb;
        for (int k = k0 + tid; k < k1; k += kThreads) s += static_cast<double>(__ldcg(d.ws_blocksum + k));
        s = block_sum(s, sm);
        if (tid == 0) {
            *sqrt_sum = static_cast<float>(sqrt(s));
            d.cnt[d.n_rb + d.n_cb] = 0u;
            if (done_flag) publish_flag(done_flag, epoch);   // everything of this factor pair is final
        }
    }
}

// Eq. 1: the last part to arrive adds all partial sums of u^2 in a fixed order
// and stores kappa = 1 / max(1, RMS(u)/d), RMS over all rows*cols components.
__device__ __forceinline__ void finalize_kappa(const TensorDev& d, int part, float partial,
                                               double clip_d, Shared& sm,
                                               unsigned* done_flag = nullptr, unsigned epoch = 0u)
{
    const int tid = threadIdx.x;
    if (tid == 0) d.ws_usq[part] = partial;
    __threadfence();
    block_sync();
    if (tid == 0) {
        const unsigned a = atomicAdd(&d.cnt[d.n_rb + d.n_cb + 1], 1u);
        sm.flag[3] = (a == static_cast<unsigned>(d.n_parts - 1));
    }
    block_sync();
    if (!sm.flag[3]) return;
    __threadfence();
    double s = 0.0;
    for (int k = tid; k < d.n_parts; k += kThreads) s += static_cast<double>(__ldcg(d.ws_usq + k));
    s = block_sum(s, sm);
    if (tid == 0) {
        const double rms = sqrt(s / (static_cast<double>(d.rows) * static_cast<double>(d.cols)));
        d.scal[1] = static_cast<float>(1.0 / fmax(1.0, rms / clip_d));
        d.cnt[d.n_rb + d.n_cb + 1] = 0u;
        if (done_flag) publish_flag(done_flag, epoch);
    }
}

// ---------------------------------------------------------------------------
// tile geometry shared by the four matrix phases
// ---------------------------------------------------------------------------
struct Geo {
    int tx, ty, TY, seg;
    long long col, row0, row1;
    bool colok;
    bool skip;        // debug build only: the tile indices themselves are out of range
};

// Debug build (-DCAME_DEBUG_BOUNDS): every tile's geometry is checked against the tensor and
// the launch plan before anything is accessed.  A violation is recorded in a device error
// word (first one wins, all are counted) and the offending accesses are masked out; nothing
// traps, so the context stays usable and the host reads the record afterwards.
#ifdef CAME_DEBUG_BOUNDS
enum : unsigned { kDbgRowBlock = 1u, kDbgColBlock = 2u, kDbgSegment = 3u, kDbgVectorTail = 4u, kDbgRowRange = 5u };
__device__ unsigned g_debug_bounds[8];   // [0] code of the first violation  [1] rb  [2] cb  [3] rows  [4] cols
                                         // [5] number of violating threads
__device__ __forceinline__ void debug_report(unsigned code, const TensorDev& d, int rb, int cb)
{
    atomicAdd(&g_debug_bounds[5], 1u);
    if (atomicCAS(&g_debug_bounds[0], 0u, code) == 0u) {
        g_debug_bounds[1] = static_cast<unsigned>(rb);
        g_debug_bounds[2] = static_cast<unsigned>(cb);
        g_debug_bounds[3] = static_cast<unsigned>(d.rows);
        g_debug_bounds[4] = static_cast<unsigned>(d.cols);
    }
}
#define CAME_DEBUG_SKIP_TILE(q) do { if ((q).skip) return; } while (0)
#else
#define CAME_DEBUG_SKIP_TILE(q) do { } while (0)
#endif

template <int VEC>
__device__ __forceinline__ Geo make_geo(const TensorDev& d, int rb, int cb)
{
    Geo q;
    const int tid = threadIdx.x;
    const int TX = 1 << d.tx_log2;
    q.tx = tid & (TX - 1);
    q.ty = tid >> d.tx_log2;
    q.TY = kThreads >> d.tx_log2;
    q.col = (static_cast<long long>(cb) * TX + q.tx) * VEC;
    q.colok = q.col < d.cols;
    q.row0 = static_cast<long long>(rb) * d.tr;
    q.row1 = min(d.rows, q.row0 + d.tr);
    q.seg = cb * (TX >> 5) + (q.tx >> 5);
    q.skip = false;
#ifdef CAME_DEBUG_BOUNDS
    unsigned bad = 0u;
    if (rb < 0 || rb >= d.n_rb || q.row0 >= d.rows) bad = kDbgRowBlock;            // block-uniform
    else if (cb < 0 || cb >= d.n_cb) bad = kDbgColBlock;                            // block-uniform
    else if (q.row1 > d.rows || q.row1 - q.row0 > d.tr) bad = kDbgRowRange;         // block-uniform
    else if (q.seg < 0 || q.seg >= d.n_seg) bad = kDbgSegment;                      // warp-uniform
    else if (q.colok && q.col + VEC > d.cols) bad = kDbgVectorTail;                 // per thread
    if (bad != 0u) {
        debug_report(bad, d, rb, cb);
        q.colok = false;                                     // this thread loads and stores nothing
        if (bad != kDbgVectorTail) q.row1 = q.row0;          // whole warp: no rows, no row partials
        q.skip = bad == kDbgRowBlock || bad == kDbgColBlock || bad == kDbgRowRange;
    }
#endif
    return q;
}

// raw gradient words of one thread-row: kept packed until they are used
template <int KIND> struct Raw;
template <> struct Raw<kF32x4>  { float4 v; };
template <> struct Raw<kBF16x8> { uint4 v; };
template <> struct Raw<kF32x8>  { float v[8]; };
template <> struct Raw<kF32x1>  { float v; };
template <> struct Raw<kBF16x1> { uint16_t v; };

template <int KIND>
__device__ __forceinline__ void load_raw(const char* p, Raw<KIND>& r)
{
    if constexpr (KIND == kF32x4) r.v = __ldg(reinterpret_cast<const float4*>(p));
    else if constexpr (KIND == kBF16x8) r.v = __ldg(reinterpret_cast<const uint4*>(p));
    else if constexpr (KIND == kF32x8) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]),
                       "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7]) : "l"(p));
    }
    else if constexpr (KIND == kF32x1) r.v = __ldg(reinterpret_cast<const float*>(p));
    else r.v = __ldg(reinterpret_cast<const uint16_t*>(p));
}

template <int KIND>
__device__ __forceinline__ void zero_raw(Raw<KIND>& r)
{
    if constexpr (KIND == kF32x4) r.v = make_float4(0.f, 0.f, 0.f, 0.f);
    else if constexpr (KIND == kBF16x8) r.v = make_uint4(0u, 0u, 0u, 0u);
    else if constexpr (KIND == kF32x8) {
#pragma unroll
        for (int j = 0; j < 8; ++j) r.v[j] = 0.f;
    }
    else if constexpr (KIND == kF32x1) r.v = 0.f;
    else r.v = 0;
}

template <int KIND>
__device__ __forceinline__ void unpack(const Raw<KIND>& r, float (&x)[Traits<KIND>::VEC])
{
    if constexpr (KIND == kF32x4) { x[0] = r.v.x; x[1] = r.v.y; x[2] = r.v.z; x[3] = r.v.w; }
    else if constexpr (KIND == kF32x8) {
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = r.v[j];
    } else if constexpr (KIND == kBF16x8) {
        x[0] = bf16lo(r.v.x); x[1] = bf16hi(r.v.x); x[2] = bf16lo(r.v.y); x[3] = bf16hi(r.v.y);
        x[4] = bf16lo(r.v.z); x[5] = bf16hi(r.v.z); x[6] = bf16lo(r.v.w); x[7] = bf16hi(r.v.w);
    } else if constexpr (KIND == kF32x1) x[0] = r.v;
    else x[0] = __uint_as_float(static_cast<uint32_t>(r.v) << 16);
}

template <int KIND> __device__ __forceinline__ constexpr int grad_elem_bytes()
{
    return (KIND == kF32x4 || KIND == kF32x1 || KIND == kF32x8) ? 4 : 2;
}

// write this tile's column partial sums (summed over the block's row groups in a fixed order)
template <int VEC>
__device__ __forceinline__ void write_col_partials(const TensorDev& d, const Geo& q, int rb,
                                                   const float (&cacc)[VEC], Shared& sm)
{
    float out[VEC];
    if (q.TY > 1) {
        const int TXV = (1 << d.tx_log2) * VEC;
#pragma unroll
        for (int v = 0; v < VEC; ++v) sm.colred[q.ty * TXV + q.tx * VEC + v] = cacc[v];
        block_sync();
        if (q.ty != 0) return;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            float s = 0.f;
            for (int y = 0; y < q.TY; ++y) s += sm.colred[y * TXV + q.tx * VEC + v];
            out[v] = s;
        }
    } else {
#pragma unroll
        for (int v = 0; v < VEC; ++v) out[v] = cacc[v];
    }
    if (q.colok) store_f<VEC>(d.ws_colpart + static_cast<long long>(rb) * d.cols + q.col, out);
}

// Row partial sums of U consecutive thread-rows (rows rbase + k*TY): reduced across the warp
// in one batch; lane (k << (5 - log2 U)) stores row k's partial for this warp's column segment.
template <int U>
__device__ __forceinline__ void store_row_partials(float (&rs)[U], float* __restrict__ rowpart_seg,
                                                   long long rbase, int TY, long long row1, int lane)
{
    constexpr int SH = 5 - Log2<U>::v;
    const float tot = multi_row_warp_sum<U>(rs, lane);
    if ((lane & ((1 << SH) - 1)) == 0) {
        const long long row = rbase + static_cast<long long>(lane >> SH) * TY;
        if (row < row1) rowpart_seg[row] = tot;
    }
}

// ---------------------------------------------------------------------------
// P1 (Algorithm 2: r_t, c_t): row and column sums of g^2
// ---------------------------------------------------------------------------
template <int KIND, int UU = 0>
__device__ __forceinline__ void p1_tile(const TensorDev& d, int rb, int cb, const StepConsts& hc,
                                        Shared& sm, unsigned* done_flag = nullptr, unsigned epoch = 0u)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = UU > 0 ? UU : ((KIND == kF32x8) ? CAME_P12_U / 2 : CAME_P12_U);   // 32 raw registers either way
    const Geo q = make_geo<VEC>(d, rb, cb);
    CAME_DEBUG_SKIP_TILE(q);
    const int lane = threadIdx.x & 31;
    const long long stride = static_cast<long long>(q.TY) * d.cols * grad_elem_bytes<KIND>();
    const char* gp = static_cast<const char*>(d.g) +
                     ((q.row0 + q.ty) * d.cols + q.col) * grad_elem_bytes<KIND>();
    float* const rowpart_seg = d.ws_rowpart + q.seg * d.rows;
    float cacc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) cacc[v] = 0.f;

    for (long long rbase = q.row0 + q.ty; rbase < q.row1; rbase += static_cast<long long>(q.TY) * U) {
        Raw<KIND> raw[U];
        const bool full = rbase + static_cast<long long>(U - 1) * q.TY < q.row1;
        if (full && q.colok) {
#pragma unroll
            for (int k = 0; k < U; ++k) load_raw<KIND>(gp + k * stride, raw[k]);
        } else {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                if (q.colok && rbase + static_cast<long long>(k) * q.TY < q.row1)
                    load_raw<KIND>(gp + k * stride, raw[k]);
                else zero_raw<KIND>(raw[k]);
            }
        }
        gp += U * stride;
        float rs[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float x[VEC];
            unpack<KIND>(raw[k], x);
            float s = 0.f;
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                cacc[v] = fmaf(x[v], x[v], cacc[v]);
                s = fmaf(x[v], x[v], s);
            }
            rs[k] = s;
        }
        store_row_partials<U>(rs, rowpart_seg, rbase, q.TY, q.row1, lane);
    }
    write_col_partials<VEC>(d, q, rb, cacc, sm);
    finalize_factors(d, rb, cb, hc.beta2, hc.omb2, hc.eps1, hc.gscale2, d.r, d.c, d.scal + 0, sm,
                     done_flag, epoch);
}

// ---------------------------------------------------------------------------
// P2 (Algorithm 2: v_t, u_t; Eq. 1): sum of u^2 -> kappa
// ---------------------------------------------------------------------------
template <int KIND, int UU = 0>
__device__ __forceinline__ void p2_tile(const TensorDev& d, int rb, int cb, const StepConsts& hc,
                                        Shared& sm, unsigned* done_flag = nullptr, unsigned epoch = 0u)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = UU > 0 ? UU : ((KIND == kF32x8) ? CAME_P12_U / 2 : CAME_P12_U);   // 32 raw registers either way
    const Geo q = make_geo<VEC>(d, rb, cb);
    CAME_DEBUG_SKIP_TILE(q);
    const long long stride = static_cast<long long>(q.TY) * d.cols * grad_elem_bytes<KIND>();
    const char* gp = static_cast<const char*>(d.g) +
                     ((q.row0 + q.ty) * d.cols + q.col) * grad_elem_bytes<KIND>();
    const float* ap = d.ws_rowscale + q.row0 + q.ty;
    const float ssr = __ldcg(d.scal + 0) * hc.gscale;          // sqrt(sum r) * gradient pre-scale
    float b[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) b[v] = q.colok ? __ldcg(d.ws_colscale + q.col + v) : 0.f;
    float acc = 0.f;

    for (long long rbase = q.row0 + q.ty; rbase < q.row1; rbase += static_cast<long long>(q.TY) * U) {
        Raw<KIND> raw[U];
        float a[U];
        const bool full = rbase + static_cast<long long>(U - 1) * q.TY < q.row1;
        if (full && q.colok) {
#pragma unroll
            for (int k = 0; k < U; ++k) { load_raw<KIND>(gp + k * stride, raw[k]); a[k] = __ldcg(ap + k * q.TY); }
        } else {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                if (q.colok && rbase + static_cast<long long>(k) * q.TY < q.row1) {
                    load_raw<KIND>(gp + k * stride, raw[k]); a[k] = __ldcg(ap + k * q.TY);
                } else { zero_raw<KIND>(raw[k]); a[k] = 0.f; }
            }
        }
        gp += U * stride;
        ap += U * q.TY;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float x[VEC];
            unpack<KIND>(raw[k], x);
            const float ai = a[k] * ssr;
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                const float u = (x[v] * b[v]) * ai;
                acc = fmaf(u, u, acc);
            }
        }
    }
    acc = block_sum(acc, sm);
    finalize_kappa(d, rb * d.n_cb + cb, acc, hc.clip_d, sm, done_flag, epoch);
}

// ---------------------------------------------------------------------------
// P3 (Algorithm 2: uhat_t, m_t, U_t, R_t, C_t).
// With e = uhat_t - m_{t-1}:  m_t = m_{t-1} + (1-beta1) e  and  uhat_t - m_t = beta1 e,
// so U_t = beta1^2 e^2; the factor beta1^2 is applied once to the finished sums.
// ---------------------------------------------------------------------------
template <int KIND, int UU = 0>
__device__ __forceinline__ void p3_tile(const TensorDev& d, int rb, int cb, const StepConsts& hc,
                                        Shared& sm, unsigned* done_flag = nullptr, unsigned epoch = 0u)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = UU > 0 ? UU : CAME_P34_U;
    const Geo q = make_geo<VEC>(d, rb, cb);
    CAME_DEBUG_SKIP_TILE(q);
    const int lane = threadIdx.x & 31;
    const long long first = (q.row0 + q.ty) * d.cols + q.col;
    const long long gstride = static_cast<long long>(q.TY) * d.cols * grad_elem_bytes<KIND>();
    const long long mstride = static_cast<long long>(q.TY) * d.cols;
    const char* gp = static_cast<const char*>(d.g) + first * grad_elem_bytes<KIND>();
    float* mp = d.m + first;
    const float* ap = d.ws_rowscale + q.row0 + q.ty;
    float* const rowpart_seg = d.ws_rowpart + q.seg * d.rows;
    const float ssr_k = __ldcg(d.scal + 0) * __ldcg(d.scal + 1) * hc.gscale;   // sqrt(sum r) * kappa * pre-scale
    const float omb1 = hc.omb1;
    float b[VEC], cacc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
        b[v] = q.colok ? __ldcg(d.ws_colscale + q.col + v) : 0.f;
        cacc[v] = 0.f;
    }

    for (long long rbase = q.row0 + q.ty; rbase < q.row1; rbase += static_cast<long long>(q.TY) * U) {
        Raw<KIND> raw[U];
        float mo[U][VEC], a[U];
        const bool full = rbase + static_cast<long long>(U - 1) * q.TY < q.row1;
        if (full && q.colok) {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                load_raw<KIND>(gp + k * gstride, raw[k]);
                load_f<VEC>(mp + k * mstride, mo[k]);
                a[k] = __ldcg(ap + k * q.TY);
            }
        } else {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                if (q.colok && rbase + static_cast<long long>(k) * q.TY < q.row1) {
                    load_raw<KIND>(gp + k * gstride, raw[k]);
                    load_f<VEC>(mp + k * mstride, mo[k]);
                    a[k] = __ldcg(ap + k * q.TY);
                } else {
                    zero_raw<KIND>(raw[k]);
                    a[k] = 0.f;
#pragma unroll
                    for (int v = 0; v < VEC; ++v) mo[k][v] = 0.f;
                }
            }
        }
        float rs[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float x[VEC];
            unpack<KIND>(raw[k], x);
            const float ai = a[k] * ssr_k;
            float s = 0.f;
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                const float uh = (x[v] * b[v]) * ai;
                const float e = uh - mo[k][v];
                mo[k][v] = fmaf(omb1, e, mo[k][v]);
                cacc[v] = fmaf(e, e, cacc[v]);
                s = fmaf(e, e, s);
            }
            rs[k] = s;
            if (q.colok && (full || rbase + static_cast<long long>(k) * q.TY < q.row1))
                store_f<VEC>(mp + k * mstride, mo[k]);
        }
        gp += U * gstride;
        mp += U * mstride;
        ap += U * q.TY;
        store_row_partials<U>(rs, rowpart_seg, rbase, q.TY, q.row1, lane);
    }
    write_col_partials<VEC>(d, q, rb, cacc, sm);
    finalize_factors(d, rb, cb, hc.beta3, hc.omb3, hc.eps2, hc.b1sq, d.R, d.C, d.scal + 2, sm,
                     done_flag, epoch);
}

// ---------------------------------------------------------------------------
// P4 (Algorithm 2: S_t and the parameter line, plus decoupled decay):
//   theta -= lr * (m * rsqrt(R_i) * sqrt(sum R) * rsqrt(C_j) + wd * theta)
// ---------------------------------------------------------------------------
template <int KIND, int UU = 0>
__device__ __forceinline__ void p4_tile(const TensorDev& d, int rb, int cb, const StepConsts& hc)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = UU > 0 ? UU : CAME_P34_U;
    const Geo q = make_geo<VEC>(d, rb, cb);
    CAME_DEBUG_SKIP_TILE(q);
    if (!q.colok) return;
    const long long first = (q.row0 + q.ty) * d.cols + q.col;
    const long long stride = static_cast<long long>(q.TY) * d.cols;
    const float* mp = d.m + first;
    float* pp = d.p + first;
    uint16_t* hp16 = d.p_bf16 ? d.p_bf16 + first : nullptr;
    const float* ap = d.ws_rowscale + q.row0 + q.ty;
    const float ssR = __ldcg(d.scal + 2);
    const float wd = (d.flags & kFlagNoWd) ? 0.f : hc.wd;
    const float nlr = -hc.lr;
    float B[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) B[v] = __ldcg(d.ws_colscale + q.col + v);

    for (long long rbase = q.row0 + q.ty; rbase < q.row1; rbase += static_cast<long long>(q.TY) * U) {
        float mo[U][VEC], th[U][VEC], a[U];
        const bool full = rbase + static_cast<long long>(U - 1) * q.TY < q.row1;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (full || rbase + static_cast<long long>(k) * q.TY < q.row1) {
                load_f<VEC>(mp + k * stride, mo[k]);
                load_f<VEC>(pp + k * stride, th[k]);
                a[k] = __ldcg(ap + k * q.TY);
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (full || rbase + static_cast<long long>(k) * q.TY < q.row1) {
                const float Ai = a[k] * ssR;
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                    const float upd = fmaf(wd, th[k][v], (mo[k][v] * B[v]) * Ai);
                    th[k][v] = fmaf(nlr, upd, th[k][v]);
                }
                store_f<VEC>(pp + k * stride, th[k]);
                if (hp16) store_bf16<VEC>(hp16 + k * stride, th[k]);
            }
        }
        mp += U * stride;
        pp += U * stride;
        if (hp16) hp16 += U * stride;
        ap += U * q.TY;
    }
}

// ---------------------------------------------------------------------------
// Algorithm 1 (Adafactor with momentum), the lines after the clip: with kappa known there is
// no further tensor-wide dependency, so momentum and parameter update are one pass:
//   m_t = m_{t-1} + (1-beta1)(uhat_t - m_{t-1});  theta -= lr * (m_t + wd * theta)
// ---------------------------------------------------------------------------
template <int KIND, int UU = 0>
__device__ __forceinline__ void p34_adafactor_tile(const TensorDev& d, int rb, int cb,
                                                   const StepConsts& hc)
{
    constexpr int VEC = Traits<KIND>::VEC;
    constexpr int U = UU > 0 ? UU : ((KIND == kF32x8) ? CAME_P34_U / 2 : CAME_P34_U);   // 24 registers per thread-row there
    const Geo q = make_geo<VEC>(d, rb, cb);
    CAME_DEBUG_SKIP_TILE(q);
    if (!q.colok) return;
    const long long first = (q.row0 + q.ty) * d.cols + q.col;
    const long long gstride = static_cast<long long>(q.TY) * d.cols * grad_elem_bytes<KIND>();
    const long long stride = static_cast<long long>(q.TY) * d.cols;
    const char* gp = static_cast<const char*>(d.g) + first * grad_elem_bytes<KIND>();
    float* mp = d.m + first;
    float* pp = d.p + first;
    uint16_t* hp16 = d.p_bf16 ? d.p_bf16 + first : nullptr;
    const float* ap = d.ws_rowscale + q.row0 + q.ty;
    const float ssr_k = __ldcg(d.scal + 0) * __ldcg(d.scal + 1) * hc.gscale;
    const float wd = (d.flags & kFlagNoWd) ? 0.f : hc.wd;
    const float nlr = -hc.lr, omb1 = hc.omb1;
    float b[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) b[v] = __ldcg(d.ws_colscale + q.col + v);

    for (long long rbase = q.row0 + q.ty; rbase < q.row1; rbase += static_cast<long long>(q.TY) * U) {
        Raw<KIND> raw[U];
        float mo[U][VEC], th[U][VEC], a[U];
        const bool full = rbase + static_cast<long long>(U - 1) * q.TY < q.row1;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (full || rbase + static_cast<long long>(k) * q.TY < q.row1) {
                load_raw<KIND>(gp + k * gstride, raw[k]);
                load_f<VEC>(mp + k * stride, mo[k]);
                load_f<VEC>(pp + k * stride, th[k]);
                a[k] = __ldcg(ap + k * q.TY);
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (full || rbase + static_cast<long long>(k) * q.TY < q.row1) {
                float x[VEC];
                unpack<KIND>(raw[k], x);
                const float ai = a[k] * ssr_k;
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                    const float uh = (x[v] * b[v]) * ai;
                    mo[k][v] = fmaf(omb1, uh - mo[k][v], mo[k][v]);
                    th[k][v] = fmaf(nlr, fmaf(wd, th[k][v], mo[k][v]), th[k][v]);
                }
                store_f<VEC>(mp + k * stride, mo[k]);
                store_f<VEC>(pp + k * stride, th[k]);
                if (hp16) store_bf16<VEC>(hp16 + k * stride, th[k]);
            }
        }
        gp += U * gstride;
        mp += U * stride;
        pp += U * stride;
        if (hp16) hp16 += U * stride;
        ap += U * q.TY;
    }
}

// ---------------------------------------------------------------------------
// vectors: the unfactored path.  A vector is cut into chunks of kVecChunk elements that ride
// in the tile list: the first half runs in P1's grid, the second (after kappa) in P3's.
// Each thread owns kVecPerThread elements and issues all their loads before using any.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float load_grad_scalar(const TensorDev& d, long long i)
{
    if (d.kind == kBF16x1 || d.kind == kBF16x8)
        return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const uint16_t*>(d.g) + i)) << 16);
    return __ldg(static_cast<const float*>(d.g) + i);
}

// v_t = beta2 v + (1-beta2)(g^2 + eps1);  partial sum of u^2 = g^2 / v_t;  kappa when complete
__device__ __forceinline__ void vec_second_moment_chunk(const TensorDev& d, int chunk,
                                                        const StepConsts& hc, Shared& sm,
                                                        unsigned* done_flag = nullptr,
                                                        unsigned epoch = 0u)
{
    const long long i0 = static_cast<long long>(chunk) * kVecChunk + threadIdx.x;
    float g[kVecPerThread], v[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const long long i = i0 + k * kThreads;
        const bool ok = i < d.rows;
        g[k] = ok ? load_grad_scalar(d, i) * hc.gscale : 0.f;
        v[k] = ok ? __ldcg(d.r + i) : 1.f;
    }
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const long long i = i0 + k * kThreads;
        if (i < d.rows) {
            const float vn = fmaf(hc.beta2, v[k], hc.omb2 * fmaf(g[k], g[k], hc.eps1));
            d.r[i] = vn;
            const float u = g[k] * __frsqrt_rn(vn);
            acc = fmaf(u, u, acc);
        }
    }
    acc = block_sum(acc, sm);
    finalize_kappa(d, chunk, acc, hc.clip_d, sm, done_flag, epoch);
}

// uhat, m_t, S_t, theta_t (S and the confidence term skipped for kFlagVecNoConf)
__device__ __forceinline__ void vec_apply_chunk(const TensorDev& d, int chunk, const StepConsts& hc)
{
    const long long i0 = static_cast<long long>(chunk) * kVecChunk + threadIdx.x;
    const float kappa = __ldcg(d.scal + 1);
    const float wd = (d.flags & kFlagNoWd) ? 0.f : hc.wd;
    const bool noconf = (d.flags & kFlagVecNoConf) != 0;
    float g[kVecPerThread], v[kVecPerThread], mo[kVecPerThread], th[kVecPerThread], S[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const long long i = i0 + k * kThreads;
        const bool ok = i < d.rows;
        g[k] = ok ? load_grad_scalar(d, i) * hc.gscale : 0.f;
        v[k] = ok ? __ldcg(d.r + i) : 1.f;
        mo[k] = ok ? __ldcg(d.m + i) : 0.f;
        th[k] = ok ? __ldcg(d.p + i) : 0.f;
        S[k] = (ok && !noconf) ? __ldcg(d.R + i) : 1.f;
    }
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
        const long long i = i0 + k * kThreads;
        if (i < d.rows) {
            const float uh = (g[k] * __frsqrt_rn(v[k])) * kappa;
            const float e = uh - mo[k];
            const float mn = fmaf(hc.omb1, e, mo[k]);
            d.m[i] = mn;
            float dir;
            if (noconf) {
                dir = mn;
            } else {
                const float Sn = fmaf(hc.beta3, S[k], hc.omb3 * fmaf(hc.b1sq * e, e, hc.eps2));
                d.R[i] = Sn;
                dir = mn * __frsqrt_rn(Sn);
            }
            const float tn = fmaf(-hc.lr, fmaf(wd, th[k], dir), th[k]);
            d.p[i] = tn;
            if (d.p_bf16) d.p_bf16[i] = static_cast<uint16_t>(pack_bf16x2(tn, 0.f) & 0xffffu);
        }
    }
}

// ---------------------------------------------------------------------------
// kernels: one block per tile, block-uniform dispatch on the tensor's kind
// ---------------------------------------------------------------------------
#define CAME_DISPATCH(FN, ...)                                         \
    switch (d.kind) {                                                  \
        case kF32x4:  FN<kF32x4>(__VA_ARGS__);  break;                 \
        case kBF16x8: FN<kBF16x8>(__VA_ARGS__); break;                 \
        case kF32x8:  FN<kF32x8>(__VA_ARGS__);  break;                 \
        case kF32x1:  FN<kF32x1>(__VA_ARGS__);  break;                 \
        default:      FN<kBF16x1>(__VA_ARGS__); break;                 \
    }

__device__ __forceinline__ Tile fetch_tile(const Tile* tiles, int ntiles, int reverse)
{
    const int b = static_cast<int>(blockIdx.x);
    return tiles[reverse ? (ntiles - 1 - b) : b];
}

// Programmatic dependent launch: the phase kernels are launched with stream serialisation
// relaxed, so the next phase's blocks may be scheduled while this phase's last blocks are still
// running.  A block lets its dependents go at once (they hold no resources this grid still
// needs: every block of this grid has started by then) and, after reading only the tile list
// and the tensor table (written by copies, never by a kernel), waits for the whole previous
// grid, memory included, before it touches anything a kernel produced.
__device__ __forceinline__ void pdl_release_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait_for_previous_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, CAME_P1_MINB)
k_p1_reduce_g2(const TensorDev* __restrict__ T, const Tile* __restrict__ tiles, int ntiles,
               int reverse, StepConsts hc)
{
    __shared__ Shared sm;
    pdl_release_dependents();
    const Tile t = fetch_tile(tiles, ntiles, reverse);
    const TensorDev d = T[t.tensor];       // by value: descriptor fields live in registers
    pdl_wait_for_previous_grid();
    if (d.ndim == 1) { vec_second_moment_chunk(d, t.rb, hc, sm); return; }
    CAME_DISPATCH(p1_tile, d, t.rb, t.cb, hc, sm)
}

__global__ void __launch_bounds__(kThreads, CAME_P2_MINB)
k_p2_sum_u2(const TensorDev* __restrict__ T, const Tile* __restrict__ tiles, int ntiles,
            int reverse, StepConsts hc)
{
    __shared__ Shared sm;
    pdl_release_dependents();
    const Tile t = fetch_tile(tiles, ntiles, reverse);
    const TensorDev d = T[t.tensor];
    pdl_wait_for_previous_grid();
    if (d.ndim == 1) return;               // vectors have no second reduction pass
    CAME_DISPATCH(p2_tile, d, t.rb, t.cb, hc, sm)
}

__global__ void __launch_bounds__(kThreads, CAME_P3_MINB)
k_p3_momentum_instability(const TensorDev* __restrict__ T, const Tile* __restrict__ tiles,
                          int ntiles, int reverse, StepConsts hc)
{
    __shared__ Shared sm;
    pdl_release_dependents();
    const Tile t = fetch_tile(tiles, ntiles, reverse);
    const TensorDev d = T[t.tensor];
    pdl_wait_for_previous_grid();
    if (d.ndim == 1) { vec_apply_chunk(d, t.rb, hc); return; }
    CAME_DISPATCH(p3_tile, d, t.rb, t.cb, hc, sm)
}

__global__ void __launch_bounds__(kThreads, CAME_P4_MINB)
k_p4_apply(const TensorDev* __restrict__ T, const Tile* __restrict__ tiles, int ntiles,
           int reverse, StepConsts hc)
{
    pdl_release_dependents();
    const Tile t = fetch_tile(tiles, ntiles, reverse);
    const TensorDev d = T[t.tensor];
    pdl_wait_for_previous_grid();
    if (d.ndim == 1) return;               // vectors finished in P3's grid
    CAME_DISPATCH(p4_tile, d, t.rb, t.cb, hc)
}

__global__ void __launch_bounds__(kThreads, 2)
k_p34_adafactor_apply(const TensorDev* __restrict__ T, const Tile* __restrict__ tiles, int ntiles,
                      int reverse, StepConsts hc)
{
    pdl_release_dependents();
    const Tile t = fetch_tile(tiles, ntiles, reverse);
    const TensorDev d = T[t.tensor];
    pdl_wait_for_previous_grid();
    if (d.ndim == 1) { vec_apply_chunk(d, t.rb, hc); return; }
    CAME_DISPATCH(p34_adafactor_tile, d, t.rb, t.cb, hc)
}

}  // namespace came
