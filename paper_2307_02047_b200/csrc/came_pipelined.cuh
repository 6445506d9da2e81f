// Pipelined schedule of the CAME step for sm_100a: the whole step (Algorithm 2, all four phases
// over all tensors) as one persistent grid with per-tensor "phase done" flags.  The ordering
// argument and the bounded waits are described at the top of came_kernels.cuh, whose tile
// routines, reductions and flag helpers this file uses.
#pragma once
#include "came_kernels.cuh"

namespace came {

// ---------------------------------------------------------------------------
// Pipelined schedule: the whole step in one persistent grid (see the top of this file).
// `adafactor` selects Algorithm 1 (phase 2 is then the fused momentum + apply pass and there
// is no phase 3).  `wait_limit_ns` bounds every wait for a flag.
//
// A block is kThreads tile threads plus one helper warp.  The helper runs ahead of the tile
// threads through a two-slot ring in shared memory: it draws the next ticket, fetches the item
// and its tensor descriptor into the free slot, waits (bounded) for the flag the item needs,
// and only then hands the slot over.  The round trips to the L2 that each of these steps
// costs are thus spent while the tile threads stream the previous tile.  Hand-over uses the
// hardware barriers 2,3 (slot filled) and 4,5 (slot free); every path of the helper ends in a
// hand-over (a real item, "no more items", or "give up"), so the tile threads never wait for
// something that does not come.
// ---------------------------------------------------------------------------
#ifndef CAME_PIPE_MAXREG
#define CAME_PIPE_MAXREG 80                // two blocks of 288 threads per SM (registers are granted per 4 warps)
#endif
#ifndef CAME_PIPE_U12
#define CAME_PIPE_U12 0
#endif
#ifndef CAME_PIPE_U3
#define CAME_PIPE_U3 1
#endif
#ifndef CAME_PIPE_U4
#define CAME_PIPE_U4 1
#endif
#ifndef CAME_PIPE_U34A
#define CAME_PIPE_U34A 1
#endif
constexpr int kPipeThreads = kThreads + kHelperThreads;
constexpr int kPipeSlots = 2;

struct PipeSlot {
    TensorDev d;
    Item it;             // it.phase < 0: -1 = no more items, -2 = a wait ran out
};

// Hand-over barriers of the ring (all kPipeThreads threads take part: one side arrives, the
// other waits).  The barrier numbers are literals so that the kernel is charged for the six
// hardware barriers it uses and no more.
static_assert(kPipeThreads == 288 && kPipeSlots == 2, "the barrier instructions below name these");
__device__ __forceinline__ void slot_filled_arrive(int s)
{
    if (s == 0) asm volatile("bar.arrive 2, 288;" ::: "memory"); else asm volatile("bar.arrive 3, 288;" ::: "memory");
}
__device__ __forceinline__ void slot_filled_wait(int s)
{
    if (s == 0) asm volatile("bar.sync 2, 288;" ::: "memory"); else asm volatile("bar.sync 3, 288;" ::: "memory");
}
__device__ __forceinline__ void slot_free_arrive(int s)
{
    if (s == 0) asm volatile("bar.arrive 4, 288;" ::: "memory"); else asm volatile("bar.arrive 5, 288;" ::: "memory");
}
__device__ __forceinline__ void slot_free_wait(int s)
{
    if (s == 0) asm volatile("bar.sync 4, 288;" ::: "memory"); else asm volatile("bar.sync 5, 288;" ::: "memory");
}

#define CAME_DISPATCH_U(FN, UU, ...)                                       \
    switch (d.kind) {                                                      \
        case kF32x4:  FN<kF32x4, UU>(__VA_ARGS__);  break;                 \
        case kBF16x8: FN<kBF16x8, UU>(__VA_ARGS__); break;                 \
        case kF32x8:  FN<kF32x8, UU>(__VA_ARGS__);  break;                 \
        case kF32x1:  FN<kF32x1, UU>(__VA_ARGS__);  break;                 \
        default:      FN<kBF16x1, UU>(__VA_ARGS__); break;                 \
    }

__global__ void __maxnreg__(CAME_PIPE_MAXREG)
k_step_pipelined(const TensorDev* __restrict__ T, const Item* __restrict__ items, int nitems,
                 PipeSync* __restrict__ sync, StepConsts hc, int adafactor,
                 unsigned long long wait_limit_ns)
{
    __shared__ Shared sm;
    __shared__ PipeSlot slot[kPipeSlots];
    __shared__ unsigned s_ctl[2];          // [0] error word at entry  [1] epoch of this step
    const int tid = threadIdx.x;
    if (tid == 0) {
        s_ctl[0] = load_acquire(&sync->error);
        s_ctl[1] = load_acquire(&sync->epoch) + 1u;
    }
    __syncthreads();                        // all kPipeThreads threads: the only use of barrier 0
    // a grid that starts with the error word set hands out no ticket and changes nothing
    if (s_ctl[0] != 0u) return;
    const unsigned epoch = s_ctl[1];

    if (tid >= kThreads) {
        // ---------------- helper warp ----------------
        const int lane = tid - kThreads;
        unsigned next_ticket = 0u;
        if (lane == 0) next_ticket = atomicAdd(&sync->ticket, 1u);
        for (unsigned k = 0;; ++k) {
            const int s = static_cast<int>(k % kPipeSlots);
            // this item's ticket was requested one round ago; the request for the next one is
            // issued now, so its round trip overlaps this round's fetches and waits
            const unsigned ticket = __shfl_sync(0xffffffffu, next_ticket, 0);
            if (lane == 0 && ticket < static_cast<unsigned>(nitems)) next_ticket = atomicAdd(&sync->ticket, 1u);
            if (k >= kPipeSlots) slot_free_wait(s);      // the tile threads are done with it
            int outcome = 0;                                            // 0 go, -1 no more items, -2 give up
            if (ticket >= static_cast<unsigned>(nitems)) {
                outcome = -1;
            } else {
                const Item it = items[ticket];
                const unsigned* src = reinterpret_cast<const unsigned*>(T + it.tensor);
                unsigned* dst = reinterpret_cast<unsigned*>(&slot[s].d);
                constexpr int kWords = static_cast<int>(sizeof(TensorDev) / 4);
                for (int w = lane; w < kWords; w += 32) dst[w] = __ldg(src + w);
                if (lane == 0) slot[s].it = it;
                __syncwarp();
                // tensor-wide results the item needs: P2 <- r,c ; P3 (vector apply) <- kappa ; P4 <- R,C
                if (it.phase > 0) {
                    int ok = 1;
                    if (lane == 0)
                        ok = wait_for_flag(slot[s].d.done + (it.phase - 1), epoch, &sync->error,
                                           &sync->err_item, ticket, wait_limit_ns) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) outcome = -2;
                }
            }
            if (outcome != 0 && lane == 0) slot[s].it.phase = outcome;
            __threadfence_block();
            slot_filled_arrive(s);
            if (outcome != 0) break;
        }
        return;
    }

    // ---------------- tile threads ----------------
    bool failed = false;
    for (unsigned k = 0;; ++k) {
        const int s = static_cast<int>(k % kPipeSlots);
        slot_filled_wait(s);                                            // the helper's hand-over
        const TensorDev& d = slot[s].d;
        const int phase = slot[s].it.phase, rb = slot[s].it.rb, cb = slot[s].it.cb;
        if (phase < 0) { failed = (phase == -2); break; }
        if (d.ndim == 1) {
            if (phase == 0) vec_second_moment_chunk(d, rb, hc, sm, d.done + 1, epoch);
            else vec_apply_chunk(d, rb, hc);
        } else {
            switch (phase) {
                case 0: CAME_DISPATCH_U(p1_tile, CAME_PIPE_U12, d, rb, cb, hc, sm, d.done + 0, epoch) break;
                case 1: CAME_DISPATCH_U(p2_tile, CAME_PIPE_U12, d, rb, cb, hc, sm, d.done + 1, epoch) break;
                case 2:
                    if (adafactor) { CAME_DISPATCH_U(p34_adafactor_tile, CAME_PIPE_U34A, d, rb, cb, hc) }
                    else { CAME_DISPATCH_U(p3_tile, CAME_PIPE_U3, d, rb, cb, hc, sm, d.done + 2, epoch) }
                    break;
                default: CAME_DISPATCH_U(p4_tile, CAME_PIPE_U4, d, rb, cb, hc) break;
            }
        }
        block_sync();                       // every tile thread is done with the slot and the scratch
        slot_free_arrive(s);
    }

    // leave: the last block out re-arms the control block for the next step
    block_sync();
    if (tid == 0) {
        __threadfence();
        const unsigned e = atomicAdd(&sync->exited, 1u);
        if (e == gridDim.x - 1u) {
            sync->ticket = 0u;
            sync->exited = 0u;
            if (!failed && load_acquire(&sync->error) == 0u) sync->epoch = epoch;
            __threadfence();
        }
    }
}

// Runs the bounded wait of the pipelined schedule on a flag that nothing ever sets, so that
// the time-out path can be exercised on its own: words[3] receives 1 if the wait reported a
// time-out (and set the error word), 0 if it claimed the flag had arrived.
__global__ void k_wait_probe(unsigned* words /* [0] flag (stays 0) [1] error [2] err_item [3] status */,
                             unsigned long long limit_ns)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        const bool ok = wait_for_flag(words + 0, 1u, words + 1, words + 2, 7u, limit_ns);
        words[3] = ok ? 0u : 1u;
    }
}

}  // namespace came
