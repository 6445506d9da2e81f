/*
 * came_b200.h -- C ABI of the B200 (sm_100a) CAME optimizer step.
 *
 * The library performs one thing: the per-step parameter update of the CAME
 * optimizer ("CAME: Confidence-guided Adaptive Memory Efficient Optimization",
 * Algorithm 2) over a list of parameter tensors resident on one GPU.
 *
 * For a matrix parameter theta (n rows x m columns, row-major) with gradient g,
 * one step computes, in the notation of Algorithm 2 (all matrix squares,
 * divisions and roots element-wise, 1_n / 1_m all-ones vectors):
 *
 *   r_t = beta2 r_{t-1} + (1-beta2) (g^2 + eps1 1_n 1_m^T) 1_m        row sums
 *   c_t = beta2 c_{t-1} + (1-beta2) 1_n^T (g^2 + eps1 1_n 1_m^T)      column sums
 *   v_t = r_t c_t / 1_n^T r_t                                         (Eq. 2, rank one)
 *   u_t = g / sqrt(v_t)
 *   uhat_t = u_t / max(1, RMS(u_t)/d)                                 (Eq. 1)
 *   m_t = beta1 m_{t-1} + (1-beta1) uhat_t
 *   U_t = (uhat_t - m_t)^2
 *   R_t = beta3 R_{t-1} + (1-beta3) (U_t + eps2 1_n 1_m^T) 1_m
 *   C_t = beta3 C_{t-1} + (1-beta3) 1_n^T (U_t + eps2 1_n 1_m^T)
 *   S_t = R_t C_t / 1_n^T R_t
 *   theta_t = theta_{t-1} - eta (m_t / sqrt(S_t) + lambda theta_{t-1})
 *
 * r, c, R, C are EMAs of SUMS (not means), exactly as printed in Algorithm 2; a
 * caller that keeps means converts with r_mean = r / m, c_mean = c / n.
 * lambda (decoupled weight decay) is an extension: the paper has none, and
 * lambda = 0 gives Algorithm 2 exactly.
 *
 * A vector parameter (ndim == 1) takes the unfactored path: v (stored in `r`)
 * and S (stored in `R`) are full-length element-wise EMAs,
 *   v_t = beta2 v + (1-beta2)(g^2 + eps1), u = g/sqrt(v_t), clip as above,
 *   m_t as above, S_t = beta3 S + (1-beta3)((uhat - m_t)^2 + eps2),
 *   theta_t = theta_{t-1} - eta (m_t / sqrt(S_t) + lambda theta_{t-1}),
 * which is what Algorithm 2 yields for an n x 1 matrix.
 *
 * Initial state (inputs of Algorithm 2): m_0 = r_0 = c_0 = 0; R_0 = C_0 = 0 by
 * the same convention.  came_create zero-fills the state unless told to keep it.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device addresses on the context's GPU; "host"
 *     pointers are ordinary process memory.  Each argument says which.
 *   - The caller owns every tensor buffer it passes in; the library owns the
 *     context and its internal device tables and reduction workspace.
 *   - Every function returns a came_status; nothing is launched when
 *     validation fails.  No exceptions, no abort.  came_last_error gives text.
 *   - came_step enqueues work on the caller's stream and returns without
 *     synchronising.  A context is not re-entrant: one thread at a time.  The
 *     context's device must be the calling thread's current device (checked:
 *     CAME_ERR_DEVICE, nothing launched), and the stream must belong to it.
 */
#ifndef CAME_B200_H
#define CAME_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct came_ctx came_ctx;   /* opaque */

typedef enum {
    CAME_OK = 0,
    CAME_ERR_NULL = 1,        /* a required pointer is NULL */
    CAME_ERR_SHAPE = 2,       /* rows/cols/ndim/count out of range */
    CAME_ERR_DTYPE = 3,       /* unknown gradient dtype */
    CAME_ERR_ALIGN = 4,       /* a tensor pointer is not 16-byte aligned */
    CAME_ERR_HPARAM = 5,      /* hyper-parameter out of range or not finite */
    CAME_ERR_STEP_ORDER = 6,  /* step is not previous step + 1 */
    CAME_ERR_DEVICE = 7,      /* bad device ordinal / no usable CUDA device */
    CAME_ERR_OOM = 8,         /* host or device allocation failed */
    CAME_ERR_CUDA = 9,        /* a CUDA runtime call failed; see came_last_error */
    CAME_ERR_INTERNAL = 10,
    CAME_ERR_UNSUPPORTED = 11,/* request outside what this entry point handles */
    CAME_ERR_OVERLAP = 12     /* two of the buffers passed to came_create share memory */
} came_status;

typedef enum { CAME_F32 = 0, CAME_BF16 = 1 } came_dtype;   /* gradient storage type */

/* per-tensor flags */
enum {
    CAME_T_NO_WEIGHT_DECAY   = 1u << 0,  /* lambda treated as 0 for this tensor */
    CAME_T_VEC_NO_CONFIDENCE = 1u << 1   /* vectors only: theta -= eta (m_t + lambda theta), i.e.
                                            the last line of Algorithm 1; S is left untouched */
};

/* came_create flags */
enum {
    CAME_CREATE_KEEP_STATE = 1u << 0,    /* resume: do not zero m, r, c, R, C */
    CAME_CREATE_ADAFACTOR  = 1u << 1     /* run Algorithm 1 (Adafactor with momentum) instead of
                                            Algorithm 2: the same lines up to m_t, then
                                            theta_t = theta_{t-1} - eta (m_t + lambda theta_{t-1});
                                            R and C are not used and may be NULL */
};

/* One parameter tensor.  All pointers are DEVICE pointers, 16-byte aligned,
 * to contiguous, non-overlapping buffers that stay valid until came_destroy
 * (came_create compares every buffer of every tensor with every other and answers
 * CAME_ERR_OVERLAP if two share a byte; gradient pointers swapped in later through
 * came_step are the caller's responsibility). */
typedef struct {
    float*       param;   /* fp32 [rows*cols], row-major; updated in place              */
    const void*  grad;    /* grad_dtype [rows*cols], same layout; read only             */
    float*       m;       /* fp32 [rows*cols]  momentum of the clipped update           */
    float*       r;       /* matrix: fp32 [rows] row factor of g^2 | vector: v [rows]    */
    float*       c;       /* matrix: fp32 [cols] column factor     | vector: NULL        */
    float*       R;       /* matrix: fp32 [rows] row factor of U   | vector: S [rows]    */
    float*       C;       /* matrix: fp32 [cols] column factor     | vector: NULL        */
                          /* R (and C) may be NULL where they are not used: Algorithm 1 mode,
                             or a vector flagged CAME_T_VEC_NO_CONFIDENCE */
    int64_t      rows;    /* >= 1 */
    int64_t      cols;    /* >= 1; must be 1 when ndim == 1 */
    int32_t      ndim;    /* 1 = vector, 2 = matrix; other ranks are not defined by the paper */
    int32_t      grad_dtype;  /* came_dtype */
    uint32_t     flags;   /* CAME_T_* */
    uint32_t     reserved;    /* must be 0 */
    void*        param_bf16;  /* optional DEVICE bf16 [rows*cols], 16-byte aligned: receives the
                                 updated parameters rounded to nearest-even bf16 in the same pass
                                 that writes `param` (the copy the next forward pass reads);
                                 NULL = none.  Not part of the paper's algorithm. */
} came_tensor;

/* Hyper-parameters of one step (doubles: 1-beta is formed in double, then each
 * constant is rounded to fp32 once).  Symbols as in the inputs of Algorithm 2. */
typedef struct {
    double  lr;            /* eta    >= 0                                  */
    double  beta1;         /* in [0,1)                                     */
    double  beta2;         /* in [0,1)                                     */
    double  beta3;         /* in [0,1)                                     */
    double  eps1;          /* >= 0, regulariser of g^2 (Algorithm 2 uses 1e-30).  With 0 a row
                              or column of g that is entirely zero gives r_i = 0 (c_j = 0) and
                              u = 0 / sqrt(0) = NaN there, exactly as Algorithm 2 evaluated
                              literally does; keep it > 0 unless no such row can occur */
    double  eps2;          /* >= 0, regulariser of the instability U (1e-16); 0 has the same
                              consequence for S_t when uhat_t = m_t on a whole row or column */
    double  clip_d;        /* d > 0, RMS clipping threshold (Eq. 1)         */
    double  weight_decay;  /* lambda >= 0 (extension; 0 = the paper)        */
    int64_t step;          /* t >= 1; must be previous + 1 after the first call.  Not used
                              in the arithmetic (Algorithm 2 has no bias correction). */
    double  grad_scale;    /* s > 0: the step uses g_t = s * (gradient buffer), e.g. 1/(number of
                              accumulation steps) or 1/(loss scale); 0 means 1.  Folded into the
                              per-tensor scalars, so it costs no pass and no per-element work. */
} came_hparams;

/* came_query selectors */
enum {
    CAME_Q_NUMEL = 0,            /* total parameter elements                                    */
    CAME_Q_STATE_BYTES = 1,      /* bytes of optimizer state m, r, c, R, C                       */
    CAME_Q_STREAM_BYTES = 2,     /* algorithmic bytes per step when no tensor stays on chip      */
    CAME_Q_COMPULSORY_BYTES = 3, /* floor: g, m, theta read once; m, theta written once          */
    CAME_Q_WORKSPACE_BYTES = 4,  /* device bytes the context allocated                           */
    CAME_Q_NUM_TILES = 5,        /* tiles in the launch plan (matrix tiles + vector chunks)      */
    CAME_Q_LAUNCHES_PER_STEP = 6,/* kernels one came_step enqueues                               */
    CAME_Q_LAST_STEP = 7,        /* last step accepted (0 before the first)                      */
    CAME_Q_NUM_PHASES = 8,       /* entries came_get_phase_ms reports                            */
    CAME_Q_MATRIX_NUMEL = 9,     /* elements that live in matrices (the four-phase path)         */
    CAME_Q_SCHEDULE = 10,        /* 0 = one grid per phase, 1 = pipelined persistent grid        */
    CAME_Q_PIPE_GROUPS = 11,     /* pipelined schedule: tensor groups (pipeline stages)          */
    CAME_Q_PIPE_GRID = 12,       /* pipelined schedule: blocks of the persistent grid            */
    CAME_Q_DEVICE_ERROR = 13,    /* pipelined schedule: 0, or the error word a step left on the
                                    device (low 8 bits: 1 = a bounded wait ran out; upper bits:
                                    the work item that gave up).  SYNCHRONISES the device. */
    CAME_Q_P1_STREAM_GRID = 14   /* blocks of the persistent streaming form of the first phase
                                    (0 = the context uses the one-block-per-tile form)          */
};

/* Algorithm 2, set-up.  Validates `t[0..n)` (HOST array of descriptors holding
 * DEVICE pointers), selects `device`, builds the launch plan, allocates the
 * context's device tables and reduction workspace, and zero-fills the state
 * buffers (m_0 = r_0 = c_0 = R_0 = C_0 = 0) unless CAME_CREATE_KEEP_STATE.
 * Synchronises the device once.  On failure *out is NULL. */
came_status came_create(came_ctx** out, const came_tensor* t, int32_t n, int32_t device,
                        uint32_t flags);

/* Algorithm 2, one pass of the loop body over every tensor of the context.
 * `hp`: HOST pointer.  `grads`: HOST array of n DEVICE gradient pointers that
 * replace the ones given at create for this and later steps, or NULL to keep
 * them.  A replacement must be aligned like the pointer it replaces was used: the
 * launch plan is fixed at create, so where create found an fp32 gradient (with
 * cols % 8 == 0 and param, m, grad all 32-byte aligned) and planned 256-bit loads,
 * the replacement must be 32-byte aligned too (came_required_grad_alignment);
 * everywhere else 16 bytes.  A pointer that is not gives CAME_ERR_ALIGN and
 * nothing is launched.  `cuda_stream`: the caller's cudaStream_t (NULL = default
 * stream).  Asynchronous; allocates nothing. */
came_status came_step(came_ctx* ctx, const came_hparams* hp, const void* const* grads,
                      void* cuda_stream);

/* Same step, fed from and drained to HOST memory: for every tensor i copies
 * host_grads[i] (HOST, grad_dtype [rows*cols], ideally pinned) into the tensor's
 * device gradient buffer, runs the step, then, where host_params_out is not NULL
 * and host_params_out[i] is not NULL, copies the updated parameters back (HOST,
 * fp32 [rows*cols]).  Tensors are independent in Algorithm 2, so the work is
 * pipelined over groups of consecutive tensors on two internal copy streams:
 * uploads, the step and downloads of different groups overlap.  Everything is
 * ordered after the work already on `cuda_stream`, and `cuda_stream` waits for the
 * last download, so synchronising it is enough.  Asynchronous for pinned memory. */
came_status came_step_host(came_ctx* ctx, const came_hparams* hp, const void* const* host_grads,
                           void* const* host_params_out, void* cuda_stream);

/* Frees the context's device and host memory.  Caller's tensors are untouched.
 * The caller must have synchronised every stream it passed to came_step. */
came_status came_destroy(came_ctx* ctx);

/* Text of the last error on this context (or of the last failed came_create
 * when ctx is NULL).  HOST string owned by the library. */
const char* came_last_error(const came_ctx* ctx);

/* Name of a status code.  HOST string, static. */
const char* came_status_string(came_status s);

/* Facts about the context; `what` is a CAME_Q_* selector, *out a HOST int64. */
came_status came_query(const came_ctx* ctx, int32_t what, int64_t* out);

/* The pipelined schedule waits, inside its one grid, for per-tensor "phase done" flags; each
 * wait is bounded (CAME_TUNE_PIPE_WAIT_NS, 2 s by default).  If a wait ever runs out, the grid
 * records an error word and returns; later steps of the context then do nothing (they leave
 * every buffer untouched) until the caller, having seen CAME_Q_DEVICE_ERROR != 0, calls
 * came_clear_device_error, which re-zeroes the context's counters, flags and control block
 * on `cuda_stream`.  State tensors may hold a partly applied step at that point: restore them
 * from the caller's last checkpoint.  Harmless on a context that uses the other schedule. */
came_status came_clear_device_error(came_ctx* ctx, void* cuda_stream);

/* Self-test of that bounded wait, without a context: one thread waits, with the limit given
 * (1 us .. 1 s), for a flag that nothing sets.  Outputs (HOST): whether the wait reported a
 * time-out (1 expected), the error word it left (1 expected), and the device time the kernel
 * took.  Allocates and frees 16 bytes of device memory; synchronises. */
came_status came_selftest_wait_timeout(int32_t device, int64_t limit_ns, int32_t* out_timed_out,
                                       int32_t* out_error_word, float* out_elapsed_ms);

/* Debug build only (the library compiled with -DCAME_DEBUG_BOUNDS; paper_2307_02047_b200/build.py
 * builds it as libcame_b200_debug.so): every tile's index arithmetic is checked on the device
 * against the tensor's shape and the launch plan before anything is accessed.  A violation
 * never traps: the offending accesses are masked out and a record is kept on the device.
 * came_debug_bounds copies that record to `out6` (HOST, six words: code of the first violation
 * -- 0 none, 1 row block, 2 column block, 3 row-partial segment, 4 vector access past the end
 * of a row, 5 row range -- then its rb, cb, the tensor's rows and cols, and the number of
 * violating threads) and synchronises the device.  In the ordinary build it writes zeros and
 * returns CAME_ERR_UNSUPPORTED. */
came_status came_debug_bounds(int32_t device, uint32_t* out6);

/* Per-phase device timing.  When enabled, came_step records CUDA events on the
 * caller's stream between its kernels (no synchronisation); switching it on
 * restarts the average.  came_get_phase_ms synchronises on the last recorded
 * event and writes up to `cap` durations in milliseconds (HOST floats), each the
 * mean over the profiled steps (the most recent 128), in launch order; names via
 * came_phase_name. */
came_status came_set_profiling(came_ctx* ctx, int32_t enabled);
came_status came_get_phase_ms(came_ctx* ctx, float* out_ms, int32_t cap, int32_t* out_count);
const char* came_phase_name(const came_ctx* ctx, int32_t phase);

/* Launch-plan geometry of one tensor, computed on the host without touching
 * the GPU (the same routine came_create uses).  Outputs (HOST): elements per
 * thread per load (1, 4 or 8), threads across columns, rows per tile, number of
 * row blocks and column blocks.  `aligned32` says whether param and m are
 * 32-byte aligned; `tile_elems_target` <= 0 selects the default.  (came_create runs a
 * matrix with cols == 1 as its 1 x rows view, the same memory with the roles of the row and
 * column factors exchanged, so that every lane has work: ask for the plan of that view.) */
came_status came_plan_tensor(int64_t rows, int64_t cols, int32_t ndim, int32_t grad_dtype,
                             int32_t aligned32, int64_t tile_elems_target, int32_t* out_vec,
                             int32_t* out_threads_x, int32_t* out_tile_rows, int32_t* out_n_rb,
                             int32_t* out_n_cb);

/* Host-only helpers (no CUDA call).
 * came_required_grad_alignment: bytes a gradient pointer must be aligned to for a tensor
 * whose plan reads `vec` elements per thread (came_plan_tensor's out_vec): 32 for fp32
 * gradients with vec == 8, else 16.
 * came_device_status: the comparison came_step makes before it launches anything --
 * CAME_OK when `current_device` (the calling thread's cudaGetDevice) is the device the
 * context was created on, else CAME_ERR_DEVICE.
 * came_lr_warmup: the learning rate of step `step` (1-based) under the warm-up the paper's
 * experiments use (Section 4.1, "Implementation Detail": start from a smaller rate and
 * increase gradually to eta).  The paper does not give the shape of the ramp; this one is
 * linear: lr_start + (lr_peak - lr_start) * step / warmup_steps for step < warmup_steps,
 * lr_peak from then on (and for warmup_steps <= 0).  The value goes into came_hparams.lr. */
int32_t     came_required_grad_alignment(int32_t grad_dtype, int32_t vec);
came_status came_device_status(int32_t context_device, int32_t current_device);
double      came_lr_warmup(double lr_peak, double lr_start, int64_t step, int64_t warmup_steps);

/* Allocation-free factor update (the paper has no counterpart: this exists for callers of
 * this library that are not allowed to allocate device memory).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a memory pool or
 * framework allocator that owns the whole device heap, in a latency-critical loop where an
 * allocation's implicit synchronisation is unacceptable, or under a fixed memory budget
 * audited at start-up.  Such a caller cannot use came_create, which allocates the context's
 * tables and reduction workspace.
 *
 * What it does: the first two lines of Algorithm 2 for ONE matrix,
 *   r = beta2 r + (1-beta2)(g^2 + eps1 1 1^T) 1_m,   c = beta2 c + (1-beta2) 1_n^T (g^2 + eps1 1 1^T),
 * with the same tile kernel as came_step's first phase.  `grad` (DEVICE, grad_dtype
 * [rows*cols], row-major, 16-byte aligned, read only), `r` (DEVICE fp32 [rows], in/out),
 * `c` (DEVICE fp32 [cols], in/out); `out_sqrt_sum_r` (DEVICE fp32 [1], may be NULL)
 * receives sqrt(1_n^T r).  The partial sums live in a fixed array of
 * CAME_STATIC_SCRATCH_BYTES inside the library image (every GPU that loads the library
 * holds that much until the process exits).  A matrix whose partial sums do not fit is
 * rejected with CAME_ERR_UNSUPPORTED and a message naming the bytes needed; nothing is
 * launched.  Calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * The first call on each device looks up the device address of the scratch array (a
 * cudaGetSymbolAddress with `device` current); make that first call outside any stream
 * capture.  Every call uses the same scratch array and clears the part that must start at
 * zero, so two calls whose GPU work overlaps (different streams, or different host threads)
 * race: serialise them on one stream.  Asynchronous on `cuda_stream`. */
#define CAME_STATIC_SCRATCH_BYTES (8u << 20)
came_status came_factor_update_static(const void* grad, int32_t grad_dtype, int64_t rows,
                                      int64_t cols, float* r, float* c, double beta2,
                                      double eps1, float* out_sqrt_sum_r, int32_t device,
                                      void* cuda_stream);

/* Host-only companion of came_factor_update_static: runs the same argument checks and the
 * same planning, touches no GPU, launches nothing.  Outputs (HOST, may be NULL): elements per
 * thread per gradient load (8 = 256-bit loads of fp32, chosen only when `grad` is 32-byte
 * aligned; 4 = 128-bit; bf16 reads 8 per 128-bit load) and the bytes of the built-in
 * scratch the call would use.  Returns what the real call would return for these arguments. */
came_status came_factor_update_static_plan(const void* grad, int32_t grad_dtype, int64_t rows,
                                           int64_t cols, const float* r, const float* c,
                                           double beta2, double eps1, int32_t device,
                                           int32_t* out_vec, int64_t* out_scratch_bytes);

/* Process-wide tuning knobs, read by later came_create calls (each knob is an atomic, so any
 * thread may set one; a context takes the values in force while it is being created, so set
 * them before the contexts they are meant for).  CAME_TUNE_TILE_ELEMS:
 * elements per matrix tile (0 restores the default, which scales with the size
 * of the parameter set).  They change scheduling only, never results beyond the
 * order of the partial sums. */
enum {
    CAME_TUNE_TILE_ELEMS = 0,
    CAME_TUNE_SCHED_GROUP_BYTES = 1,  /* > 0: came_step runs all phases of one group of consecutive
                                         tensors (about this many bytes of g, m and theta) before
                                         the next group, instead of one grid per phase over all
                                         tensors; per-phase timing is then not reported.  0 = off. */
    CAME_TUNE_HOST_GROUP_BYTES = 2,   /* bytes of gradients + parameters per pipeline stage of
                                         came_step_host (default 1 GiB) */
    CAME_TUNE_PDL = 3,                /* 1 (default): phase kernels use programmatic dependent
                                         launch, so a phase's blocks are scheduled during the
                                         previous phase's tail; 0: plain stream order.  Read at
                                         every step. */
    CAME_TUNE_F32_VEC8 = 4,           /* 1 (default): fp32 gradients are read 8 per thread with
                                         256-bit loads when rows are 32-byte aligned; 0: 4 per
                                         thread (128-bit) */
    CAME_TUNE_SCHEDULE = 5,           /* schedule of contexts created afterwards: 0 = the default
                                         (one grid per phase), 1 = one grid per phase (four launches),
                                         2 = pipelined: the whole step is ONE persistent grid whose
                                         blocks draw (tensor, tile, phase) items in an order that
                                         sends L2-sized groups of tensors through the phases one
                                         pipeline stage apart, so a group's gradient is read from
                                         HBM once and its momentum is still in the L2 when the last
                                         phase reads it.  Same arithmetic, same results; measured
                                         slower than the phase grids on B200, hence not the default. */
    CAME_TUNE_PIPE_TILE_ELEMS = 6,    /* pipelined schedule: elements per tile (0 = default 32768) */
    CAME_TUNE_PIPE_GROUP_BYTES = 7,   /* pipelined schedule: bytes of gradient + momentum per
                                         tensor group (0 = default 48 MiB) */
    CAME_TUNE_PIPE_WAIT_NS = 8,       /* pipelined schedule: limit of every wait for a flag, in
                                         nanoseconds (0 = default 2 s) */
    CAME_TUNE_PIPE_ORDER = 9,         /* pipelined schedule: 0 = groups one stage apart (default),
                                         1 = each group's phases back to back */
    CAME_TUNE_P1_STREAM = 10,         /* first phase (r_t, c_t) as a persistent grid that stages the
                                         gradient through per-thread rings of asynchronous copies
                                         in shared memory, so that loads stay in flight across
                                         the per-tile epilogue: 0 or 1 = off (default), 2 = for
                                         every matrix whose rows load in 16-byte pieces.  Same
                                         sums in the same order: results are bit-identical either
                                         way.  Measured slower on B200 (the phase is bound by
                                         instruction issue once the latency is hidden), hence off. */
    CAME_TUNE_P1_STREAM_RING = 11     /* batches of 8 x 16 bytes per thread in that ring
                                         (1..4; 0 = default 2, i.e. 64 KB per block) */
};
came_status came_tune(int32_t key, int64_t value);

#ifdef __cplusplus
}
#endif
#endif /* CAME_B200_H */
