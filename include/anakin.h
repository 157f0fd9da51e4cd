/*
 * anakin.h -- C ABI of the Anakin hot path on one NVIDIA B200 (sm_100a).
 *
 * The library runs the co-located loop of the Anakin architecture (Podracer paper, Section 3.1 "Online
 * Learning with Anakin"; Figure 2, top): a batch of environments written as array code is stepped on the
 * accelerator next to the agent for T interactions, then one parameter update is computed from those
 * interactions and averaged over the batch.  Nothing crosses the host/device boundary inside the loop
 * (Section 3.1: the host only schedules); the workload is self-contained and deterministic given a seed
 * (Section 3.1).
 *
 * Workload (Section 4.1 of the paper describes it only as small networks on grid-world environments; the
 * concrete rules are this library's):
 *   env      N x N integer gridworld per env, C = N*N cells; per-env wall mask, start and goal cell drawn from the
 *            seed; actions 0 up (row-1), 1 right (col+1), 2 down (row+1), 3 left (col-1); a move into a wall or
 *            off the grid leaves the agent in place; reaching the goal pays +1 and ends the episode, the step cap
 *            ends it with 0; an ended episode restarts from the seeded start cell inside the same step.
 *   obs      three one-hot planes (walls, agent, goal) flattened to D = 3C values; never stored, rebuilt from state.
 *   agent    MLP D-H-H with ReLU, a head of 4 action logits and 1 value; categorical sampling by inverse CDF
 *            with a Philox4x32-10 uniform keyed by (seed) and counted by (env, global step).
 *   update   GAE(gamma, lambda) advantages, A2C loss  -mean(A log pi) + value_coef mean((V-ret)^2)
 *            - entropy_coef mean(entropy), gradient = mean over all B*T rows, one Adam step.
 *
 * Conventions
 *   - Every call returns int: ANAKIN_OK (0) or a negative ANAKIN_E_* code.  Nothing throws or aborts.
 *   - The caller owns ALL device memory: one workspace of anakin_workspace_bytes() bytes, 256-byte aligned,
 *     allocated by the caller (e.g. a torch uint8 tensor) and alive until anakin_destroy().  The library
 *     allocates no device memory.  The handle itself is host memory owned by the library.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work is
 *     enqueued on it.  reset/rollout/learn/run are asynchronous; anakin_get with a HOST pointer and
 *     anakin_status synchronise the stream before returning; anakin_set with a HOST pointer is enqueued (pageable
 *     memory is staged by the runtime before the call returns; a page-locked source buffer must stay unchanged until
 *     the stream has run the copy).
 *   - A handle is not thread-safe.  Different handles (different workspaces) are independent.
 *   - Unsupported shapes are refused with ANAKIN_E_UNSUPPORTED_CFG; there is no CPU fallback.
 *
 * Flat parameter order (PARAMS, GRADS, ADAM_M, ADAM_V; fp32):
 *   W1[D][H], b1[H], W2[H][H], b2[H], Wh[H][5] (columns 0..3 logits, 4 value), bh[5];
 *   P = D*H + H + H*H + H + 5*H + 5.
 * Trajectory arrays are time-major: element (t, b) at index t*B + b.
 *
 * Many policies (anakin_cfg.n_policies = K >= 2).  Every kernel runs with one grid slice per policy on that policy's
 * own sub-workspace; per policy the arithmetic is exactly the single-policy one (its gradient is the mean over ITS
 * B_p*T rows, its Adam state is its own; parameter i of policy p is initialised from Philox counter (i, p, 0), so
 * policy 0 is the single-policy initialisation).  Blobs then hold the K policies one after the other: PARAMS, GRADS,
 * ADAM_M, ADAM_V as [K][P]; STATS as K anakin_stats; per-env blobs [B] in global env order; per-step blobs as K
 * consecutive blocks, block p = the single-policy blob of policy p ([T][B_p], values [T+1][B_p]); forced actions
 * likewise.  Supported: fp32, H in {64, 128} (small networks), every policy non-empty ((K-1)*Bp < B), K <= 65535; reset, rollout,
 * rollout_forced, gae, update, learn, run, grads, apply_grads, get/set, status.  anakin_learn_ppo, anakin_learn_vtrace
 * and the no-allocation rollout return ANAKIN_E_UNSUPPORTED_CFG.
 */
#ifndef ANAKIN_H_
#define ANAKIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct anakin_handle anakin_t;

enum {
    ANAKIN_OK = 0,
    ANAKIN_E_INVALID_ARG = -1,
    ANAKIN_E_BAD_STATE = -2,           /* e.g. learn() with no rollout pending, rollout() before reset() */
    ANAKIN_E_WORKSPACE_TOO_SMALL = -3,
    ANAKIN_E_UNSUPPORTED_CFG = -4,
    ANAKIN_E_CUDA = -5,                /* a CUDA runtime call failed; see anakin_last_cuda_error() */
    ANAKIN_E_DEVICE_STATUS = -6        /* the sticky device status word is non-zero */
};

enum { ANAKIN_PRECISION_FP32 = 0, ANAKIN_PRECISION_BF16 = 1 };

/* Plain-old-data configuration.  struct_size must be sizeof(anakin_cfg) (ABI versioning). */
/* Environments (Section 3.1: any `initial_state` / `step` written as array code).  GRID: a move off the board or into a
 * wall leaves the agent in place.  TORUS: a move off an edge re-enters at the opposite edge; walls still block. */
#define ANAKIN_ENV_GRID 0
#define ANAKIN_ENV_TORUS 1

typedef struct anakin_cfg {
    uint32_t struct_size;
    int32_t B;            /* environments, >= 1 */
    int32_t N;            /* grid side, 2..16 (cells fit a uint8) */
    int32_t H;            /* hidden width, multiple of 32, 32..1024 */
    int32_t T_max;        /* largest rollout length, >= 1 */
    int32_t episode_cap;  /* 1..255 */
    double wall_density;  /* [0, 1); a cell is a wall when its 32-bit draw is below floor(wall_density * 2^32) */
    float gamma, gae_lambda, entropy_coef, value_coef;
    float lr, adam_b1, adam_b2, adam_eps;
    int32_t precision;    /* ANAKIN_PRECISION_*: BF16 = bf16 weights/activations as GEMM inputs, fp32 accumulate,
                             fp32 master parameters in Adam */
    int32_t device;       /* CUDA device ordinal the workspace lives on */
    int32_t debug_logits; /* non-zero: debug records -- rollouts also store the 4 logits of every (t, b), updates
                             also store the ReLU gates of every row (DEBUG_LOGITS / DEBUG_GATES blobs) */
    int32_t env_offset;   /* global index of this handle's first env, >= 0 (0 on a single device).  Env b draws its
                             initial state and its action noise from the Philox counters of env env_offset + b, so
                             that G handles with B/G envs each and offsets 0, B/G, ... hold exactly the envs of one
                             handle with B envs (the replicas of Section 3.1, Figure 2 bottom) */
    int32_t env_kind;     /* ANAKIN_ENV_*: which `step` the envs run (same state, same observation planes) */
    int32_t n_policies;   /* 0 or 1: one policy.  K >= 2: K independent networks trained side by side (the shape of the
                             paper's meta-learning use case, Section 4.1: many small policies on one accelerator);
                             policy p acts in and learns from envs [p*Bp, min(B, (p+1)*Bp)), Bp = ceil(B/K), and nothing
                             couples the policies.  See "Many policies" below. */
} anakin_cfg;

/* Blob selectors for anakin_get / anakin_set.  Sizes in bytes for the LAST rollout length T (or T_max where noted). */
enum {
    ANAKIN_PARAMS = 0,       /* f32[P]                       get/set */
    ANAKIN_GRADS = 1,        /* f32[P]   last batch-mean gradient      get/set (set: before anakin_apply_grads) */
    ANAKIN_ADAM_M = 2,       /* f32[P]                       get/set */
    ANAKIN_ADAM_V = 3,       /* f32[P]                       get/set */
    ANAKIN_ADAM_STEP = 4,    /* i64[1]  host-side counter; pointer must be HOST   get/set */
    ANAKIN_ENV_WALLS = 5,    /* u32[B][ceil(C/32)] bit c of an env = cell c is a wall   get/set */
    ANAKIN_ENV_START = 6,    /* u8[B]                        get/set */
    ANAKIN_ENV_GOAL = 7,     /* u8[B]                        get/set */
    ANAKIN_ENV_POS = 8,      /* u8[B]   agent cell            get/set */
    ANAKIN_ENV_TEP = 9,      /* u8[B]   steps into the episode get/set */
    ANAKIN_GLOBAL_STEP = 10, /* i64[1]  env steps since reset (the Philox step counter); HOST pointer   get/set */
    ANAKIN_TRAJ_POS = 11,    /* u8[T][B]  state the action was taken in   get/set */
    ANAKIN_TRAJ_ACTION = 12, /* i8[T][B]                     get/set */
    ANAKIN_TRAJ_DONE = 13,   /* u8[T][B]                     get/set */
    ANAKIN_TRAJ_REWARD = 14, /* f32[T][B]                    get/set */
    ANAKIN_TRAJ_VALUE = 15,  /* f32[T+1][B]  row T = bootstrap value of the state after the last step   get/set */
    ANAKIN_TRAJ_LOGP = 16,   /* f32[T][B]  log pi(a_t|s_t)   get/set */
    ANAKIN_ADV = 17,         /* f32[T][B]                    get/set */
    ANAKIN_RET = 18,         /* f32[T][B]                    get/set */
    ANAKIN_STATS = 19,       /* anakin_stats                 get */
    ANAKIN_DEBUG_LOGITS = 20, /* f32[T][B][4], only with cfg.debug_logits   get */
    ANAKIN_DEBUG_GATES = 21   /* u32[2][T*B][H/32], only with cfg.debug_logits: bit j%32 of word [layer][row][j/32] is
                                 set when hidden unit j of that layer was active (h > 0) in the last update   get */
};

/* Counters since reset plus the loss terms of the last update. */
typedef struct anakin_stats {
    uint64_t frames;         /* env steps taken (B per step) */
    uint64_t episodes;       /* episodes finished (goal or cap) */
    uint64_t goals;          /* episodes that ended at the goal = sum of rewards */
    uint64_t episode_steps;  /* sum of the lengths of finished episodes */
    float loss_total, loss_pg, loss_value, entropy;
} anakin_stats;

/* Size of the device workspace a configuration needs.  Validates cfg. */
int anakin_workspace_bytes(const anakin_cfg* cfg, size_t* bytes);

/*
 * Creates a handle over a caller-provided DEVICE workspace (256-byte aligned, >= anakin_workspace_bytes()).
 * No device memory is allocated and nothing is enqueued.  The state is undefined until anakin_reset().
 * Errors: INVALID_ARG (null / misaligned / bad struct_size), UNSUPPORTED_CFG, WORKSPACE_TOO_SMALL, CUDA.
 */
int anakin_create(const anakin_cfg* cfg, void* dev_workspace, size_t bytes, void* cuda_stream, anakin_t** out);

/* Frees the host handle.  The workspace stays the caller's.  Does not synchronise. */
int anakin_destroy(anakin_t* h);

/*
 * The paper's `initial_state` for all B envs (Section 3.1) plus agent initialisation: draws walls, start and
 * goal of every env from the seed, puts every agent on its start cell, draws Xavier-uniform weights (zero
 * biases), zeroes the Adam moments, the step counters and the statistics.  Enqueued on the stream.
 */
int anakin_reset(anakin_t* h, uint64_t seed);

/*
 * T interactions of every env with the current policy (Figure 2, top: "a sequence of interactions"), 1 <= T <= T_max,
 * continuing from the current env state: per step, observation from state -> MLP -> sample -> env `step`; records
 * pos, action, done, reward, value, logp (time-major) and the bootstrap value row T.  Advances GLOBAL_STEP by T.
 * Errors: BAD_STATE before reset, INVALID_ARG for T out of range.
 */
int anakin_rollout(anakin_t* h, int T);

/*
 * Same kernel path with sampling overridden by dev_actions (DEVICE pointer, i8[T][B], values 0..3): the env is
 * "driven by the same action sequence" for transition parity tests.  logp is that of the forced action.
 */
int anakin_rollout_forced(anakin_t* h, int T, const int8_t* dev_actions);

/*
 * The parameter update of the minimal unit (Section 3.1; Figure 2, top): GAE over the last rollout, A2C loss,
 * backward through the MLP on all B*T rows (the env and the sampled actions carry no gradient), batch mean of
 * the gradient (the single-device form of the cross-core average), one Adam step.  Consumes the pending
 * rollout.  Errors: BAD_STATE if no rollout is pending.
 */
int anakin_learn(anakin_t* h);

/* Only the update's first half: fills ADV and RET from the pending rollout (for stage-wise parity tests). */
int anakin_gae(anakin_t* h);

/* Only the update's second half: loss, backward, batch mean and Adam from the ADV and RET blobs as they stand
 * (anakin_learn == anakin_gae followed by anakin_update).  Consumes the pending rollout. */
int anakin_update(anakin_t* h);

/*
 * The update split at the point where the paper averages gradients across devices (Section 3.1: the update computed on
 * each core's batch is averaged with a collective before it is applied).
 *   anakin_grads        everything anakin_learn does up to and including the batch mean over this handle's B*T rows:
 *                       fills GRADS and the loss statistics, consumes the pending rollout, leaves parameters and Adam
 *                       state untouched.  Errors: BAD_STATE if no rollout is pending.
 *   anakin_apply_grads  one Adam step with the GRADS blob as it stands (after the caller has averaged it over the
 *                       replicas, on this stream).  Errors: BAD_STATE before the first anakin_reset.
 *   anakin_apply_grads_mean   the same step for a GRADS blob that holds the SUM of the replicas' gradients (what a
 *                       sum all-reduce leaves): the kernel divides by n_replicas first and stores the mean back into
 *                       GRADS, so the caller's exchange needs no arithmetic of its own.  n_replicas = 1 is
 *                       anakin_apply_grads.  Errors: INVALID_ARG for n_replicas < 1.
 * anakin_grads followed by anakin_apply_grads gives bitwise the result of anakin_learn.
 */
int anakin_grads(anakin_t* h);
int anakin_apply_grads(anakin_t* h);
int anakin_apply_grads_mean(anakin_t* h, int n_replicas);

/*
 * Another objective over the same trajectory buffers (Section 3.2 leaves the choice of objective open; this one is the
 * clipped surrogate of PPO, Schulman et al. 2017, Eq. 7): GAE once, then `epochs` full-batch Adam steps in which the
 * policy term of a row is -min(r A, clip(r, 1-clip_eps, 1+clip_eps) A), r = pi(a|s) / pi_old(a|s) from the recorded
 * TRAJ_LOGP; value and entropy terms as in anakin_learn.  Every epoch after the first recomputes the forward pass of
 * the recorded rows with the current parameters.  The first epoch equals anakin_learn's step (r = 1 everywhere).
 * Consumes the pending rollout.  Errors: BAD_STATE if none is pending; INVALID_ARG for epochs < 1 or clip_eps <= 0.
 */
int anakin_learn_ppo(anakin_t* h, int epochs, float clip_eps);

/*
 * A third objective over the same buffers: the off-policy correction of the paper's other agent (Section 3.2 names
 * V-trace; defined in Espeholt et al. 2018, "IMPALA", Eq. 1).  The pending trajectory was generated by the policy whose
 * log-probabilities are in TRAJ_LOGP (the behaviour policy mu); the policy being updated (pi) is the handle's current
 * parameters, which differ from mu's after an earlier epoch, after anakin_set(PARAMS), or when the trajectory was
 * written with anakin_set.  Each of the `epochs` steps
 *   1. takes the head outputs of the recorded rows under the current parameters (the rollout's saved ones when the
 *      parameters have not changed since; otherwise the forward pass is recomputed, including the value of the state
 *      after the last step = the env state as it stands, ENV_POS),
 *   2. fills ADV and RET by the reverse scan   w = pi(a|s)/mu(a|s), rho = min(rho_bar, w), c = min(c_bar, w), d = 1 - done,
 *      delta = rho (r + gamma d V' - V),  v - V = delta + gamma d c (v' - V'),  RET = v,  ADV = rho (r + gamma d v' - V),
 *   3. runs the update of anakin_update (policy gradient with ADV, value regression to RET, entropy bonus, Adam).
 * With pi = mu and both levels >= 1 it is the A2C update with GAE at lambda = 1.  Consumes the pending rollout.
 * Errors: BAD_STATE if none is pending; INVALID_ARG for epochs < 1 or a negative level; UNSUPPORTED_CFG on hidden widths
 * whose rollout does not save the head outputs (the generic non-tensor path).
 */
int anakin_learn_vtrace(anakin_t* h, int epochs, float rho_bar, float c_bar);

/* iters x ( anakin_rollout(T_max); anakin_learn() ), enqueue-only: no copy and no synchronisation. */
int anakin_run(anakin_t* h, int iters);

/*
 * Copy a blob out of / into the workspace.  `ptr` is a host pointer (ptr_is_device = 0; anakin_get synchronises the
 * stream, anakin_set only enqueues: see the conventions above) or a device pointer (ptr_is_device = 1; asynchronous
 * on the stream), or a PAGE-LOCKED host pointer (ptr_is_device = 2; asynchronous on the stream in both directions: the
 * data of an anakin_get is there once the caller has synchronised the stream, e.g. with anakin_status).  `bytes` must equal the blob's
 * size.  Setting any TRAJ_* / ADV / RET blob marks a rollout of the last used length as pending, so the stages
 * can be driven with the other side's data.  Errors: INVALID_ARG (unknown blob, wrong size, read-only blob).
 */
int anakin_get(anakin_t* h, int which, void* ptr, size_t bytes, int ptr_is_device);
int anakin_set(anakin_t* h, int which, const void* ptr, size_t bytes, int ptr_is_device);

/* Size in bytes of a blob for the current rollout length (0 if unknown). */
size_t anakin_blob_bytes(anakin_t* h, int which);

/* Synchronises the stream and returns the sticky device status word (0 = clean) in *device_status. */
int anakin_status(anakin_t* h, int* device_status);

/*
 * Self-test of the bounded device-side waits.  Every wait inside the tensor-core kernels (on an mbarrier that a TMA
 * copy, an MMA or a peer CTA completes) gives up after a clock limit, raises bit 4 (a bounded wait gave up) in the
 * sticky status word and lets the kernel return.  This call enqueues a one-CTA kernel that waits, with the given limit
 * in SM clocks (1 .. 2e9), on a barrier nobody arrives on: afterwards anakin_status reports bit 4 and every other call
 * works as before (anakin_reset clears the word).  It never spins past the limit and never traps.
 */
int anakin_selftest_wait_timeout(anakin_t* h, int64_t limit_clocks);

/* Number of kernel launches enqueued by this handle since creation (host-side counter). */
uint64_t anakin_launch_count(anakin_t* h);

/*
 * Per-kernel timing with CUDA events recorded on the handle's stream around every launch (off by default; the
 * events add a little launch overhead while on).  anakin_profile_read synchronises the stream, writes the summed
 * duration in milliseconds and the number of launches of each kernel id (0 .. anakin_kernel_count()-1) since the
 * last read into total_ms[] / counts[] (both of n_ids >= anakin_kernel_count() entries), and clears the records.
 */
int anakin_profile_enable(anakin_t* h, int on);
int anakin_profile_read(anakin_t* h, int n_ids, double* total_ms, uint64_t* counts);
int anakin_kernel_count(void);
const char* anakin_kernel_name(int id);

/*
 * anakin_rollout_noalloc -- a rollout for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Some callers cannot call cudaMalloc, and so cannot size and provide the workspace the handle-based calls need:
 * a control loop whose memory budget is fixed at start-up, a plug-in inside an application that owns the
 * allocator, a process that must never synchronise the device (cudaMalloc and cudaFree may).  This call needs no
 * handle and no workspace.  The caller passes the rollout's inputs and outputs as DEVICE pointers; the only
 * scratch the rollout uses (B*H floats, plus two 256 KiB repacked copies of the second-layer weights) is a fixed
 * array compiled into the library, so
 *     B * H  <=  ANAKIN_NOALLOC_MAX_BH  (1,048,576 floats = 4 MiB),
 * and every GPU that loads the library holds those 4.5 MiB until the process exits.  Larger sizes return
 * ANAKIN_E_WORKSPACE_TOO_SMALL (with a message on stderr); precision must be ANAKIN_PRECISION_FP32
 * (ANAKIN_E_UNSUPPORTED_CFG otherwise).  The call itself calls no cudaMalloc / cudaFree and no allocating library
 * routine; it enqueues one small memset and up to three kernels on `cuda_stream` and returns without synchronising.
 *
 * It computes exactly what anakin_rollout(h, T) computes on a handle with the same cfg, seed, GLOBAL_STEP, PARAMS
 * and env blobs: same kernels, same results.
 *   in      dev_params f32[P]; dev_walls u32[B][ceil(C/32)]; dev_start, dev_goal u8[B]   (read only)
 *   in/out  dev_pos, dev_tep u8[B]   (env dynamic state, advanced by T steps)
 *   out     dev_traj_pos u8[T][B]; dev_traj_action i8[T][B]; dev_traj_done u8[T][B]; dev_traj_reward f32[T][B];
 *           dev_traj_value f32[T+1][B]; dev_traj_logp f32[T][B]
 *   global_step   env steps taken since the seed's reset (the caller adds T after each call); 1 <= T <= cfg->T_max
 * All buffers are the caller's and must stay alive until the stream has run the call.
 *
 * Set-up: the FIRST call on each device looks up the array's device address (cudaGetSymbolAddress) with that
 * device current; make that first call outside any stream capture.  The device that is current at the call must be
 * the one the pointers and the stream belong to.
 * Sharing: every call on a device uses the same array, which keeps the previous call's contents; the call
 * overwrites or clears all of it that it reads, so sequential calls are independent, but two calls that overlap
 * on the GPU (different streams, or different threads) race on it.  Not thread-safe.
 */
#define ANAKIN_NOALLOC_MAX_BH 1048576
int anakin_rollout_noalloc(const anakin_cfg* cfg, uint64_t seed, int64_t global_step, int T,
                           const float* dev_params, const uint32_t* dev_walls, const uint8_t* dev_start,
                           const uint8_t* dev_goal, uint8_t* dev_pos, uint8_t* dev_tep,
                           uint8_t* dev_traj_pos, int8_t* dev_traj_action, uint8_t* dev_traj_done,
                           float* dev_traj_reward, float* dev_traj_value, float* dev_traj_logp,
                           void* cuda_stream);

/*
 * Device status of the last anakin_rollout_noalloc call on the current device.  (No counterpart in the paper either.)
 * That call has no handle, so anakin_status cannot serve it: its sticky status word (0 = clean; the same bits as
 * anakin_status reports: a start position outside the grid or on a wall, a bounded device-side wait that gave up)
 * sits in the library's built-in array.  This call copies the word out on `cuda_stream` -- pass the stream the rollout
 * was enqueued on -- and SYNCHRONISES that stream; it allocates nothing.  Returns ANAKIN_OK with *device_status = 0,
 * or ANAKIN_E_DEVICE_STATUS with the word: then the trajectory the rollout wrote is not to be trusted.  The next
 * anakin_rollout_noalloc call clears the word, so read it before enqueueing another one.
 */
int anakin_noalloc_status(void* cuda_stream, int* device_status);

/* Static description of an error code. */
const char* anakin_strerror(int code);

/* Text of the last CUDA runtime error seen by this handle ("" if none). */
const char* anakin_last_cuda_error(anakin_t* h);

#ifdef __cplusplus
}
#endif
#endif /* ANAKIN_H_ */
