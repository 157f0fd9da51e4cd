// Shared device/host declarations of the Anakin library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <type_traits>
#include <vector>

#include "anakin.h"

namespace anakin {

// Sticky device status bits (anakin_status).
enum : int {
    DEV_OK = 0,
    DEV_E_BAD_ACTION = 1,   // a forced action outside 0..3
    DEV_E_BAD_STATE = 2,    // an env position outside the grid or on a wall
    DEV_E_WAIT_TIMEOUT = 4  // a bounded wait gave up
};

struct Dims {
    int B, N, C, D, H, W, Tmax;  // envs, grid side, cells, obs features, hidden, wall words per env, max T
    int env0;                    // global index of env 0 (Philox counters use env0 + b)
    size_t oW1, ob1, oW2, ob2, oWh, obh, P;
    // Many policies (independent networks side by side): npol sub-workspaces of identical layout, pstride bytes apart;
    // policy p owns envs [env0 + p*B, ...): B envs each, B_last for the last policy.  npol <= 1: one policy.
    int npol, B_last;
    size_t pstride;
};

inline Dims make_dims(int B, int N, int H, int Tmax) {
    Dims d;
    d.env0 = 0;
    d.npol = 1; d.B_last = B; d.pstride = 0;
    d.B = B; d.N = N; d.C = N * N; d.D = 3 * d.C; d.H = H; d.W = (d.C + 31) / 32; d.Tmax = Tmax;
    d.oW1 = 0;
    d.ob1 = d.oW1 + (size_t)d.D * H;
    d.oW2 = d.ob1 + H;
    d.ob2 = d.oW2 + (size_t)H * H;
    d.oWh = d.ob2 + H;
    d.obh = d.oWh + (size_t)H * 5;
    d.P = d.obh + 5;
    return d;
}

// Every sub-buffer of the caller's workspace.
struct Buffers {
    float* theta;    // fp32 master parameters [P]
    float* theta_c;  // parameters the network computes with: == theta (fp32) or bf16-rounded weights (bf16 mode)
    float* grads;    // [P]
    float* adam_m;   // [P]
    float* adam_v;   // [P]
    uint32_t* walls; // [B][W]
    uint8_t* start;  // [B]
    uint8_t* goal;   // [B]
    uint8_t* pos;    // [B]
    uint8_t* tep;    // [B]
    uint8_t* tpos;   // [Tmax][B]
    int8_t* tact;    // [Tmax][B]
    uint8_t* tdone;  // [Tmax][B]
    float* trew;     // [Tmax][B]
    float* tval;     // [Tmax+1][B]
    float* tlogp;    // [Tmax][B]
    float* adv;      // [Tmax][B]
    float* ret;      // [Tmax][B]
    float* dbg_logits;  // [Tmax][B][4] or null
    uint32_t* dbg_gates;  // [2][R][H/32] or null: ReLU gates of the last update
    float* base;     // [B][H]  b1 + sum of W1 rows of the wall cells + W1 row of the goal cell
    uint2* w2f_hi;   // [H*H/4] W2 as mma.sync B fragments, high parts (null: the warp-level rollout kernel is not used)
    uint2* w2f_lo;   // [H*H/4] bf16 low parts
    uint16_t* w2p_hi;  // [H][H] W2 row-major as 16-bit hi / lo planes (B operand of the dh1 kernel)
    uint16_t* w2p_lo;
    float* h1;       // [R][H]
    uint8_t* gate1;  // [R][H/8] layer-1 ReLU gates of every recorded row: bit j%8 of byte j/8 = the 16-bit hi term of h1[j] is not zero (null: not kept)
    float* h2;       // [R][H]
    float* out5;     // [R][8] head outputs (4 logits, value) of every recorded row, saved by the tensor-pipe rollout
    float* vboot;    // [B] value of the state after the last recorded step under the CURRENT parameters (replay mode 2)
    float* dh2;      // [R][H]
    float* dh1;      // [R][H]
    float* dout;     // [R][8]  (5 used)
    float* S;        // [B][H]  sum over t of dh1
    float* part;     // [NS][P] split-K partial gradients
    float* loss_part;  // [LOSS_BLOCKS][4]
    anakin_stats* stats;
    int* status;
};

constexpr int LOSS_BLOCKS = 592;

// ---- many policies: a kernel launched with one grid slice per policy moves every workspace pointer to its policy ----
#ifdef __CUDACC__
template <class T> __device__ __forceinline__ void shift_ptr(T*& p, size_t off) {
    if (p) p = reinterpret_cast<T*>(reinterpret_cast<unsigned char*>(const_cast<typename std::remove_const<T>::type*>(p)) + off);
}
// All sub-buffers of a policy lie at the same offsets inside its sub-workspace.  The status word stays the first
// policy's: one sticky word for the whole handle.
__device__ __forceinline__ void shift_buffers(Buffers& b, size_t off) {
    shift_ptr(b.theta, off); shift_ptr(b.theta_c, off); shift_ptr(b.grads, off); shift_ptr(b.adam_m, off); shift_ptr(b.adam_v, off);
    shift_ptr(b.walls, off); shift_ptr(b.start, off); shift_ptr(b.goal, off); shift_ptr(b.pos, off); shift_ptr(b.tep, off);
    shift_ptr(b.tpos, off); shift_ptr(b.tact, off); shift_ptr(b.tdone, off); shift_ptr(b.trew, off); shift_ptr(b.tval, off);
    shift_ptr(b.tlogp, off); shift_ptr(b.adv, off); shift_ptr(b.ret, off); shift_ptr(b.dbg_logits, off); shift_ptr(b.dbg_gates, off);
    shift_ptr(b.base, off); shift_ptr(b.w2f_hi, off); shift_ptr(b.w2f_lo, off);
    shift_ptr(b.w2p_hi, off); shift_ptr(b.w2p_lo, off); shift_ptr(b.h1, off); shift_ptr(b.gate1, off); shift_ptr(b.h2, off); shift_ptr(b.out5, off);
    shift_ptr(b.vboot, off); shift_ptr(b.dh2, off); shift_ptr(b.dh1, off); shift_ptr(b.dout, off); shift_ptr(b.S, off);
    shift_ptr(b.part, off); shift_ptr(b.loss_part, off); shift_ptr(b.stats, off);
}
__device__ __forceinline__ void select_policy(Dims& d, Buffers& b, int pol) {
    shift_buffers(b, (size_t)pol * d.pstride);
    d.env0 += pol * d.B;
    if (pol == d.npol - 1) d.B = d.B_last;
}
#endif

// ---- Philox4x32-10 (Salmon et al., SC'11) ----
struct U4 { uint32_t x, y, z, w; };

__host__ __device__ inline U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t pa = (uint64_t)0xD2511F53u * c0;
        const uint64_t pb = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(pb >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(pa >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)pb;
        c3 = (uint32_t)pa;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return U4{c0, c1, c2, c3};
}

enum : uint32_t { STREAM_ENV = 1, STREAM_PARAM = 2, STREAM_ACT = 3 };

__device__ inline float uniform24(uint32_t x) { return (float)(x >> 8) * (1.0f / 16777216.0f); }

__device__ inline float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
template <int PREC> __device__ inline float rnd(float x) { return PREC == 1 ? round_bf16(x) : x; }

// Policy term of one row.  Adds the term to l_pg and returns the factor f with d(term)/d(logit k) = -A f (1{k=a} - p_k).
//   clip <= 0: plain policy gradient  -A log pi(a|s)                                   f = 1
//   clip  > 0: clipped surrogate (PPO, Schulman et al. 2017, Eq. 7)  -min(r A, clip(r, 1-clip, 1+clip) A),
//              r = exp(log pi(a|s) - logp_old);  f = r where the unclipped product is the smaller one (ties included), else 0
__device__ __forceinline__ float policy_term(float A, float lpa, float logp_old, float clip, float& l_pg) {
    if (clip <= 0.f) {
        l_pg += -A * lpa;
        return 1.f;
    }
    const float r = expf(lpa - logp_old), rc = fminf(fmaxf(r, 1.f - clip), 1.f + clip);
    const float u = r * A, c = rc * A;
    l_pg += -fminf(u, c);
    return u <= c ? r : 0.f;
}

// launch parameter blocks --------------------------------------------------------------------------
struct RolloutArgs {
    Dims d;
    Buffers b;
    int T;
    int cap;
    uint32_t gstep0;
    uint32_t key0, key1;
    int env_kind;          // ANAKIN_ENV_*: the transition rule (env_step.cuh)
    const int8_t* forced;  // nullable
    int replay;            // 1: recompute and save the activations of the recorded rows only (no sampling, no env step);
                           // 2: the same, plus one forward of the current env state whose value goes to Buffers::vboot
    int fuse_gae;          // 1: after the last step each env's owner thread also runs the GAE scan (fills ADV, RET)
    float gamma, lambda;
    int gae_smem;          // set by the tensor-pipe rollout's launcher: the fused scan reads its inputs from shared memory
};

// One parameter range and where its split-K partial sums live: partial s of parameter i is part[s*stride + (i - start)].
struct PartRegion {
    const float* part;
    int ns;
    size_t stride;
    size_t start;
};

struct LearnArgs {
    static constexpr int NREG = 8;
    Dims d;
    Buffers b;
    int T;
    int NS;  // split-K factor of the weight-gradient GEMMs (FFMA path)
    float c_v, c_e;
    float lr, beta1, beta2, eps;
    int adam_k;  // step index after the increment
    float bc1, bc2;  // Adam's bias corrections 1 - beta1^k, 1 - beta2^k (evaluated in double on the host)
    int phase;   // 0: reduce the partials and apply Adam; 1: reduce only (GRADS and loss statistics)
    float grad_div;  // Adam-only launch: > 1 = GRADS holds a sum over this many replicas, divided here into their mean
    float ppo_clip;  // > 0: the policy term is the clipped surrogate over the recorded log-probabilities (TRAJ_LOGP)
    // tensor-pipe path
    int ts;               // t-slices of the dh1 kernel: S holds ts*B rows (slice z, env b at row z*B + b)
    float gscale, inv_gscale;  // power of two carried by every gradient-side tensor, divided out in the reduction
    float* part_small;    // per (CTA, row group) partials of dWh | db2 | dbh
    size_t small_stride;
    PartRegion reg[NREG];
};

#ifdef __CUDACC__
// One Adam step of one parameter (Kingma & Ba, Algorithm 1):
//   m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;  theta -= lr (m/(1-b1^k)) / (sqrt(v/(1-b2^k)) + eps)
// Every product and sum is rounded on its own (no contraction into fused multiply-adds), so that every kernel that
// takes the step gets the same bits, whatever surrounds the call.
struct AdamIn { float m, v, theta; };
__device__ __forceinline__ AdamIn adam_arith(const LearnArgs& a, const AdamIn& in, float g) {
    AdamIn o;
    o.m = __fadd_rn(__fmul_rn(a.beta1, in.m), __fmul_rn(1.f - a.beta1, g));
    o.v = __fadd_rn(__fmul_rn(a.beta2, in.v), __fmul_rn(__fmul_rn(1.f - a.beta2, g), g));
    const float mhat = __fdiv_rn(o.m, a.bc1), vhat = __fdiv_rn(o.v, a.bc2);
    o.theta = __fsub_rn(in.theta, __fdiv_rn(__fmul_rn(a.lr, mhat), __fadd_rn(__fsqrt_rn(vhat), a.eps)));
    return o;
}
__device__ __forceinline__ void select_policy(RolloutArgs& a, int pol) {
    if (a.forced) a.forced += (size_t)pol * a.T * a.d.B;  // forced actions come as one [T][B_p] block per policy
    select_policy(a.d, a.b, pol);
}
__device__ __forceinline__ void select_policy(LearnArgs& a, int pol) {
    // (the partial regions reg[] stay as passed: the reduction kernel indexes them dynamically, reads them from the launch
    // parameters and adds the policy's offset itself)
    shift_ptr(a.part_small, (size_t)pol * a.d.pstride);
    select_policy(a.d, a.b, pol);
}
// What a kernel body works with: the launch parameters themselves (GROUPED = false: nothing is copied), or a copy moved
// to the policy of this grid slice.
template <bool GROUPED, class A> struct PolicyArgs;
template <class A> struct PolicyArgs<false, A> {
    const A& a;
    __device__ __forceinline__ PolicyArgs(const A& in, int) : a(in) {}
};
template <class A> struct PolicyArgs<true, A> {
    A a;
    __device__ __forceinline__ PolicyArgs(const A& in, int pol) : a(in) { select_policy(a, pol); }
};
struct DimsBuffers {
    Dims d;
    Buffers b;
};
__device__ __forceinline__ void select_policy(DimsBuffers& v, int pol) { select_policy(v.d, v.b, pol); }
#endif

// Split counts and partial-buffer layout of the tensor-pipe learner (a pure function of the sizes).
struct LearnPlan {
    int ns_w2, ns_agent, ns_env, ns_small, loss_blocks, heads_grid;
    size_t small_stride, off_w2, off_agent, off_walls, off_goal, off_small, part_floats;
};
void learn_mma_plan(const Dims& d, LearnPlan* p);

// Kernel identifiers (anakin_kernel_name / anakin_profile_read index by these).
enum KernelId : int {
    K_RESET_ENV = 0, K_RESET_PARAMS, K_REFRESH_PARAMS, K_ENV_BASE, K_ROLLOUT, K_GAE, K_H1, K_FWD2, K_HEADS_LOSS, K_DH1,
    K_DW2, K_COLSUMS, K_SUM_OVER_T, K_DW1_AGENT, K_DW1_WALLS, K_DW1_GOAL, K_REDUCE_ADAM, K_LOSS_TOTAL, K_PACK_GATES, K_PACK_W2, K_HEADS_BWD, K_REPLAY, K_VTRACE, K_COUNT
};

// Optional per-kernel timing with CUDA events on the launching stream (off by default).
struct Profiler {
    struct Rec { int id; cudaEvent_t a, b; };
    bool on = false;
    std::vector<Rec> recs;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t take() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
};

// What a launch site needs: the stream, the launch counter and the profiler.
struct Ctx {
    cudaStream_t s;
    uint64_t* launches;
    Profiler* prof;
};

// Counts one kernel launch and, when profiling, brackets it with two events.
struct Scope {
    const Ctx c;  // by value: launch sites may pass a temporary
    cudaEvent_t b = nullptr;
    Scope(const Ctx& ctx, int id) : c(ctx) {
        ++*c.launches;
        if (c.prof && c.prof->on) {
            Profiler::Rec r{id, c.prof->take(), c.prof->take()};
            cudaEventRecord(r.a, c.s);
            b = r.b;
            c.prof->recs.push_back(r);
        }
    }
    ~Scope() { if (b) cudaEventRecord(b, c.s); }
};

// Operands of the split-K "TN" GEMMs  C[m][n] = sum_k A[k][m] B[k][n]  (weight gradients).
enum : int { A_PLANES = 0, A_ONEHOT = 1, A_WALLS = 2, A_ENV = 3 };  // A_ENV: row tile 0 = A_WALLS, row tile 1 = A_ONEHOT of idx2

struct GemmTnArgs {
    int M, N, K, klen;
    const __nv_bfloat16 *Ahi, *Alo;  // A_PLANES: [K][lda]
    int lda;
    const uint8_t* idx;              // A_ONEHOT: A[k][m] = (idx[k % kmod] == m)   (kmod = 0: idx[k])
    int kmod;                        // rows of A repeat with this period (S holds several t-slices of B envs)
    const uint32_t* walls;           // A_WALLS: A[k][m] = bit m of env k % kmod (m < ones_row), 1 for m == ones_row
    int W, ones_row;
    const __nv_bfloat16 *Bhi, *Blo;  // [K][ldb]
    int ldb;
    float* part;                     // out: part[split*stride + off + m*ldc + n]; row ones_row goes to off_ones + n
    size_t stride, off, off_ones;
    int ldc;
    // A_ENV only: the second row tile is the one-hot of idx2 (M2 rows), written to part2[split*stride2 + m*ldc + n]
    const uint8_t* idx2;
    int M2;
    float* part2;
    size_t stride2;
    // many policies (npol > 1): grid.z = policy * nsplit + split; every pointer above moves by pstride bytes per policy;
    // the last policy has K_last rows (period kmod_last)
    int npol, nsplit, K_last, kmod_last;
    size_t pstride;
    size_t alo_off_last, blo_off_last;  // Alo - Ahi and Blo - Bhi (elements) in the last policy's more compact planes
};
#ifdef __CUDACC__
__device__ __forceinline__ void select_policy(GemmTnArgs& g, int pol) {
    const size_t off = (size_t)pol * g.pstride;
    shift_ptr(g.Ahi, off); shift_ptr(g.Alo, off); shift_ptr(g.idx, off); shift_ptr(g.walls, off); shift_ptr(g.Bhi, off);
    shift_ptr(g.Blo, off); shift_ptr(g.part, off); shift_ptr(g.idx2, off); shift_ptr(g.part2, off);
    if (pol == g.npol - 1) {
        g.K = g.K_last;
        g.kmod = g.kmod_last;
        if (g.Alo) g.Alo = g.Ahi + g.alo_off_last;
        if (g.Blo) g.Blo = g.Bhi + g.blo_off_last;
    }
}
#endif

// tcgen05 version (tensor memory accumulators, TMA-fed); cudaErrorNotSupported when the shape is not covered.
cudaError_t launch_gemm_tn_tc(const GemmTnArgs& g, int amode, int apl, int bpl, int prec, int splits, int* status, cudaStream_t s);

// kernels (defined in the .cu files) ----------------------------------------------------------------
cudaError_t launch_reset(const Dims& d, const Buffers& b, uint64_t seed, double density, int prec, const Ctx& c);
cudaError_t launch_env_base(const Dims& d, const Buffers& b, const Ctx& c);
cudaError_t launch_rollout(const RolloutArgs& a, int prec, const Ctx& c);
cudaError_t launch_rollout_mma(const RolloutArgs& a, int prec, cudaStream_t s);  // cudaErrorNotSupported if not covered
bool rollout_mma_supported(int H);
bool rollout_uses_fragments(int H, int prec);  // the warp-level kernel (and with it the fragment copies of W2) serves this shape
cudaError_t launch_rollout_tc128(const RolloutArgs& a, cudaStream_t s);  // two-group tcgen05 rollout (H = 128, fp32, large batches); cudaErrorNotSupported otherwise
cudaError_t launch_rollout_pair2(const RolloutArgs& a, cudaStream_t s);  // two env groups per CTA pair (H = 256, fp32, large batches); cudaErrorNotSupported otherwise
cudaError_t launch_rollout_pair(const RolloutArgs& a, cudaStream_t s);  // CTA-pair tcgen05 rollout (H = 256, fp32); cudaErrorNotSupported otherwise
bool wide_supported(int H, int prec);         // bf16 workload with a hidden layer too wide for the persistent rollout
bool tensor_path_supported(int H, int prec);  // either tensor-core path: the update reuses activations the rollout saved
cudaError_t launch_rollout_wide(const RolloutArgs& a, const Ctx& c);  // T+1 forward passes, or the replay of recorded rows
cudaError_t launch_pack_w2_wide(const Dims& d, const Buffers& b, const Ctx& c);
cudaError_t launch_dh1_wide(const LearnArgs& a, const Ctx& c);
cudaError_t launch_env_base_wide(const Dims& d, const Buffers& b, const Ctx& c);  // cudaErrorNotSupported if not covered
cudaError_t launch_pack_w2(const Dims& d, const Buffers& b, int prec, const Ctx& c);
cudaError_t launch_gae(const Dims& d, const Buffers& b, int T, float gamma, float lambda, const Ctx& c);
// V-trace scan over the recorded rows: current-policy logits and values from out5, bootstrap values from `boot` [B].
cudaError_t launch_vtrace(const Dims& d, const Buffers& b, int T, float gamma, float rho_bar, float c_bar, const float* boot, const Ctx& c);
cudaError_t launch_learn(const LearnArgs& a, int prec, const Ctx& c);
cudaError_t launch_learn_mma(const LearnArgs& a, int prec, const Ctx& c);
cudaError_t launch_adam_only(const LearnArgs& a, int prec, const Ctx& c);  // Adam from GRADS as they stand
constexpr int DH1A_UNITS = 128;  // hidden units (columns of dh1) one CTA of the fused dh1 + agent-plane kernel owns
bool dh1_agent_tc_supported(const Dims& d);
// dh1, S and the agent plane of dW1 in one tcgen05 kernel; cudaErrorNotSupported if not covered
cudaError_t launch_dh1_agent_tc(const LearnArgs& a, int prec, int grid_x, float* part_agent, size_t part_stride, cudaStream_t s);
cudaError_t launch_dh1_tc(const LearnArgs& a, int prec, cudaStream_t s);  // tcgen05 dh1 kernel; cudaErrorNotSupported if not covered  // needs the activations the rollout saved
cudaError_t launch_selftest_wait(int* status, long long limit_clocks, long long* waited_clocks, cudaStream_t s);
cudaError_t launch_refresh_compute_params(const Dims& d, const Buffers& b, int prec, const Ctx& c);

}  // namespace anakin
