// Per-env part of one interaction (Podracer paper, Section 3.1: `step` maps a state and an action to a new state
// and a reward): categorical sampling from the 4 logits, the integer gridworld step, and the time-major records.
// One thread owns one env for the whole rollout; its dynamic state lives in that thread's registers.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace anakin {

struct EnvLane {
    int pos, tep, start, goal;
    unsigned long long n_episodes, n_goals, n_epsteps;
    int bad;
};

// The part of an interaction that does not depend on the policy's output: the Philox uniform of (env, step) and, for
// each of the four actions, the cell the agent would end up in.  A kernel can compute it while it waits for memory or
// for the tensor pipe, so that only the softmax and the selection remain once the logits are known.
struct StepPre {
    float u;
    int np[4];  // 0 up, 1 right, 2 down, 3 left; blocked moves stay in place
};

// The env's movement rule as a compile-time plug-in: target(row, col, action, N) = the cell the move aims at, or -1
// when it leaves the board.  Everything else of `step` (walls, clock, goal, restart, records) is shared.
struct GridMoves {  // borders block
    static __device__ __forceinline__ int target(int row, int col, int act, int N) {
        const int nr = act == 0 ? row - 1 : act == 2 ? row + 1 : row, nc = act == 1 ? col + 1 : act == 3 ? col - 1 : col;
        return (nr >= 0 && nr < N && nc >= 0 && nc < N) ? nr * N + nc : -1;
    }
};
struct TorusMoves {  // borders wrap around
    static __device__ __forceinline__ int target(int row, int col, int act, int N) {
        int nr = act == 0 ? row - 1 : act == 2 ? row + 1 : row, nc = act == 1 ? col + 1 : act == 3 ? col - 1 : col;
        nr = nr < 0 ? N - 1 : nr >= N ? 0 : nr;
        nc = nc < 0 ? N - 1 : nc >= N ? 0 : nc;
        return nr * N + nc;
    }
};

// A state handed in from outside (anakin_set, the handle-less rollout) may not be a legal one.  Start, goal and agent
// must be cells of the board, and the agent does not stand on a wall: anything else raises DEV_E_BAD_STATE and is
// replaced (start and goal by cell 0, the agent by the start cell), so that every later index stays inside its array.
// walls: this env's wall words.
__device__ __forceinline__ void check_env_state(EnvLane& s, int C, const uint32_t* walls) {
    if (s.start >= C) { s.bad |= DEV_E_BAD_STATE; s.start = 0; }
    if (s.goal >= C) { s.bad |= DEV_E_BAD_STATE; s.goal = 0; }
    if (s.pos >= C || ((walls[s.pos >> 5] >> (s.pos & 31)) & 1u)) { s.bad |= DEV_E_BAD_STATE; s.pos = s.start; }
}

// walls: this env's wall words (shared memory), 8 words.
template <class Moves>
__device__ __forceinline__ StepPre step_prepare_t(const EnvLane& s, const RolloutArgs& a, int env, int t, const uint32_t* walls) {
    StepPre p;
    const U4 r = philox4x32_10((uint32_t)(a.d.env0 + env), a.gstep0 + (uint32_t)t, 0, STREAM_ACT, a.key0, a.key1);
    p.u = uniform24(r.x);
    const int N = a.d.N;
    const int row = s.pos / N, col = s.pos - row * N;
#pragma unroll
    for (int act = 0; act < 4; ++act) {
        const int cand = Moves::target(row, col, act, N);
        int np = s.pos;
        if (cand >= 0 && !((walls[cand >> 5] >> (cand & 31)) & 1u)) np = cand;
        p.np[act] = np;
    }
    return p;
}
__device__ __forceinline__ StepPre step_prepare(const EnvLane& s, const RolloutArgs& a, int env, int t, const uint32_t* walls) {
    return a.env_kind == ANAKIN_ENV_TORUS ? step_prepare_t<TorusMoves>(s, a, env, t, walls) : step_prepare_t<GridMoves>(s, a, env, t, walls);
}

// Categorical sampling from the 4 logits (inverse CDF against the prepared uniform) and the env transition, in two parts
// so that a kernel can publish the new position before it spends time on the records:
//   act_decide   softmax terms, the sampled (or forced) action, the transition; updates the env state in `s`
//   act_record   log-probability and the time-major records of the step
struct ActOut {
    float la_mx, Z, rew;  // logit of the action minus the maximum, softmax denominator, reward
    int act, done, pos0;  // action, episode ended at this step, the state the action was taken in
};
__device__ __forceinline__ ActOut act_decide(EnvLane& s, const RolloutArgs& a, int env, int t, float l0, float l1, float l2, float l3,
                                             const StepPre& pre) {
    const size_t i = (size_t)t * a.d.B + env;
    // softmax and inverse CDF: c0 = p0, c1 = c0 + p1, c2 = c1 + p2; a = [u>=c0] + [u>=c1] + [u>=c2]
    const float mx = fmaxf(fmaxf(l0, l1), fmaxf(l2, l3));
    const float x0 = expf(l0 - mx), x1 = expf(l1 - mx), x2 = expf(l2 - mx), x3 = expf(l3 - mx);
    const float Z = ((x0 + x1) + x2) + x3;
    // the comparisons u >= c_k are taken as u Z >= x0 + .. + x_k: no division, and the same decision except within
    // rounding (1e-7) of a boundary
    const float s01 = x0 + x1, s012 = s01 + x2;
    const float uz = pre.u * Z;
    int act = (uz >= x0) + (uz >= s01) + (uz >= s012);
    if (a.forced) {
        act = a.forced[i];
        if (act < 0 || act > 3) { s.bad |= DEV_E_BAD_ACTION; act &= 3; }
    }
    ActOut o;
    o.la_mx = (act == 0 ? l0 : act == 1 ? l1 : act == 2 ? l2 : l3) - mx;
    o.Z = Z;
    o.act = act;
    o.pos0 = s.pos;
    const int np = act == 0 ? pre.np[0] : act == 1 ? pre.np[1] : act == 2 ? pre.np[2] : pre.np[3];
    const int te = s.tep + 1;
    o.rew = 0.f;
    o.done = 0;
    if (np == s.goal) { o.rew = 1.f; o.done = 1; }
    else if (te >= a.cap) { o.done = 1; }
    if (o.done) {
        s.n_episodes += 1;
        s.n_goals += (np == s.goal);
        s.n_epsteps += te;
        s.pos = s.start;
        s.tep = 0;
    } else {
        s.pos = np;
        s.tep = te;
    }
    return o;
}
__device__ __forceinline__ void act_record(const RolloutArgs& a, int env, int t, float l0, float l1, float l2, float l3, const ActOut& o) {
    const Buffers& b = a.b;
    const size_t i = (size_t)t * a.d.B + env;
    b.tlogp[i] = o.la_mx - logf(o.Z);
    b.tpos[i] = (uint8_t)o.pos0;
    b.tact[i] = (int8_t)o.act;
    if (b.dbg_logits) reinterpret_cast<float4*>(b.dbg_logits)[i] = make_float4(l0, l1, l2, l3);
    b.trew[i] = o.rew;
    b.tdone[i] = (uint8_t)o.done;
}
// Both parts at once.  Returns bit 0 = the episode ended at this step, bit 1 = it ended at the goal (reward 1).
__device__ __forceinline__ int act_and_step_pre(EnvLane& s, const RolloutArgs& a, int env, int t, float l0, float l1, float l2,
                                                float l3, const StepPre& pre) {
    const ActOut o = act_decide(s, a, env, t, l0, l1, l2, l3, pre);
    act_record(a, env, t, l0, l1, l2, l3, o);
    return o.done | (o.rew != 0.f ? 2 : 0);
}

__device__ __forceinline__ void act_and_step(EnvLane& s, const RolloutArgs& a, int env, int t, float l0, float l1, float l2,
                                             float l3, const uint32_t* walls) {
    const StepPre pre = step_prepare(s, a, env, t, walls);
    act_and_step_pre(s, a, env, t, l0, l1, l2, l3, pre);
}

// An owner warp folds its lanes' per-env counters and adds them with integer atomics (order-free totals); the frame count
// is added once per launch (by one warp of CTA 0: count_frames).
__device__ __forceinline__ void flush_env_stats(EnvLane& s, const RolloutArgs& a, bool count_frames = true) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s.n_episodes += __shfl_xor_sync(0xFFFFFFFFu, s.n_episodes, off);
        s.n_goals += __shfl_xor_sync(0xFFFFFFFFu, s.n_goals, off);
        s.n_epsteps += __shfl_xor_sync(0xFFFFFFFFu, s.n_epsteps, off);
        s.bad |= __shfl_xor_sync(0xFFFFFFFFu, s.bad, off);
    }
    if ((threadIdx.x & 31) == 0) {
        const Buffers& b = a.b;
        if (s.n_episodes) atomicAdd((unsigned long long*)&b.stats->episodes, s.n_episodes);
        if (s.n_goals) atomicAdd((unsigned long long*)&b.stats->goals, s.n_goals);
        if (s.n_epsteps) atomicAdd((unsigned long long*)&b.stats->episode_steps, s.n_epsteps);
        if (blockIdx.x == 0 && count_frames) atomicAdd((unsigned long long*)&b.stats->frames, (unsigned long long)a.d.B * a.T);
        if (s.bad) atomicOr(b.status, s.bad);
    }
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(gsrc), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// GAE reverse scan of one env (explicit rounding intrinsics: the standalone kernel and the fused learner agree bitwise):
//   d_t = 1 - done_t; delta_t = r_t + gamma d_t V_{t+1} - V_t; A_t = delta_t + gamma lambda d_t A_{t+1}; ret_t = A_t + V_t
__device__ __forceinline__ void gae_scan_env(const Buffers& b, int B, int T, int env, float gamma, float lambda) {
    float A = 0.f;
    float vnext = b.tval[(size_t)T * B + env];
    const float gl = __fmul_rn(gamma, lambda);
    // eight steps at a time: all loads of a chunk are issued before its stores, so the scan pays one memory round trip
    // per chunk instead of one per step
    for (int tb = T; tb > 0; tb -= 8) {
        float v[8], r[8], nd[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int t = tb - 1 - q;
            if (t >= 0) {
                const size_t i = (size_t)t * B + env;
                v[q] = b.tval[i];
                r[q] = b.trew[i];
                nd[q] = b.tdone[i] ? 0.f : 1.f;
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int t = tb - 1 - q;
            if (t >= 0) {
                const size_t i = (size_t)t * B + env;
                const float delta = __fsub_rn(__fmaf_rn(__fmul_rn(gamma, nd[q]), vnext, r[q]), v[q]);
                A = __fmaf_rn(__fmul_rn(gl, nd[q]), A, delta);
                b.adv[i] = A;
                b.ret[i] = __fadd_rn(A, v[q]);
                vnext = v[q];
            }
        }
    }
}

// The same scan over a copy of one CTA's values and outcomes kept in shared memory by the rollout (value row t of the
// CTA's env e at sv[t*ME + e], outcome code of act_and_step_pre at sc[t*ME + e]): no global load on the serial chain.
// Same operations in the same order as gae_scan_env, so the results are bitwise equal.
__device__ __forceinline__ void gae_scan_env_smem(const Buffers& b, int B, int T, int env, float gamma, float lambda, const float* sv,
                                                  const uint8_t* sc, int ME, int e) {
    float A = 0.f;
    float vnext = sv[T * ME + e];
    const float gl = __fmul_rn(gamma, lambda);
    for (int t = T - 1; t >= 0; --t) {
        const size_t i = (size_t)t * B + env;
        const float v = sv[t * ME + e];
        const int code = sc[t * ME + e];
        const float nd = (code & 1) ? 0.f : 1.f, r = (code & 2) ? 1.f : 0.f;
        const float delta = __fsub_rn(__fmaf_rn(__fmul_rn(gamma, nd), vnext, r), v);
        A = __fmaf_rn(__fmul_rn(gl, nd), A, delta);
        b.adv[i] = A;
        b.ret[i] = __fadd_rn(A, v);
        vnext = v;
    }
}

// ---- warp-level tensor-core helpers (mma.sync m16n8k16, bf16 inputs, fp32 accumulate) ----
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_ptr) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_ptr) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Operand formats of the tensor-pipe kernels.
//   PREC 0 (fp32 workloads): every fp32 operand is split into two fp16 terms, x ~= hi + lo with hi = fp16(x),
//     lo = fp16(x - hi): 22 significand bits.  Three fp16 products hi*hi + lo*hi + hi*lo accumulated in fp32 reproduce
//     the fp32 product to about 2^-21.  (A bf16 split keeps only 16 bits, which is not enough for the 1e-4 parity
//     bound on the weight gradients.)  fp16 has a narrow exponent range, so gradient-side tensors are carried
//     multiplied by a power of two (LearnArgs::gscale) that is divided out exactly when the partials are reduced.
//   PREC 1 (bf16 workload): operands are bf16 values already; one bf16 product, no lo term.
// pack2<PREC> rounds two consecutive elements to the 16-bit format: the lower-index element goes to the low half.
template <int PREC>
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    if (PREC == 1) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);  // one packed conversion; .x (low half) = x0
        hi = *reinterpret_cast<const uint32_t*>(&h);
        lo = 0u;
    } else {
        const __half2 h = __floats2half2_rn(x0, x1);
        const float2 hf = __half22float2(h);
        const __half2 l = __floats2half2_rn(x0 - hf.x, x1 - hf.y);
        hi = *reinterpret_cast<const uint32_t*>(&h);
        lo = *reinterpret_cast<const uint32_t*>(&l);
    }
}
template <int PREC>
__device__ __forceinline__ void split1(float x, uint16_t& hi, uint16_t& lo) {
    if (PREC == 1) {
        hi = __bfloat16_as_ushort(__float2bfloat16_rn(x));
        lo = 0;
    } else {
        const __half h = __float2half_rn(x);
        hi = __half_as_ushort(h);
        lo = __half_as_ushort(__float2half_rn(x - __half2float(h)));
    }
}
template <int PREC>
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if (PREC == 1) mma_bf16(d, a, b0, b1);
    else mma_f16(d, a, b0, b1);
}
// Two-term bf16 split (used for fp32 sums that feed a bf16 product in the bf16 workload).
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
__device__ __forceinline__ uint32_t pack_bf16(__nv_bfloat16 lo_elem, __nv_bfloat16 hi_elem) {
    return (uint32_t)__bfloat16_as_ushort(lo_elem) | ((uint32_t)__bfloat16_as_ushort(hi_elem) << 16);
}
// One bit per 16-bit element of v that is not a (signed) zero; element 0 = the low half of v.x = bit 0.
__device__ __forceinline__ uint32_t nonzero_bits16(const uint4& v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) m |= ((w[i] & 0x00007FFFu) ? 1u : 0u) << (2 * i) | ((w[i] & 0x7FFF0000u) ? 2u : 0u) << (2 * i);
    return m;
}
// 1.0 in the 16-bit operand format
template <int PREC> __device__ __forceinline__ uint32_t one16() { return PREC == 1 ? 0x3F80u : 0x3C00u; }

}  // namespace anakin
