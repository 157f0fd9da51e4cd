// Acting half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top): T interactions of
// every env with the policy, fused into one persistent kernel.  A CTA owns ME envs for the whole rollout,
// so there is no inter-CTA dependency and no grid-wide wait anywhere.
#include "env_step.cuh"

namespace anakin {

// base[b][j] = b1[j] + sum over wall cells c (ascending) of W1[c][j] + W1[2C+goal_b][j].
// The wall and goal planes of the observation do not change during an env's life, so their contribution
// to the first layer is computed once per parameter version instead of once per step.
// One thread owns four hidden units of one env; the W1 rows are fetched eight at a time (independent loads) and added in
// ascending cell order, the goal row last.
template <bool GROUPED>
__global__ void __launch_bounds__(256) k_env_base(DimsBuffers in) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);  // many policies: grid.y = policy
    const Dims& d = pa.a.d;
    const Buffers& b = pa.a.b;
    const int H4 = d.H / 4;
    const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (size_t)d.B * H4) return;
    const int e = (int)(idx / H4), j4 = (int)(idx - (size_t)e * H4);
    const uint32_t* w = b.walls + (size_t)e * d.W;
    const float4* W1 = reinterpret_cast<const float4*>(b.theta_c + d.oW1) + j4;
    const int goal_row = 2 * d.C + min((int)b.goal[e], d.C - 1);  // (the rollout flags a goal outside the board)
    float4 acc = reinterpret_cast<const float4*>(b.theta_c + d.ob1)[j4];
    int wi = 0;
    uint32_t bits = w[0];
    bool goal_done = false;
    auto next_row = [&]() -> int {  // next wall cell in ascending order, then the goal row, then -1
        while (!bits && wi + 1 < d.W) bits = w[++wi];
        if (bits) {
            const int c = wi * 32 + (__ffs(bits) - 1);
            bits &= bits - 1;
            return c;
        }
        if (!goal_done) { goal_done = true; return goal_row; }
        return -1;
    };
    for (;;) {
        int rows[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) rows[q] = next_row();
        float4 v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = rows[q] >= 0 ? __ldg(W1 + (size_t)rows[q] * H4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            if (rows[q] >= 0) { acc.x += v[q].x; acc.y += v[q].y; acc.z += v[q].z; acc.w += v[q].w; }
        }
        if (rows[7] < 0) break;
    }
    reinterpret_cast<float4*>(b.base)[idx] = acc;
}

cudaError_t launch_env_base(const Dims& d, const Buffers& b, const Ctx& c) {
    if (d.npol <= 1) {
        const cudaError_t ew = launch_env_base_wide(d, b, c);  // tensor-core form where it applies
        if (ew != cudaErrorNotSupported) return ew;
    }
    Scope sc(c, K_ENV_BASE);
    const unsigned nb = (unsigned)(((size_t)d.B * (d.H / 4) + 255) / 256);
    if (d.npol > 1) k_env_base<true><<<dim3(nb, d.npol), 256, 0, c.s>>>(DimsBuffers{d, b});
    else k_env_base<false><<<nb, 256, 0, c.s>>>(DimsBuffers{d, b});
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// Persistent rollout.  256 threads = 8 warps; H = 32*HJ hidden units; ME = 8*RR envs per CTA.
// Per step: h1 = relu(base + W1[agent row]) -> h2 = relu(h1 W2 + b2) (register-tiled FFMA, W2 streamed through
// L1/L2) -> 5 head outputs by warp reduction -> one thread per env: softmax, inverse-CDF sample with the
// Philox uniform of (env, global step), env step, coalesced time-major stores.
// ----------------------------------------------------------------------------------------------------
template <int HJ, int RR, int PREC>
__global__ void __launch_bounds__(256) k_rollout(RolloutArgs a) {
    constexpr int H = 32 * HJ, ME = 8 * RR;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* s_base = reinterpret_cast<float*>(smem_raw);  // [ME][H]
    float* s_h1 = s_base + ME * H;                       // [ME][H]
    float* s_h2 = s_h1 + ME * H;                         // [ME][H]
    float* s_out = s_h2 + ME * H;                        // [ME][8]
    uint32_t* s_walls = reinterpret_cast<uint32_t*>(s_out + ME * 8);  // [ME][8]
    int* s_pos = reinterpret_cast<int*>(s_walls + ME * 8);            // [ME]

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int e0 = blockIdx.x * ME;
    const int B = d.B, C = d.C;
    const float* W1 = b.theta_c + d.oW1;
    const float* W2 = b.theta_c + d.oW2;
    const float* b2 = b.theta_c + d.ob2;
    const float* Wh = b.theta_c + d.oWh;
    const float* bh = b.theta_c + d.obh;

    for (int idx = tid; idx < ME * H; idx += 256) {
        const int e = idx / H, j = idx - e * H;
        s_base[idx] = (e0 + e < B) ? b.base[(size_t)(e0 + e) * H + j] : 0.f;
    }
    // per-env state lives in the registers of thread `tid` (tid < ME)
    int my_pos = 0, my_tep = 0, my_start = 0, my_goal = 0;
    const bool owner = tid < ME && e0 + tid < B;
    if (tid < ME) {
        if (owner) {
            my_pos = b.pos[e0 + tid];
            my_tep = b.tep[e0 + tid];
            my_start = b.start[e0 + tid];
            my_goal = b.goal[e0 + tid];
            for (int wi = 0; wi < 8; ++wi) s_walls[tid * 8 + wi] = wi < d.W ? b.walls[(size_t)(e0 + tid) * d.W + wi] : 0u;
        }
    }
    unsigned long long n_episodes = 0, n_goals = 0, n_epsteps = 0;
    int bad = 0;
    if (tid < ME) {
        if (owner) {
            EnvLane es;
            es.pos = my_pos; es.tep = my_tep; es.start = my_start; es.goal = my_goal;
            es.bad = 0;
            check_env_state(es, C, s_walls + tid * 8);
            my_pos = es.pos; my_start = es.start; my_goal = es.goal;
            bad |= es.bad;
        }
        s_pos[tid] = my_pos;
    }
    __syncthreads();

    for (int t = 0; t <= a.T; ++t) {
        // ---- layer 1: only the agent plane changes from step to step
        for (int idx = tid; idx < ME * H; idx += 256) {
            const int e = idx / H, j = idx - e * H;
            const float z = s_base[idx] + W1[(size_t)(C + s_pos[e]) * H + j];
            s_h1[idx] = rnd<PREC>(fmaxf(z, 0.f));
        }
        __syncthreads();
        // ---- layer 2: thread (wid, lane) owns rows wid+8*rr and columns lane+32*jj
        {
            float acc[RR][HJ];
#pragma unroll
            for (int rr = 0; rr < RR; ++rr)
#pragma unroll
                for (int jj = 0; jj < HJ; ++jj) acc[rr][jj] = 0.f;
#pragma unroll 2
            for (int k = 0; k < H; ++k) {
                float w[HJ];
#pragma unroll
                for (int jj = 0; jj < HJ; ++jj) w[jj] = __ldg(W2 + (size_t)k * H + lane + 32 * jj);
#pragma unroll
                for (int rr = 0; rr < RR; ++rr) {
                    const float x = s_h1[(wid + 8 * rr) * H + k];
#pragma unroll
                    for (int jj = 0; jj < HJ; ++jj) acc[rr][jj] = fmaf(x, w[jj], acc[rr][jj]);
                }
            }
#pragma unroll
            for (int jj = 0; jj < HJ; ++jj) {
                const float bias = __ldg(b2 + lane + 32 * jj);
#pragma unroll
                for (int rr = 0; rr < RR; ++rr)
                    s_h2[(wid + 8 * rr) * H + lane + 32 * jj] = rnd<PREC>(fmaxf(acc[rr][jj] + bias, 0.f));
            }
        }
        __syncthreads();
        // ---- heads: warp `wid` reduces its RR envs
#pragma unroll
        for (int rr = 0; rr < RR; ++rr) {
            const int e = wid + 8 * rr;
            float o[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
            for (int k = lane; k < H; k += 32) {
                const float x = s_h2[e * H + k];
#pragma unroll
                for (int c = 0; c < 5; ++c) o[c] = fmaf(x, __ldg(Wh + k * 5 + c), o[c]);
            }
#pragma unroll
            for (int c = 0; c < 5; ++c) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) o[c] += __shfl_xor_sync(0xFFFFFFFFu, o[c], off);
            }
            if (lane < 5) s_out[e * 8 + lane] = o[lane] + __ldg(bh + lane);
        }
        __syncthreads();
        // ---- one thread per env: value, sample, env step, records
        if (owner) {
            const int env = e0 + tid;
            const float l0 = s_out[tid * 8 + 0], l1 = s_out[tid * 8 + 1], l2 = s_out[tid * 8 + 2], l3 = s_out[tid * 8 + 3];
            b.tval[(size_t)t * B + env] = s_out[tid * 8 + 4];
            if (t < a.T) {  // the shared per-env step (env_step.cuh): sample, transition rule of the configured env, records
                EnvLane es;
                es.pos = my_pos; es.tep = my_tep; es.start = my_start; es.goal = my_goal;
                es.n_episodes = es.n_goals = es.n_epsteps = 0;
                es.bad = 0;
                act_and_step(es, a, env, t, l0, l1, l2, l3, s_walls + tid * 8);
                my_pos = es.pos;
                my_tep = es.tep;
                n_episodes += es.n_episodes;
                n_goals += es.n_goals;
                n_epsteps += es.n_epsteps;
                bad |= es.bad;
                s_pos[tid] = my_pos;
            }
        }
        __syncthreads();
    }
    if (owner) {
        b.pos[e0 + tid] = (uint8_t)my_pos;
        b.tep[e0 + tid] = (uint8_t)my_tep;
    }
    // statistics: integer atomics only, so totals do not depend on arrival order
    if (tid < 32) {
        // ME <= 32: all owners are in warp 0
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            n_episodes += __shfl_xor_sync(0xFFFFFFFFu, n_episodes, off);
            n_goals += __shfl_xor_sync(0xFFFFFFFFu, n_goals, off);
            n_epsteps += __shfl_xor_sync(0xFFFFFFFFu, n_epsteps, off);
            bad |= __shfl_xor_sync(0xFFFFFFFFu, bad, off);
        }
        if (tid == 0) {
            if (n_episodes) atomicAdd((unsigned long long*)&b.stats->episodes, n_episodes);
            if (n_goals) atomicAdd((unsigned long long*)&b.stats->goals, n_goals);
            if (n_epsteps) atomicAdd((unsigned long long*)&b.stats->episode_steps, n_epsteps);
            if (blockIdx.x == 0) atomicAdd((unsigned long long*)&b.stats->frames, (unsigned long long)B * a.T);
            if (bad) atomicOr(b.status, bad);
        }
    }
}

template <int HJ, int RR, int PREC>
static cudaError_t launch_rollout_t(const RolloutArgs& a, cudaStream_t s) {
    constexpr int H = 32 * HJ, ME = 8 * RR;
    const size_t smem = (size_t)(3 * ME * H + ME * 8) * sizeof(float) + ME * 8 * sizeof(uint32_t) + ME * sizeof(int);
    cudaError_t e = cudaFuncSetAttribute(k_rollout<HJ, RR, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_rollout<HJ, RR, PREC><<<(a.d.B + ME - 1) / ME, 256, smem, s>>>(a);
    return cudaGetLastError();
}

template <int PREC>
static cudaError_t launch_rollout_p(const RolloutArgs& a, cudaStream_t s) {
    switch (a.d.H / 32) {
        case 1: return launch_rollout_t<1, 4, PREC>(a, s);
        case 2: return launch_rollout_t<2, 4, PREC>(a, s);
        case 3: return launch_rollout_t<3, 4, PREC>(a, s);
        case 4: return launch_rollout_t<4, 4, PREC>(a, s);
        case 6: return launch_rollout_t<6, 4, PREC>(a, s);
        case 8: return launch_rollout_t<8, 4, PREC>(a, s);
        case 12: return launch_rollout_t<12, 4, PREC>(a, s);
        case 16: return launch_rollout_t<16, 2, PREC>(a, s);
        case 24: return launch_rollout_t<24, 2, PREC>(a, s);
        case 32: return launch_rollout_t<32, 2, PREC>(a, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_rollout(const RolloutArgs& a, int prec, const Ctx& c) {
    if (wide_supported(a.d.H, prec) && a.b.w2p_hi) return launch_rollout_wide(a, c);  // three launches per step
    Scope sc(c, K_ROLLOUT);
    const cudaError_t e = launch_rollout_mma(a, prec, c.s);  // tensor-pipe kernel where the shape is covered
    if (e != cudaErrorNotSupported) return e;
    return prec == 1 ? launch_rollout_p<1>(a, c.s) : launch_rollout_p<0>(a, c.s);
}

// ----------------------------------------------------------------------------------------------------
// GAE reverse scan: lane = env, so every load and store of a warp is one contiguous segment per t.
//   d_t = 1 - done_t; delta_t = r_t + gamma d_t V_{t+1} - V_t; A_t = delta_t + gamma lambda d_t A_{t+1}; ret = A + V
// ----------------------------------------------------------------------------------------------------
template <bool GROUPED>
__global__ void __launch_bounds__(128) k_gae(DimsBuffers in, int T, float gamma, float lambda) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);
    const Dims& d = pa.a.d;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= d.B) return;
    gae_scan_env(pa.a.b, d.B, T, e, gamma, lambda);
}

cudaError_t launch_gae(const Dims& d, const Buffers& b, int T, float gamma, float lambda, const Ctx& c) {
    Scope sc(c, K_GAE);
    if (d.npol > 1) k_gae<true><<<dim3((d.B + 127) / 128, d.npol), 128, 0, c.s>>>(DimsBuffers{d, b}, T, gamma, lambda);
    else k_gae<false><<<(d.B + 127) / 128, 128, 0, c.s>>>(DimsBuffers{d, b}, T, gamma, lambda);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// V-trace targets (Espeholt et al. 2018, IMPALA, Eq. 1; recursive form), lane = env, reverse scan over t.  mu = the policy
// that acted (recorded log-probabilities), pi = the current parameters (head outputs of the recorded rows in out5):
//   w = exp(logp_pi - logp_mu); rho = min(rho_bar, w); c = min(c_bar, w); d = 1 - done
//   delta = rho (r + gamma d V' - V);  e = delta + gamma d c e';  ret = V + e;  adv = rho (r + gamma d (V' + e') - V)
// Four steps per memory round trip.
// ----------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_vtrace(Dims d, Buffers b, int T, float gamma, float rho_bar, float c_bar, const float* boot) {
    const int env = blockIdx.x * blockDim.x + threadIdx.x;
    if (env >= d.B) return;
    const int B = d.B;
    float e_next = 0.f, v_next = boot[env];
    for (int tb = T; tb > 0; tb -= 4) {
        float4 lg[4];
        float v[4], r[4], nd[4], lmu[4];
        int act[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = tb - 1 - q;
            if (t >= 0) {
                const size_t i = (size_t)t * B + env;
                const float4* o = reinterpret_cast<const float4*>(b.out5 + i * 8);
                lg[q] = o[0];
                v[q] = o[1].x;
                r[q] = b.trew[i];
                nd[q] = b.tdone[i] ? 0.f : 1.f;
                lmu[q] = b.tlogp[i];
                act[q] = b.tact[i];
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int t = tb - 1 - q;
            if (t >= 0) {
                const size_t i = (size_t)t * B + env;
                const float l0 = lg[q].x, l1 = lg[q].y, l2 = lg[q].z, l3 = lg[q].w;
                const float mx = fmaxf(fmaxf(l0, l1), fmaxf(l2, l3));
                const float Z = ((expf(l0 - mx) + expf(l1 - mx)) + expf(l2 - mx)) + expf(l3 - mx);
                const float la = act[q] == 0 ? l0 : act[q] == 1 ? l1 : act[q] == 2 ? l2 : l3;
                const float lpi = (la - mx) - logf(Z);
                const float w = expf(lpi - lmu[q]);
                const float rho = fminf(rho_bar, w), c = fminf(c_bar, w);
                const float gd = gamma * nd[q];
                const float delta = rho * ((r[q] + gd * v_next) - v[q]);
                const float e = delta + gd * c * e_next;
                b.adv[i] = rho * ((r[q] + gd * (v_next + e_next)) - v[q]);
                b.ret[i] = v[q] + e;
                e_next = e;
                v_next = v[q];
            }
        }
    }
}

cudaError_t launch_vtrace(const Dims& d, const Buffers& b, int T, float gamma, float rho_bar, float c_bar, const float* boot, const Ctx& c) {
    Scope sc(c, K_VTRACE);
    k_vtrace<<<(d.B + 127) / 128, 128, 0, c.s>>>(d, b, T, gamma, rho_bar, c_bar, boot);
    return cudaGetLastError();
}

}  // namespace anakin
