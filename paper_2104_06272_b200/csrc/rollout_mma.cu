// Persistent rollout on the tensor pipe (warp-level mma.sync), second-layer weights resident on chip.
//
// Acting half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top).  A CTA owns 32 envs for all
// T+1 forward passes of a rollout; nothing is exchanged between CTAs.  Per step:
//   layer 1   h1 = relu(base + W1[agent row])            gather-add, written to smem as 16-bit (hi, lo) planes
//   layer 2   h2 = relu(h1 W2 + b2)                      mma.sync m16n8k16; warp w owns output columns [NC*w, NC*w+NC)
//   heads     out = h2 Wh + bh                           fp32 FMA on the accumulator fragments, fixed-order reduction
//   env       softmax, Philox inverse-CDF sample, gridworld step, time-major records   (one thread per env)
// fp32 workloads use a two-term fp16 split of both operands and three MMAs per product (hi*hi + lo*hi + hi*lo,
// fp32 accumulate).  W2's "hi" B-fragments stay in shared memory and its "lo" B-fragments in registers for the
// whole kernel (H = 256: 128 KB + 128 KB), so after the prologue the loop touches no weight bytes beyond the
// agent's W1 row.  The bf16 workload needs one MMA per product and no lo planes.
#include "env_step.cuh"

namespace anakin {

// B fragments of W2 for mma.m16n8k16 (.col B): entry [(ks*(H/8) + nt)*32 + lane] holds, for g = lane/4, t = lane%4,
// n = 8*nt + g:  x = {W2[16ks+2t][n], W2[16ks+2t+1][n]},  y = {W2[16ks+2t+8][n], W2[16ks+2t+9][n]}  (low half first).
template <int PREC, bool GROUPED>
__global__ void __launch_bounds__(256) k_pack_w2(DimsBuffers in) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);  // many policies: grid.y = policy
    const Dims& d = pa.a.d;
    const Buffers& b = pa.a.b;
    const int H = d.H;
    const int total = H * H / 4;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int lane = idx & 31, nt = (idx >> 5) % (H / 8), ks = (idx >> 5) / (H / 8);
    const int g = lane >> 2, t = lane & 3;
    const int n = nt * 8 + g, k0 = ks * 16 + 2 * t;
    const float* W2 = b.theta_c + d.oW2;
    if (b.w2f_hi) {
        const int ks4[4] = {k0, k0 + 1, k0 + 8, k0 + 9};
        uint2 hi, lo;
        split2<PREC>(W2[(size_t)ks4[0] * H + n], W2[(size_t)ks4[1] * H + n], hi.x, lo.x);
        split2<PREC>(W2[(size_t)ks4[2] * H + n], W2[(size_t)ks4[3] * H + n], hi.y, lo.y);
        b.w2f_hi[idx] = hi;
        b.w2f_lo[idx] = lo;
    }
    // and W2 itself as row-major hi / lo planes: this thread covers elements 4*idx .. 4*idx+3
    if (!b.w2p_hi || !b.w2p_lo) return;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint16_t h16, l16;
        split1<PREC>(W2[(size_t)4 * idx + q], h16, l16);
        b.w2p_hi[(size_t)4 * idx + q] = h16;
        b.w2p_lo[(size_t)4 * idx + q] = l16;
    }
}

cudaError_t launch_pack_w2(const Dims& d, const Buffers& b, int prec, const Ctx& c) {
    if (!b.w2f_hi && !b.w2p_hi) return cudaSuccess;
    Scope sc(c, K_PACK_W2);
    const unsigned nb = (d.H * d.H / 4 + 255) / 256;
    if (d.npol > 1) {
        if (prec == 1) return cudaErrorNotSupported;
        k_pack_w2<0, true><<<dim3(nb, d.npol), 256, 0, c.s>>>(DimsBuffers{d, b});
    } else if (prec == 1) k_pack_w2<1, false><<<nb, 256, 0, c.s>>>(DimsBuffers{d, b});
    else k_pack_w2<0, false><<<nb, 256, 0, c.s>>>(DimsBuffers{d, b});
    return cudaGetLastError();
}

template <int H, int NW, int PREC>
struct RolloutMmaCfg {
    static constexpr int ME = 32;            // envs per CTA (two m16 tiles)
    static constexpr int NC = H / NW;        // output columns per warp
    static constexpr int NT = NC / 8;        // n8 tiles per warp
    static constexpr int KS = H / 16;        // k16 steps
    static constexpr int LD = H + 8;         // bf16 row pitch of the h1 planes (16-byte skew: conflict-free ldmatrix)
    static constexpr int PLANES = PREC == 1 ? 1 : 2;
    static constexpr size_t smem_bytes =
        (size_t)H * H * 2                    // W2 hi fragments
        + (size_t)ME * H * 4                 // base
        + (size_t)PLANES * ME * LD * 2       // h1 hi (and lo)
        + (size_t)NW * ME * 5 * 4            // per-warp head partials
        + (size_t)(H * 5 + H + 8) * 4        // Wh, b2, bh
        + (size_t)ME * 8 * 4 + ME * 4        // walls, pos
        + (size_t)ME * 8;                    // prepared half of the next interaction
    // values and outcomes of the CTA's envs for the GAE scan at the end (only when the scan is fused and they fit)
    static constexpr size_t gae_bytes(int T) { return (size_t)(T + 1) * ME * 4 + (size_t)T * ME; }
};

template <int H, int NW, int PREC, bool GROUPED>
__global__ void __launch_bounds__(NW * 32, (H <= 128 ? 2 : 1)) k_rollout_mma(RolloutArgs a_in) {
    const PolicyArgs<GROUPED, RolloutArgs> pa(a_in, blockIdx.y);  // many policies: grid.y = policy
    const RolloutArgs& a = pa.a;
    using Cfg = RolloutMmaCfg<H, NW, PREC>;
    constexpr int ME = Cfg::ME, NT = Cfg::NT, KS = Cfg::KS, LD = Cfg::LD, NTHREADS = NW * 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint2* s_w2hi = reinterpret_cast<uint2*>(smem_raw);                        // [KS][H/8][32]
    float* s_base = reinterpret_cast<float*>(smem_raw + (size_t)H * H * 2);    // [ME][H]
    __nv_bfloat16* s_h1hi = reinterpret_cast<__nv_bfloat16*>(s_base + ME * H); // [ME][LD]
    __nv_bfloat16* s_h1lo = s_h1hi + (PREC == 1 ? 0 : ME * LD);               // [ME][LD] (fp32 workloads only)
    float* s_red = reinterpret_cast<float*>(s_h1hi + Cfg::PLANES * ME * LD);   // [NW][ME][5]
    float* s_wh = s_red + NW * ME * 5;                                         // [H][5]
    float* s_b2 = s_wh + H * 5;                                                // [H]
    float* s_bh = s_b2 + H;                                                    // [8]
    uint32_t* s_walls = reinterpret_cast<uint32_t*>(s_bh + 8);                 // [ME][8]
    int* s_pos = reinterpret_cast<int*>(s_walls + ME * 8);                     // [ME]
    uint2* s_pre = reinterpret_cast<uint2*>(s_pos + ME);                       // [ME]
    float* s_gv = reinterpret_cast<float*>(s_pre + ME);                        // [T+1][ME] (a.gae_smem only)
    uint8_t* s_gc = reinterpret_cast<uint8_t*>(s_gv + (a.T + 1) * ME);         // [T][ME]

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t4 = lane & 3;
    const int e0 = blockIdx.x * ME;
    const int B = d.B, C = d.C;
    const float* W1 = b.theta_c + d.oW1;

    // ---- prologue: weights and per-env constants on chip
    // asynchronous copies: every 16-byte chunk is in flight at once, nothing is staged in registers
    for (int i = tid; i < H * H * 2 / 16; i += NTHREADS) cp_async16(reinterpret_cast<uint4*>(s_w2hi) + i, reinterpret_cast<const uint4*>(b.w2f_hi) + i, 16);
    for (int i = tid; i < ME * H / 4; i += NTHREADS) {
        const int e = i / (H / 4), j = 4 * (i - e * (H / 4));
        const bool ok = e0 + e < B;
        cp_async16(s_base + e * H + j, b.base + (size_t)(ok ? e0 + e : 0) * H + j, ok ? 16 : 0);
    }
    cp_async_commit();
    for (int i = tid; i < H * 5; i += NTHREADS) s_wh[i] = b.theta_c[d.oWh + i];
    for (int i = tid; i < H; i += NTHREADS) s_b2[i] = b.theta_c[d.ob2 + i];
    if (tid < 5) s_bh[tid] = b.theta_c[d.obh + tid];
    uint2 blo[PREC == 1 ? 1 : KS][NT];
    if (PREC == 0) {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int j = 0; j < NT; ++j) blo[ks][j] = b.w2f_lo[(ks * (H / 8) + wid * NT + j) * 32 + lane];
    }
    EnvLane s;
    s.pos = s.tep = s.start = s.goal = 0;
    s.n_episodes = s.n_goals = s.n_epsteps = 0;
    s.bad = 0;
    const bool owner = tid < ME && e0 + tid < B;
    if (tid < ME) {
        for (int wi = 0; wi < 8; ++wi) s_walls[tid * 8 + wi] = (owner && wi < d.W) ? b.walls[(size_t)(e0 + tid) * d.W + wi] : 0u;
        if (owner) {
            s.pos = b.pos[e0 + tid];
            s.tep = b.tep[e0 + tid];
            s.start = b.start[e0 + tid];
            s.goal = b.goal[e0 + tid];
            check_env_state(s, C, s_walls + tid * 8);
        }
        s_pos[tid] = s.pos;
    }
    cp_async_wait<0>();
    __syncthreads();

    // Saved activations (the update reuses the policy's forward pass: Section 3.1): row i = t*B + env.
    __nv_bfloat16* g_h1hi = reinterpret_cast<__nv_bfloat16*>(b.h1);
    __nv_bfloat16* g_h1lo = g_h1hi + (size_t)B * d.Tmax * H;
    const int t_end = a.replay == 1 ? a.T - 1 : a.T;  // replay recomputes the T recorded rows (mode 2: and the current state)
    for (int t = 0; t <= t_end; ++t) {
        if (a.replay) {  // positions come from the recorded trajectory (row T: the env state as it stands)
            if (tid < ME) s_pos[tid] = owner ? min((int)(t < a.T ? b.tpos[(size_t)t * B + e0 + tid] : b.pos[e0 + tid]), C - 1) : 0;
            __syncthreads();
        }
        // ---- layer 1: eight consecutive hidden units per thread and trip.  All gathers of the agent's W1 row are issued
        // before any is used (one L2 round trip per step, not one per trip); the fp16 planes go to shared memory for
        // the MMAs and, for the update's reuse, straight to global memory (16 bytes per lane).
        {
            constexpr int TRIPS = ME * H / 8 / NTHREADS;
            static_assert(TRIPS * NTHREADS == ME * H / 8, "layer-1 trips must tile the h1 block");
            const bool save_h1 = b.h1 != nullptr && t < a.T;
            float4 w[TRIPS][2];
#pragma unroll
            for (int i = 0; i < TRIPS; ++i) {
                const int p = tid + i * NTHREADS;
                const int e = p / (H / 8), k = 8 * (p - e * (H / 8));
                const float4* wp = reinterpret_cast<const float4*>(W1 + (size_t)(C + s_pos[e]) * H + k);
                w[i][0] = __ldg(wp);
                w[i][1] = __ldg(wp + 1);
            }
#pragma unroll
            for (int i = 0; i < TRIPS; ++i) {
                const int p = tid + i * NTHREADS;
                const int e = p / (H / 8), k = 8 * (p - e * (H / 8));
                const float4 b0 = *reinterpret_cast<const float4*>(s_base + e * H + k);
                const float4 b1 = *reinterpret_cast<const float4*>(s_base + e * H + k + 4);
                uint4 hi, lo;
                split2<PREC>(fmaxf(b0.x + w[i][0].x, 0.f), fmaxf(b0.y + w[i][0].y, 0.f), hi.x, lo.x);
                split2<PREC>(fmaxf(b0.z + w[i][0].z, 0.f), fmaxf(b0.w + w[i][0].w, 0.f), hi.y, lo.y);
                split2<PREC>(fmaxf(b1.x + w[i][1].x, 0.f), fmaxf(b1.y + w[i][1].y, 0.f), hi.z, lo.z);
                split2<PREC>(fmaxf(b1.z + w[i][1].z, 0.f), fmaxf(b1.w + w[i][1].w, 0.f), hi.w, lo.w);
                if (PREC == 0) *reinterpret_cast<uint4*>(s_h1lo + e * LD + k) = lo;
                *reinterpret_cast<uint4*>(s_h1hi + e * LD + k) = hi;
                if (save_h1 && e0 + e < B) {
                    const size_t gi = ((size_t)t * B + e0 + e) * H + k;
                    *reinterpret_cast<uint4*>(g_h1hi + gi) = hi;
                    if (PREC == 0) *reinterpret_cast<uint4*>(g_h1lo + gi) = lo;
                    if (b.gate1) b.gate1[gi >> 3] = (uint8_t)nonzero_bits16(hi);  // the gates of these eight units
                }
            }
        }
        __syncthreads();
        // The logits-independent half of the interaction (the Philox uniform, the four candidate cells) is taken by the
        // owner threads now, under the other warps' tensor work, so that only softmax and selection follow the heads.
        // It waits in shared memory (two words per env) rather than in registers, which the MMA loop needs.
        const bool acting = owner && !a.replay && t < a.T;
        if (acting) {
            const StepPre pre = step_prepare(s, a, e0 + tid, t, s_walls + tid * 8);
            s_pre[tid] = make_uint2(__float_as_uint(pre.u), (uint32_t)pre.np[0] | ((uint32_t)pre.np[1] << 8) | ((uint32_t)pre.np[2] << 16) | ((uint32_t)pre.np[3] << 24));
        }
        // ---- layer 2 on the tensor pipe: acc[mt][j] = rows 16mt.. x columns 8(wid*NT+j)..
        float acc[2][NT][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[mt][j][q] = 0.f;
        {
            const int arow = (lane & 7) + ((lane >> 3) & 1) * 8, acol = (lane >> 4) * 8;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t ahi[2][4], alo[2][4];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    ldmatrix_x4(ahi[mt], s_h1hi + (16 * mt + arow) * LD + 16 * ks + acol);
                    if (PREC == 0) ldmatrix_x4(alo[mt], s_h1lo + (16 * mt + arow) * LD + 16 * ks + acol);
                }
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const uint2 bhi = s_w2hi[(ks * (H / 8) + wid * NT + j) * 32 + lane];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        if (PREC == 0) {
                            mma16816<PREC>(acc[mt][j], alo[mt], bhi.x, bhi.y);
                            mma16816<PREC>(acc[mt][j], ahi[mt], blo[ks][j].x, blo[ks][j].y);
                        }
                        mma16816<PREC>(acc[mt][j], ahi[mt], bhi.x, bhi.y);
                    }
                }
            }
        }
        // ---- epilogue: bias, ReLU, head partials over this warp's columns
        {
            float ps[4][5];  // rows g, g+8, 16+g, 24+g
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 5; ++c) ps[r][c] = 0.f;
            const bool save_h2 = b.h2 != nullptr && t < a.T;
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                const int col0 = (wid * NT + j) * 8 + 2 * t4;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const float bias = s_b2[col0 + cc];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) acc[mt][j][2 * hh + cc] = rnd<PREC>(fmaxf(acc[mt][j][2 * hh + cc] + bias, 0.f));
                }
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int row = 16 * mt + 8 * hh + g;
                        if (save_h2 && e0 + row < B)
                            *reinterpret_cast<float2*>(b.h2 + ((size_t)t * B + e0 + row) * H + col0) =
                                make_float2(acc[mt][j][2 * hh], acc[mt][j][2 * hh + 1]);
                    }
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    float wh[5];
#pragma unroll
                    for (int c = 0; c < 5; ++c) wh[c] = s_wh[(col0 + cc) * 5 + c];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const float h2 = acc[mt][j][2 * hh + cc];
#pragma unroll
                            for (int c = 0; c < 5; ++c) ps[2 * mt + hh][c] = fmaf(h2, wh[c], ps[2 * mt + hh][c]);
                        }
                }
            }
            // sum over the four lanes of a quad with a transposing exchange: after two rounds lane t4 holds the total
            // of ONE of the four rows (15 shuffles instead of 40), and every lane stores its row
            float q2[2][5];
            const bool b0 = t4 & 1, b1 = t4 & 2;
#pragma unroll
            for (int c = 0; c < 5; ++c) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float send = b0 ? ps[i][c] : ps[2 + i][c];
                    const float keep = b0 ? ps[2 + i][c] : ps[i][c];
                    q2[i][c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
                }
            }
            const int r = (b0 ? 2 : 0) + (b1 ? 1 : 0);
            const int row = 16 * (r >> 1) + 8 * (r & 1) + g;
#pragma unroll
            for (int c = 0; c < 5; ++c) {
                const float send = b1 ? q2[0][c] : q2[1][c];
                const float keep = b1 ? q2[1][c] : q2[0][c];
                s_red[(wid * ME + row) * 5 + c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
            }
        }
        __syncthreads();
        // ---- one thread per env: fixed-order sum of the warps' partials, then act and step
        if (owner) {
            float o[5];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] = 0.f;
            for (int w = 0; w < NW; ++w)
#pragma unroll
                for (int c = 0; c < 5; ++c) o[c] += s_red[(w * ME + tid) * 5 + c];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] += s_bh[c];
            const int env = e0 + tid;
            if (b.out5 && t < a.T) {  // the update reuses the head outputs of every recorded row
                float4* o5 = reinterpret_cast<float4*>(b.out5 + ((size_t)t * B + env) * 8);
                o5[0] = make_float4(o[0], o[1], o[2], o[3]);
                o5[1] = make_float4(o[4], 0.f, 0.f, 0.f);
            }
            if (a.replay == 2 && t == a.T) b.vboot[env] = o[4];
            if (!a.replay) {
                b.tval[(size_t)t * B + env] = o[4];
                if (a.gae_smem) s_gv[t * ME + tid] = o[4];
                if (acting) {
                    const uint2 pk = s_pre[tid];
                    StepPre pre;
                    pre.u = __uint_as_float(pk.x);
#pragma unroll
                    for (int q = 0; q < 4; ++q) pre.np[q] = (pk.y >> (8 * q)) & 0xFF;
                    const int code = act_and_step_pre(s, a, env, t, o[0], o[1], o[2], o[3], pre);
                    if (a.gae_smem) s_gc[t * ME + tid] = (uint8_t)code;
                    s_pos[tid] = s.pos;
                }
            }
        }
        __syncthreads();
    }
    if (a.replay) return;
    if (owner) {
        b.pos[e0 + tid] = (uint8_t)s.pos;
        b.tep[e0 + tid] = (uint8_t)s.tep;
        // the owner thread wrote this env's rewards, values and done flags itself: it can scan them right away
        if (a.gae_smem) gae_scan_env_smem(b, B, a.T, e0 + tid, a.gamma, a.lambda, s_gv, s_gc, ME, tid);
        else if (a.fuse_gae) gae_scan_env(b, B, a.T, e0 + tid, a.gamma, a.lambda);
    }
    if (tid < 32) flush_env_stats(s, a);
}

constexpr size_t MAX_DYN_SMEM = 232448;  // 227 KB of dynamic shared memory per CTA

template <int H, int NW, int PREC, bool GROUPED = false>
static cudaError_t launch_t(const RolloutArgs& a0, cudaStream_t s) {
    using Cfg = RolloutMmaCfg<H, NW, PREC>;
    RolloutArgs a = a0;
    size_t smem = Cfg::smem_bytes;
    a.gae_smem = 0;
    if (a.fuse_gae && !a.replay && smem + Cfg::gae_bytes(a.T) <= MAX_DYN_SMEM) {
        a.gae_smem = 1;
        smem += Cfg::gae_bytes(a.T);
    }
    cudaError_t e = cudaFuncSetAttribute(k_rollout_mma<H, NW, PREC, GROUPED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MAX_DYN_SMEM);
    if (e != cudaSuccess) return e;
    const dim3 grid((a.d.B + Cfg::ME - 1) / Cfg::ME, GROUPED ? a.d.npol : 1);
    k_rollout_mma<H, NW, PREC, GROUPED><<<grid, NW * 32, smem, s>>>(a);
    return cudaGetLastError();
}

bool rollout_mma_supported(int H) { return H == 64 || H == 128 || H == 256; }
// fp32 at H = 256 runs the CTA-pair tcgen05 kernel, which reads the row-major planes of W2 only.
bool rollout_uses_fragments(int H, int prec) { return rollout_mma_supported(H) && !(H == 256 && prec == 0); }

// Returns cudaErrorNotSupported when the shape is not covered by the tensor-pipe kernel.
cudaError_t launch_rollout_mma(const RolloutArgs& a, int prec, cudaStream_t s) {
    if (!rollout_mma_supported(a.d.H)) return cudaErrorNotSupported;
    if (prec == 0 && a.d.npol <= 1 && a.d.H == 256) {  // the CTA-pair kernels on the 5th-generation tensor cores
        const cudaError_t e = launch_rollout_pair2(a, s);  // large batches: two env groups per pair
        if (e != cudaErrorNotSupported) return e;
        return launch_rollout_pair(a, s);
    }
    if (prec == 0 && a.d.npol <= 1 && a.d.H == 128) {  // large batches: two env groups per CTA on the 5th-generation tensor cores
        const cudaError_t e = launch_rollout_tc128(a, s);
        if (e != cudaErrorNotSupported) return e;
    }
    if (!a.b.w2f_hi) return cudaErrorNotSupported;
    if (a.d.npol > 1) {  // many policies: one grid slice per policy, each with its own weights on chip
        if (prec != 0) return cudaErrorNotSupported;
        switch (a.d.H) {
            case 64: return launch_t<64, 4, 0, true>(a, s);
            case 128: return launch_t<128, 8, 0, true>(a, s);
        }
        return cudaErrorNotSupported;
    }
    if (prec == 1) {
        switch (a.d.H) {
            case 64: return launch_t<64, 4, 1>(a, s);
            case 128: return launch_t<128, 8, 1>(a, s);
            case 256: return launch_t<256, 16, 1>(a, s);
        }
    } else {
        switch (a.d.H) {
            case 64: return launch_t<64, 4, 0>(a, s);
            case 128: return launch_t<128, 8, 0>(a, s);
        }
    }
    return cudaErrorNotSupported;
}

}  // namespace anakin
