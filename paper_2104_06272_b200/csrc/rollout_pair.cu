// Persistent rollout on the 5th-generation tensor cores: a pair of CTAs (a cluster of two, on neighbouring SMs) owns
// 64 envs for all T+1 forward passes of a rollout and shares the second-layer weights between its two SMs.
//
// Acting half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top), hidden width 256, fp32 workloads.
// The second layer is computed transposed,  D[j][env] = sum_k W2[k][j] h1[env][k],  as tcgen05.mma.cta_group::2 with
// M = 256 hidden units, so that each CTA keeps only ITS 128 columns of W2 on chip (two fp16 planes, 128 KB, loaded once
// by TMA) and builds only the h1 rows of ITS 32 envs; the tensor cores of the pair read both CTAs' h1 rows, and each
// CTA receives its 128 hidden units x all 64 envs in its own tensor memory.  Per step:
//   layer 1   h1 = relu(base + W1[agent row])       gather-add; the fp16 (hi, lo) terms go straight into the swizzled
//                                                   K-major operand tile [32 hi rows | 32 lo rows] x 256 k
//   layer 2   two MMAs per k16:  W2hi x [h1hi | h1lo]  (N = 128 over the pair)  and  W2lo x h1hi  (N = 64), fp32
//             accumulators in tensor memory; one thread of the leader CTA issues them for the pair
//   heads     a thread = one hidden unit j: bias, ReLU, h2 stores (one 128-byte line per env and warp); the warp's
//             32 units x 32 envs go to shared memory as fp16 (hi, lo) terms and come back transposed (ldmatrix.trans)
//             as A fragments of warp-level MMAs against Wh: out[env][c] = sum_j h2[j][env] Wh[j][c]; the eight 32-unit
//             partials of an env meet in the shared memory of the CTA that owns it, sent as asynchronous remote stores
//             that count their bytes on the owner's mbarrier
//   env       (ninth warp) one thread per env: softmax, Philox inverse-CDF sample, gridworld step, time-major records
// Inside a step the CTAs of a pair meet only through mbarriers (operand blocks written -> issuer; MMAs finished ->
// workers; partials landed -> owners) and each CTA has one barrier of its own (new positions); the cluster barrier is
// used at start and exit only.  Every mbarrier wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the threads keep
// walking through the barriers to the exit, where tensor memory is freed.
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

struct PairCfg {
    static constexpr int H = 256, ME = 32, NWORK = 8, THREADS = (NWORK + 1) * 32;
    static constexpr int BOX = 64 * 64 * 2;                   // one 64 x 64 box of 16-bit elements
    static constexpr int A_PLANE = (128 / 64) * (H / 64) * BOX;  // this CTA's 128 columns of W2, all k: 64 KB
    static constexpr int B_CHUNK = 64 * 128;                  // 64 operand rows (32 hi + 32 lo) x 64 k
    static constexpr int B_BYTES = (H / 64) * B_CHUNK;        // 32 KB
    static constexpr int TMEM_COLS = 256;                     // [0,128): W2hi x [hi|lo] of both CTAs, [128,192): W2lo x hi
    static constexpr size_t fixed_bytes =
        2 * (size_t)A_PLANE + B_BYTES + (size_t)ME * H * 4    // W2 planes, operand tile, base
        + 64                                                  // barriers, tensor-memory slot
        + (size_t)8 * ME * 5 * 4                              // head partials: 8 blocks of 32 hidden units
        + 8 * 4 + (size_t)ME * 8 * 4 + ME * 4;                // bh, walls, pos
    static constexpr size_t gae_bytes(int T) { return (size_t)(T + 1) * ME * 4 + (size_t)T * ME; }
};

struct PairMaps {
    CUtensorMap w_hi, w_lo;  // W2 row-major [k][j] as fp16 planes, boxes of 64 j x 64 k
};

// Asynchronous store of one float into the shared memory of a CTA of the cluster; when it has landed it counts its
// four bytes on the mbarrier (same CTA as the destination), so the reader needs no fence from the writer.
__device__ __forceinline__ void st_async_f32(uint32_t cluster_addr, float v, uint32_t cluster_bar_addr) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(cluster_addr), "f"(v),
                 "r"(cluster_bar_addr)
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairCfg::THREADS, 1) k_rollout_pair(const __grid_constant__ PairMaps maps, RolloutArgs a) {
    using Cfg = PairCfg;
    constexpr int H = Cfg::H, ME = Cfg::ME, NWT = Cfg::NWORK * 32;
    extern __shared__ unsigned char smem_raw[];
    // the dynamic shared memory starts at the same offset in both CTAs, so the rounded base does too
    unsigned char* sm = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* s_ahi = sm;
    unsigned char* s_alo = s_ahi + Cfg::A_PLANE;
    unsigned char* s_bop = s_alo + Cfg::A_PLANE;
    float* s_base = reinterpret_cast<float*>(s_bop + Cfg::B_BYTES);                 // [ME][H]
    uint64_t* wbar = reinterpret_cast<uint64_t*>(s_base + ME * H);                  // weights landed
    uint64_t* tfull = wbar + 1;                                                     // this step's MMAs finished
    uint64_t* ready = tfull + 1;   // [4] leader's copy: k block kb of both CTAs' operand rows written (16 warps arrive)
    uint64_t* pfull = ready + 4;   // the eight head partials of this CTA's envs have landed (counted in bytes)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pfull + 1);
    float* s_red = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(wbar) + 64);  // [8][ME][5]
    float* s_bh = s_red + 8 * ME * 5;                                               // [8]
    uint32_t* s_walls = reinterpret_cast<uint32_t*>(s_bh + 8);                      // [ME][8]
    int* s_pos = reinterpret_cast<int*>(s_walls + ME * 8);                          // [ME]
    float* s_gv = reinterpret_cast<float*>(s_pos + ME);                             // [T+1][ME] (a.gae_smem only)
    uint8_t* s_gc = reinterpret_cast<uint8_t*>(s_gv + (a.T + 1) * ME);              // [T][ME]

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t rank = tc::cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int e0 = pair * 2 * ME + (int)rank * ME;  // this CTA's first env
    const int B = d.B, C = d.C;
    const float* W1 = b.theta_c + d.oW1;
    const bool worker = wid < Cfg::NWORK;

    // ---- prologue
    if (tid == 0) {
        tc::mbar_init(wbar, 1);
        tc::mbar_init(tfull, 1);
        for (int kb = 0; kb < 4; ++kb) tc::mbar_init(&ready[kb], 2 * Cfg::NWORK);
        tc::mbar_init(pfull, 1);
        tc::mbar_fence_init();
    }
    if (wid == Cfg::NWORK) tc::tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (tid == NWT) {  // this CTA's 128 columns of W2: box (kb, bx) = k rows 64kb.., columns 128 rank + 64 bx..
        tc::mbar_expect_tx(wbar, 2 * Cfg::A_PLANE);
#pragma unroll
        for (int kb = 0; kb < H / 64; ++kb)
#pragma unroll
            for (int bx = 0; bx < 2; ++bx) {
                tc::tma_load_2d(s_ahi + (kb * 2 + bx) * Cfg::BOX, &maps.w_hi, wbar, 128 * (int)rank + 64 * bx, 64 * kb);
                tc::tma_load_2d(s_alo + (kb * 2 + bx) * Cfg::BOX, &maps.w_lo, wbar, 128 * (int)rank + 64 * bx, 64 * kb);
            }
    }
    // hidden unit of this thread in the heads phase, and its constants
    const int q = wid & 3, rE = (wid >> 2) & 1;  // accumulator lanes 32q.., envs of CTA rE
    const int j = 128 * (int)rank + 32 * q + lane;
    float b2j = 0.f;
    uint32_t whf_hi[2][2], whf_lo[2][2];  // Wh rows of this warp's 32 hidden units as mma B fragments (k16 x n8), two k steps
    EnvLane s;
    s.pos = s.tep = s.start = s.goal = 0;
    s.n_episodes = s.n_goals = s.n_epsteps = 0;
    s.bad = 0;
    const int ow = tid - NWT;  // warp 8: lane = env of this CTA (its lane 0 also issues the pair's MMAs)
    const bool owner = ow >= 0 && e0 + ow < B;
    if (worker) {
        for (int i = tid; i < ME * H / 4; i += NWT) {
            const int e = i / (H / 4), k = 4 * (i - e * (H / 4));
            const bool okb = e0 + e < B;
            cp_async16(s_base + e * H + k, b.base + (size_t)(okb ? e0 + e : 0) * H + k, okb ? 16 : 0);
        }
        cp_async_commit();
        b2j = b.theta_c[d.ob2 + j];
        {   // fragment element (k, n): lane = 4n + t holds k = 2t, 2t+1 (first register) and 2t+8, 2t+9 (second)
            const int n = lane >> 2, t4 = lane & 3;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int jj = 128 * (int)rank + 32 * q + 16 * ks + 8 * hh + 2 * t4;
                    const float w0 = n < 5 ? b.theta_c[d.oWh + (size_t)jj * 5 + n] : 0.f;
                    const float w1 = n < 5 ? b.theta_c[d.oWh + (size_t)(jj + 1) * 5 + n] : 0.f;
                    split2<0>(w0, w1, whf_hi[ks][hh], whf_lo[ks][hh]);
                }
        }
        if (tid < 5) s_bh[tid] = b.theta_c[d.obh + tid];
        cp_async_wait<0>();
    } else {
        for (int wi = 0; wi < 8; ++wi) s_walls[ow * 8 + wi] = (owner && wi < d.W) ? b.walls[(size_t)(e0 + ow) * d.W + wi] : 0u;
        if (owner) {
            s.pos = b.pos[e0 + ow];
            s.tep = b.tep[e0 + ow];
            s.start = b.start[e0 + ow];
            s.goal = b.goal[e0 + ow];
            check_env_state(s, C, s_walls + ow * 8);
        }
        s_pos[ow] = s.pos;
    }
    bool ok = true;
    if (tid == NWT) ok = tc::mbar_wait(wbar, 0);  // the issuer's thread vouches for the weights of its CTA
    __syncthreads();
    tc::cluster_sync_all();  // both CTAs' barriers, tensor memory and weights exist before the first MMA

    __nv_bfloat16* g_h1hi = reinterpret_cast<__nv_bfloat16*>(b.h1);
    __nv_bfloat16* g_h1lo = g_h1hi + (size_t)B * d.Tmax * H;
    const uint32_t idesc_w = tc::umma_idesc<0>(256, 128, true, false), idesc_n = tc::umma_idesc<0>(256, 64, true, false);

    const int t_end = a.replay == 1 ? a.T - 1 : a.T;  // replay recomputes the T recorded rows (mode 2: and the current state)
    for (int t = 0; t <= t_end; ++t) {
        if (a.replay) {  // positions come from the recorded trajectory
            if (ow >= 0) s_pos[ow] = owner ? min((int)(t < a.T ? b.tpos[(size_t)t * B + e0 + ow] : b.pos[e0 + ow]), C - 1) : 0;
            __syncthreads();
        }
        if (tid == NWT) tc::mbar_expect_tx(pfull, 8 * ME * 5 * 4);  // this step's head partials, counted as they land
        // ---- layer 1 (workers): 16-byte chunks of eight hidden units; all gathers of the agent's W1 row are in flight
        // before any is used.  Trip kb covers k block kb (64 hidden units of layer 1) of all 32 envs: chunk c8 of env e goes
        // to operand row e (hi) and 32 + e (lo) of that block, at the 16-byte position c8 ^ (e % 8) of the 128-byte row
        // (the 128-byte swizzle of a K-major operand).  Each finished block is announced to the issuer at once, so the
        // tensor cores start on block 0 while the later blocks are still being written.
        if (worker) {
            const int e = tid >> 3, c8 = tid & 7;
            uint4 hi[4], lo[4];
            const float* wrow = W1 + (size_t)(C + s_pos[e]) * H + 8 * c8;
            float4 w[4][2];
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                const float4* wp = reinterpret_cast<const float4*>(wrow + 64 * kb);
                w[kb][0] = __ldg(wp);
                w[kb][1] = __ldg(wp + 1);
            }
            tc::tc_fence_before();  // this thread's reads of last step's accumulators precede the arrivals below
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                const int k = 64 * kb + 8 * c8;
                const float4 b0 = *reinterpret_cast<const float4*>(s_base + e * H + k);
                const float4 b1 = *reinterpret_cast<const float4*>(s_base + e * H + k + 4);
                split2<0>(fmaxf(b0.x + w[kb][0].x, 0.f), fmaxf(b0.y + w[kb][0].y, 0.f), hi[kb].x, lo[kb].x);
                split2<0>(fmaxf(b0.z + w[kb][0].z, 0.f), fmaxf(b0.w + w[kb][0].w, 0.f), hi[kb].y, lo[kb].y);
                split2<0>(fmaxf(b1.x + w[kb][1].x, 0.f), fmaxf(b1.y + w[kb][1].y, 0.f), hi[kb].z, lo[kb].z);
                split2<0>(fmaxf(b1.z + w[kb][1].z, 0.f), fmaxf(b1.w + w[kb][1].w, 0.f), hi[kb].w, lo[kb].w);
                unsigned char* row = s_bop + kb * Cfg::B_CHUNK + e * 128 + ((c8 ^ (e & 7)) << 4);
                *reinterpret_cast<uint4*>(row) = hi[kb];
                *reinterpret_cast<uint4*>(row + ME * 128) = lo[kb];
                tc::fence_proxy_async();  // ordinary stores -> visible to the tensor cores
                __syncwarp();
                if (lane == 0) tc::mbar_arrive_remote_cta_release(tc::mapa(tc::smem_u32(&ready[kb]), 0));
            }
            // the copies for the update leave after the arrivals (their CTA-scope release does not wait for global stores)
            if (b.h1 != nullptr && t < a.T && e0 + e < B) {
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    const size_t gi = ((size_t)t * B + e0 + e) * H + 64 * kb + 8 * c8;
                    *reinterpret_cast<uint4*>(g_h1hi + gi) = hi[kb];
                    *reinterpret_cast<uint4*>(g_h1lo + gi) = lo[kb];
                    if (b.gate1) b.gate1[gi >> 3] = (uint8_t)nonzero_bits16(hi[kb]);  // the gates of these eight units
                }
            }
        }
        // the logits-independent half of the interaction, taken by the owner warp while the workers gather
        const bool acting = owner && !a.replay && t < a.T;
        StepPre pre;
        if (acting) pre = step_prepare(s, a, e0 + ow, t, s_walls + ow * 8);
        // ---- layer 2: the leader's issuer thread drives both tensor cores, k block by k block.  A block's sixteen
        // arrivals also say that those warps have read last step's accumulators.
        if (tid == NWT && rank == 0) {
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                if (ok) ok = tc::mbar_wait_cluster(&ready[kb], (uint32_t)t & 1u);
                tc::tc_fence_after();
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16) {
                    // A (MN-major): 16 k rows = 2048 bytes into each box, 8192 bytes between the two 64-column boxes
                    const uint64_t ahi = tc::umma_desc(s_ahi + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                    const uint64_t alo = tc::umma_desc(s_alo + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                    // B (K-major): 16 k = 32 bytes along the swizzled rows, 1024 bytes between 8-row groups
                    const uint64_t bd = tc::umma_desc(s_bop + kb * Cfg::B_CHUNK + k16 * 32, 16, 1024);
                    tc::umma_pair(tmem, ahi, bd, idesc_w, (kb | k16) ? 1u : 0u);
                    tc::umma_pair(tmem + 128u, alo, bd, idesc_n, (kb | k16) ? 1u : 0u);
                }
            }
            tc::umma_commit_pair(tfull, 3);
        }
        // ---- heads (workers): thread = hidden unit j, 32 envs of CTA rE
        if (worker) {
            if (ok) ok = tc::mbar_wait(tfull, (uint32_t)t & 1u);
            tc::tc_fence_after();
            float v[32];
            {
                uint32_t r0[32], r1[32], r2[32];
                const uint32_t lanes = tmem + ((uint32_t)(32 * q) << 16);
                tc::tmem_ld32_nowait(lanes + (uint32_t)(64 * rE), r0);        // W2hi x h1hi
                tc::tmem_ld32_nowait(lanes + (uint32_t)(64 * rE + 32), r1);   // W2hi x h1lo
                tc::tmem_ld32_nowait(lanes + 128u + (uint32_t)(32 * rE), r2); // W2lo x h1hi
                tc::tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = fmaxf(((__uint_as_float(r0[e]) + __uint_as_float(r1[e])) + __uint_as_float(r2[e])) + b2j, 0.f);
            }
            // head partials over this warp's 32 hidden units on the warp-level tensor path.  The operand tile is free
            // once the step's MMAs have finished: warp w keeps [32 units][32 envs] fp16 hi and lo planes in its 4 KB of it,
            // rows of 64 bytes whose 16-byte chunks are XOR-swizzled by (row / 2) % 4 (conflict-free both ways).
            unsigned char* wsm = s_bop + wid * 4096;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint4 hi, lo;
                split2<0>(v[8 * c4 + 0], v[8 * c4 + 1], hi.x, lo.x);
                split2<0>(v[8 * c4 + 2], v[8 * c4 + 3], hi.y, lo.y);
                split2<0>(v[8 * c4 + 4], v[8 * c4 + 5], hi.z, lo.z);
                split2<0>(v[8 * c4 + 6], v[8 * c4 + 7], hi.w, lo.w);
                const int off = lane * 64 + ((c4 ^ ((lane >> 1) & 3)) << 4);
                *reinterpret_cast<uint4*>(wsm + off) = hi;
                *reinterpret_cast<uint4*>(wsm + 2048 + off) = lo;
            }
            __syncwarp();
            float acc[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
            {
                // A fragment (row = env, k = unit) from the [unit][env] tile: matrix i of the x4 load covers units
                // 16ks + 8(i/2) .., envs 16mt + 8(i%2) ..; the transposing load hands out the fragment's register order
                const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    const int krow = 16 * ks + 8 * (mi >> 1) + r8;
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        const int chunk = 2 * mt + (mi & 1);
                        const int off = krow * 64 + ((chunk ^ ((krow >> 1) & 3)) << 4);
                        uint32_t ahi[4], alo[4];
                        ldmatrix_x4_trans(ahi, wsm + off);
                        ldmatrix_x4_trans(alo, wsm + 2048 + off);
                        // the x4 order above is (k lo, m lo), (k lo, m hi), (k hi, m lo), (k hi, m hi) = a0, a1, a2, a3
                        mma_f16(acc[mt], alo, whf_hi[ks][0], whf_hi[ks][1]);
                        mma_f16(acc[mt], ahi, whf_lo[ks][0], whf_lo[ks][1]);
                        mma_f16(acc[mt], ahi, whf_hi[ks][0], whf_hi[ks][1]);
                    }
                }
            }
            // accumulator element (row g + 8hh of tile mt, column 2 t4 + cc) = (env 16mt + 8hh + g, head 2 t4 + cc)
            {
                const int g = lane >> 2, t4 = lane & 3;
                const uint32_t pbar = tc::mapa(tc::smem_u32(pfull), (uint32_t)rE);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int e = 16 * mt + 8 * hh + g;
                        const uint32_t dst = tc::mapa(tc::smem_u32(s_red + ((4 * (int)rank + q) * ME + e) * 5 + 2 * t4), (uint32_t)rE);
                        if (t4 < 3) st_async_f32(dst, acc[mt][2 * hh], pbar);
                        if (t4 < 2) st_async_f32(dst + 4u, acc[mt][2 * hh + 1], pbar);
                    }
            }
            // h2 for the update: one 128-byte line per env
            const int env0 = pair * 2 * ME + rE * ME;  // first env of the block this warp holds
            if (b.h2 != nullptr && t < a.T) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (env0 + e < B) b.h2[((size_t)t * B + env0 + e) * H + j] = v[e];
            }
        }
        // ---- one thread per env: once the eight partials are in, their fixed-order sum, then act and step
        if (!worker && ok) ok = tc::mbar_wait_cluster(pfull, (uint32_t)t & 1u);
        // The new positions are all the next step's gather needs: the owners publish them and release the workers (named
        // barrier 1: the workers wait on it, the owner warp only arrives, once and as a whole warp) before they write the
        // step's records.
        if (!worker) {
            float o[5];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] = 0.f;
            ActOut ao;
            ao.la_mx = ao.Z = ao.rew = 0.f;
            ao.act = ao.done = ao.pos0 = 0;
            const int env = e0 + ow;
            if (owner) {
#pragma unroll
                for (int blk = 0; blk < 8; ++blk)
#pragma unroll
                    for (int c = 0; c < 5; ++c) o[c] += s_red[(blk * ME + ow) * 5 + c];
#pragma unroll
                for (int c = 0; c < 5; ++c) o[c] += s_bh[c];
                if (acting) {
                    ao = act_decide(s, a, env, t, o[0], o[1], o[2], o[3], pre);
                    s_pos[ow] = s.pos;
                }
            }
            __syncwarp();
            asm volatile("bar.arrive 1, %0;" ::"n"(Cfg::THREADS) : "memory");
            if (owner) {
                if (b.out5 && t < a.T) {  // the update reuses the head outputs of every recorded row
                    float4* o5 = reinterpret_cast<float4*>(b.out5 + ((size_t)t * B + env) * 8);
                    o5[0] = make_float4(o[0], o[1], o[2], o[3]);
                    o5[1] = make_float4(o[4], 0.f, 0.f, 0.f);
                }
                if (a.replay == 2 && t == a.T) b.vboot[env] = o[4];
                if (!a.replay) {
                    b.tval[(size_t)t * B + env] = o[4];
                    if (a.gae_smem) s_gv[t * ME + ow] = o[4];
                }
                if (acting) {
                    act_record(a, env, t, o[0], o[1], o[2], o[3], ao);
                    if (a.gae_smem) s_gc[t * ME + ow] = (uint8_t)(ao.done | (ao.rew != 0.f ? 2 : 0));
                }
            }
        } else {
            // every worker is done with its staging area in the operand tile, and the positions are in place
            asm volatile("bar.sync 1, %0;" ::"n"(Cfg::THREADS) : "memory");
        }
    }
    if (owner && !a.replay) {
        b.pos[e0 + ow] = (uint8_t)s.pos;
        b.tep[e0 + ow] = (uint8_t)s.tep;
        if (a.gae_smem) gae_scan_env_smem(b, B, a.T, e0 + ow, a.gamma, a.lambda, s_gv, s_gc, ME, ow);
        else if (a.fuse_gae) gae_scan_env(b, B, a.T, e0 + ow, a.gamma, a.lambda);
    }
    if (!worker && !a.replay) flush_env_stats(s, a);
    if (!ok && lane == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
    // neither CTA frees tensor memory or leaves while the other may still signal it
    tc::tc_fence_before();
    __syncthreads();
    tc::cluster_sync_all();
    if (wid == Cfg::NWORK) tc::tmem_dealloc_pair(tmem, Cfg::TMEM_COLS);
}

}  // namespace

// Covers hidden width 256 with fp32 parameters (two-term fp16 operands) when the row-major 16-bit planes of W2 exist;
// anything else returns cudaErrorNotSupported and the caller takes the warp-level kernel.
cudaError_t launch_rollout_pair(const RolloutArgs& a0, cudaStream_t s) {
    using Cfg = PairCfg;
    if (a0.d.H != Cfg::H || !a0.b.w2p_hi || !a0.b.w2p_lo || !a0.b.base) return cudaErrorNotSupported;
    RolloutArgs a = a0;
    size_t smem = Cfg::fixed_bytes + 1024;  // alignment slack
    a.gae_smem = 0;
    if (a.fuse_gae && !a.replay && smem + Cfg::gae_bytes(a.T) <= 232448) {
        a.gae_smem = 1;
        smem += Cfg::gae_bytes(a.T);
    }
    PairMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.w_hi, a.b.w2p_hi, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_lo, a.b.w2p_lo, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    const cudaError_t e = cudaFuncSetAttribute(k_rollout_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    const int pairs = (a.d.B + 2 * Cfg::ME - 1) / (2 * Cfg::ME);
    k_rollout_pair<<<2 * pairs, Cfg::THREADS, smem, s>>>(maps, a);
    return cudaGetLastError();
}

}  // namespace anakin
