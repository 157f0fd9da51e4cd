// Persistent rollout on the 5th-generation tensor cores for hidden width 256 and large batches: a pair of CTAs (a
// cluster of two, on neighbouring SMs) owns 128 envs for all T+1 forward passes, in TWO independent groups of 64.
//
// Acting half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top), fp32 workloads.  The layout of one
// group is that of the one-group CTA-pair kernel: layer 2 transposed, D[j][env] = sum_k W2[k][j] h1[env][k], as
// tcgen05.mma.cta_group::2 with M = 256 hidden units, each CTA keeping ITS 128 columns of W2 on chip (two fp16 planes,
// 128 KB, loaded once by TMA) and building the h1 rows of ITS 32 envs of the group.  With many envs per SM the rollout is a
// throughput problem, but one group walks a strictly serial chain per step (gather -> tensor cores -> heads -> sample);
// so a CTA holds two groups, each with eight worker warps and an owner warp of its own, and one group's tensor-core and
// sampling phases fall into the other's gather and heads phases.  Per group and step:
//   layer 1   h1 = relu(base + W1[agent row])       gather-add (base read from L2: shared memory holds W2 and two
//                                                   operand tiles); fp16 (hi, lo) terms straight into the swizzled
//                                                   K-major operand tile [32 hi rows | 32 lo rows] x 256 k
//   layer 2   two MMAs per k16:  W2hi x [h1hi | h1lo]  (N = 128 over the pair)  and  W2lo x h1hi  (N = 64), fp32
//             accumulators in tensor memory; one thread of the leader CTA's issuer warp drives both groups
//   heads     a worker thread = one hidden unit j: bias, ReLU, h2 stores, then 32 units x 32 envs through shared memory
//             (ldmatrix.trans) into warp-level MMAs against Wh; the eight 32-unit partials of an env meet in the shared
//             memory of the CTA that owns it, sent as asynchronous remote stores that count their bytes on its mbarrier
//   env       (owner warps) one thread per env: softmax, Philox inverse-CDF sample, gridworld step, time-major records;
//             the new position is published before the records are written
// The phases meet through mbarriers only; the cluster barrier is used at start and exit.  Every wait is bounded; a timeout
// raises DEV_E_WAIT_TIMEOUT and the threads keep walking through the barriers to the exit, where tensor memory is freed.
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

struct Pair2Cfg {
    static constexpr int H = 256, ME = 32, NG = 2, NWORK = 8;       // ME envs per CTA and group, NWORK worker warps per group
    static constexpr int NWT = NG * NWORK * 32;                     // worker threads
    static constexpr int NOWN = NG * ME;                            // owner threads: one per env of this CTA
    static constexpr int THREADS = NWT + NOWN + 32;                 // + the issuer warp
    static constexpr int BOX = 64 * 64 * 2;                         // one 64 x 64 box of 16-bit elements
    static constexpr int A_PLANE = (128 / 64) * (H / 64) * BOX;     // this CTA's 128 columns of W2, all k: 64 KB
    static constexpr int B_CHUNK = 64 * 128;                        // 64 operand rows (32 hi + 32 lo) x 64 k
    static constexpr int B_BYTES = (H / 64) * B_CHUNK;              // a group's operand tile: 32 KB
    static constexpr int ACC = 192;                                 // TMEM columns of a group
    static constexpr int TMEM_COLS = 512;
    static constexpr size_t fixed_bytes =
        2 * (size_t)A_PLANE + (size_t)NG * B_BYTES                  // W2 planes, operand tiles
        + 256                                                       // barriers, tensor-memory slot
        + (size_t)NG * 8 * ME * 5 * 4                               // head partials: 8 blocks of 32 hidden units per group
        + 8 * 4 + (size_t)NOWN * 8 * 4 + NOWN * 4;                  // bh, walls, pos
    static constexpr size_t gae_bytes(int T) { return (size_t)(T + 1) * NOWN * 4 + (size_t)T * NOWN; }
};

struct Pair2Maps {
    CUtensorMap w_hi, w_lo;  // W2 row-major [k][j] as fp16 planes, boxes of 64 j x 64 k
};

// Asynchronous store of one float into the shared memory of a CTA of the cluster; when it has landed it counts its
// four bytes on the mbarrier (same CTA as the destination), so the reader needs no fence from the writer.
__device__ __forceinline__ void st_async_f32_2(uint32_t cluster_addr, float v, uint32_t cluster_bar_addr) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(cluster_addr), "f"(v),
                 "r"(cluster_bar_addr)
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Pair2Cfg::THREADS, 1) k_rollout_pair2(const __grid_constant__ Pair2Maps maps, RolloutArgs a) {
    using Cfg = Pair2Cfg;
    constexpr int H = Cfg::H, ME = Cfg::ME, NG = Cfg::NG, NWT = Cfg::NWT, NOWN = Cfg::NOWN;
    extern __shared__ unsigned char smem_raw[];
    // the dynamic shared memory starts at the same offset in both CTAs, so the rounded base does too
    unsigned char* sm = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* s_ahi = sm;
    unsigned char* s_alo = s_ahi + Cfg::A_PLANE;
    unsigned char* s_bop = s_alo + Cfg::A_PLANE;                                     // [NG] operand tiles
    uint64_t* wbar = reinterpret_cast<uint64_t*>(s_bop + NG * Cfg::B_BYTES);         // weights landed
    uint64_t* tfull = wbar + 1;      // [NG] this step's MMAs of the group finished
    uint64_t* ready = tfull + NG;    // [NG][4] leader's copy: k block of both CTAs' operand rows written (16 warps arrive)
    uint64_t* pfull = ready + NG * 4;  // [NG] the eight head partials of this CTA's envs of the group have landed (bytes)
    uint64_t* posrdy = pfull + NG;     // [NG] this CTA's positions of the group for the next step are published
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(posrdy + NG);
    float* s_red = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(wbar) + 256);  // [NG][8][ME][5]
    float* s_bh = s_red + NG * 8 * ME * 5;                                           // [8]
    uint32_t* s_walls = reinterpret_cast<uint32_t*>(s_bh + 8);                       // [NOWN][8]
    int* s_pos = reinterpret_cast<int*>(s_walls + NOWN * 8);                         // [NOWN]
    float* s_gv = reinterpret_cast<float*>(s_pos + NOWN);                            // [T+1][NOWN] (a.gae_smem only)
    uint8_t* s_gc = reinterpret_cast<uint8_t*>(s_gv + (a.T + 1) * NOWN);             // [T][NOWN]

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t rank = tc::cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    // the pair owns envs pair*128 ..: group g has 64 of them, CTA `rank` the 32 at pair*128 + g*64 + rank*32
    const int B = d.B, C = d.C;
    const float* W1 = b.theta_c + d.oW1;
    const bool worker = tid < NWT;
    const bool ownerw = tid >= NWT && tid < NWT + NOWN;
    const int iwarp = (NWT + NOWN) / 32;           // the issuer warp
    const bool issuer = tid == NWT + NOWN;

    // ---- prologue
    if (tid == 0) {
        tc::mbar_init(wbar, 1);
        for (int g = 0; g < NG; ++g) {
            tc::mbar_init(&tfull[g], 1);
            for (int kb = 0; kb < 4; ++kb) tc::mbar_init(&ready[4 * g + kb], 2 * Cfg::NWORK);
            tc::mbar_init(&pfull[g], 1);
            tc::mbar_init(&posrdy[g], 1);
        }
        tc::mbar_fence_init();
    }
    if (wid == iwarp) tc::tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (issuer) {  // this CTA's 128 columns of W2: box (kb, bx) = k rows 64kb.., columns 128 rank + 64 bx..
        tc::mbar_expect_tx(wbar, 2 * Cfg::A_PLANE);
#pragma unroll
        for (int kb = 0; kb < H / 64; ++kb)
#pragma unroll
            for (int bx = 0; bx < 2; ++bx) {
                tc::tma_load_2d(s_ahi + (kb * 2 + bx) * Cfg::BOX, &maps.w_hi, wbar, 128 * (int)rank + 64 * bx, 64 * kb);
                tc::tma_load_2d(s_alo + (kb * 2 + bx) * Cfg::BOX, &maps.w_lo, wbar, 128 * (int)rank + 64 * bx, 64 * kb);
            }
    }
    // worker constants
    const int wg = worker ? wid / Cfg::NWORK : 0;   // the worker's group
    const int wl = wid % Cfg::NWORK;                // its warp within the group
    const int tidg = tid % (Cfg::NWORK * 32);       // its thread index within the group
    const int q = wl & 3, rE = (wl >> 2) & 1;       // accumulator lanes 32q.., envs of CTA rE
    const int j = 128 * (int)rank + 32 * q + lane;  // hidden unit of this thread in the heads phase
    float b2j = 0.f;
    uint32_t whf_hi[2][2], whf_lo[2][2];  // Wh rows of this warp's 32 hidden units as mma B fragments (k16 x n8), two k steps
    EnvLane s;
    s.pos = s.tep = s.start = s.goal = 0;
    s.n_episodes = s.n_goals = s.n_epsteps = 0;
    s.bad = 0;
    const int ow = tid - NWT;                  // owner threads: index into this CTA's envs, group ow / ME
    const int og = ownerw ? ow / ME : 0;
    const int oe = ow - og * ME;               // env index within the group's 32 of this CTA
    const int oenv = pair * (2 * NG * ME) + og * (2 * ME) + (int)rank * ME + oe;  // global env of an owner thread
    const bool owner = ownerw && oenv < B;
    if (worker) {
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
    } else if (ownerw) {
        for (int wi = 0; wi < 8; ++wi) s_walls[ow * 8 + wi] = (owner && wi < d.W) ? b.walls[(size_t)oenv * d.W + wi] : 0u;
        if (owner) {
            s.pos = b.pos[oenv];
            s.tep = b.tep[oenv];
            s.start = b.start[oenv];
            s.goal = b.goal[oenv];
            check_env_state(s, C, s_walls + ow * 8);
            if (a.replay) s.pos = min((int)(a.T > 0 ? b.tpos[oenv] : b.pos[oenv]), C - 1);  // row 0 of the recorded positions
        }
        s_pos[ow] = s.pos;
    }
    bool ok = true;
    if (issuer) ok = tc::mbar_wait(wbar, 0);  // the issuer's thread vouches for the weights of its CTA
    __syncthreads();
    tc::cluster_sync_all();  // both CTAs' barriers, tensor memory and weights exist before the first MMA

    __nv_bfloat16* g_h1hi = reinterpret_cast<__nv_bfloat16*>(b.h1);
    __nv_bfloat16* g_h1lo = g_h1hi + (size_t)B * d.Tmax * H;
    const int t_end = a.replay == 1 ? a.T - 1 : a.T;  // replay recomputes the T recorded rows (mode 2: and the current state)

    if (wid == iwarp) {
        // ---- layer 2: one thread of the leader CTA drives both tensor cores for both groups, k block by k block, in the
        // order the groups' operand blocks are written.  A block's sixteen arrivals also say that those warps have read
        // the group's accumulators of the step before.
        if (issuer && rank == 0) {
            const uint32_t idesc_w = tc::umma_idesc<0>(256, 128, true, false), idesc_n = tc::umma_idesc<0>(256, 64, true, false);
            for (int t = 0; t <= t_end; ++t) {
                for (int g = 0; g < NG; ++g) {
                    const uint32_t acc = tmem + (uint32_t)(g * Cfg::ACC);
                    unsigned char* bop = s_bop + g * Cfg::B_BYTES;
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb) {
                        if (ok) ok = tc::mbar_wait_cluster(&ready[4 * g + kb], (uint32_t)t & 1u);
                        tc::tc_fence_after();
#pragma unroll
                        for (int k16 = 0; k16 < 4; ++k16) {
                            // A (MN-major): 16 k rows = 2048 bytes into each box, 8192 bytes between the two 64-column boxes
                            const uint64_t ahi = tc::umma_desc(s_ahi + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                            const uint64_t alo = tc::umma_desc(s_alo + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                            // B (K-major): 16 k = 32 bytes along the swizzled rows, 1024 bytes between 8-row groups
                            const uint64_t bd = tc::umma_desc(bop + kb * Cfg::B_CHUNK + k16 * 32, 16, 1024);
                            tc::umma_pair(acc, ahi, bd, idesc_w, (kb | k16) ? 1u : 0u);
                            tc::umma_pair(acc + 128u, alo, bd, idesc_n, (kb | k16) ? 1u : 0u);
                        }
                    }
                    tc::umma_commit_pair(&tfull[g], 3);
                }
            }
        }
    } else if (worker) {
        // ---- layer 1 of group g for step t: 16-byte chunks of eight hidden units; all gathers are in flight before any is
        // used.  Thread (e, c8) covers chunk c8 of the four k blocks of env e: the chunk goes to operand row e (hi) and
        // 32 + e (lo) of its block, at the 16-byte position c8 ^ (e % 8) of the 128-byte row (the 128-byte swizzle of a
        // K-major operand).  Each finished block is announced to the leader's issuer at once.
        auto gather = [&](int g, int t) {
            const int e = tidg >> 3, c8 = tidg & 7;
            const int env = pair * (2 * NG * ME) + g * (2 * ME) + (int)rank * ME + e;
            unsigned char* bop = s_bop + g * Cfg::B_BYTES;
            const float* wrow = W1 + (size_t)(C + s_pos[g * ME + e]) * H + 8 * c8;
            const float* brow = b.base + (size_t)(env < B ? env : 0) * H + 8 * c8;
            uint4 hi[4], lo[4];
#pragma unroll
            for (int half = 0; half < 2; ++half) {  // two k blocks at a time (registers)
                float4 w[2][2], bs[2][2];
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int kb = 2 * half + kk;
                    const float4* wp = reinterpret_cast<const float4*>(wrow + 64 * kb);
                    const float4* bp = reinterpret_cast<const float4*>(brow + 64 * kb);
                    w[kk][0] = __ldg(wp);
                    w[kk][1] = __ldg(wp + 1);
                    bs[kk][0] = __ldg(bp);
                    bs[kk][1] = __ldg(bp + 1);
                }
                if (half == 0) tc::tc_fence_before();  // this thread's reads of the group's accumulators precede the arrivals below
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int kb = 2 * half + kk;
                    const float4 b0 = bs[kk][0], b1 = bs[kk][1], w0 = w[kk][0], w1 = w[kk][1];
                    split2<0>(fmaxf(b0.x + w0.x, 0.f), fmaxf(b0.y + w0.y, 0.f), hi[kb].x, lo[kb].x);
                    split2<0>(fmaxf(b0.z + w0.z, 0.f), fmaxf(b0.w + w0.w, 0.f), hi[kb].y, lo[kb].y);
                    split2<0>(fmaxf(b1.x + w1.x, 0.f), fmaxf(b1.y + w1.y, 0.f), hi[kb].z, lo[kb].z);
                    split2<0>(fmaxf(b1.z + w1.z, 0.f), fmaxf(b1.w + w1.w, 0.f), hi[kb].w, lo[kb].w);
                    unsigned char* row = bop + kb * Cfg::B_CHUNK + e * 128 + ((c8 ^ (e & 7)) << 4);
                    *reinterpret_cast<uint4*>(row) = hi[kb];
                    *reinterpret_cast<uint4*>(row + ME * 128) = lo[kb];
                    tc::fence_proxy_async();  // ordinary stores -> visible to the tensor cores
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive_remote_cta_release(tc::mapa(tc::smem_u32(&ready[4 * g + kb]), 0));
                }
            }
            // the copies for the update leave after the arrivals (their CTA-scope release does not wait for global stores)
            if (b.h1 != nullptr && t < a.T && env < B) {
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    const size_t gi = ((size_t)t * B + env) * H + 64 * kb + 8 * c8;
                    *reinterpret_cast<uint4*>(g_h1hi + gi) = hi[kb];
                    *reinterpret_cast<uint4*>(g_h1lo + gi) = lo[kb];
                    if (b.gate1) b.gate1[gi >> 3] = (uint8_t)nonzero_bits16(hi[kb]);  // the gates of these eight units
                }
            }
        };
        // ---- heads of group g for step t: thread = hidden unit j, the group's 32 envs of CTA rE
        auto heads = [&](int g, int t) {
            if (ok) ok = tc::mbar_wait(&tfull[g], (uint32_t)t & 1u);
            tc::tc_fence_after();
            // sixteen envs at a time (registers): accumulator columns -> bias, ReLU -> the h2 rows for the update -> the
            // fp16 (hi, lo) terms for the head products.  The group's operand tile is free once the step's MMAs have
            // finished: warp w keeps [32 units][32 envs] fp16 hi and lo planes in its 4 KB of it, rows of 64 bytes whose
            // 16-byte chunks are XOR-swizzled by (row / 2) % 4 (conflict-free both ways).
            unsigned char* wsm = s_bop + g * Cfg::B_BYTES + wl * 4096;
            const int env0 = pair * (2 * NG * ME) + g * (2 * ME) + rE * ME;  // first env of the block this warp holds
            const bool save_h2 = b.h2 != nullptr && t < a.T;
            const uint32_t lanes = tmem + (uint32_t)(g * Cfg::ACC) + ((uint32_t)(32 * q) << 16);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float v[16];
                {
                    uint32_t r0[16], r1[16], r2[16];
                    tc::tmem_ld16_nowait(lanes + (uint32_t)(64 * rE + 16 * hf), r0);         // W2hi x h1hi
                    tc::tmem_ld16_nowait(lanes + (uint32_t)(64 * rE + 32 + 16 * hf), r1);    // W2hi x h1lo
                    tc::tmem_ld16_nowait(lanes + 128u + (uint32_t)(32 * rE + 16 * hf), r2);  // W2lo x h1hi
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = fmaxf(((__uint_as_float(r0[e]) + __uint_as_float(r1[e])) + __uint_as_float(r2[e])) + b2j, 0.f);
                }
                if (save_h2) {  // one 128-byte line per env and warp
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        if (env0 + 16 * hf + e < B) b.h2[((size_t)t * B + env0 + 16 * hf + e) * H + j] = v[e];
                }
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    const int c4 = 2 * hf + c2;
                    uint4 hi, lo;
                    split2<0>(v[8 * c2 + 0], v[8 * c2 + 1], hi.x, lo.x);
                    split2<0>(v[8 * c2 + 2], v[8 * c2 + 3], hi.y, lo.y);
                    split2<0>(v[8 * c2 + 4], v[8 * c2 + 5], hi.z, lo.z);
                    split2<0>(v[8 * c2 + 6], v[8 * c2 + 7], hi.w, lo.w);
                    const int off = lane * 64 + ((c4 ^ ((lane >> 1) & 3)) << 4);
                    *reinterpret_cast<uint4*>(wsm + off) = hi;
                    *reinterpret_cast<uint4*>(wsm + 2048 + off) = lo;
                }
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
                        mma_f16(acc[mt], alo, whf_hi[ks][0], whf_hi[ks][1]);
                        mma_f16(acc[mt], ahi, whf_lo[ks][0], whf_lo[ks][1]);
                        mma_f16(acc[mt], ahi, whf_hi[ks][0], whf_hi[ks][1]);
                    }
                }
            }
            // every warp of the group is done with its staging area before any of them writes the operand tile again (the
            // partials below only tell an owner about the four warps of each CTA that hold ITS envs); named barrier 1 + g
            asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "n"(Cfg::NWORK * 32) : "memory");
            // accumulator element (row g8 + 8hh of tile mt, column 2 t4 + cc) = (env 16mt + 8hh + g8 of CTA rE's block, head 2 t4 + cc)
            {
                const int g8 = lane >> 2, t4 = lane & 3;
                const uint32_t pbar = tc::mapa(tc::smem_u32(&pfull[g]), (uint32_t)rE);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int e = 16 * mt + 8 * hh + g8;
                        const uint32_t dst = tc::mapa(tc::smem_u32(s_red + (((g * 8) + 4 * (int)rank + q) * ME + e) * 5 + 2 * t4), (uint32_t)rE);
                        if (t4 < 3) st_async_f32_2(dst, acc[mt][2 * hh], pbar);
                        if (t4 < 2) st_async_f32_2(dst + 4u, acc[mt][2 * hh + 1], pbar);
                    }
            }
        };
        // a group's eight warps walk its steps on their own
        gather(wg, 0);
        for (int t = 0; t <= t_end; ++t) {
            heads(wg, t);
            if (t < t_end) {
                if (ok) ok = tc::mbar_wait(&posrdy[wg], (uint32_t)t & 1u);  // the owners have published the positions after step t
                gather(wg, t + 1);
            }
        }
    } else if (ownerw) {
        // ---- one thread per env of this CTA (owner warp og serves group og)
        for (int t = 0; t <= t_end; ++t) {
            if (lane == 0) tc::mbar_expect_tx(&pfull[og], 8 * ME * 5 * 4);  // this step's head partials, counted as they land
            const bool acting = owner && !a.replay && t < a.T;
            StepPre pre;
            if (acting) pre = step_prepare(s, a, oenv, t, s_walls + ow * 8);
            if (ok) ok = tc::mbar_wait_cluster(&pfull[og], (uint32_t)t & 1u);
            float o[5];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] = 0.f;
            ActOut ao;
            ao.la_mx = ao.Z = ao.rew = 0.f;
            ao.act = ao.done = ao.pos0 = 0;
            if (owner) {
#pragma unroll
                for (int blk = 0; blk < 8; ++blk)
#pragma unroll
                    for (int c = 0; c < 5; ++c) o[c] += s_red[((og * 8 + blk) * ME + oe) * 5 + c];
#pragma unroll
                for (int c = 0; c < 5; ++c) o[c] += s_bh[c];
                if (acting) {
                    ao = act_decide(s, a, oenv, t, o[0], o[1], o[2], o[3], pre);
                    s_pos[ow] = s.pos;
                } else if (a.replay && t < t_end) {  // positions come from the recorded trajectory (row T: the env state as it stands)
                    s_pos[ow] = min((int)(t + 1 < a.T ? b.tpos[(size_t)(t + 1) * B + oenv] : b.pos[oenv]), C - 1);
                }
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&posrdy[og]);  // the group's workers of this CTA may gather the next step
            if (owner) {
                if (b.out5 && t < a.T) {  // the update reuses the head outputs of every recorded row
                    float4* o5 = reinterpret_cast<float4*>(b.out5 + ((size_t)t * B + oenv) * 8);
                    o5[0] = make_float4(o[0], o[1], o[2], o[3]);
                    o5[1] = make_float4(o[4], 0.f, 0.f, 0.f);
                }
                if (a.replay == 2 && t == a.T) b.vboot[oenv] = o[4];
                if (!a.replay) {
                    b.tval[(size_t)t * B + oenv] = o[4];
                    if (a.gae_smem) s_gv[t * NOWN + ow] = o[4];
                }
                if (acting) {
                    act_record(a, oenv, t, o[0], o[1], o[2], o[3], ao);
                    if (a.gae_smem) s_gc[t * NOWN + ow] = (uint8_t)(ao.done | (ao.rew != 0.f ? 2 : 0));
                }
            }
        }
        if (owner && !a.replay) {
            b.pos[oenv] = (uint8_t)s.pos;
            b.tep[oenv] = (uint8_t)s.tep;
            if (a.gae_smem) gae_scan_env_smem(b, B, a.T, oenv, a.gamma, a.lambda, s_gv, s_gc, NOWN, ow);
            else if (a.fuse_gae) gae_scan_env(b, B, a.T, oenv, a.gamma, a.lambda);
        }
        if (!a.replay) flush_env_stats(s, a, wid == NWT / 32);
    }
    if (!ok && lane == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
    // neither CTA frees tensor memory or leaves while the other may still signal it
    tc::tc_fence_before();
    __syncthreads();
    tc::cluster_sync_all();
    if (wid == iwarp) tc::tmem_dealloc_pair(tmem, Cfg::TMEM_COLS);
}

}  // namespace

// Covers hidden width 256 with fp32 parameters on batches large enough to give every SM pair a cluster of 128 envs;
// anything else returns cudaErrorNotSupported and the caller takes the one-group CTA-pair kernel.
cudaError_t launch_rollout_pair2(const RolloutArgs& a0, cudaStream_t s) {
    using Cfg = Pair2Cfg;
    constexpr int PER_PAIR = 2 * Cfg::NG * Cfg::ME;
    if (a0.d.H != Cfg::H || !a0.b.w2p_hi || !a0.b.w2p_lo || !a0.b.base || a0.d.npol > 1) return cudaErrorNotSupported;
    if (a0.d.B < 74 * PER_PAIR) return cudaErrorNotSupported;
    RolloutArgs a = a0;
    size_t smem = Cfg::fixed_bytes + 1024;  // alignment slack
    a.gae_smem = 0;
    if (a.fuse_gae && !a.replay && smem + Cfg::gae_bytes(a.T) <= 232448) {
        a.gae_smem = 1;
        smem += Cfg::gae_bytes(a.T);
    }
    Pair2Maps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.w_hi, a.b.w2p_hi, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_lo, a.b.w2p_lo, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    const cudaError_t e = cudaFuncSetAttribute(k_rollout_pair2, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    const int pairs = (a.d.B + PER_PAIR - 1) / PER_PAIR;
    k_rollout_pair2<<<2 * pairs, Cfg::THREADS, smem, s>>>(maps, a);
    return cudaGetLastError();
}

}  // namespace anakin
