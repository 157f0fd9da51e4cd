// Persistent rollout on the 5th-generation tensor cores for hidden width 128 and large batches: one CTA owns 128 envs
// for all T+1 forward passes of a rollout and keeps the whole second layer on chip.
//
// Acting half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top), fp32 workloads.  With many envs per
// SM the rollout is a throughput problem, but a single env group still walks a strictly serial chain per step (gather the
// agent's first-layer row -> tensor cores -> heads -> sample -> next gather).  The CTA therefore holds TWO independent
// groups of 64 envs, each with eight worker warps of its own, so that one group's tensor-core phase and sampling phase
// fall into the other group's gather and heads phases.  Per group and step:
//   layer 1   h1 = relu(base + W1[agent row])       gather-add; the fp16 (hi, lo) terms go straight into the swizzled
//                                                   K-major operand tile [64 hi rows | 64 lo rows] x 128 k
//   layer 2   transposed, D[j][env] = sum_k W2[k][j] h1[env][k], M = 128 hidden units: two tcgen05 MMAs per k16,
//             W2hi x [h1hi | h1lo] (N = 128) and W2lo x h1hi (N = 64), fp32 accumulators in tensor memory; both fp16
//             planes of W2 (64 KB) are loaded once by TMA; one thread of a dedicated warp issues the MMAs of both groups
//   heads     a worker thread = one hidden unit j (its accumulator lane): bias, ReLU, h2 stores (one 128-byte line per
//             env and warp); the warp's 32 units x 32 envs go to shared memory as fp16 (hi, lo) terms and come back
//             transposed (ldmatrix.trans) as A fragments of warp-level MMAs against Wh; the four 32-unit partials of an
//             env are summed by its owner thread in a fixed order
//   env       (owner warps) one thread per env: softmax, Philox inverse-CDF sample, gridworld step, time-major records;
//             the new position is published before the records are written
// The phases meet through mbarriers only (operand blocks written -> issuer; MMAs finished -> workers; partials stored ->
// owners; positions published -> workers).  Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the threads
// keep walking through the barriers to the exit, where tensor memory is freed.
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

struct Tc128Cfg {
    static constexpr int H = 128, NE = 64, NG = 2, NWORK = 8;   // NWORK worker warps per group
    static constexpr int NWT = NG * NWORK * 32;                 // worker threads
    static constexpr int NOWN = NG * NE;                        // owner threads: one per env
    static constexpr int THREADS = NWT + NOWN + 32;             // + the issuer warp
    static constexpr int BOX = 64 * 64 * 2;                     // one 64 x 64 box of 16-bit elements
    static constexpr int A_PLANE = (H / 64) * (H / 64) * BOX;   // all of W2 as one fp16 plane: 32 KB
    static constexpr int B_CHUNK = 2 * NE * 128;                // 128 operand rows (64 hi + 64 lo) x 64 k: 16 KB
    static constexpr int B_BYTES = (H / 64) * B_CHUNK;          // a group's operand tile: 32 KB
    static constexpr int ACC = 192;                             // TMEM columns of a group: [0,128) W2hi x [hi|lo], [128,192) W2lo x hi
    static constexpr int TMEM_COLS = 512;
    static constexpr size_t fixed_bytes =
        2 * (size_t)A_PLANE + (size_t)NG * B_BYTES + (size_t)NG * NE * H * 4  // W2 planes, operand tiles, base
        + 256                                                                 // barriers, tensor-memory slot
        + (size_t)NG * 4 * NE * 5 * 4                                         // head partials: 4 blocks of 32 hidden units
        + 8 * 4 + (size_t)NOWN * 8 * 4 + NOWN * 4;                            // bh, walls, pos
    static constexpr size_t gae_bytes(int T) { return (size_t)(T + 1) * NOWN * 4 + (size_t)T * NOWN; }
};

struct Tc128Maps {
    CUtensorMap w_hi, w_lo;  // W2 row-major [k][j] as fp16 planes, boxes of 64 j x 64 k
};

__global__ void __launch_bounds__(Tc128Cfg::THREADS, 1) k_rollout_tc128(const __grid_constant__ Tc128Maps maps, RolloutArgs a) {
    using Cfg = Tc128Cfg;
    constexpr int H = Cfg::H, NE = Cfg::NE, NG = Cfg::NG, NWT = Cfg::NWT, NOWN = Cfg::NOWN;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // the swizzle needs 1024-byte alignment
    unsigned char* s_ahi = sm;
    unsigned char* s_alo = s_ahi + Cfg::A_PLANE;
    unsigned char* s_bop = s_alo + Cfg::A_PLANE;                                     // [NG] operand tiles
    float* s_base = reinterpret_cast<float*>(s_bop + NG * Cfg::B_BYTES);             // [NG][NE][H]
    uint64_t* wbar = reinterpret_cast<uint64_t*>(s_base + NG * NE * H);              // weights landed
    uint64_t* tfull = wbar + 1;     // [NG] this step's MMAs of the group finished
    uint64_t* ready = tfull + NG;   // [NG][2] k block of the group's operand rows written (8 worker warps arrive)
    uint64_t* pdone = ready + NG * 2;  // [NG] the four head partials of every env of the group are stored (8 warps arrive)
    uint64_t* posrdy = pdone + NG;     // [NG] the group's positions for the next step are published (2 owner warps arrive)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(posrdy + NG);
    float* s_red = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(wbar) + 256);  // [NG][4][NE][5]
    float* s_bh = s_red + NG * 4 * NE * 5;                                           // [8]
    uint32_t* s_walls = reinterpret_cast<uint32_t*>(s_bh + 8);                       // [NOWN][8]
    int* s_pos = reinterpret_cast<int*>(s_walls + NOWN * 8);                         // [NOWN]
    float* s_gv = reinterpret_cast<float*>(s_pos + NOWN);                            // [T+1][NOWN] (a.gae_smem only)
    uint8_t* s_gc = reinterpret_cast<uint8_t*>(s_gv + (a.T + 1) * NOWN);             // [T][NOWN]

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int e0 = blockIdx.x * NOWN;  // this CTA's first env; group g owns envs e0 + g*NE ..
    const int B = d.B, C = d.C;
    const float* W1 = b.theta_c + d.oW1;
    const bool worker = tid < NWT;
    const bool ownerw = tid >= NWT && tid < NWT + NOWN;  // a thread of the owner warps
    const bool issuer = tid == NWT + NOWN;               // lane 0 of the last warp

    // ---- prologue
    if (tid == 0) {
        tc::mbar_init(wbar, 1);
        for (int g = 0; g < NG; ++g) {
            tc::mbar_init(&tfull[g], 1);
            tc::mbar_init(&ready[2 * g], Cfg::NWORK);
            tc::mbar_init(&ready[2 * g + 1], Cfg::NWORK);
            tc::mbar_init(&pdone[g], Cfg::NWORK);
            tc::mbar_init(&posrdy[g], NE / 32);
        }
        tc::mbar_fence_init();
    }
    if (wid == (NWT + NOWN) / 32) tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (issuer) {  // all of W2: box (kb, bx) = k rows 64kb.., columns 64bx..
        tc::mbar_expect_tx(wbar, 2 * Cfg::A_PLANE);
#pragma unroll
        for (int kb = 0; kb < H / 64; ++kb)
#pragma unroll
            for (int bx = 0; bx < H / 64; ++bx) {
                tc::tma_load_2d(s_ahi + (kb * (H / 64) + bx) * Cfg::BOX, &maps.w_hi, wbar, 64 * bx, 64 * kb);
                tc::tma_load_2d(s_alo + (kb * (H / 64) + bx) * Cfg::BOX, &maps.w_lo, wbar, 64 * bx, 64 * kb);
            }
    }
    // worker constants: hidden unit of this thread in the heads phase (its accumulator lane) and the env half it reads
    const int wg = worker ? wid / Cfg::NWORK : 0;   // the worker's group
    const int wl = wid % Cfg::NWORK;                // its warp within the group
    const int tidg = tid % (Cfg::NWORK * 32);       // its thread index within the group
    const int q = wl & 3, half = (wl >> 2) & 1;
    const int j = 32 * q + lane;
    float b2j = 0.f;
    uint32_t whf_hi[2][2], whf_lo[2][2];  // Wh rows of this warp's 32 hidden units as mma B fragments (k16 x n8), two k steps
    EnvLane s;
    s.pos = s.tep = s.start = s.goal = 0;
    s.n_episodes = s.n_goals = s.n_epsteps = 0;
    s.bad = 0;
    const int ow = tid - NWT;              // owner threads: env e0 + ow, group ow / NE
    const int og = ownerw ? ow / NE : 0;   // the owner's group
    const bool owner = ownerw && e0 + ow < B;
    if (worker) {
        for (int i = tid; i < NG * NE * H / 4; i += NWT) {
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
                    const int jj = 32 * q + 16 * ks + 8 * hh + 2 * t4;
                    const float w0 = n < 5 ? b.theta_c[d.oWh + (size_t)jj * 5 + n] : 0.f;
                    const float w1 = n < 5 ? b.theta_c[d.oWh + (size_t)(jj + 1) * 5 + n] : 0.f;
                    split2<0>(w0, w1, whf_hi[ks][hh], whf_lo[ks][hh]);
                }
        }
        if (tid < 5) s_bh[tid] = b.theta_c[d.obh + tid];
        cp_async_wait<0>();
    } else if (ownerw) {
        for (int wi = 0; wi < 8; ++wi) s_walls[ow * 8 + wi] = (owner && wi < d.W) ? b.walls[(size_t)(e0 + ow) * d.W + wi] : 0u;
        if (owner) {
            s.pos = b.pos[e0 + ow];
            s.tep = b.tep[e0 + ow];
            s.start = b.start[e0 + ow];
            s.goal = b.goal[e0 + ow];
            check_env_state(s, C, s_walls + ow * 8);
            if (a.replay) s.pos = min((int)(a.T > 0 ? b.tpos[e0 + ow] : b.pos[e0 + ow]), C - 1);  // row 0 of the recorded positions
        }
        s_pos[ow] = s.pos;
    }
    bool ok = true;
    if (issuer) ok = tc::mbar_wait(wbar, 0);
    __syncthreads();

    __nv_bfloat16* g_h1hi = reinterpret_cast<__nv_bfloat16*>(b.h1);
    __nv_bfloat16* g_h1lo = g_h1hi + (size_t)B * d.Tmax * H;
    const int t_end = a.replay == 1 ? a.T - 1 : a.T;  // replay recomputes the T recorded rows (mode 2: and the current state)

    if (issuer) {
        // ---- layer 2: one thread drives the tensor core for both groups, k block by k block, in the order the groups'
        // operand blocks are written (group 0, then group 1, every step).  A block's eight arrivals also say that those
        // warps have read the group's accumulators of the step before.
        const uint32_t idesc_w = tc::umma_idesc<0>(128, 128, true, false), idesc_n = tc::umma_idesc<0>(128, 64, true, false);
        for (int t = 0; t <= t_end; ++t) {
            for (int g = 0; g < NG; ++g) {
                const uint32_t acc = tmem + (uint32_t)(g * Cfg::ACC);
                unsigned char* bop = s_bop + g * Cfg::B_BYTES;
#pragma unroll
                for (int kb = 0; kb < 2; ++kb) {
                    if (ok) ok = tc::mbar_wait(&ready[2 * g + kb], (uint32_t)t & 1u);
                    tc::tc_fence_after();
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        // A (MN-major): 16 k rows = 2048 bytes into each box, one box further per 64 columns
                        const uint64_t ahi = tc::umma_desc(s_ahi + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                        const uint64_t alo = tc::umma_desc(s_alo + kb * 2 * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                        // B (K-major): 16 k = 32 bytes along the swizzled rows, 1024 bytes between 8-row groups
                        const uint64_t bd = tc::umma_desc(bop + kb * Cfg::B_CHUNK + k16 * 32, 16, 1024);
                        tc::umma(acc, ahi, bd, idesc_w, (kb | k16) ? 1u : 0u);
                        tc::umma(acc + 128u, alo, bd, idesc_n, (kb | k16) ? 1u : 0u);
                    }
                }
                tc::umma_commit(&tfull[g]);
            }
        }
    } else if (worker) {
        // ---- layer 1 of group g for step t: 16-byte chunks of eight hidden units; all gathers of the agents' W1 rows are
        // in flight before any is used.  Thread (e, c8) covers chunk c8 of both k blocks of envs e and e + 32 (eight lanes
        // read 256 contiguous bytes of one row): chunk c8 goes to operand row (hi) and 64 + row (lo) of its block, at the
        // 16-byte position c8 ^ (row % 8) of the 128-byte row (the 128-byte swizzle of a K-major operand).  Each finished
        // block is announced to the issuer at once.
        auto gather = [&](int g, int t) {
            const int e = tidg >> 3, c8 = tidg & 7;
            unsigned char* bop = s_bop + g * Cfg::B_BYTES;
            float4 w[2][2][2];
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const float* wrow = W1 + (size_t)(C + s_pos[g * NE + e + 32 * p]) * H + 8 * c8;
#pragma unroll
                for (int kb = 0; kb < 2; ++kb) {
                    const float4* wp = reinterpret_cast<const float4*>(wrow + 64 * kb);
                    w[kb][p][0] = __ldg(wp);
                    w[kb][p][1] = __ldg(wp + 1);
                }
            }
            tc::tc_fence_before();  // this thread's reads of the group's accumulators precede the arrivals below
            uint4 hi[2][2], lo[2][2];
#pragma unroll
            for (int kb = 0; kb < 2; ++kb) {
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    const int er = e + 32 * p, k = 64 * kb + 8 * c8;  // row within the group
                    const float* bp = s_base + (g * NE + er) * H + k;
                    const float4 b0 = *reinterpret_cast<const float4*>(bp);
                    const float4 b1 = *reinterpret_cast<const float4*>(bp + 4);
                    const float4 w0 = w[kb][p][0], w1 = w[kb][p][1];
                    split2<0>(fmaxf(b0.x + w0.x, 0.f), fmaxf(b0.y + w0.y, 0.f), hi[kb][p].x, lo[kb][p].x);
                    split2<0>(fmaxf(b0.z + w0.z, 0.f), fmaxf(b0.w + w0.w, 0.f), hi[kb][p].y, lo[kb][p].y);
                    split2<0>(fmaxf(b1.x + w1.x, 0.f), fmaxf(b1.y + w1.y, 0.f), hi[kb][p].z, lo[kb][p].z);
                    split2<0>(fmaxf(b1.z + w1.z, 0.f), fmaxf(b1.w + w1.w, 0.f), hi[kb][p].w, lo[kb][p].w);
                    unsigned char* row = bop + kb * Cfg::B_CHUNK + er * 128 + ((c8 ^ (er & 7)) << 4);
                    *reinterpret_cast<uint4*>(row) = hi[kb][p];
                    *reinterpret_cast<uint4*>(row + NE * 128) = lo[kb][p];
                }
                tc::fence_proxy_async();  // ordinary stores -> visible to the tensor core
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&ready[2 * g + kb]);
            }
            // the copies for the update leave after the arrivals
            if (b.h1 != nullptr && t < a.T) {
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    const int env = e0 + g * NE + e + 32 * p;
                    if (env < B) {
#pragma unroll
                        for (int kb = 0; kb < 2; ++kb) {
                            const size_t gi = ((size_t)t * B + env) * H + 64 * kb + 8 * c8;
                            *reinterpret_cast<uint4*>(g_h1hi + gi) = hi[kb][p];
                            *reinterpret_cast<uint4*>(g_h1lo + gi) = lo[kb][p];
                            if (b.gate1) b.gate1[gi >> 3] = (uint8_t)nonzero_bits16(hi[kb][p]);  // the gates of these eight units
                        }
                    }
                }
            }
        };
        // ---- heads of group g for step t: thread = hidden unit j, the 32 envs of its half of the group
        auto heads = [&](int g, int t) {
            if (ok) ok = tc::mbar_wait(&tfull[g], (uint32_t)t & 1u);
            tc::tc_fence_after();
            // sixteen envs at a time (registers): accumulator columns -> bias, ReLU -> the h2 rows for the update -> the
            // fp16 (hi, lo) terms for the head products.  The group's operand tile is free once the step's MMAs have
            // finished: warp w keeps [32 units][32 envs] fp16 hi and lo planes in its 4 KB of it, rows of 64 bytes whose
            // 16-byte chunks are XOR-swizzled by (row / 2) % 4 (conflict-free both ways).
            unsigned char* wsm = s_bop + g * Cfg::B_BYTES + wl * 4096;
            const int env0 = e0 + g * NE + 32 * half;  // first env of the block this warp holds
            const bool save_h2 = b.h2 != nullptr && t < a.T;
            const uint32_t lanes = tmem + (uint32_t)(g * Cfg::ACC) + ((uint32_t)(32 * q) << 16);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float v[16];
                {
                    uint32_t r0[16], r1[16], r2[16];
                    tc::tmem_ld16_nowait(lanes + (uint32_t)(32 * half + 16 * hf), r0);         // W2hi x h1hi
                    tc::tmem_ld16_nowait(lanes + (uint32_t)(NE + 32 * half + 16 * hf), r1);    // W2hi x h1lo
                    tc::tmem_ld16_nowait(lanes + 128u + (uint32_t)(32 * half + 16 * hf), r2);  // W2lo x h1hi
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
            // accumulator element (row g8 + 8hh of tile mt, column 2 t4 + cc) = (env 16mt + 8hh + g8 of this half, head 2 t4 + cc)
            {
                const int g8 = lane >> 2, t4 = lane & 3;
                float* red = s_red + ((g * 4 + q) * NE + 32 * half) * 5;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int e = 16 * mt + 8 * hh + g8;
                        if (t4 < 3) red[e * 5 + 2 * t4] = acc[mt][2 * hh];
                        if (t4 < 2) red[e * 5 + 2 * t4 + 1] = acc[mt][2 * hh + 1];
                    }
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&pdone[g]);
        };
        // a group's eight warps walk its steps on their own; the two groups drift apart by themselves, so that one group's
        // tensor-core and sampling phases fall into the other's gather and heads phases
        gather(wg, 0);
        for (int t = 0; t <= t_end; ++t) {
            heads(wg, t);
            if (t < t_end) {
                if (ok) ok = tc::mbar_wait(&posrdy[wg], (uint32_t)t & 1u);  // the owners have published the positions after step t
                gather(wg, t + 1);
            }
        }
    } else if (ownerw) {
        // ---- one thread per env
        const int env = e0 + ow;
        const int oe = ow - og * NE;  // env index within the group
        for (int t = 0; t <= t_end; ++t) {
            // the logits-independent half of the interaction, while the workers gather and the tensor core runs
            const bool acting = owner && !a.replay && t < a.T;
            StepPre pre;
            if (acting) pre = step_prepare(s, a, env, t, s_walls + ow * 8);
            if (ok) ok = tc::mbar_wait(&pdone[og], (uint32_t)t & 1u);
            float o[5];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] = 0.f;
            ActOut ao;
            ao.la_mx = ao.Z = ao.rew = 0.f;
            ao.act = ao.done = ao.pos0 = 0;
            if (owner) {
#pragma unroll
                for (int blk = 0; blk < 4; ++blk)
#pragma unroll
                    for (int c = 0; c < 5; ++c) o[c] += s_red[((og * 4 + blk) * NE + oe) * 5 + c];
#pragma unroll
                for (int c = 0; c < 5; ++c) o[c] += s_bh[c];
                if (acting) {
                    ao = act_decide(s, a, env, t, o[0], o[1], o[2], o[3], pre);
                    s_pos[ow] = s.pos;
                } else if (a.replay && t < t_end) {  // positions come from the recorded trajectory (row T: the env state as it stands)
                    s_pos[ow] = min((int)(t + 1 < a.T ? b.tpos[(size_t)(t + 1) * B + env] : b.pos[env]), C - 1);
                }
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&posrdy[og]);  // the workers may gather the group's next step
            if (owner) {
                if (b.out5 && t < a.T) {  // the update reuses the head outputs of every recorded row
                    float4* o5 = reinterpret_cast<float4*>(b.out5 + ((size_t)t * B + env) * 8);
                    o5[0] = make_float4(o[0], o[1], o[2], o[3]);
                    o5[1] = make_float4(o[4], 0.f, 0.f, 0.f);
                }
                if (a.replay == 2 && t == a.T) b.vboot[env] = o[4];
                if (!a.replay) {
                    b.tval[(size_t)t * B + env] = o[4];
                    if (a.gae_smem) s_gv[t * NOWN + ow] = o[4];
                }
                if (acting) {
                    act_record(a, env, t, o[0], o[1], o[2], o[3], ao);
                    if (a.gae_smem) s_gc[t * NOWN + ow] = (uint8_t)(ao.done | (ao.rew != 0.f ? 2 : 0));
                }
            }
        }
        if (owner && !a.replay) {
            b.pos[env] = (uint8_t)s.pos;
            b.tep[env] = (uint8_t)s.tep;
            if (a.gae_smem) gae_scan_env_smem(b, B, a.T, env, a.gamma, a.lambda, s_gv, s_gc, NOWN, ow);
            else if (a.fuse_gae) gae_scan_env(b, B, a.T, env, a.gamma, a.lambda);
        }
        if (!a.replay) flush_env_stats(s, a, wid == NWT / 32);
    }
    if (!ok && lane == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
    tc::tc_fence_before();
    __syncthreads();
    if (wid == (NWT + NOWN) / 32) tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
}

}  // namespace

// Covers hidden width 128 with fp32 parameters (two-term fp16 operands) on batches large enough to give every SM a CTA
// of 128 envs; anything else returns cudaErrorNotSupported and the caller takes the warp-level kernel.
cudaError_t launch_rollout_tc128(const RolloutArgs& a0, cudaStream_t s) {
    using Cfg = Tc128Cfg;
    if (a0.d.H != Cfg::H || !a0.b.w2p_hi || !a0.b.w2p_lo || !a0.b.base || a0.d.npol > 1) return cudaErrorNotSupported;
    if (a0.d.B < 148 * Cfg::NOWN) return cudaErrorNotSupported;
    RolloutArgs a = a0;
    size_t smem = Cfg::fixed_bytes + 1024;  // alignment slack
    a.gae_smem = 0;
    if (a.fuse_gae && !a.replay && smem + Cfg::gae_bytes(a.T) <= 232448) {
        a.gae_smem = 1;
        smem += Cfg::gae_bytes(a.T);
    }
    Tc128Maps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.w_hi, a.b.w2p_hi, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_lo, a.b.w2p_lo, Cfg::H, Cfg::H, 64, false)) return cudaErrorNotSupported;
    const cudaError_t e = cudaFuncSetAttribute(k_rollout_tc128, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    k_rollout_tc128<<<(a.d.B + Cfg::NOWN - 1) / Cfg::NOWN, Cfg::THREADS, smem, s>>>(maps, a);
    return cudaGetLastError();
}

}  // namespace anakin
