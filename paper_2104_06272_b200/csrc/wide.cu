// Wide-network path (bf16 workload, hidden width 512 / 1024 / 2048): the layer-2 products of the Anakin minimal unit
// (Podracer paper, Section 3.1; Figure 2, top) as large GEMMs on the 5th-generation tensor cores.
//
// With a hidden layer this wide W2 no longer fits on chip next to a CTA's activations, so the acting half runs as three
// launches per environment step instead of one persistent kernel:
//   k_h1_wide      h1 = bf16(relu(base[env] + W1[agent row]))                  gather-add, HBM-bound
//   k_gemm_nt_tc   h2 = bf16(relu(h1 W2 + b2))                                 tcgen05, persistent, bias/ReLU epilogue
//   k_heads_wide   out = h2 Wh + bh, then softmax / Philox sample / env step   warp per env, then thread per env
// h1 and h2 of every recorded row stay in HBM as bf16 for the update, which calls k_gemm_nt_tc once more for
// dh1 = (dh2 W2^T) gated by h1 > 0 over all B*T rows, and k_sum_t_wide for S = sum over t of dh1.
//
// k_gemm_nt_tc: C[m][n] = sum_k A[m][k] Bop[k][n] with A row-major (K-major for the MMA).  One persistent CTA per SM walks
// 128 x 256 output tiles (n fastest, so that the CTAs running together share A tiles through L2):
//   warp 0 (one lane)  TMA producer: 64-wide k chunks of A (128 rows) and B (256 columns) into a 3-stage ring
//   warp 1 (one lane)  tcgen05.mma issuer, four k16 MMAs per chunk into one of two 256-column fp32 accumulators in TMEM
//   warps 2-9          epilogue of tile i while the MMAs of tile i+1 run: tcgen05.ld, bias + ReLU (or gate), bf16, store
// B is either K-major (rows = n: W2 as stored, for dh2 W2^T) or MN-major (rows = k: W2 as stored, for h1 W2).
// Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the CTA unwinds (tensor memory freed).
#include <cstring>

#include "wide_gemm.cuh"

namespace anakin {

bool wide_supported(int H, int prec) { return prec == 1 && (H == 512 || H == 1024 || H == 2048); }
bool tensor_path_supported(int H, int prec) { return rollout_mma_supported(H) || wide_supported(H, prec); }

namespace {

using namespace widegemm;

struct NtCfg {
    static constexpr int BM = 128, BN = NT_BN, KC = 64, STAGES = 3, THREADS = 320, MAXN = NT_MAXN;
    static constexpr int A_BYTES = BM * KC * 2, B_BYTES = BN * KC * 2, STAGE = A_BYTES + B_BYTES;
    static constexpr size_t smem_bytes = (size_t)STAGES * STAGE + 1024 /*alignment slack*/ + 256 /*barriers, tmem slot*/ + MAXN * 4 + NT_EPI_WARPS * NT_STAGE_BYTES;
};

template <int EPI, bool B_MN>
__global__ void __launch_bounds__(320, 1) k_gemm_nt_tc(const __grid_constant__ NtMaps maps, NtArgs g) {
    using Cfg = NtCfg;
    constexpr int BM = Cfg::BM, BN = Cfg::BN, KC = Cfg::KC, STAGES = Cfg::STAGES;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // the swizzle needs 1024-byte alignment
    uint64_t* bars = (uint64_t*)(base + STAGES * Cfg::STAGE);
    uint64_t* full = bars;                // [STAGES]
    uint64_t* empty = bars + STAGES;      // [STAGES]
    uint64_t* tfull = bars + 2 * STAGES;  // [2] accumulator written
    uint64_t* tempty = tfull + 2;         // [2] accumulator drained (4 epilogue warps arrive)
    uint32_t* tmem_slot = (uint32_t*)(tempty + 2);
    float* s_bias = (float*)(base + STAGES * Cfg::STAGE + 256);
    unsigned char* s_stage = (unsigned char*)(s_bias + NT_MAXN);  // [NT_EPI_WARPS][NT_STAGE_BYTES]
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int nt = g.N / BN, mt = (g.M + BM - 1) / BM, ntiles = mt * nt, nch = g.K / KC;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&tfull[i], 1); tc::mbar_init(&tempty[i], NT_EPI_WARPS); }
        tc::mbar_fence_init();
    }
    if (EPI != EPI_GATE)
        for (int i = tid; i < g.N; i += Cfg::THREADS) s_bias[i] = g.bias[i];
    if (wid == 2) tc::tmem_alloc(tmem_slot, 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer
            int c = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int m0 = (tile / nt) * BM, n0 = (tile % nt) * BN;
                for (int kc = 0; kc < nch; ++kc, ++c) {
                    const int s = c % STAGES;
                    if (c >= STAGES) ok = tc::mbar_wait(&empty[s], ((c / STAGES) - 1) & 1);
                    if (!ok) break;
                    unsigned char* sa = base + s * Cfg::STAGE;
                    unsigned char* sb = sa + Cfg::A_BYTES;
                    tc::mbar_expect_tx(&full[s], Cfg::STAGE);
                    // rows past M belong to later rows of the buffer or are zero-filled; the epilogue drops them
                    tc::tma_load_2d(sa, &maps.a, &full[s], kc * KC, g.row0 + m0);
                    if (B_MN) {
#pragma unroll
                        for (int bx = 0; bx < BN / 64; ++bx) tc::tma_load_2d(sb + bx * 8192, &maps.b, &full[s], n0 + 64 * bx, kc * KC);
                    } else {
                        tc::tma_load_2d(sb, &maps.b, &full[s], kc * KC, n0);  // two boxes of 128 rows (n)
                        tc::tma_load_2d(sb + Cfg::B_BYTES / 2, &maps.b, &full[s], kc * KC, n0 + BN / 2);
                    }
                }
            }
            if (!ok) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0) {  // ---- MMA issuer
            const uint32_t idesc = tc::umma_idesc<1>(BM, BN, false, B_MN);
            int c = 0, u = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++u) {
                const int buf = u & 1;
                if (u >= 2) ok = tc::mbar_wait(&tempty[buf], ((u >> 1) - 1) & 1);  // the epilogue of tile u-2 has drained it
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + (uint32_t)(buf * BN);
                for (int kc = 0; kc < nch; ++kc, ++c) {
                    const int s = c % STAGES;
                    ok = tc::mbar_wait(&full[s], (c / STAGES) & 1);
                    if (!ok) break;
                    tc::tc_fence_after();
                    unsigned char* sa = base + s * Cfg::STAGE;
                    unsigned char* sb = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < KC / 16; ++k16) {
                        // K-major: 16 k = 32 bytes along the swizzled 128-byte rows; MN-major: 16 k rows = 2048 bytes
                        const uint64_t ad = tc::umma_desc(sa + k16 * 32, 16, 1024);
                        const uint64_t bd = B_MN ? tc::umma_desc(sb + k16 * 2048, 8192, 1024) : tc::umma_desc(sb + k16 * 32, 16, 1024);
                        tc::umma(acc, ad, bd, idesc, (kc > 0 || k16 > 0) ? 1u : 0u);
                    }
                    tc::umma_commit(&empty[s]);
                }
                if (ok) tc::umma_commit(&tfull[buf]);
            }
            if (!ok) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- epilogue warps: accumulator lanes 32*(wid%4)..+31 = output rows
        const int q = wid & 3, half = (wid - 2) >> 2;
        int u = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++u) {
            const int buf = u & 1;
            const int m0 = (tile / nt) * BM, n0 = (tile % nt) * BN;
            const int m = m0 + 32 * q + lane;
            const bool valid = m < g.M;
            const size_t gi = ((size_t)g.row0 + (valid ? m : 0)) * g.N + n0;
            if (EPI == EPI_GATE && valid) nt_prefetch_gate(g, gi);  // towards L2 while the MMAs run
            ok = tc::mbar_wait(&tfull[buf], (u >> 1) & 1);
            if (!ok) break;
            tc::tc_fence_after();
            nt_epilogue_warp<EPI>(g, s_bias, s_stage + (wid - 2) * NT_STAGE_BYTES, tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * BN), m - lane, n0, lane,
                                  half * (BN / 2), (half + 1) * (BN / 2));
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&tempty[buf]);  // the issuer may overwrite this accumulator now
        }
        if (!ok && lane == 0) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (wid == 2) tc::tmem_dealloc(tmem, 512);
}

template <int EPI, bool B_MN>
cudaError_t launch_nt(const NtMaps& maps, const NtArgs& g, cudaStream_t s) {
    if (g.N % NtCfg::BN != 0 || g.K % NtCfg::KC != 0 || g.N > NtCfg::MAXN || g.M < 1) return cudaErrorNotSupported;
    if (g.M >= 2 * NtCfg::BM) {  // the CTA-pair kernel (256 x 256 tiles) where there are rows for it
        const cudaError_t ep = launch_nt_pair(EPI, B_MN, maps, g, s);
        if (ep != cudaErrorNotSupported) return ep;
    }
    const cudaError_t e = cudaFuncSetAttribute(k_gemm_nt_tc<EPI, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)NtCfg::smem_bytes);
    if (e != cudaSuccess) return e;
    const int ntiles = ((g.M + NtCfg::BM - 1) / NtCfg::BM) * (g.N / NtCfg::BN);
    const int grid = ntiles < 148 ? ntiles : 148;
    k_gemm_nt_tc<EPI, B_MN><<<grid, NtCfg::THREADS, NtCfg::smem_bytes, s>>>(maps, g);
    return cudaGetLastError();
}

// h1 rows: 8 hidden units per thread.  pos[i] is the agent cell of row i (env = i mod B).
__global__ void __launch_bounds__(256) k_h1_wide(Dims d, Buffers b, const uint8_t* pos, size_t rows, size_t row0) {
    const int H = d.H, H8 = H / 8;
    const float* W1a = b.theta_c + d.oW1 + (size_t)d.C * H;  // agent plane of W1
    uint4* out = reinterpret_cast<uint4*>(b.h1) + row0 * H8;
    const size_t total = rows * H8;
    for (size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (size_t)gridDim.x * 256) {
        const size_t i = idx / H8;
        const int j8 = (int)(idx - i * H8);
        const int env = (int)(i % d.B);
        const int p = min((int)pos[i], d.C - 1);  // a position handed in from outside stays inside the plane
        const float4* bp = reinterpret_cast<const float4*>(b.base + (size_t)env * H) + 2 * j8;
        const float4* wp = reinterpret_cast<const float4*>(W1a + (size_t)p * H) + 2 * j8;
        const float4 b0 = bp[0], b1 = bp[1], w0 = __ldg(wp), w1 = __ldg(wp + 1);
        uint4 o;
        o.x = pack_bf16(__float2bfloat16_rn(fmaxf(b0.x + w0.x, 0.f)), __float2bfloat16_rn(fmaxf(b0.y + w0.y, 0.f)));
        o.y = pack_bf16(__float2bfloat16_rn(fmaxf(b0.z + w0.z, 0.f)), __float2bfloat16_rn(fmaxf(b0.w + w0.w, 0.f)));
        o.z = pack_bf16(__float2bfloat16_rn(fmaxf(b1.x + w1.x, 0.f)), __float2bfloat16_rn(fmaxf(b1.y + w1.y, 0.f)));
        o.w = pack_bf16(__float2bfloat16_rn(fmaxf(b1.z + w1.z, 0.f)), __float2bfloat16_rn(fmaxf(b1.w + w1.w, 0.f)));
        out[idx] = o;
    }
}

// Heads, sampling and env step for 32 rows per CTA: eight warps take four rows each for the head products, then warp 0
// takes one row per lane for the per-env part (its env state and wall words were requested at kernel start).
//   mode 0: step t of the rollout (row = env): saves the head outputs and the value, samples, steps the env, records.
//   mode 1: bootstrap forward after the last step: saves the value only.
//   mode 2: replay of recorded rows (row = t*B + env): saves the head outputs only.
//   mode 3: forward of the current env state under the current parameters: saves the value to vboot.
constexpr int HW_ROWS = 32;

template <int H>
__global__ void __launch_bounds__(256) k_heads_wide(RolloutArgs a, int t, int mode, size_t rows, size_t row0) {
    constexpr int TRIPS = H / 128;   // a lane covers four consecutive hidden units per trip
    extern __shared__ __align__(16) float s_wh[];  // [H][5] as stored
    __shared__ float s_out[HW_ROWS][8];
    __shared__ uint32_t s_walls[HW_ROWS][8];
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const size_t i0 = (size_t)blockIdx.x * HW_ROWS;
    {   // Wh: straight 16-byte copies (the parameter block starts on a 16-byte boundary for these H)
        const float4* src = reinterpret_cast<const float4*>(b.theta_c + d.oWh);
        float4* dst = reinterpret_cast<float4*>(s_wh);
#pragma unroll
        for (int q = 0; q < (5 * H / 4 + 255) / 256; ++q)
            if (tid + 256 * q < 5 * H / 4) dst[tid + 256 * q] = __ldg(src + tid + 256 * q);
    }
    EnvLane es;
    es.pos = es.tep = es.start = es.goal = 0;
    if (mode == 0) {
        if (tid < HW_ROWS && i0 + tid < rows) {
            es.pos = b.pos[i0 + tid];
            es.tep = b.tep[i0 + tid];
            es.start = b.start[i0 + tid];
            es.goal = b.goal[i0 + tid];
        }
        for (int idx = tid; idx < HW_ROWS * d.W; idx += 256) {
            const int e = idx / d.W, wi = idx - e * d.W;
            if (i0 + e < rows) s_walls[e][wi] = b.walls[(i0 + e) * d.W + wi];
        }
    }
    const uint16_t* h2b = reinterpret_cast<const uint16_t*>(b.h2);
    // a warp walks rows wid, wid+8, ...; the loads of the next row are in flight while this row is reduced
    uint2 v[TRIPS], vn[TRIPS];
    auto load_row = [&](int r, uint2 (&dst)[TRIPS]) {
        const size_t i = i0 + r;
        const uint2* hp = reinterpret_cast<const uint2*>(h2b + (row0 + (i < rows ? i : 0)) * H);
#pragma unroll
        for (int q = 0; q < TRIPS; ++q) dst[q] = (r < HW_ROWS && i < rows) ? __ldg(hp + lane + 32 * q) : make_uint2(0u, 0u);
    };
    load_row(wid, v);
    __syncthreads();
#pragma unroll 1
    for (int r = wid; r < HW_ROWS; r += 8) {
        load_row(r + 8, vn);
        float acc[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < TRIPS; ++q) {
            const float x[4] = {__uint_as_float(v[q].x << 16), __uint_as_float(v[q].x & 0xFFFF0000u), __uint_as_float(v[q].y << 16),
                                __uint_as_float(v[q].y & 0xFFFF0000u)};
            // this lane's four units are 20 consecutive floats of Wh (80-byte lane stride: conflict-free 16-byte reads)
            const float4* wp = reinterpret_cast<const float4*>(s_wh + 20 * (lane + 32 * q));
            float w[20];
#pragma unroll
            for (int j = 0; j < 5; ++j) {
                const float4 f = wp[j];
                w[4 * j] = f.x; w[4 * j + 1] = f.y; w[4 * j + 2] = f.z; w[4 * j + 3] = f.w;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int c = 0; c < 5; ++c) acc[c] = fmaf(x[u], w[5 * u + c], acc[c]);
        }
#pragma unroll
        for (int c = 0; c < 5; ++c)
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[c] += __shfl_xor_sync(0xFFFFFFFFu, acc[c], off);
        if (lane == 0) {
#pragma unroll
            for (int c = 0; c < 5; ++c) s_out[r][c] = acc[c] + b.theta_c[d.obh + c];
        }
#pragma unroll
        for (int q = 0; q < TRIPS; ++q) v[q] = vn[q];
    }
    __syncthreads();
    __shared__ int s_pos[HW_ROWS];
    if (tid < HW_ROWS) {
    const size_t i = i0 + tid;
    const bool valid = i < rows;
    unsigned long long n_ep = 0, n_goal = 0, n_steps = 0;
    int bad = 0;
    if (valid) {
        const float o0 = s_out[tid][0], o1 = s_out[tid][1], o2 = s_out[tid][2], o3 = s_out[tid][3], v4 = s_out[tid][4];
        if (mode == 1) {
            b.tval[(size_t)a.T * d.B + i] = v4;
        } else if (mode == 3) {
            b.vboot[i] = v4;
        } else {
            const size_t row = mode == 0 ? (size_t)t * d.B + i : i;
            float4* o = reinterpret_cast<float4*>(b.out5 + row * 8);
            o[0] = make_float4(o0, o1, o2, o3);
            o[1] = make_float4(v4, 0.f, 0.f, 0.f);
            if (mode == 0) {
                b.tval[row] = v4;
                const int env = (int)i;
                es.n_episodes = es.n_goals = es.n_epsteps = 0;
                es.bad = 0;
                check_env_state(es, d.C, s_walls[tid]);
                act_and_step(es, a, env, t, o0, o1, o2, o3, s_walls[tid]);
                b.pos[env] = (uint8_t)es.pos;
                b.tep[env] = (uint8_t)es.tep;
                s_pos[tid] = es.pos;
                n_ep = es.n_episodes; n_goal = es.n_goals; n_steps = es.n_epsteps; bad = es.bad;
            }
        }
    }
    if (mode == 0) {
    // fold the warp's counters and add them with integer atomics (order-free totals)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        n_ep += __shfl_xor_sync(0xFFFFFFFFu, n_ep, off);
        n_goal += __shfl_xor_sync(0xFFFFFFFFu, n_goal, off);
        n_steps += __shfl_xor_sync(0xFFFFFFFFu, n_steps, off);
        bad |= __shfl_xor_sync(0xFFFFFFFFu, bad, off);
    }
    if (lane == 0) {
        if (n_ep) atomicAdd((unsigned long long*)&b.stats->episodes, n_ep);
        if (n_goal) atomicAdd((unsigned long long*)&b.stats->goals, n_goal);
        if (n_steps) atomicAdd((unsigned long long*)&b.stats->episode_steps, n_steps);
        if (blockIdx.x == 0 && tid == 0) atomicAdd((unsigned long long*)&b.stats->frames, (unsigned long long)d.B);
        if (bad) atomicOr(b.status, bad);
    }
    }
    }
    if (mode != 0) return;
    // ---- layer 1 of the NEXT step for this CTA's envs, from the positions just produced (rows (t+1)*B + env):
    // 8 threads per env, 16-byte chunks interleaved so that a row's lanes read and write contiguous memory
    __syncthreads();
    {
        const int rl = tid >> 3, q = tid & 7;
        const size_t env = i0 + rl;
        if (env < rows) {
            const float4* bp = reinterpret_cast<const float4*>(b.base + env * H);
            const float4* wp = reinterpret_cast<const float4*>(b.theta_c + d.oW1 + ((size_t)d.C + s_pos[rl]) * H);
            uint4* out = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(b.h1) + ((size_t)(t + 1) * d.B + env) * H);
#pragma unroll 4
            for (int ch = q; ch < H / 8; ch += 8) {
                const float4 b0 = bp[2 * ch], b1 = bp[2 * ch + 1], w0 = __ldg(wp + 2 * ch), w1 = __ldg(wp + 2 * ch + 1);
                uint4 o;
                o.x = pack_bf16(__float2bfloat16_rn(fmaxf(b0.x + w0.x, 0.f)), __float2bfloat16_rn(fmaxf(b0.y + w0.y, 0.f)));
                o.y = pack_bf16(__float2bfloat16_rn(fmaxf(b0.z + w0.z, 0.f)), __float2bfloat16_rn(fmaxf(b0.w + w0.w, 0.f)));
                o.z = pack_bf16(__float2bfloat16_rn(fmaxf(b1.x + w1.x, 0.f)), __float2bfloat16_rn(fmaxf(b1.y + w1.y, 0.f)));
                o.w = pack_bf16(__float2bfloat16_rn(fmaxf(b1.z + w1.z, 0.f)), __float2bfloat16_rn(fmaxf(b1.w + w1.w, 0.f)));
                out[ch] = o;
            }
        }
    }
}

// S[env][j] = sum over t of dh1[t*B + env][j], kept as two bf16 terms (hi and lo planes) for the K = B GEMMs of dW1.
__global__ void __launch_bounds__(256) k_sum_t_wide(Dims d, Buffers b, int T) {
    const int H8 = d.H / 8;
    const size_t total = (size_t)d.B * H8;
    const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= total) return;
    const uint4* src = reinterpret_cast<const uint4*>(b.dh1) + idx;
    float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int t0 = 0; t0 < T; t0 += 8) {  // eight loads in flight
        uint4 v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = t0 + q < T ? __ldg(src + (size_t)(t0 + q) * total) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                s[2 * e] += __uint_as_float(w[e] << 16);
                s[2 * e + 1] += __uint_as_float(w[e] & 0xFFFF0000u);
            }
        }
    }
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        __nv_bfloat16 h0, l0, h1, l1;
        split_bf16(s[2 * e], h0, l0);
        split_bf16(s[2 * e + 1], h1, l1);
        hi[e] = pack_bf16(h0, h1);
        lo[e] = pack_bf16(l0, l1);
    }
    uint4* S_hi = reinterpret_cast<uint4*>(b.S);
    uint4* S_lo = S_hi + total;
    S_hi[idx] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    S_lo[idx] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

// W2 as a row-major bf16 plane (the values are bf16 already in this workload).
__global__ void __launch_bounds__(256) k_pack_w2_wide(Dims d, Buffers b) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i < (size_t)d.H * d.H) b.w2p_hi[i] = __bfloat16_as_ushort(__float2bfloat16_rn(b.theta_c[d.oW2 + i]));
}

// Operands of the base GEMM: X[env][c] = 1 where cell c of the env is a wall (bf16), and the wall plane of W1 as bf16
// (exact: the weights are bf16 values in this workload).
__global__ void __launch_bounds__(256) k_expand_walls(Dims d, Buffers b, uint16_t* X, uint16_t* W1w) {
    const size_t nx = (size_t)d.B * (d.C / 8), nw = (size_t)d.C * d.H;
    for (size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x; idx < nx + nw; idx += (size_t)gridDim.x * 256) {
        if (idx < nx) {
            const size_t e = idx / (d.C / 8);
            const int c8 = (int)(idx - e * (d.C / 8));
            const uint32_t bits = (b.walls[e * d.W + (c8 >> 2)] >> ((c8 & 3) * 8)) & 0xFFu;
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) o[q] = ((bits >> (2 * q)) & 1u ? 0x3F80u : 0u) | ((bits >> (2 * q + 1)) & 1u ? 0x3F800000u : 0u);
            reinterpret_cast<uint4*>(X)[idx] = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            const size_t i = idx - nx;
            W1w[i] = __bfloat16_as_ushort(__float2bfloat16_rn(b.theta_c[d.oW1 + i]));
        }
    }
}

#define CKW(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

cudaError_t heads_wide(const RolloutArgs& a, int t, int mode, size_t rows, size_t row0, cudaStream_t s) {
    const size_t smem = (size_t)5 * a.d.H * sizeof(float);
    const unsigned grid = (unsigned)((rows + HW_ROWS - 1) / HW_ROWS);
    switch (a.d.H) {
        case 512: k_heads_wide<512><<<grid, 256, smem, s>>>(a, t, mode, rows, row0); break;
        case 1024: k_heads_wide<1024><<<grid, 256, smem, s>>>(a, t, mode, rows, row0); break;
        case 2048: k_heads_wide<2048><<<grid, 256, smem, s>>>(a, t, mode, rows, row0); break;
        default: return cudaErrorNotSupported;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pack_w2_wide(const Dims& d, const Buffers& b, const Ctx& c) {
    Scope sc(c, K_PACK_W2);
    k_pack_w2_wide<<<(unsigned)(((size_t)d.H * d.H + 255) / 256), 256, 0, c.s>>>(d, b);
    return cudaGetLastError();
}

// base = b1 + walls x W1[wall plane] + W1[goal row] as one GEMM (K = C cells).  Applies to the buffers of the wide path
// (bf16 workload: the products 1 x w are exact and the accumulation is fp32); cudaErrorNotSupported otherwise.
// Uses the dh1 buffer, which is dead outside the update, as scratch for the two bf16 operands.
cudaError_t launch_env_base_wide(const Dims& d, const Buffers& b, const Ctx& c) {
    const bool wide_buffers = b.w2p_hi && d.H >= 512;  // (narrower layers keep fp32-sized activation buffers)
    if (!wide_buffers || d.C % 64 != 0 || d.H % NtCfg::BN != 0 || d.H > NtCfg::MAXN) return cudaErrorNotSupported;
    uint16_t* X = reinterpret_cast<uint16_t*>(b.dh1);
    uint16_t* W1w = X + (size_t)d.B * d.C;
    NtMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.a, X, d.B, d.C, 128, true)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.b, W1w, d.C, d.H, 64, true)) return cudaErrorNotSupported;
    {
        Scope sc(c, K_ENV_BASE);
        k_expand_walls<<<148 * 8, 256, 0, c.s>>>(d, b, X, W1w);
        CKW(cudaGetLastError());
    }
    Scope sc(c, K_ENV_BASE);
    NtArgs g;
    memset(&g, 0, sizeof(g));
    g.M = d.B; g.N = d.H; g.K = d.C; g.row0 = 0;
    g.bias = b.theta_c + d.ob1;
    g.outf = b.base;
    g.addrows = b.theta_c + d.oW1;
    g.addidx = b.goal;
    g.addrow0 = 2 * d.C;
    g.status = b.status;
    return launch_nt<EPI_BASE, true>(maps, g, c.s);
}

// T+1 forward passes (or, in replay mode, one pass over the recorded rows).
cudaError_t launch_rollout_wide(const RolloutArgs& a, const Ctx& c) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int H = d.H, B = d.B;
    const size_t cap_rows = (size_t)2 * B * d.Tmax;  // the fp32-sized h1 / h2 buffers hold this many bf16 rows
    NtMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.a, b.h1, cap_rows, H, 128, true)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.b, b.w2p_hi, H, H, 64, true)) return cudaErrorNotSupported;
    NtArgs g;
    memset(&g, 0, sizeof(g));
    g.N = H; g.K = H;
    g.out = reinterpret_cast<uint16_t*>(b.h2);
    g.bias = b.theta_c + d.ob2;
    g.status = b.status;
    auto h1_grid = [](size_t rows, int H) { return (unsigned)((rows * (H / 8) + 255) / 256); };
    if (a.replay) {
        const size_t R = (size_t)B * a.T;
        {
            Scope sc(c, K_REPLAY);
            k_h1_wide<<<h1_grid(R, H), 256, 0, c.s>>>(d, b, b.tpos, R, 0);
            CKW(cudaGetLastError());
        }
        {
            Scope sc(c, K_REPLAY);
            g.M = (int)R; g.row0 = 0;
            CKW((launch_nt<EPI_FWD, true>(maps, g, c.s)));
        }
        {
            Scope sc(c, K_REPLAY);
            CKW(heads_wide(a, 0, 2, R, 0, c.s));
        }
        if (a.replay == 2) {  // one more forward on the env state as it stands, in the B rows after the recorded ones
            {
                Scope sc(c, K_REPLAY);
                k_h1_wide<<<h1_grid(B, H), 256, 0, c.s>>>(d, b, b.pos, B, R);
                CKW(cudaGetLastError());
            }
            {
                Scope sc(c, K_REPLAY);
                g.M = B; g.row0 = (int)R;
                CKW((launch_nt<EPI_FWD, true>(maps, g, c.s)));
            }
            Scope sc(c, K_REPLAY);
            return heads_wide(a, 0, 3, B, R, c.s);
        }
        return cudaSuccess;
    }
    for (int t = 0; t <= a.T; ++t) {
        const size_t row0 = (size_t)t * B;
        if (t == 0) {  // later steps: the heads kernel of step t-1 writes the h1 rows of step t
            Scope sc(c, K_H1);
            k_h1_wide<<<h1_grid(B, H), 256, 0, c.s>>>(d, b, b.pos, B, row0);
            CKW(cudaGetLastError());
        }
        {
            Scope sc(c, K_FWD2);
            g.M = B; g.row0 = (int)row0;
            CKW((launch_nt<EPI_FWD, true>(maps, g, c.s)));
        }
        {
            Scope sc(c, K_ROLLOUT);
            CKW(heads_wide(a, t, t == a.T ? 1 : 0, B, row0, c.s));
        }
    }
    return cudaSuccess;
}

// dh1 = (dh2 W2^T) gated by h1 > 0 over all R rows, then S = sum over t of dh1.
cudaError_t launch_dh1_wide(const LearnArgs& a, const Ctx& c) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int H = d.H;
    const size_t R = (size_t)d.B * a.T;
    NtMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_tensor_map_2d(&maps.a, b.dh2, R, H, 128, true)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.b, b.w2p_hi, H, H, 128, true)) return cudaErrorNotSupported;
    NtArgs g;
    memset(&g, 0, sizeof(g));
    g.M = (int)R; g.N = H; g.K = H; g.row0 = 0;
    g.out = reinterpret_cast<uint16_t*>(b.dh1);
    g.gate = reinterpret_cast<const uint16_t*>(b.h1);
    g.status = b.status;
    {
        Scope sc(c, K_DH1);
        CKW((launch_nt<EPI_GATE, false>(maps, g, c.s)));
    }
    {
        Scope sc(c, K_SUM_OVER_T);
        k_sum_t_wide<<<(unsigned)(((size_t)d.B * (H / 8) + 255) / 256), 256, 0, c.s>>>(d, b, a.T);
        CKW(cudaGetLastError());
    }
    return cudaSuccess;
}

}  // namespace anakin
