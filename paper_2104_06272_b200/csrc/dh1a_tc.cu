// dh1 = (dh2 W2^T) gated by h1 > 0, S = sum over t of dh1, AND the agent plane of dW1 = onehot(pos)^T dh1, in one
// tcgen05 kernel: dh1 never goes to HBM.
//
// Backward pass through the second layer of the policy/value MLP and the first-layer weight gradient of the rows the
// agent's position selects (the update half of the Anakin minimal unit, Podracer paper, Section 3.1; Figure 2, top).
// A CTA owns 64 output columns and walks tiles of 128 envs (tile index blockIdx.x, blockIdx.x + gridDim.x, ...) and, per
// tile, the steps t of its slice:
//   warp 0 (one lane)  TMA producer: W2's 64-column slice once (resident), then the dh2 planes of every step through a
//                      ring of 128 x 64 K-major boxes
//   warp 1 (one lane)  tcgen05.mma issuer.  Per step: the dh1 product (K = H, three fp16 terms per k16, one in the bf16
//                      workload) into one of two 64-column accumulators; then, for the step before, the agent-plane
//                      product  D[cell][col] += sum over the 128 envs of onehot[env][cell] * dh1[env][col]  (K = 128,
//                      both operands MN-major tiles that the epilogue warps wrote) into a third accumulator that lives
//                      for the whole kernel
//   warps 2-5          epilogue, thread = env: tcgen05.ld, gate, S +=, 16-bit split; writes its dh1 row (hi and lo
//                      planes) and its one-hot element into the two operand tiles in the 128-byte-swizzled layout
// At the end the epilogue warps store S (two 16-bit planes) and the agent accumulator (rows = cells) as one split-K
// partial per (env tile, t slice).  Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the CTA unwinds.
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

template <int H, int PREC>
struct Dh1aCfg {
    static constexpr int BM = 128, BN = 64, KC = 64, THREADS = 192;
    static constexpr int PL = PREC == 1 ? 1 : 2;
    static constexpr int NCH = H / KC;
    static constexpr int W_BOX = BN * 128;               // 64 n-rows x 64 k (8 KB), K-major
    static constexpr int W_BYTES = PL * NCH * W_BOX;     // resident W2 slice
    static constexpr int A_BOX = BM * 128;               // 128 env rows x 64 k (16 KB), K-major
    static constexpr int A_STAGE = PL * A_BOX;
    static constexpr int D_TILE = PL * BM * 128;         // dh1 tile: 128 k-rows (envs) x 64 cols, MN-major, hi (and lo)
    static constexpr int O_TILE = 2 * BM * 128;          // one-hot tile: 128 k-rows (envs) x 128 cells (two 64-wide boxes)
    static constexpr int ACCW = PL * BN;                 // accumulator width: the hi x lo term has its own 64 columns
    static constexpr int TMEM_COLS = 3 * ACCW <= 256 ? 256 : 512;
    static constexpr int BARS = 256;
    static constexpr int MAX_SMEM = 232448 - 1024;       // 227 KB per CTA minus alignment slack
    static constexpr int RING = MAX_SMEM - BARS - W_BYTES - D_TILE - O_TILE;
    static constexpr int STAGES = RING / A_STAGE >= 6 ? 6 : RING / A_STAGE;
    static_assert(STAGES >= 2, "the dh2 ring needs two stages");
    static constexpr size_t smem_bytes = (size_t)W_BYTES + (size_t)STAGES * A_STAGE + D_TILE + O_TILE + BARS + 1024;
};

struct Dh1aMaps {
    CUtensorMap a_hi, a_lo, w_hi, w_lo;
};

template <int H, int PREC>
__global__ void __launch_bounds__(192, 1) k_dh1a_tc(const __grid_constant__ Dh1aMaps maps, LearnArgs a, float* part_agent, size_t part_stride) {
    using Cfg = Dh1aCfg<H, PREC>;
    constexpr int BM = Cfg::BM, BN = Cfg::BN, KC = Cfg::KC, PL = Cfg::PL, NCH = Cfg::NCH, STAGES = Cfg::STAGES;
    constexpr int PREFETCH = 3 * NCH;  // chunks between the L2 prefetch of a box and its load (three steps)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sW = base;                                   // [NCH][PL] boxes: the lo box follows the hi box of its k chunk
    unsigned char* sA = sW + Cfg::W_BYTES;                      // [STAGES][PL] boxes
    unsigned char* sD = sA + STAGES * Cfg::A_STAGE;             // dh1 tile, hi plane then lo plane
    unsigned char* sO = sD + Cfg::D_TILE;                       // one-hot tile, two boxes of 64 cells
    uint64_t* bars = (uint64_t*)(sO + Cfg::O_TILE);
    uint64_t* full = bars;                  // [STAGES]
    uint64_t* empty = full + STAGES;        // [STAGES]
    uint64_t* tfull = empty + STAGES;       // [2] dh1 accumulator written
    uint64_t* tempty = tfull + 2;           // [2] dh1 accumulator drained (4 epilogue warps arrive)
    uint64_t* wfull = tempty + 2;           // W2 slice landed
    uint64_t* tiles_full = wfull + 1;       // operand tiles of a step written (128 epilogue threads arrive)
    uint64_t* tiles_free = tiles_full + 1;  // the agent MMAs that read them have finished
    uint32_t* tmem_slot = (uint32_t*)(tiles_free + 1);

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int B = d.B, T = a.T, C = d.C;
    const int n0 = blockIdx.y * BN;
    const int m_tiles = (B + BM - 1) / BM;
    int* status = b.status;
    const int tl = (T + a.ts - 1) / a.ts;  // this CTA's slice of the steps
    const int t0 = blockIdx.z * tl, t1 = min(T, t0 + tl);
    const int nsteps = t1 > t0 ? t1 - t0 : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&tfull[i], 1); tc::mbar_init(&tempty[i], 4); }
        tc::mbar_init(wfull, 1);
        tc::mbar_init(tiles_full, 128);
        tc::mbar_init(tiles_free, 1);
        tc::mbar_fence_init();
    }
    if (wid == 2) tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    // the one-hot tile starts all zero; every step clears the element it set the step before
    for (int i = tid; i < Cfg::O_TILE / 16; i += Cfg::THREADS) reinterpret_cast<uint4*>(sO)[i] = make_uint4(0u, 0u, 0u, 0u);
    tc::fence_proxy_async();
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    constexpr int ACCW = Cfg::ACCW;
    const uint32_t acc_agent = tmem + 2 * ACCW;
    int my_tiles = 0;  // env tiles this CTA walks
    for (int mt = blockIdx.x; mt < m_tiles; mt += gridDim.x) ++my_tiles;
    const int G = my_tiles * nsteps;  // steps of this CTA, all env tiles together (the pipelines run across tiles)
    bool ok = true;

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer
            tc::mbar_expect_tx(wfull, Cfg::W_BYTES);
#pragma unroll
            for (int kc = 0; kc < NCH; ++kc) {
                tc::tma_load_2d(sW + PL * kc * Cfg::W_BOX, &maps.w_hi, wfull, kc * KC, n0);
                if (PL == 2) tc::tma_load_2d(sW + (PL * kc + 1) * Cfg::W_BOX, &maps.w_lo, wfull, kc * KC, n0);
            }
            for (int c = 0; c < G * NCH && ok; ++c) {
                const int s = c % STAGES, g = c / NCH, kc = c - g * NCH;
                const int e0 = ((int)blockIdx.x + (g / nsteps) * (int)gridDim.x) * BM, t = t0 + g % nsteps;
                {   // pull the boxes of a later chunk towards L2 now, so that their TMA load is an L2 hit
                    const int cp = c + PREFETCH;
                    if (cp < G * NCH) {
                        const int gp = cp / NCH, kp = cp - gp * NCH;
                        const int ep = ((int)blockIdx.x + (gp / nsteps) * (int)gridDim.x) * BM, tp = t0 + gp % nsteps;
                        tc::tma_prefetch_2d(&maps.a_hi, kp * KC, tp * B + ep);
                        if (PL == 2) tc::tma_prefetch_2d(&maps.a_lo, kp * KC, tp * B + ep);
                    }
                }
                if (c >= STAGES) ok = tc::mbar_wait(&empty[s], ((c / STAGES) - 1) & 1);
                if (!ok) break;
                tc::mbar_expect_tx(&full[s], Cfg::A_STAGE);
                // rows t*B + e0 .. +127 of the dh2 planes (rows past the batch end belong to the next step or are
                // zero-filled past the last row; their results are discarded by the epilogue)
                tc::tma_load_2d(sA + s * Cfg::A_STAGE, &maps.a_hi, &full[s], kc * KC, t * B + e0);
                if (PL == 2) tc::tma_load_2d(sA + s * Cfg::A_STAGE + Cfg::A_BOX, &maps.a_lo, &full[s], kc * KC, t * B + e0);
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0) {  // ---- MMA issuer
            // Operand fetch from shared memory bounds these MMAs, so terms that share an A operand are issued as ONE
            // instruction over a wider B: [W_hi | W_lo] (N = 128) for a_hi, and [dh1_hi | dh1_lo] for the one-hot.
            const uint32_t idesc = tc::umma_idesc<PREC>(BM, BN, false, false);
            const uint32_t idesc_w = tc::umma_idesc<PREC>(BM, ACCW, false, false);
            const uint32_t idesc_agent = tc::umma_idesc<PREC>(128, ACCW, true, true);
            // agent-plane product of step v: 8 k16 steps over the 128 envs (the one-hot is exact; columns 64.. of the
            // accumulator collect the dh1 lo plane's share)
            auto agent_mma = [&](int v) {
                ok = tc::mbar_wait(tiles_full, (uint32_t)v & 1u);
                if (!ok) return;
                tc::tc_fence_after();
#pragma unroll
                for (int k16 = 0; k16 < BM / 16; ++k16) {
                    const uint64_t od = tc::umma_desc(sO + k16 * 2048, BM * 128, 1024);  // cells 64.. are one box further
                    const uint64_t dh = tc::umma_desc(sD + k16 * 2048, BM * 128, 1024);  // the lo plane is the next box
                    tc::umma(acc_agent, od, dh, idesc_agent, (v > 0 || k16 > 0) ? 1u : 0u);
                }
                tc::umma_commit(tiles_free);
            };
            ok = tc::mbar_wait(wfull, 0);
            for (int u = 0; u < G && ok; ++u) {
                const int buf = u & 1;
                if (u >= 2) ok = tc::mbar_wait(&tempty[buf], ((u >> 1) - 1) & 1);  // epilogue of step u-2 has drained it
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + (uint32_t)(buf * ACCW);
                for (int kc = 0; kc < NCH && ok; ++kc) {
                    const int c = u * NCH + kc, s = c % STAGES;
                    ok = tc::mbar_wait(&full[s], (c / STAGES) & 1);
                    if (!ok) break;
                    tc::tc_fence_after();
                    unsigned char* sa = sA + s * Cfg::A_STAGE;
#pragma unroll
                    for (int k16 = 0; k16 < KC / 16; ++k16) {
                        // K-major operands: 16 k = 32 bytes further along the swizzled 128-byte rows
                        const uint64_t a_hi = tc::umma_desc(sa + k16 * 32, 16, 1024);
                        const uint64_t w_hi = tc::umma_desc(sW + PL * kc * Cfg::W_BOX + k16 * 32, 16, 1024);  // lo rows follow
                        const uint32_t accum = (kc > 0 || k16 > 0) ? 1u : 0u;
                        tc::umma(acc, a_hi, w_hi, idesc_w, accum);  // columns 0-63: hi x hi; 64-127: hi x lo
                        if (PL == 2) tc::umma(acc, tc::umma_desc(sa + Cfg::A_BOX + k16 * 32, 16, 1024), w_hi, idesc, 1u);  // lo x hi
                    }
                    tc::umma_commit(&empty[s]);
                }
                if (!ok) break;
                tc::umma_commit(&tfull[buf]);
                if (u >= 1) agent_mma(u - 1);  // queued behind this step's product: the tensor pipe stays busy
            }
            if (ok && G > 0) agent_mma(G - 1);
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- epilogue warps: thread = env (accumulator lane 32*(wid%4) + lane), all 64 columns of the tile
        const int q = wid & 3, row = 32 * q + lane;
        const uint16_t* g_h1hi = reinterpret_cast<const uint16_t*>(b.h1);
        unsigned char* drow = sD + row * 128;
        int prev_off = -1;  // byte offset of the one-hot element this thread set the step before
        int g = 0;          // running step index of this CTA
        for (int mt = blockIdx.x; mt < m_tiles && ok; mt += gridDim.x) {
            const int env = mt * BM + row;
            const bool valid = env < B;
            float s_acc[64];
#pragma unroll
            for (int j = 0; j < 64; ++j) s_acc[j] = 0.f;
            if (valid && nsteps > 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(g_h1hi + ((size_t)t0 * B + env) * H + n0));
            for (int t = t0; t < t1; ++t, ++g) {
                const int buf = g & 1;
                const size_t gi = ((size_t)t * B + (valid ? env : 0)) * H + n0;
                if (valid && t + 1 < t1) asm volatile("prefetch.global.L2 [%0];" ::"l"(g_h1hi + gi + (size_t)B * H));
                // this row's layer-1 gates (64 units x 16 bit) and position, fetched before the accumulator is waited for
                uint4 gate[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) gate[j] = valid ? __ldg(reinterpret_cast<const uint4*>(g_h1hi + gi) + j) : make_uint4(0u, 0u, 0u, 0u);
                const int cell = valid ? (int)b.tpos[(size_t)t * B + env] : -1;
                if (ok) ok = tc::mbar_wait(&tfull[buf], (g >> 1) & 1);
                if (!ok) break;
                tc::tc_fence_after();
                uint32_t r0[32], r1[32];
                const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * ACCW);
                tc::tmem_ld32(taddr, r0);
                tc::tmem_ld32(taddr + 32, r1);
                if (PL == 2) {  // add the hi x lo term
                    uint32_t r2[32];
                    tc::tmem_ld32(taddr + 64, r2);
#pragma unroll
                    for (int j = 0; j < 32; ++j) r0[j] = __float_as_uint(__uint_as_float(r0[j]) + __uint_as_float(r2[j]));
                    tc::tmem_ld32(taddr + 96, r2);
#pragma unroll
                    for (int j = 0; j < 32; ++j) r1[j] = __float_as_uint(__uint_as_float(r1[j]) + __uint_as_float(r2[j]));
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&tempty[buf]);  // the issuer may overwrite this accumulator now
                // the operand tiles are free once the agent MMAs of the step before have finished
                if (g >= 1) ok = tc::mbar_wait(tiles_free, (uint32_t)(g - 1) & 1u);
                if (!ok) break;
                const uint32_t* gw = reinterpret_cast<const uint32_t*>(gate);
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {  // 16-byte chunks of 8 columns
                    uint32_t phi[4], plo[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int col = 8 * c8 + 2 * j;
                        const uint32_t gt = gw[4 * c8 + j];  // units col, col+1; h1 >= 0, so "h1 > 0" is "any magnitude bit set"
                        const float x0 = __uint_as_float(col < 32 ? r0[col] : r1[col - 32]);
                        const float x1 = __uint_as_float(col < 32 ? r0[col + 1] : r1[col - 31]);
                        const float v0 = rnd<PREC>((gt & 0x00007FFFu) ? x0 : 0.f);
                        const float v1 = rnd<PREC>((gt & 0x7FFF0000u) ? x1 : 0.f);
                        s_acc[col] += v0;
                        s_acc[col + 1] += v1;
                        split2<PREC>(v0, v1, phi[j], plo[j]);  // rows past the batch end have all-zero gates
                    }
                    // element (k = row, n) of the MN-major tile: byte k*128 + ((n/8) ^ (k%8))*16 + (n%8)*2
                    const int off = (c8 ^ (row & 7)) << 4;
                    *reinterpret_cast<uint4*>(drow + off) = make_uint4(phi[0], phi[1], phi[2], phi[3]);
                    if (PL == 2) *reinterpret_cast<uint4*>(drow + BM * 128 + off) = make_uint4(plo[0], plo[1], plo[2], plo[3]);
                }
                if (prev_off >= 0) *reinterpret_cast<uint16_t*>(sO + prev_off) = 0;
                prev_off = -1;
                if (cell >= 0 && cell < 128) {
                    prev_off = (cell >> 6) * (BM * 128) + row * 128 + ((((cell & 63) >> 3) ^ (row & 7)) << 4) + (cell & 7) * 2;
                    *reinterpret_cast<uint16_t*>(sO + prev_off) = (uint16_t)one16<PREC>();
                }
                tc::fence_proxy_async();  // generic-proxy stores -> visible to the tensor core
                tc::mbar_arrive(tiles_full);
            }
            // S (sum over t of dh1) as two 16-bit planes [ts*B][H]: an fp32 sum keeps two terms in either workload
            if (valid && ok) {
                uint16_t* S_hi = reinterpret_cast<uint16_t*>(b.S);
                uint16_t* S_lo = S_hi + (size_t)a.ts * B * H;
                const size_t si = ((size_t)blockIdx.z * B + env) * H + n0;  // an empty slice writes zeros
                uint32_t phi[32], plo[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (PREC == 1) {
                        __nv_bfloat16 h0, l0, h1v, l1;
                        split_bf16(s_acc[2 * j], h0, l0);
                        split_bf16(s_acc[2 * j + 1], h1v, l1);
                        phi[j] = pack_bf16(h0, h1v);
                        plo[j] = pack_bf16(l0, l1);
                    } else {
                        split2<0>(s_acc[2 * j], s_acc[2 * j + 1], phi[j], plo[j]);
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    reinterpret_cast<uint4*>(S_hi + si)[j] = make_uint4(phi[4 * j], phi[4 * j + 1], phi[4 * j + 2], phi[4 * j + 3]);
                    reinterpret_cast<uint4*>(S_lo + si)[j] = make_uint4(plo[4 * j], plo[4 * j + 1], plo[4 * j + 2], plo[4 * j + 3]);
                }
            }
        }
        if (!ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        // agent-plane partial of this (env tile, t slice): accumulator lane = cell
        bool got = ok;
        if (got && G > 0) got = tc::mbar_wait(tiles_free, (uint32_t)(G - 1) & 1u);
        if (!got && ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        tc::tc_fence_after();
        __syncwarp();
        const int cellr = 32 * q + lane;
        float* part = part_agent + (size_t)(blockIdx.z * gridDim.x + blockIdx.x) * part_stride;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t r[32];
            if (got && G > 0) {
                tc::tmem_ld32(acc_agent + ((uint32_t)(32 * q) << 16) + (uint32_t)(32 * half), r);
                if (PL == 2) {  // the dh1 lo plane's share
                    uint32_t r2[32];
                    tc::tmem_ld32(acc_agent + ((uint32_t)(32 * q) << 16) + (uint32_t)(64 + 32 * half), r2);
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;  // an empty slice contributes zeros
            }
            if (cellr < C) {
                float4* dst = reinterpret_cast<float4*>(part + (size_t)cellr * H + n0 + 32 * half);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                         __uint_as_float(r[4 * j + 3]));
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (wid == 2) tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
}

template <int H, int PREC>
cudaError_t launch_t(const LearnArgs& a, int grid_x, float* part_agent, size_t part_stride, cudaStream_t s) {
    using Cfg = Dh1aCfg<H, PREC>;
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const size_t R = (size_t)d.B * a.T, RH = (size_t)d.B * d.Tmax * H;
    const bool bf = PREC == 1;
    Dh1aMaps maps;
    memset(&maps, 0, sizeof(maps));
    const uint16_t* dh2hi = reinterpret_cast<const uint16_t*>(b.dh2);
    if (!make_tensor_map_2d(&maps.a_hi, dh2hi, R, H, 128, bf)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_hi, b.w2p_hi, H, H, 64, bf)) return cudaErrorNotSupported;
    if (Cfg::PL == 2) {
        if (!make_tensor_map_2d(&maps.a_lo, dh2hi + RH, R, H, 128, bf)) return cudaErrorNotSupported;
        if (!make_tensor_map_2d(&maps.w_lo, b.w2p_lo, H, H, 64, bf)) return cudaErrorNotSupported;
    }
    cudaError_t e = cudaFuncSetAttribute(k_dh1a_tc<H, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
    if (e != cudaSuccess) return e;
    dim3 grid(grid_x, H / Cfg::BN, a.ts);
    k_dh1a_tc<H, PREC><<<grid, Cfg::THREADS, Cfg::smem_bytes, s>>>(maps, a, part_agent, part_stride);
    return cudaGetLastError();
}

}  // namespace

bool dh1_agent_tc_supported(const Dims& d) { return (d.H == 128 || d.H == 256) && d.C <= 128; }

// grid_x CTAs share the 128-env tiles (grid_x <= ceil(B/128)); a.ts slices the steps.  The agent-plane partials go to
// part_agent[split * part_stride + cell * H + col] with split = t slice * grid_x + blockIdx.x: grid_x * a.ts splits.
// cudaErrorNotSupported when the shape is not covered.
cudaError_t launch_dh1_agent_tc(const LearnArgs& a, int prec, int grid_x, float* part_agent, size_t part_stride, cudaStream_t s) {
    if (!dh1_agent_tc_supported(a.d) || !a.b.w2p_hi || (prec != 1 && !a.b.w2p_lo)) return cudaErrorNotSupported;
    if (a.d.H == 256) return prec == 1 ? launch_t<256, 1>(a, grid_x, part_agent, part_stride, s) : launch_t<256, 0>(a, grid_x, part_agent, part_stride, s);
    return prec == 1 ? launch_t<128, 1>(a, grid_x, part_agent, part_stride, s) : launch_t<128, 0>(a, grid_x, part_agent, part_stride, s);
}

}  // namespace anakin
