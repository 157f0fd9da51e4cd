// dh1 = (dh2 W2^T) gated by h1 > 0, and S = sum over t of dh1, on the 5th-generation tensor cores.
//
// Backward pass through the second layer of the policy/value MLP (the update half of the Anakin minimal unit, Podracer
// paper, Section 3.1; Figure 2, top).  A CTA owns 128 envs x 128 output columns and walks t = 0..T-1, so S accumulates in
// registers.  Its slice of W2 (128 rows, all of K, hi and lo planes) is TMA-loaded once and stays in shared memory; the
// dh2 planes stream through a TMA ring of 128 x 64 K-major boxes that runs across the t boundaries without draining.
//   warp 0 (one lane)  TMA producer
//   warp 1 (one lane)  tcgen05.mma issuer: per k16 three MMAs (lo*hi, hi*lo, hi*hi fp16 terms; one bf16 MMA in the bf16
//                      workload) into one of two 128-column fp32 accumulators in tensor memory
//   warps 2-9          epilogue of step t while the MMAs of step t+1 run: tcgen05.ld, gate, S += , split, store dh1 planes
// Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the CTA unwinds (tensor memory freed).
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

template <int H, int PREC>
struct Dh1TcCfg {
    static constexpr int BM = 128, BN = 128, KC = 64, THREADS = 320;
    static constexpr int PL = PREC == 1 ? 1 : 2;
    static constexpr int NCH = H / KC;
    static constexpr int BOX = 128 * 64 * 2;                      // one 128-row x 64-k box (16 KB)
    static constexpr int W_BYTES = PL * NCH * BOX;                // resident W2 slice
    static constexpr int A_STAGE = PL * BOX;
    static constexpr int MAX_SMEM = 232448 - 1024 - 256;         // 227 KB per CTA, minus alignment slack and barriers
    static constexpr int STAGES = (MAX_SMEM - W_BYTES) / A_STAGE >= 6 ? 6 : (MAX_SMEM - W_BYTES) / A_STAGE;
    static constexpr size_t smem_bytes = (size_t)W_BYTES + (size_t)STAGES * A_STAGE + 1024 + 256;
};

struct Dh1TcMaps {
    CUtensorMap a_hi, a_lo, w_hi, w_lo;
};

template <int H, int PREC>
__global__ void __launch_bounds__(320, 1) k_dh1_tc(const __grid_constant__ Dh1TcMaps maps, LearnArgs a) {
    using Cfg = Dh1TcCfg<H, PREC>;
    constexpr int BM = Cfg::BM, BN = Cfg::BN, KC = Cfg::KC, PL = Cfg::PL, NCH = Cfg::NCH, STAGES = Cfg::STAGES, BOX = Cfg::BOX;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sW = base;                       // [PL][NCH] boxes
    unsigned char* sA = base + Cfg::W_BYTES;        // [STAGES][PL] boxes
    uint64_t* bars = (uint64_t*)(sA + STAGES * Cfg::A_STAGE);
    uint64_t* full = bars;                 // [STAGES]
    uint64_t* empty = bars + STAGES;       // [STAGES]
    uint64_t* tfull = bars + 2 * STAGES;   // [2] accumulator buffer written
    uint64_t* tempty = tfull + 2;          // [2] accumulator buffer drained (8 epilogue warps arrive)
    uint64_t* wfull = tempty + 2;          // W2 slice landed
    uint32_t* tmem_slot = (uint32_t*)(wfull + 1);

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int B = d.B, T = a.T;
    const int e0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const size_t RH = (size_t)B * d.Tmax * H;
    int* status = b.status;
    // this CTA's slice of the steps
    const int tl = (T + a.ts - 1) / a.ts;
    const int t0 = blockIdx.z * tl, t1 = min(T, t0 + tl);
    const int nsteps = t1 > t0 ? t1 - t0 : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&tfull[i], 1); tc::mbar_init(&tempty[i], 8); }
        tc::mbar_init(wfull, 1);
        tc::mbar_fence_init();
    }
    if (wid == 2) tc::tmem_alloc(tmem_slot, 256);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int nchunks = nsteps * NCH;
    bool ok = true;

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer
            tc::mbar_expect_tx(wfull, Cfg::W_BYTES);
#pragma unroll
            for (int kc = 0; kc < NCH; ++kc) {
                tc::tma_load_2d(sW + kc * BOX, &maps.w_hi, wfull, kc * KC, n0);
                if (PL == 2) tc::tma_load_2d(sW + (NCH + kc) * BOX, &maps.w_lo, wfull, kc * KC, n0);
            }
            for (int c = 0; c < nchunks && ok; ++c) {
                const int s = c % STAGES, u = c / NCH, kc = c - u * NCH, t = t0 + u;
                if (c >= STAGES) ok = tc::mbar_wait(&empty[s], ((c / STAGES) - 1) & 1);
                if (!ok) break;
                tc::mbar_expect_tx(&full[s], Cfg::A_STAGE);
                // rows t*B + e0 .. +127 of the dh2 planes (rows past the batch end belong to the next step or are
                // zero-filled past the last row; their results are discarded by the epilogue)
                tc::tma_load_2d(sA + s * Cfg::A_STAGE, &maps.a_hi, &full[s], kc * KC, t * B + e0);
                if (PL == 2) tc::tma_load_2d(sA + s * Cfg::A_STAGE + BOX, &maps.a_lo, &full[s], kc * KC, t * B + e0);
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0) {  // ---- MMA issuer
            const uint32_t idesc = tc::umma_idesc<PREC>(BM, BN, false, false);
            ok = tc::mbar_wait(wfull, 0);
            for (int u = 0; u < nsteps && ok; ++u) {
                const int buf = u & 1;
                if (u >= 2) ok = tc::mbar_wait(&tempty[buf], ((u >> 1) - 1) & 1);  // epilogue of step u-2 has drained it
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + (uint32_t)(buf * BN);
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
                        const uint64_t w_hi = tc::umma_desc(sW + kc * BOX + k16 * 32, 16, 1024);
                        uint32_t accum = (kc > 0 || k16 > 0) ? 1u : 0u;
                        if (PL == 2) {
                            tc::umma(acc, tc::umma_desc(sa + BOX + k16 * 32, 16, 1024), w_hi, idesc, accum);
                            tc::umma(acc, a_hi, tc::umma_desc(sW + (NCH + kc) * BOX + k16 * 32, 16, 1024), idesc, 1u);
                            accum = 1u;
                        }
                        tc::umma(acc, a_hi, w_hi, idesc, accum);
                    }
                    tc::umma_commit(&empty[s]);
                }
                if (ok) tc::umma_commit(&tfull[buf]);
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- epilogue warps: accumulator lanes 32*(wid%4)..+31 (= envs), column half (wid-2)/4 of the 128-wide tile
        const int q = wid & 3, ch = (wid - 2) >> 2;
        const int env = e0 + 32 * q + lane;
        const bool valid = env < B;
        const int col0 = n0 + 64 * ch;
        const uint16_t* g_h1hi = reinterpret_cast<const uint16_t*>(b.h1);
        uint16_t* g_dh1hi = reinterpret_cast<uint16_t*>(b.dh1);
        float s_acc[64];
#pragma unroll
        for (int j = 0; j < 64; ++j) s_acc[j] = 0.f;
        if (valid && nsteps > 0) {  // first two gate lines
            asm volatile("prefetch.global.L2 [%0];" ::"l"(g_h1hi + ((size_t)t0 * B + env) * H + col0));
            if (nsteps > 1) asm volatile("prefetch.global.L2 [%0];" ::"l"(g_h1hi + ((size_t)(t0 + 1) * B + env) * H + col0));
        }
        for (int t = t0; t < t1; ++t) {
            const int u = t - t0, buf = u & 1;
            const size_t gi = ((size_t)t * B + (valid ? env : 0)) * H + col0;
            // pull the gate line of step t+2 towards L2 now (one 128-byte line per thread), so that the load below
            // costs an L2 hit by the time it is issued
            if (valid && t + 2 < t1)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(g_h1hi + gi + (size_t)2 * B * H));
            // this row's layer-1 gates (64 units x 16 bit), fetched before the accumulator is waited for
            uint4 gate[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) gate[j] = valid ? __ldg(reinterpret_cast<const uint4*>(g_h1hi + gi) + j) : make_uint4(0u, 0u, 0u, 0u);
            if (ok) ok = tc::mbar_wait(&tfull[buf], (u >> 1) & 1);
            if (!ok) break;
            tc::tc_fence_after();
            uint32_t r0[32], r1[32];
            const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * BN + 64 * ch);
            tc::tmem_ld32(taddr, r0);
            tc::tmem_ld32(taddr + 32, r1);
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&tempty[buf]);  // the issuer may overwrite this accumulator now
            const uint32_t* gw = reinterpret_cast<const uint32_t*>(gate);
            // two halves of 32 columns each, to keep the live register set small
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t phi[16], plo[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const uint32_t gt = gw[16 * half + j];  // units 2j, 2j+1; h1 >= 0, so "h1 > 0" is "any bit of the high part set"
                    const float x0 = __uint_as_float(half == 0 ? r0[2 * j] : r1[2 * j]);
                    const float x1 = __uint_as_float(half == 0 ? r0[2 * j + 1] : r1[2 * j + 1]);
                    const float v0 = rnd<PREC>((gt & 0x0000FFFFu) ? x0 : 0.f);
                    const float v1 = rnd<PREC>((gt & 0xFFFF0000u) ? x1 : 0.f);
                    s_acc[32 * half + 2 * j] += v0;
                    s_acc[32 * half + 2 * j + 1] += v1;
                    split2<PREC>(v0, v1, phi[j], plo[j]);
                }
                if (valid) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        reinterpret_cast<uint4*>(g_dh1hi + gi)[4 * half + j] = make_uint4(phi[4 * j], phi[4 * j + 1], phi[4 * j + 2], phi[4 * j + 3]);
                        if (PL == 2)
                            reinterpret_cast<uint4*>(g_dh1hi + RH + gi)[4 * half + j] = make_uint4(plo[4 * j], plo[4 * j + 1], plo[4 * j + 2], plo[4 * j + 3]);
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        // S (sum over t of dh1) as two 16-bit planes [B][H]: an fp32 sum keeps two terms in either workload
        if (valid) {
            uint16_t* S_hi = reinterpret_cast<uint16_t*>(b.S);
            uint16_t* S_lo = S_hi + (size_t)a.ts * B * H;
            const size_t si = ((size_t)blockIdx.z * B + env) * H + col0;  // an empty slice writes zeros
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
    tc::tc_fence_before();
    __syncthreads();
    if (wid == 2) tc::tmem_dealloc(tmem, 256);
}

template <int H, int PREC>
static cudaError_t launch_t(const LearnArgs& a, cudaStream_t s) {
    using Cfg = Dh1TcCfg<H, PREC>;
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const size_t R = (size_t)d.B * a.T, RH = (size_t)d.B * d.Tmax * H;
    const bool bf = PREC == 1;
    Dh1TcMaps maps;
    memset(&maps, 0, sizeof(maps));
    const uint16_t* dh2hi = reinterpret_cast<const uint16_t*>(b.dh2);
    if (!make_tensor_map_2d(&maps.a_hi, dh2hi, R, H, 128, bf)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_hi, b.w2p_hi, H, H, 128, bf)) return cudaErrorNotSupported;
    if (Cfg::PL == 2) {
        if (!make_tensor_map_2d(&maps.a_lo, dh2hi + RH, R, H, 128, bf)) return cudaErrorNotSupported;
        if (!make_tensor_map_2d(&maps.w_lo, b.w2p_lo, H, H, 128, bf)) return cudaErrorNotSupported;
    }
    cudaError_t e = cudaFuncSetAttribute(k_dh1_tc<H, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
    if (e != cudaSuccess) return e;
    dim3 grid((d.B + Cfg::BM - 1) / Cfg::BM, H / Cfg::BN, a.ts);
    k_dh1_tc<H, PREC><<<grid, Cfg::THREADS, Cfg::smem_bytes, s>>>(maps, a);
    return cudaGetLastError();
}

// Covered: H = 128 or 256.  cudaErrorNotSupported otherwise (the caller falls back to the mma.sync kernel).
cudaError_t launch_dh1_tc(const LearnArgs& a, int prec, cudaStream_t s) {
    if (a.d.H == 256) return prec == 1 ? launch_t<256, 1>(a, s) : launch_t<256, 0>(a, s);
    if (a.d.H == 128) return prec == 1 ? launch_t<128, 1>(a, s) : launch_t<128, 0>(a, s);
    return cudaErrorNotSupported;
}

}  // namespace anakin
