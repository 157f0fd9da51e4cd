// CTA-pair version of the wide-path GEMM  C[m][n] = sum_k A[m][k] Bop[k][n]  (bf16, fp32 accumulate in tensor memory):
// the layer-2 products of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top) for wide hidden layers.
//
// Operand fetch from shared memory bounds a one-CTA tcgen05 MMA: a 128 x 256 tile reads 12 KB per k16 step.  Here two
// CTAs (a cluster of two, on neighbouring SMs) own one 256 x 256 output tile: each CTA stages ITS 128 rows of A and ITS
// 128 columns of B (32 KB per 64-wide k chunk instead of 48 KB), one thread of the leader CTA issues
// tcgen05.mma.cta_group::2 instructions that run on both tensor cores and read both CTAs' shared memory, and each CTA
// ends up with its 128 rows x 256 columns of the accumulator in its own tensor memory.
//   warp 0 (one lane, both CTAs)   TMA producer of its CTA's halves; the byte counts of both CTAs are credited to the
//                                  LEADER's "full" barrier, which the leader's producer arms for both
//   warp 1 (one lane, leader only) MMA issuer; commits are multicast to the "empty" / "accumulator full" barriers of both CTAs
//   warps 2-9 (both CTAs)          epilogue of tile i under the MMAs of tile i+1 (two 256-column accumulators); their
//                                  "accumulator drained" arrivals all go to the leader's barrier
// Tensor memory is allocated and freed by one warp of each CTA.  Every wait is bounded (a timeout raises
// DEV_E_WAIT_TIMEOUT and the CTA walks to the exit); the two cluster barriers at start and exit are unconditional.
#include <cstring>

#include "wide_gemm.cuh"

namespace anakin {
namespace widegemm {

namespace {

struct PairCfg {
    static constexpr int BM = 128, PM = 256, BN = NT_BN, BNH = 128, KC = 64, STAGES = 5, THREADS = 320;
    static constexpr int A_BYTES = BM * KC * 2, B_BYTES = BNH * KC * 2, STAGE = A_BYTES + B_BYTES;
    static constexpr size_t smem_bytes = (size_t)STAGES * STAGE + 1024 /*alignment slack*/ + 256 /*barriers, tmem slot*/ + NT_MAXN * 4 + NT_EPI_WARPS * NT_STAGE_BYTES;
};

template <int EPI, bool B_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(320, 1) k_gemm_nt_pair(const __grid_constant__ NtMaps maps, NtArgs g) {
    using Cfg = PairCfg;
    constexpr int BM = Cfg::BM, PM = Cfg::PM, BN = Cfg::BN, BNH = Cfg::BNH, KC = Cfg::KC, STAGES = Cfg::STAGES;
    extern __shared__ unsigned char smem_raw[];
    // the dynamic shared memory starts at the same offset in both CTAs, so the rounded base does too
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(base + STAGES * Cfg::STAGE);
    uint64_t* full = bars;                // [STAGES] leader's copy collects both CTAs' loads
    uint64_t* empty = bars + STAGES;      // [STAGES] one per CTA, signalled by the multicast commit
    uint64_t* tfull = bars + 2 * STAGES;  // [2] accumulator written (multicast commit)
    uint64_t* tempty = tfull + 2;         // [2] leader's copy: accumulator drained by the 16 epilogue warps of the pair
    uint32_t* tmem_slot = (uint32_t*)(tempty + 2);
    float* s_bias = (float*)(base + STAGES * Cfg::STAGE + 256);
    unsigned char* s_stage = (unsigned char*)(s_bias + NT_MAXN);  // [NT_EPI_WARPS][NT_STAGE_BYTES]
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const uint32_t rank = tc::cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int nt = g.N / BN, mt = (g.M + PM - 1) / PM, ntiles = mt * nt, nch = g.K / KC;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&tfull[i], 1); tc::mbar_init(&tempty[i], 2 * NT_EPI_WARPS); }
        tc::mbar_fence_init();
    }
    if (EPI != EPI_GATE)
        for (int i = tid; i < g.N; i += Cfg::THREADS) s_bias[i] = g.bias[i];
    if (wid == 2) tc::tmem_alloc_pair(tmem_slot, 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    tc::cluster_sync_all();  // both CTAs' barriers exist before either signals the other
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer of this CTA's halves
            int c = 0;
            for (int tile = pair; tile < ntiles && ok; tile += npairs) {
                const int m0 = (tile / nt) * PM + BM * (int)rank, n0 = (tile % nt) * BN + BNH * (int)rank;
                for (int kc = 0; kc < nch; ++kc, ++c) {
                    const int s = c % STAGES;
                    if (c >= STAGES) ok = tc::mbar_wait(&empty[s], ((c / STAGES) - 1) & 1);
                    if (!ok) break;
                    unsigned char* sa = base + s * Cfg::STAGE;
                    unsigned char* sb = sa + Cfg::A_BYTES;
                    if (leader) tc::mbar_expect_tx(&full[s], 2 * Cfg::STAGE);  // the loads of both CTAs
                    const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);
                    // rows past M belong to later rows of the buffer or are zero-filled; the epilogue drops them
                    tc::tma_load_2d_pair(sa, &maps.a, bar, kc * KC, g.row0 + m0);
                    if (B_MN) {
#pragma unroll
                        for (int bx = 0; bx < BNH / 64; ++bx) tc::tma_load_2d_pair(sb + bx * 8192, &maps.b, bar, n0 + 64 * bx, kc * KC);
                    } else {
                        tc::tma_load_2d_pair(sb, &maps.b, bar, kc * KC, n0);
                    }
                }
            }
            if (!ok) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0 && leader) {  // ---- MMA issuer of the pair
            const uint32_t idesc = tc::umma_idesc<1>(PM, BN, false, B_MN);
            int c = 0, u = 0;
            for (int tile = pair; tile < ntiles && ok; tile += npairs, ++u) {
                const int buf = u & 1;
                if (u >= 2) ok = tc::mbar_wait_cluster(&tempty[buf], ((u >> 1) - 1) & 1);  // both epilogues have drained tile u-2
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
                        tc::umma_pair(acc, ad, bd, idesc, (kc > 0 || k16 > 0) ? 1u : 0u);
                    }
                    tc::umma_commit_pair(&empty[s], 3);
                }
                if (ok) tc::umma_commit_pair(&tfull[buf], 3);
            }
            if (!ok) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- epilogue warps: accumulator lanes 32*(wid%4)..+31 = this CTA's output rows
        const int q = wid & 3, half = (wid - 2) >> 2;
        int u = 0;
        for (int tile = pair; tile < ntiles; tile += npairs, ++u) {
            const int buf = u & 1;
            const int m0 = (tile / nt) * PM + BM * (int)rank, n0 = (tile % nt) * BN;
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
            if (lane == 0) tc::mbar_arrive_cluster(tc::mapa(tc::smem_u32(&tempty[buf]), 0));  // the issuer may overwrite it now
        }
        if (!ok && lane == 0) atomicOr(g.status, DEV_E_WAIT_TIMEOUT);
    }
    // neither CTA leaves (or frees tensor memory) while the other may still signal it or run MMAs that touch it
    tc::tc_fence_before();
    __syncthreads();
    tc::cluster_sync_all();
    if (wid == 2) tc::tmem_dealloc_pair(tmem, 512);
}

template <int EPI, bool B_MN>
cudaError_t launch_pair_t(const NtMaps& maps, const NtArgs& g, cudaStream_t s) {
    const cudaError_t e = cudaFuncSetAttribute(k_gemm_nt_pair<EPI, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairCfg::smem_bytes);
    if (e != cudaSuccess) return e;
    const int ntiles = ((g.M + PairCfg::PM - 1) / PairCfg::PM) * (g.N / PairCfg::BN);
    const int pairs = ntiles < 74 ? ntiles : 74;
    k_gemm_nt_pair<EPI, B_MN><<<2 * pairs, PairCfg::THREADS, PairCfg::smem_bytes, s>>>(maps, g);
    return cudaGetLastError();
}

}  // namespace

// Needs: N a multiple of 256 (at most 2048), K a multiple of 64, an A map with 128-row boxes and a B map with 64 x 64
// boxes (MN-major B) or 128-row boxes (K-major B).
cudaError_t launch_nt_pair(int epi, bool b_mn, const NtMaps& maps, const NtArgs& g, cudaStream_t s) {
    if (g.N % PairCfg::BN != 0 || g.K % PairCfg::KC != 0 || g.N > NT_MAXN || g.M < 1) return cudaErrorNotSupported;
    if (epi == EPI_FWD && b_mn) return launch_pair_t<EPI_FWD, true>(maps, g, s);
    if (epi == EPI_GATE && !b_mn) return launch_pair_t<EPI_GATE, false>(maps, g, s);
    if (epi == EPI_BASE && b_mn) return launch_pair_t<EPI_BASE, true>(maps, g, s);
    return cudaErrorNotSupported;
}

}  // namespace widegemm
}  // namespace anakin
