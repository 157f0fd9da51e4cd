// dh1 = (dh2 W2^T) gated by h1 > 0, S = sum over t of dh1, AND the agent plane of dW1 = onehot(pos)^T dh1, in one
// tcgen05 kernel: dh1 never goes to HBM.
//
// Backward pass through the second layer of the policy/value MLP and the first-layer weight gradient of the rows the
// agent's position selects (the update half of the Anakin minimal unit, Podracer paper, Section 3.1; Figure 2, top).
//
// The product is taken transposed, dh1^T[unit][env] = W2[unit][:] . dh2[env][:], so that the RESIDENT operand (the
// CTA's 128 rows of W2, both 16-bit planes) is the A operand and lives in TENSOR memory for the whole kernel: an MMA
// then fetches only the streamed dh2 box from shared memory, which is what bounds a one-CTA MMA on this part.  A CTA
// owns 128 hidden units (accumulator lanes) and walks tiles of 128 envs (tile index blockIdx.x, blockIdx.x + gridDim.x,
// ...) and, per tile, the steps t of its slice:
//   warp 0 (one lane)  TMA producer: the dh2 planes of every step through a ring of 128 x 64 K-major boxes
//   warp 1 (one lane)  tcgen05.mma issuer.  Per step: the dh1 product (K = H; three fp16 terms per k16, one in the bf16
//                      workload, all into one of two 128-column accumulators); then, for the step before, the agent-plane
//                      product  D[unit][cell] += sum over the 128 envs of dh1[env][unit] * onehot[env][cell]  (K = 128,
//                      operand tiles that the epilogue warps wrote) into a third accumulator that lives for the whole
//                      kernel
//   warp 2 (one lane)  TMA loads of the layer-1 gates (the bit mask the rollout recorded, 128 envs x 16 bytes per step)
//                      into a box the epilogue reads
//   warps 3-10         epilogue, thread = (unit, half of the envs): tcgen05.ld, gate, S +=, 16-bit split; writes its
//                      dh1^T row (hi and lo planes, K-major) and the one-hot elements in the 128-byte-swizzled layout
// At the end the epilogue warps store S (two 16-bit planes) and the agent accumulator as one split-K partial per
// (env tile, t slice).  Tensor memory: [W2 planes | two dh1 accumulators | agent accumulator]; at H = 256 only the hi plane
// of W2 fits (128 + 256 + 128 = 512 columns) and the lo plane is an ordinary shared-memory operand.
//
// H = 256 runs as a CTA PAIR (a cluster of two, tcgen05 cta_group::2): the pair owns all 256 units of an env tile, each
// CTA keeps its 128 rows of W2 in its tensor memory and stages HALF of every dh2 box (64 env rows), so every element of
// dh2 is fetched by exactly one SM; one thread of the leader CTA issues the MMAs for both tensor cores, the commits are
// multicast to both CTAs' barriers, and the "drained" / "tiles written" arrivals of both CTAs go to the leader's.  In
// the agent-plane product each CTA supplies its own dh1^T rows (A) and the one-hot columns of ITS 64 cells (B).
// Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT and the CTA unwinds (the cluster barriers at start and exit
// are unconditional).
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

template <int H, int PREC>
struct Dh1aCfg {
    static constexpr bool PAIR = H == 2 * DH1A_UNITS;  // two CTAs share an env tile, 128 units each
    static constexpr int NCTA = PAIR ? 2 : 1;
    static constexpr int BM = 128;  // envs per tile (the MMAs' N)
    static constexpr int ROWS = BM / NCTA;  // env rows of a dh2 box this CTA stages
    static constexpr int BN = DH1A_UNITS;  // hidden units per CTA (the MMAs' M: accumulator lanes)
    static constexpr int KC = 64;
    static constexpr int EPI_WARPS = 8, FIRST_EPI = 3, THREADS = 32 * (FIRST_EPI + EPI_WARPS);
    static constexpr int PL = PREC == 1 ? 1 : 2;
    static constexpr int NCH = H / KC;
    static constexpr int A_BOX = ROWS * 128;             // dh2: this CTA's env rows x 64 k, K-major
    static constexpr int A_STAGE = PL * A_BOX;
    static constexpr int D_BOX = BN * 128;               // dh1^T: 128 unit rows x 64 envs (16 KB), K-major
    static constexpr int D_TILE = PL * 2 * D_BOX;        // [plane][env half]
    static constexpr int O_TILE = (2 / NCTA) * BM * 128; // one-hot: 128 k-rows (envs) x this CTA's cells (64-wide boxes), MN-major
    static constexpr int G_TILE = BM * (BN / 8);         // gates: 128 env rows x 16 bytes (one bit per unit)
    // W2 rows in tensor memory: two k per 32-bit column, hi plane then lo.  At H = 256 only the hi plane fits beside the
    // accumulators; the lo plane (needed for one of the three fp16 terms) stays in shared memory as K-major boxes.
    static constexpr bool W_LO_SMEM = PL == 2 && H == 256;
    static constexpr int WT_PL = W_LO_SMEM ? 1 : PL;     // planes of W2 held in tensor memory
    static constexpr int W_COLS = WT_PL * H / 2;
    static constexpr int ACC_COL = W_COLS, AGENT_COL = W_COLS + 2 * 128;  // two dh1 accumulators, then the agent plane's
    static constexpr int TMEM_COLS = 512;
    static_assert(AGENT_COL + 128 <= TMEM_COLS, "tensor memory: W2 planes + three 128-column accumulators");
    static constexpr int W_BOX = BN * 128;               // W2 lo: 128 unit rows x 64 k (16 KB), K-major
    static constexpr int W_BYTES = W_LO_SMEM ? NCH * W_BOX : 0;
    // the planes bound for tensor memory are staged by TMA in the (still unused) dh1^T tile where they fit
    static constexpr bool W_STAGED = WT_PL * NCH * W_BOX <= PL * 2 * BN * 128;
    static constexpr int BARS = 256;
    static constexpr int MAX_SMEM = 232448 - 1024;       // 227 KB per CTA minus alignment slack
    static constexpr int RING = MAX_SMEM - BARS - W_BYTES - D_TILE - O_TILE - G_TILE;
    static constexpr int STAGES = RING / A_STAGE >= 6 ? 6 : RING / A_STAGE;
    static_assert(STAGES >= 2, "the dh2 ring needs two stages");
    static constexpr size_t smem_bytes = (size_t)W_BYTES + (size_t)STAGES * A_STAGE + D_TILE + O_TILE + G_TILE + BARS + 1024;
};

struct Dh1aMaps {
    CUtensorMap a_hi, a_lo, gate, w_hi, w_lo;
};

template <int H, int PREC>
__device__ __forceinline__ void dh1a_body(const Dh1aMaps& maps, const LearnArgs& a, float* part_agent, size_t part_stride) {
    using Cfg = Dh1aCfg<H, PREC>;
    constexpr int BM = Cfg::BM, BN = Cfg::BN, KC = Cfg::KC, PL = Cfg::PL, NCH = Cfg::NCH, STAGES = Cfg::STAGES;
    constexpr bool PAIR = Cfg::PAIR;
    constexpr int NCTA = Cfg::NCTA;
    constexpr int PREFETCH = 3 * NCH;  // chunks between the L2 prefetch of a box and its load (three steps)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sW = base;                                   // W2 lo plane, one box per k chunk (H = 256 only)
    unsigned char* sA = sW + Cfg::W_BYTES;                      // [STAGES][PL] boxes
    unsigned char* sD = sA + STAGES * Cfg::A_STAGE;             // dh1^T tile: [plane][env half] boxes
    unsigned char* sO = sD + Cfg::D_TILE;                       // one-hot tile, two boxes of 64 cells
    unsigned char* sG = sO + Cfg::O_TILE;                       // gate tile, two boxes of 64 units
    uint64_t* bars = (uint64_t*)(sG + Cfg::G_TILE);
    uint64_t* full = bars;                  // [STAGES]
    uint64_t* empty = full + STAGES;        // [STAGES]
    uint64_t* tfull = empty + STAGES;       // [2] dh1 accumulator written
    uint64_t* tempty = tfull + 2;           // [2] dh1 accumulator drained (the epilogue warps arrive)
    uint64_t* wfull = tempty + 2;           // W2 rows are in tensor memory (the epilogue warps arrive) and its lo boxes have landed
    uint64_t* tiles_full = wfull + 1;       // operand tiles of a step written (every epilogue thread arrives)
    uint64_t* tiles_free = tiles_full + 1;  // the agent MMAs that read them have finished
    uint64_t* gfull = tiles_free + 1;       // gate tile landed
    uint64_t* gempty = gfull + 1;           // gate tile read (the epilogue warps arrive)
    uint64_t* wstage = gempty + 1;          // the W2 rows bound for tensor memory have landed in their staging boxes
    uint32_t* tmem_slot = (uint32_t*)(wstage + 1);

    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int B = d.B, T = a.T, C = d.C;
    const uint32_t rank = PAIR ? tc::cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    const int xi = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, nx = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;  // tile walker
    const int n0 = PAIR ? (int)rank * BN : (int)blockIdx.y * BN;
    const int m_tiles = (B + BM - 1) / BM;
    int* status = b.status;
    const int tl = (T + a.ts - 1) / a.ts;  // this CTA's slice of the steps
    const int t0 = blockIdx.z * tl, t1 = min(T, t0 + tl);
    const int nsteps = t1 > t0 ? t1 - t0 : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&tfull[i], 1);
            tc::mbar_init(&tempty[i], NCTA * Cfg::EPI_WARPS);  // (the leader's copy collects both CTAs' arrivals)
        }
        tc::mbar_init(wfull, NCTA * Cfg::EPI_WARPS + (Cfg::W_LO_SMEM ? 1 : 0));  // (+ the producer's expect_tx arrival)
        tc::mbar_init(tiles_full, NCTA * Cfg::EPI_WARPS);
        tc::mbar_init(tiles_free, 1);
        tc::mbar_init(gfull, 1);
        tc::mbar_init(gempty, Cfg::EPI_WARPS);
        tc::mbar_init(wstage, 1);
        tc::mbar_fence_init();
    }
    if (wid == 2) {
        if (PAIR) tc::tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
        else tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    }
    // the one-hot tile starts all zero; every step clears the elements it set the step before
    for (int i = tid; i < Cfg::O_TILE / 16; i += Cfg::THREADS) reinterpret_cast<uint4*>(sO)[i] = make_uint4(0u, 0u, 0u, 0u);
    tc::fence_proxy_async();
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (PAIR) tc::cluster_sync_all();  // both CTAs' barriers exist before either signals the other
    const uint32_t tmem = *tmem_slot;
    const uint32_t acc_agent = tmem + (uint32_t)Cfg::AGENT_COL;
    int my_tiles = 0;  // env tiles this CTA walks
    for (int mt = xi; mt < m_tiles; mt += nx) ++my_tiles;
    const int G = my_tiles * nsteps;  // steps of this CTA, all env tiles together (the pipelines run across tiles)
    bool ok = true;
    // first row (t*B + env) of running step g
    auto row_of = [&](int g) { return (t0 + g % nsteps) * B + (xi + (g / nsteps) * nx) * BM; };
    // arrival on / wait for a barrier of the leader CTA (pair: the peer's arrivals cross the cluster)
    // (release at CTA scope: what these arrivals publish is this warp's finished tensor-memory accesses and its stores to
    // its own CTA's shared memory; a cluster-scope release costs well over a thousand clocks per arrival)
    auto arrive_leader = [&](uint64_t* bar) {
        if (PAIR) tc::mbar_arrive_remote_cta_release(tc::mapa(tc::smem_u32(bar), 0));
        else tc::mbar_arrive(bar);
    };
    auto wait_leader = [&](uint64_t* bar, uint32_t parity) { return PAIR ? tc::mbar_wait_cluster(bar, parity) : tc::mbar_wait(bar, parity); };
    auto commit = [&](uint64_t* bar) {  // ... of the MMAs issued so far, to this barrier in every CTA of the pair
        if (PAIR) tc::umma_commit_pair(bar, 3);
        else tc::umma_commit(bar);
    };

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer: this CTA's rows of W2 once, then the dh2 boxes
            if (Cfg::W_STAGED) {  // the planes bound for tensor memory: box [plane][k chunk] in the dh1^T tile
                tc::mbar_expect_tx(wstage, Cfg::WT_PL * NCH * Cfg::W_BOX);
#pragma unroll
                for (int pl = 0; pl < Cfg::WT_PL; ++pl)
#pragma unroll
                    for (int kc = 0; kc < NCH; ++kc) tc::tma_load_2d(sD + (pl * NCH + kc) * Cfg::W_BOX, pl ? &maps.w_lo : &maps.w_hi, wstage, kc * KC, n0);
            }
            if (Cfg::W_LO_SMEM) {
                if (leader) tc::mbar_expect_tx(wfull, NCTA * Cfg::W_BYTES);  // the boxes of both CTAs
                const uint32_t bar = tc::mapa(tc::smem_u32(wfull), 0);
#pragma unroll
                for (int kc = 0; kc < NCH; ++kc) {
                    if (PAIR) tc::tma_load_2d_pair(sW + kc * Cfg::W_BOX, &maps.w_lo, bar, kc * KC, n0);
                    else tc::tma_load_2d(sW + kc * Cfg::W_BOX, &maps.w_lo, wfull, kc * KC, n0);
                }
            }
            for (int c = 0; c < G * NCH && ok; ++c) {
                const int s = c % STAGES, g = c / NCH, kc = c - g * NCH;
                {   // pull the boxes of a later chunk towards L2 now, so that their TMA load is an L2 hit
                    const int cp = c + PREFETCH;
                    if (cp < G * NCH) {
                        const int gp = cp / NCH, kp = cp - gp * NCH;
                        tc::tma_prefetch_2d(&maps.a_hi, kp * KC, row_of(gp) + Cfg::ROWS * (int)rank);
                        if (PL == 2) tc::tma_prefetch_2d(&maps.a_lo, kp * KC, row_of(gp) + Cfg::ROWS * (int)rank);
                    }
                }
                if (c >= STAGES) ok = tc::mbar_wait(&empty[s], ((c / STAGES) - 1) & 1);
                if (!ok) break;
                if (leader) tc::mbar_expect_tx(&full[s], NCTA * Cfg::A_STAGE);  // the loads of both CTAs
                // rows t*B + e0 .. +127 of the dh2 planes (rows past the batch end belong to the next step or are
                // zero-filled past the last row; their results are discarded by the epilogue)
                const int row = row_of(g) + Cfg::ROWS * (int)rank;
                if (PAIR) {
                    const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);
                    tc::tma_load_2d_pair(sA + s * Cfg::A_STAGE, &maps.a_hi, bar, kc * KC, row);
                    if (PL == 2) tc::tma_load_2d_pair(sA + s * Cfg::A_STAGE + Cfg::A_BOX, &maps.a_lo, bar, kc * KC, row);
                } else {
                    tc::tma_load_2d(sA + s * Cfg::A_STAGE, &maps.a_hi, &full[s], kc * KC, row);
                    if (PL == 2) tc::tma_load_2d(sA + s * Cfg::A_STAGE + Cfg::A_BOX, &maps.a_lo, &full[s], kc * KC, row);
                }
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0 && leader) {  // ---- MMA issuer (of the pair)
            const uint32_t idesc = tc::umma_idesc<PREC>(NCTA * BN, BM, false, false);
            const uint32_t idesc_agent = tc::umma_idesc<PREC>(NCTA * BN, 128, false, true);
            // agent-plane product of step v: 8 k16 steps over the 128 envs per plane of dh1 (the one-hot is exact)
            auto agent_mma = [&](int v) {
                ok = wait_leader(tiles_full, (uint32_t)v & 1u);
                if (!ok) return;
                tc::tc_fence_after();
#pragma unroll
                for (int pl = 0; pl < PL; ++pl) {
#pragma unroll
                    for (int k16 = 0; k16 < BM / 16; ++k16) {
                        // dh1^T (K-major): env half k16/4, 32 bytes per k16 along the swizzled rows; one-hot (MN-major): 16
                        // env rows = 2048 bytes further, cells 64.. one box further
                        const uint64_t dd = tc::umma_desc(sD + (pl * 2 + (k16 >> 2)) * Cfg::D_BOX + (k16 & 3) * 32, 16, 1024);
                        const uint64_t od = tc::umma_desc(sO + k16 * 2048, BM * 128, 1024);
                        const uint32_t accum = (v > 0 || pl > 0 || k16 > 0) ? 1u : 0u;
                        if (PAIR) tc::umma_pair(acc_agent, dd, od, idesc_agent, accum);
                        else tc::umma(acc_agent, dd, od, idesc_agent, accum);
                    }
                }
                commit(tiles_free);
            };
            ok = wait_leader(wfull, 0);
            for (int u = 0; u < G && ok; ++u) {
                const int buf = u & 1;
                if (u >= 2) ok = wait_leader(&tempty[buf], (uint32_t)((u >> 1) - 1) & 1u);  // the epilogues of step u-2 have drained it
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + (uint32_t)(Cfg::ACC_COL + 128 * buf);
                for (int kc = 0; kc < NCH && ok; ++kc) {
                    const int c = u * NCH + kc, s = c % STAGES;
                    ok = tc::mbar_wait(&full[s], (c / STAGES) & 1);
                    if (!ok) break;
                    tc::tc_fence_after();
                    unsigned char* sa = sA + s * Cfg::A_STAGE;
#pragma unroll
                    for (int k16 = 0; k16 < KC / 16; ++k16) {
                        // W2 rows in tensor memory: 16 k = 8 columns; dh2 (K-major): 16 k = 32 bytes along the swizzled rows
                        const uint32_t w_hi = tmem + (uint32_t)(kc * (KC / 2) + k16 * 8);
                        const uint64_t d_hi = tc::umma_desc(sa + k16 * 32, 16, 1024);
                        const uint32_t accum = (kc > 0 || k16 > 0) ? 1u : 0u;
                        // Order of the three terms: two MMAs in a row that read the SAME rows of tensor memory as their A operand
                        // measured a quarter slower than with the W lo term between them.
                        if (PAIR) {
                            tc::umma_pair_ta(acc, w_hi, d_hi, idesc, accum);  // W hi x dh2 hi
                            if (PL == 2) {
                                // W lo x dh2 hi, the lo rows from shared memory
                                if (Cfg::W_LO_SMEM) tc::umma_pair(acc, tc::umma_desc(sW + kc * Cfg::W_BOX + k16 * 32, 16, 1024), d_hi, idesc, 1u);
                                else tc::umma_pair_ta(acc, w_hi + (uint32_t)(H / 2), d_hi, idesc, 1u);
                                tc::umma_pair_ta(acc, w_hi, tc::umma_desc(sa + Cfg::A_BOX + k16 * 32, 16, 1024), idesc, 1u);  // W hi x dh2 lo
                            }
                        } else {
                            tc::umma_ta(acc, w_hi, d_hi, idesc, accum);
                            if (PL == 2) {
                                if (Cfg::W_LO_SMEM) tc::umma(acc, tc::umma_desc(sW + kc * Cfg::W_BOX + k16 * 32, 16, 1024), d_hi, idesc, 1u);
                                else tc::umma_ta(acc, w_hi + (uint32_t)(H / 2), d_hi, idesc, 1u);
                                tc::umma_ta(acc, w_hi, tc::umma_desc(sa + Cfg::A_BOX + k16 * 32, 16, 1024), idesc, 1u);
                            }
                        }
                    }
                    commit(&empty[s]);
                }
                if (!ok) break;
                commit(&tfull[buf]);
                if (u >= 1) agent_mma(u - 1);  // queued behind this step's product: the tensor pipe stays busy
            }
            if (ok && G > 0) agent_mma(G - 1);
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 2) {
        if (lane == 0) {  // ---- TMA producer of the gate tiles (rows as for dh2, units n0 .. n0+127 of the h1 hi plane)
            for (int g = 0; g < G && ok; ++g) {
                if (g + 2 < G) tc::tma_prefetch_2d(&maps.gate, n0 / 8, row_of(g + 2));
                if (g >= 1) ok = tc::mbar_wait(gempty, (uint32_t)(g - 1) & 1u);
                if (!ok) break;
                tc::mbar_expect_tx(gfull, Cfg::G_TILE);
                tc::tma_load_2d(sG, &maps.gate, gfull, n0 / 8, row_of(g));  // (x in bytes: 0 or 16)
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- epilogue warps: thread = hidden unit j (accumulator lane 32*(wid%4) + lane) x 64 of the tile's 128 envs
        const int q = wid & 3, j = 32 * q + lane, half = (wid - Cfg::FIRST_EPI) >> 2;
        const uint32_t lane_base = (uint32_t)(32 * q) << 16;
        {   // This CTA's rows of W2 go into tensor memory once: row n0 + j = lane j, two k per column (they are stored
            // that way), the hi plane in columns [0, H/2), the lo plane behind it.  The two warps of a lane quarter share the columns.
            // The rows come through shared memory (TMA boxes of 64 k, 128-byte swizzle): k chunk kc of row j is the 128
            // bytes at box kc, row j, its 16-byte pieces permuted by j % 8.
            if (!Cfg::W_STAGED) {  // (no room to stage them: straight from global memory)
#pragma unroll 1
                for (int pl = 0; pl < Cfg::WT_PL; ++pl) {
                    const uint32_t* wrow = reinterpret_cast<const uint32_t*>((pl ? b.w2p_lo : b.w2p_hi) + (size_t)(n0 + j) * H) + half * (H / 4);
#pragma unroll 1
                    for (int cc = 0; cc < H / 128; ++cc) {
                        uint32_t r[32];
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const uint4 v = __ldg(reinterpret_cast<const uint4*>(wrow + 32 * cc + c));
                            r[c] = v.x; r[c + 1] = v.y; r[c + 2] = v.z; r[c + 3] = v.w;
                        }
                        tc::tmem_st32(tmem + lane_base + (uint32_t)(pl * (H / 2) + half * (H / 4) + 32 * cc), r);
                    }
                }
            } else if ((ok = tc::mbar_wait(wstage, 0))) {
#pragma unroll 1
                for (int pl = 0; pl < Cfg::WT_PL; ++pl) {
#pragma unroll
                    for (int cc = 0; cc < H / 128; ++cc) {  // 32 columns = 64 k = one box row
                        const int kc = half * (H / 128) + cc;
                        const unsigned char* row = sD + (pl * NCH + kc) * Cfg::W_BOX + j * 128;
                        uint32_t r[32];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = *reinterpret_cast<const uint4*>(row + ((c ^ (j & 7)) << 4));
                            r[4 * c] = v.x; r[4 * c + 1] = v.y; r[4 * c + 2] = v.z; r[4 * c + 3] = v.w;
                        }
                        tc::tmem_st32(tmem + lane_base + (uint32_t)(pl * (H / 2) + kc * 32), r);
                    }
                }
            }
            tc::tmem_st_wait();
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) arrive_leader(wfull);
        }
        const uint8_t* gcol = sG + (j >> 3);  // the byte of unit j in a row of the gate box; its bit is j % 8
        const int gbit = j & 7;
        unsigned char* drow = sD + half * Cfg::D_BOX + j * 128;  // this thread's row of the dh1^T hi box of its env half
        int prev_off = -1;  // byte offset of the one-hot element this thread set the step before
        int g = 0;          // running step index of this CTA
        for (int mt = xi; mt < m_tiles && ok; mt += nx) {
            const int env0 = mt * BM + 64 * half;              // first env of this thread's half
            const int nvalid = min(64, max(0, B - env0));      // envs of the half that exist
            const int oh_env = mt * BM + j;                    // (half 0 only) the env whose one-hot row this thread keeps
            float s_acc[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) s_acc[i] = 0.f;
            for (int t = t0; t < t1; ++t, ++g) {
                const int cell = (half == 0 && oh_env < B) ? (int)b.tpos[(size_t)t * B + oh_env] : -1;
                const int buf = g & 1;
                if (ok) ok = tc::mbar_wait(&tfull[buf], (uint32_t)(g >> 1) & 1u);
                if (!ok) break;
                tc::tc_fence_after();
                uint32_t r0[32], r1[32];
                const uint32_t acc = tmem + lane_base + (uint32_t)(Cfg::ACC_COL + 128 * buf + 64 * half);
                tc::tmem_ld32_nowait(acc, r0);
                tc::tmem_ld32_nowait(acc + 32, r1);
                tc::tmem_ld_wait();
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_leader(&tempty[buf]);  // the issuer may overwrite this accumulator now
                ok = tc::mbar_wait(gfull, (uint32_t)g & 1u);
                // the operand tiles are free once the agent MMAs of the step before have finished
                if (ok && g >= 1) ok = tc::mbar_wait(tiles_free, (uint32_t)(g - 1) & 1u);
                if (!ok) break;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {  // 16-byte chunks of 8 envs
                    uint32_t phi[4], plo[4];
#pragma unroll
                    for (int p2 = 0; p2 < 4; ++p2) {
                        const int i = 8 * c8 + 2 * p2;  // envs i, i+1 of the half; gate bit (env row, unit j) of the gate box
                        const int e_a = 64 * half + i, e_b = e_a + 1;
                        const uint32_t ga = (uint32_t)gcol[e_a * (BN / 8)] >> gbit;
                        const uint32_t gb = (uint32_t)gcol[e_b * (BN / 8)] >> gbit;
                        const float x0 = __uint_as_float(i < 32 ? r0[i] : r1[i - 32]);
                        const float x1 = __uint_as_float(i < 32 ? r0[i + 1] : r1[i - 31]);
                        // rows past the batch end are another step's
                        const float v0 = rnd<PREC>((i < nvalid && (ga & 1u)) ? x0 : 0.f);
                        const float v1 = rnd<PREC>((i + 1 < nvalid && (gb & 1u)) ? x1 : 0.f);
                        s_acc[i] += v0;
                        s_acc[i + 1] += v1;
                        split2<PREC>(v0, v1, phi[p2], plo[p2]);
                    }
                    // element (m = unit j, k = env) of the K-major box: byte j*128 + ((k/8) ^ (j%8))*16 + (k%8)*2
                    const int off = (c8 ^ (j & 7)) << 4;
                    *reinterpret_cast<uint4*>(drow + off) = make_uint4(phi[0], phi[1], phi[2], phi[3]);
                    if (PL == 2) *reinterpret_cast<uint4*>(drow + 2 * Cfg::D_BOX + off) = make_uint4(plo[0], plo[1], plo[2], plo[3]);
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(gempty);  // the gate tile may be overwritten
                if (prev_off >= 0) *reinterpret_cast<uint16_t*>(sO + prev_off) = 0;
                prev_off = -1;
                if (cell >= 0 && cell < 128 && (!PAIR || (uint32_t)(cell >> 6) == rank)) {  // (pair: this CTA holds the box of its 64 cells)
                    // element (k = env j, n = cell) of the MN-major tile: byte k*128 + ((n/8) ^ (k%8))*16 + (n%8)*2
                    prev_off = (PAIR ? 0 : (cell >> 6) * (BM * 128)) + j * 128 + ((((cell & 63) >> 3) ^ (j & 7)) << 4) + (cell & 7) * 2;
                    *reinterpret_cast<uint16_t*>(sO + prev_off) = (uint16_t)one16<PREC>();
                }
                tc::fence_proxy_async();  // generic-proxy stores -> visible to the tensor cores
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) tc::mbar_arrive_remote_cta_release(tc::mapa(tc::smem_u32(tiles_full), 0));
                    else tc::mbar_arrive(tiles_full);
                }
            }
            // S (sum over t of dh1) as two 16-bit planes [ts*B][H]: an fp32 sum keeps two terms in either workload
            if (ok) {
                uint16_t* S_hi = reinterpret_cast<uint16_t*>(b.S);
                uint16_t* S_lo = S_hi + (size_t)a.ts * B * H;
                const size_t si = ((size_t)blockIdx.z * B + env0) * H + n0 + j;  // an empty slice writes zeros
#pragma unroll
                for (int i = 0; i < 64; ++i) {
                    if (i < nvalid) {
                        uint16_t hi, lo;
                        if (PREC == 1) {
                            __nv_bfloat16 h0, l0;
                            split_bf16(s_acc[i], h0, l0);
                            hi = __bfloat16_as_ushort(h0);
                            lo = __bfloat16_as_ushort(l0);
                        } else {
                            split1<0>(s_acc[i], hi, lo);
                        }
                        S_hi[si + (size_t)i * H] = hi;
                        S_lo[si + (size_t)i * H] = lo;
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        // agent-plane partial of this (env tile, t slice): accumulator lane = unit, column = cell
        bool got = ok;
        if (got && G > 0) got = tc::mbar_wait(tiles_free, (uint32_t)(G - 1) & 1u);
        if (!got && ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        tc::tc_fence_after();
        __syncwarp();
        float* part = part_agent + (size_t)(blockIdx.z * nx + xi) * part_stride + n0 + j;
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t r[32];
            if (got && G > 0) {
                tc::tmem_ld32(acc_agent + lane_base + (uint32_t)(64 * half + c0), r);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = 0u;  // an empty slice contributes zeros
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int cell = 64 * half + c0 + i;
                if (cell < C) part[(size_t)cell * H] = __uint_as_float(r[i]);
            }
        }
    }
    // (pair) neither CTA leaves or frees tensor memory while the other may still signal it or run MMAs that touch it
    tc::tc_fence_before();
    __syncthreads();
    if (PAIR) tc::cluster_sync_all();
    if (wid == 2) {
        if (PAIR) tc::tmem_dealloc_pair(tmem, Cfg::TMEM_COLS);
        else tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
    }
}

template <int H, int PREC>
__global__ void __launch_bounds__(Dh1aCfg<H, PREC>::THREADS, 1)
    k_dh1a_tc(const __grid_constant__ Dh1aMaps maps, LearnArgs a, float* part_agent, size_t part_stride) {
    dh1a_body<H, PREC>(maps, a, part_agent, part_stride);
}
template <int H, int PREC>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Dh1aCfg<H, PREC>::THREADS, 1)
    k_dh1a_pair(const __grid_constant__ Dh1aMaps maps, LearnArgs a, float* part_agent, size_t part_stride) {
    dh1a_body<H, PREC>(maps, a, part_agent, part_stride);
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
    if (!make_tensor_map_2d(&maps.a_hi, dh2hi, R, H, Cfg::ROWS, bf)) return cudaErrorNotSupported;
    if (Cfg::PL == 2 && !make_tensor_map_2d(&maps.a_lo, dh2hi + RH, R, H, Cfg::ROWS, bf)) return cudaErrorNotSupported;
    if (!b.gate1 || !make_tensor_map_u8(&maps.gate, b.gate1, R, H / 8, 128, Cfg::BN / 8)) return cudaErrorNotSupported;
    if (!make_tensor_map_2d(&maps.w_hi, b.w2p_hi, H, H, 128, bf)) return cudaErrorNotSupported;
    if (Cfg::PL == 2 && !make_tensor_map_2d(&maps.w_lo, b.w2p_lo, H, H, 128, bf)) return cudaErrorNotSupported;
    if constexpr (Cfg::PAIR) {  // the two CTAs of a pair are neighbours in x; each pair takes all H units
        cudaError_t e = cudaFuncSetAttribute(k_dh1a_pair<H, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
        if (e != cudaSuccess) return e;
        k_dh1a_pair<H, PREC><<<dim3(2 * grid_x, 1, a.ts), Cfg::THREADS, Cfg::smem_bytes, s>>>(maps, a, part_agent, part_stride);
    } else {
        cudaError_t e = cudaFuncSetAttribute(k_dh1a_tc<H, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
        if (e != cudaSuccess) return e;
        k_dh1a_tc<H, PREC><<<dim3(grid_x, H / Cfg::BN, a.ts), Cfg::THREADS, Cfg::smem_bytes, s>>>(maps, a, part_agent, part_stride);
    }
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
