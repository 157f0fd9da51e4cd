// Learning half of the Anakin minimal unit on the tensor pipe (Podracer paper, Section 3.1; Figure 2, top), for the
// hidden sizes the tensor-pipe rollout covers.  The update reuses the policy's forward pass (Section 3.1): the rollout
// kernel saved h1 (as bf16 hi/lo planes) and h2 for every recorded row, so the learner starts at the heads.
//
//   k_heads_bwd   flat 32-row tiles: saved head outputs -> softmax / loss terms -> dOut -> dh2 (fp32 FMA, HBM-bound).
//                 Emits dh2 as 16-bit hi/lo planes and per-CTA partial sums of dWh, dbh, db2 and the loss terms.
//                 At hidden width 256 (few enough rows per CTA) it also takes dW2 = h1^T dh2 for its rows: the dh2 tile it
//                 has just computed and the matching h1 tile (TMA) are the operands of tcgen05 MMAs into tensor memory,
//                 so dh2 is not read back for that product and the stand-alone dW2 GEMM is not launched.
//   k_dh1         dh1 = (dh2 W2^T) gated by h1 > 0 with mma.sync; a CTA keeps its slice of W2 in shared memory and
//                 walks t for 64 envs, so S = sum_t dh1 accumulates in registers.  Emits dh1 planes and S planes.
//   k_gemm_tn     C[m][n] = sum_k A[k][m] B[k][n] with split-K partial outputs, bf16 hi/lo planes as operands and
//                 three MMAs per product (two when A is an exact 0/1 plane, one in the bf16 workload):
//                 dW2 = h1^T dh2 (K = B*T), dW1[agent plane] = X^T dh1 (K = B*T), dW1[wall, goal planes] = X^T S
//                 (K = B; an extra all-ones row of A yields db1 = sum_b S[b]).
//   k_reduce_adam2  fixed-order sum of every region's partials (= the batch-mean gradient, the single-device form of
//                 the paper's cross-core average), Adam, loss statistics.
// No floating-point atomics: every sum has a fixed order, so runs are bitwise reproducible.
#include "tc_common.cuh"

namespace anakin {

// ----------------------------------------------------------------------------------------------------
// k_heads_bwd: softmax, loss terms, output gradients and dh2 for flat 32-row tiles (row i = t*B + env).
// The head outputs (4 logits, value) of every row were saved by the rollout, so no h2 x Wh pass is needed here.
// Persistent CTAs walk the tiles with a double-buffered cp.async stream of h2.  Per tile, every thread handles two
// adjacent hidden units of 8 rows (dh2, running sums of dWh and db2) and then, for the NEXT tile, one thread per row
// turns the saved head outputs into output gradients, so that the two phases of different warps overlap and one CTA
// barrier per tile suffices.  HBM-bound in principle: reads h2 (4 B/elt), writes the dh2 planes (2 x 2 B/elt).
// ----------------------------------------------------------------------------------------------------
// HS = width of the column slab one CTA covers (blockIdx.y picks the slab; HS = H for H <= 256); H2BF: h2 is stored as
// bf16 (the wide bf16 path) instead of fp32.
// FUSE (H = 256 only): the kernel also takes dW2 = h1^T dh2 for its rows on the tcgen05 pipe (see k_heads_bwd).
template <int H, int NW, int PREC, int HS = H, bool H2BF = false, bool FUSE = false>
struct HeadsCfg {
    static constexpr int TR = 32;  // rows per tile
    static constexpr int ESZ = H2BF ? 2 : 4;
    // the widest slab (32 KB tiles, 17 warps) runs one CTA per SM with a deep ring; the narrower ones two CTAs per SM
    static constexpr int PER_SM = TR * HS * ESZ >= 32768 ? 1 : 2;
    static constexpr int PL = PREC == 1 ? 1 : 2;
    static constexpr int BOX = TR * 128;                     // 32 rows x 64 16-bit elements, MN-major (4 KB)
    static constexpr int OP_TILE = PL * (H / 64) * BOX;      // one operand tile: [plane][64-column box]
    // two dh2 tiles; two h1 tiles where a CTA has the SM to itself, one where two CTAs share it (H = 128).  The shared
    // array is declared 128-byte aligned, so 896 bytes reach the next 1024-byte boundary.
    static constexpr int A_BUFS = PER_SM == 1 ? 2 : 1;
    static constexpr int TMEM_COLS = (H / 128) * H >= 512 ? 512 : (H / 128) * H;  // H/128 accumulators of 128 lanes x H columns
    static constexpr int FUSE_BYTES = FUSE ? (2 + A_BUFS) * OP_TILE + 896 /*alignment slack*/ + 64 /*barriers, tmem slot*/ : 0;
    static_assert(((size_t)FUSE_BYTES + (size_t)(FUSE ? 3 : 0) * TR * HS * ESZ + 2 * TR * 8 * 4 + 64) * PER_SM <= 232448, "shared memory of the fused kernel");
    static constexpr int NST = FUSE ? 3 : (PER_SM == 1 ? 6 : 4);  // depth of the h2 ring (tiles in flight = NST - 1)
    static constexpr int THREADS = NW * 32 + 32 + (FUSE ? 32 : 0);
    // FUSE, fp32 workloads: the accumulators are read out and restarted every GROUP tiles (4096 rows): the tensor core's own
    // accumulation rounds toward zero, which shows as a bias on longer sums; the groups are added with round-to-nearest
    static constexpr int GROUP = PREC == 1 ? (1 << 30) : 128;
    static constexpr size_t smem_bytes = (size_t)FUSE_BYTES + (size_t)NST * TR * HS * ESZ + (size_t)2 * TR * 8 * 4 + 64 /*barriers*/;
};

struct HeadsMaps {
    CUtensorMap h1_hi, h1_lo;  // FUSE: the h1 planes [R][H], boxes of 64 columns x 32 rows
};

template <int H, int NW, int PREC, int HS = H, bool H2BF = false, bool GROUPED = false, bool FUSE = false>
__global__ void __launch_bounds__((HeadsCfg<H, NW, PREC, HS, H2BF, FUSE>::THREADS), (HeadsCfg<H, NW, PREC, HS, H2BF, FUSE>::PER_SM))
    k_heads_bwd(LearnArgs a_in, const __grid_constant__ HeadsMaps maps) {
    const PolicyArgs<GROUPED, LearnArgs> pa(a_in, blockIdx.z);  // many policies: grid.z = policy
    const LearnArgs& a = pa.a;
    using Cfg = HeadsCfg<H, NW, PREC, HS, H2BF, FUSE>;
    constexpr int TR = Cfg::TR, NTHREADS = NW * 32, HP2 = HS / 2, ESZ = Cfg::ESZ, NST = Cfg::NST;
    static_assert(NTHREADS / HP2 == 4, "four row groups of eight rows");
    static_assert(!FUSE || (HS == H && (H == 128 || H == 256) && !H2BF && !GROUPED), "the fused dW2 product is built for the 128- and 256-wide fp32-h2 kernels");
    extern __shared__ __align__(128) unsigned char heads_smem[];
    // FUSE: the operand tiles of the dW2 MMAs first (1024-byte aligned for the 128-byte swizzle): dh2 tiles [2], h1 tiles [2]
    unsigned char* fbase = (unsigned char*)(((uintptr_t)heads_smem + 1023) & ~(uintptr_t)1023);
    unsigned char* s_t = fbase;                                  // dh2 tile, written by the column warps
    unsigned char* s_a = s_t + 2 * Cfg::OP_TILE;                 // h1 tile, by TMA
    uint64_t* fbars = reinterpret_cast<uint64_t*>(s_a + Cfg::A_BUFS * Cfg::OP_TILE);  // t_ready[2], a_full[2], mma_done[2], epi_done
    uint64_t* t_ready = fbars;
    uint64_t* a_full = fbars + 2;
    uint64_t* mma_done = fbars + 4;
    uint64_t* epi_done = fbars + 6;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(fbars + 7);
    unsigned char* s_h2 = FUSE ? fbase + (2 + Cfg::A_BUFS) * Cfg::OP_TILE + 64 : heads_smem;  // [NST][TR][HS] fp32 or bf16
    float* s_dout = reinterpret_cast<float*>(s_h2 + (size_t)NST * TR * HS * ESZ);  // [2][TR][8]
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_dout + 2 * TR * 8);              // full[2], empty[2]
    uint64_t* full = bars;
    uint64_t* empty = bars + 2;
    const int c_base = blockIdx.y * HS;  // first hidden unit of this CTA's slab
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x;
    const size_t R = (size_t)d.B * a.T;
    const size_t RH = (size_t)d.B * d.Tmax * H;
    const int ntiles = (int)((R + TR - 1) / TR);
    if (tid == 0) {
        for (int q = 0; q < 2; ++q) { tc::mbar_init(&full[q], 1); tc::mbar_init(&empty[q], NW); }
        if (FUSE) {
            for (int q = 0; q < 2; ++q) { tc::mbar_init(&t_ready[q], NW); tc::mbar_init(&a_full[q], 1); tc::mbar_init(&mma_done[q], 1); }
            tc::mbar_init(epi_done, NW);
        }
        tc::mbar_fence_init();
    }
    if (FUSE && tid >= NTHREADS + 32) tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);  // H/128 accumulators of 128 x H: dW2 rows 128 m .. +127
    if (FUSE) tc::tc_fence_before();
    __syncthreads();
    if (FUSE) tc::tc_fence_after();
    bool ok = true;
    const int my_its = (ntiles > (int)blockIdx.x) ? (ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;  // tiles of this CTA

    if (FUSE && tid >= NTHREADS + 32) {
        // ---- the MMA warp (one lane): per tile, dW2[i][j] += sum over the tile's 32 rows of h1[r][i] dh2[r][j] with the h1
        // tile (TMA, MN-major boxes) as A and the dh2 tile the column warps wrote as B; both are double-buffered.
        const uint32_t tmem = *tmem_slot;
        if (tid == NTHREADS + 32) {
            constexpr int PL = Cfg::PL;
            const uint32_t idesc = tc::umma_idesc<PREC>(128, H, true, true);
            constexpr int AB = Cfg::A_BUFS;
            auto load_h1 = [&](int it) {
                const int buf = it % AB, row = ((int)blockIdx.x + it * (int)gridDim.x) * TR;
                tc::mbar_expect_tx(&a_full[buf], Cfg::OP_TILE);
#pragma unroll
                for (int bx = 0; bx < H / 64; ++bx) {
                    tc::tma_load_2d(s_a + buf * Cfg::OP_TILE + bx * Cfg::BOX, &maps.h1_hi, &a_full[buf], 64 * bx, row);
                    if (PL == 2) tc::tma_load_2d(s_a + buf * Cfg::OP_TILE + (H / 64 + bx) * Cfg::BOX, &maps.h1_lo, &a_full[buf], 64 * bx, row);
                }
            };
            for (int q = 0; q < AB; ++q)
                if (my_its > q) load_h1(q);
            for (int it = 0; it < my_its && ok; ++it) {
                const int buf = it & 1, abuf = it % AB;
                const uint32_t ph = (uint32_t)(it >> 1) & 1u;
                ok = tc::mbar_wait(&a_full[abuf], (uint32_t)(it / AB) & 1u);
                if (ok) ok = tc::mbar_wait(&t_ready[buf], ph);
                if (!ok) break;
                tc::tc_fence_after();
                const unsigned char* ta = s_a + abuf * Cfg::OP_TILE;
                const unsigned char* tb = s_t + buf * Cfg::OP_TILE;
#pragma unroll
                for (int k16 = 0; k16 < TR / 16; ++k16) {
                    // MN-major operands: 16 k rows = 2048 bytes into each box, consecutive 64-wide boxes one box apart
                    const uint64_t b_hi = tc::umma_desc(tb + k16 * 2048, Cfg::BOX, 1024);
                    const uint64_t b_lo = tc::umma_desc(tb + (H / 64) * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
#pragma unroll
                    for (int m = 0; m < H / 128; ++m) {  // rows (units of h1) 128 m .. +127 of dW2
                        const uint64_t a_hi = tc::umma_desc(ta + 2 * m * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024);
                        const uint32_t acc = tmem + (uint32_t)(m * H);
                        uint32_t accum = (it % Cfg::GROUP > 0 || k16 > 0) ? 1u : 0u;  // (a group's first MMA restarts the sum)
                        if (PL == 2) {
                            tc::umma(acc, tc::umma_desc(ta + (H / 64 + 2 * m) * Cfg::BOX + k16 * 2048, Cfg::BOX, 1024), b_hi, idesc, accum);  // lo x hi
                            tc::umma(acc, a_hi, b_lo, idesc, 1u);                                                                        // hi x lo
                            accum = 1u;
                        }
                        tc::umma(acc, a_hi, b_hi, idesc, accum);
                    }
                }
                tc::umma_commit(&mma_done[buf]);
                if (it + AB < my_its) {  // refill this h1 buffer once the MMAs that read it have finished
                    ok = tc::mbar_wait(&mma_done[buf], ph);
                    if (ok) load_h1(it + AB);
                }
            }
            if (!ok) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
        }
        // tensor memory is freed once every column warp has read its part of the accumulators
        __syncwarp();
        const bool got = tc::mbar_wait(epi_done, 0);
        if (!got && tid == NTHREADS + 32) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
        return;
    }
    if (tid >= NTHREADS) {
        // ---- the row warp: lane = row of a tile.  It runs ahead of the column warps: the saved head outputs of a row
        // (and its advantage, return and action) become the five output gradients, written to one of two small buffers
        // that the column warps consume a tile later; the loads are requested three tiles ahead of their use.
        const int rr = tid - NTHREADS;
        const float invR = a.gscale / (float)R;  // output gradients are carried times gscale
        float a_bh[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
        float l_pg = 0.f, l_v = 0.f, l_ent = 0.f;
        struct RowIn { float4 o4; float v, adv, ret, lpo; int act; bool ok; };
        auto row_load = [&](int tile) {
            RowIn in;
            const size_t i = (size_t)tile * TR + rr;
            in.ok = tile < ntiles && i < R;
            if (in.ok) {
                in.o4 = *reinterpret_cast<const float4*>(b.out5 + i * 8);
                in.v = b.out5[i * 8 + 4];
                in.adv = b.adv[i];
                in.lpo = a.ppo_clip > 0.f ? b.tlogp[i] : 0.f;
                in.ret = b.ret[i];
                in.act = b.tact[i];
            } else {
                in.o4 = make_float4(0.f, 0.f, 0.f, 0.f);
                in.v = in.adv = in.ret = in.lpo = 0.f;
                in.act = 0;
            }
            return in;
        };
        struct RowOut { float dO[5]; };
        auto row_compute = [&](const RowIn& in) {
            RowOut out;
#pragma unroll
            for (int c = 0; c < 5; ++c) out.dO[c] = 0.f;
            if (in.ok) {
                const float o[4] = {in.o4.x, in.o4.y, in.o4.z, in.o4.w};
                const float mx = fmaxf(fmaxf(o[0], o[1]), fmaxf(o[2], o[3]));
                float ex[4], Z = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) { ex[c] = expf(o[c] - mx); Z += ex[c]; }
                const float logZ = logf(Z);
                float p[4], lp[4], ent = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) { p[c] = ex[c] / Z; lp[c] = (o[c] - mx) - logZ; ent -= p[c] * lp[c]; }
                const float A = in.adv;
                const float err = in.v - in.ret;
                const float pf = policy_term(A, in.act == 0 ? lp[0] : in.act == 1 ? lp[1] : in.act == 2 ? lp[2] : lp[3], in.lpo, a.ppo_clip, l_pg);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    out.dO[c] = rnd<PREC>((-A * pf * ((c == in.act ? 1.f : 0.f) - p[c]) + a.c_e * p[c] * (lp[c] + ent)) * invR);
                out.dO[4] = rnd<PREC>(2.f * a.c_v * err * invR);
                l_v += err * err;
                l_ent += ent;
#pragma unroll
                for (int c = 0; c < 5; ++c) a_bh[c] += out.dO[c];
            }
            return out;
        };
        const int g = (int)gridDim.x;
        RowIn in0 = row_load(blockIdx.x), in1 = row_load(blockIdx.x + g), in2 = row_load(blockIdx.x + 2 * g);
        int it = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += g, ++it) {
            const int buf = it & 1;
            const RowIn in3 = row_load(tile + 3 * g);
            const RowOut out = row_compute(in0);
            if (it >= 2 && ok) ok = tc::mbar_wait(&empty[buf], ((it >> 1) - 1) & 1);  // the column warps are done with this buffer
            float4* o4 = reinterpret_cast<float4*>(s_dout + (buf * TR + rr) * 8);
            o4[0] = make_float4(out.dO[0], out.dO[1], out.dO[2], out.dO[3]);
            o4[1] = make_float4(out.dO[4], 0.f, 0.f, 0.f);
            __syncwarp();
            if (rr == 0) tc::mbar_arrive(&full[buf]);
            in0 = in1; in1 = in2; in2 = in3;
        }
        // dbh and the loss terms of this CTA: a fixed shuffle tree over the lanes (the first slab's CTAs only)
        float vals[8] = {a_bh[0], a_bh[1], a_bh[2], a_bh[3], a_bh[4], l_pg, l_v, l_ent};
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) vals[c] += __shfl_xor_sync(0xFFFFFFFFu, vals[c], off);
        if (blockIdx.y == 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                if (rr == c) {
                    if (c < 5) {
                        for (int q = 0; q < 4; ++q) a.part_small[(size_t)(4 * blockIdx.x + q) * a.small_stride + (size_t)H * 6 + c] = q == 0 ? vals[c] : 0.f;
                    } else {
                        b.loss_part[(size_t)blockIdx.x * 4 + (c - 5)] = vals[c];
                    }
                }
            }
        }
        if (!ok && rr == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
        return;
    }

    // ---- the column warps: thread = (unit pair cp, row group rg of 8 rows)
    uint32_t* g_dh2hi = reinterpret_cast<uint32_t*>(b.dh2);  // pairs of 16-bit elements
    uint32_t* g_dh2lo = g_dh2hi + RH / 2;
    const int cp = tid % HP2, rg = tid / HP2;
    const int lane = tid & 31;
    float wh_c[2][5];
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
        for (int c = 0; c < 5; ++c) wh_c[cc][c] = b.theta_c[d.oWh + (c_base + 2 * cp + cc) * 5 + c];
    float a_wh[2][5], a_b2[2] = {0.f, 0.f};
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
        for (int c = 0; c < 5; ++c) a_wh[cc][c] = 0.f;

    // h2 tile loads: 16-byte chunks, zero-filled past the last row; a thread's chunks of one tile differ by a fixed number
    // of rows, so one address is formed per tile and the rest are constant offsets.  Always commits a group.
    constexpr int EPC = 16 / ESZ;             // elements per 16-byte chunk
    constexpr int CPR = HS / EPC;             // chunks per row
    constexpr int RPP = NTHREADS / CPR;       // rows per pass of the column warps
    static_assert(NTHREADS % CPR == 0 && TR % RPP == 0, "the tile must split into whole passes");
    const int l_r = tid / CPR, l_k = EPC * (tid % CPR);
    const unsigned char* src_base = reinterpret_cast<const unsigned char*>(b.h2) + (size_t)(c_base + l_k) * ESZ;
    auto load_tile = [&](int tile, int buf) {
        if (tile < ntiles) {
            const size_t row0 = (size_t)tile * TR + l_r;
            unsigned char* dst = s_h2 + ((size_t)(buf * TR + l_r) * HS + l_k) * ESZ;
            const unsigned char* src = src_base + row0 * H * ESZ;
#pragma unroll
            for (int j = 0; j < TR / RPP; ++j) {
                const bool okr = row0 + j * RPP < R;
                cp_async16(dst + (size_t)j * RPP * HS * ESZ, okr ? src + (size_t)j * RPP * H * ESZ : src_base, okr ? 16 : 0);
            }
        }
        cp_async_commit();
    };

    // FUSE: this CTA's partial of dW2.  Accumulator m, lane = row 128 m + lane of dW2, column = column of dW2; warp w reads
    // lane quarter w % 4 and the 64 columns of column group w / 4 (NW / 4 = H / 64 groups).  After tile `last` (the last of an
    // accumulator group): the first group writes the partial, every later one adds to what this same thread wrote.
    float* const w2part = FUSE ? const_cast<float*>(a_in.reg[4].part) + (size_t)blockIdx.x * H * H : nullptr;
    const int wq = (tid >> 5) & 3, cg = tid >> 7;
    auto dw2_out = [&](int last) -> bool {
        const bool got = tc::mbar_wait(&mma_done[last & 1], (uint32_t)(last >> 1) & 1u);
        if (!got && lane == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
        tc::tc_fence_after();
        const uint32_t tmem = *tmem_slot;
        const bool first = last / Cfg::GROUP == 0;
#pragma unroll 1
        for (int m = 0; m < H / 128; ++m) {
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t r[32];
                if (got) {
                    tc::tmem_ld32(tmem + ((uint32_t)(32 * wq) << 16) + (uint32_t)(m * H + 64 * cg + c0), r);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                float4* dst = reinterpret_cast<float4*>(w2part + (size_t)(128 * m + 32 * wq + lane) * H + 64 * cg + c0);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float4 v = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                    if (!first) {
                        const float4 o = dst[i];
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    dst[i] = v;
                }
            }
        }
        tc::tc_fence_before();
        return got;
    };
    auto dw2_zero = [&]() {  // a CTA without tiles contributes zeros
#pragma unroll 1
        for (int m = 0; m < H / 128; ++m)
            for (int i = 0; i < 16; ++i)
                reinterpret_cast<float4*>(w2part + (size_t)(128 * m + 32 * wq + lane) * H + 64 * cg)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    };
    int it = 0;
#pragma unroll
    for (int q = 0; q < NST - 1; ++q) load_tile(blockIdx.x + q * (int)gridDim.x, q);
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
        const int buf = it & 1;  // dOut buffer of this tile
        cp_async_wait<NST - 2>();
        // this tile's h2 is in place and every column warp is done with the stage that is refilled next (named barrier
        // 1: the column warps only); its output gradients come from the row warp
        asm volatile("bar.sync 1, %0;" ::"n"(NTHREADS) : "memory");
        load_tile(tile + (NST - 1) * (int)gridDim.x, (it + NST - 1) % NST);
        if (ok) ok = tc::mbar_wait(&full[buf], (it >> 1) & 1);
        // FUSE: this tile's dh2 also goes into operand tile `buf`, free once the MMAs of two tiles ago have read it
        if (FUSE && ok && it >= 2) ok = tc::mbar_wait(&mma_done[buf], ((it >> 1) - 1) & 1);
        // ---- dh2 = (dOut Wh^T) gated by h2 > 0, as 16-bit planes; running sums of dWh and db2
        const unsigned char* h2t = s_h2 + ((size_t)(it % NST) * TR + rg * 8) * HS * ESZ + (size_t)2 * cp * ESZ;
        const float* dt = s_dout + (buf * TR + rg * 8) * 8;
        const size_t i0 = (size_t)tile * TR + rg * 8;
        const int rows_left = i0 < R ? (int)((R - i0) < 8 ? (R - i0) : 8) : 0;
        uint32_t* o_hi = g_dh2hi + (i0 * H + c_base) / 2 + cp;
        uint32_t* o_lo = g_dh2lo + (i0 * H + c_base) / 2 + cp;
        const bool fullt = rows_left == 8;  // all but the last tile: stores without per-row predicates
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const float4 d0 = *reinterpret_cast<const float4*>(dt + r * 8);
            const float d0s[1][5] = {{d0.x, d0.y, d0.z, d0.w, dt[r * 8 + 4]}};
            float hv[2];
            if (H2BF) {
                const uint32_t pk = *reinterpret_cast<const uint32_t*>(h2t + (size_t)r * HS * 2);
                hv[0] = __uint_as_float(pk << 16);          // bf16 -> fp32 is a 16-bit shift
                hv[1] = __uint_as_float(pk & 0xFFFF0000u);
            } else {
                const float2 h2 = *reinterpret_cast<const float2*>(h2t + (size_t)r * HS * 4);
                hv[0] = h2.x;
                hv[1] = h2.y;
            }
            float dh[2];
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                float back = d0s[0][0] * wh_c[cc][0];
                back = fmaf(d0s[0][1], wh_c[cc][1], back);
                back = fmaf(d0s[0][2], wh_c[cc][2], back);
                back = fmaf(d0s[0][3], wh_c[cc][3], back);
                back = fmaf(d0s[0][4], wh_c[cc][4], back);
                dh[cc] = hv[cc] > 0.f ? back : 0.f;
                a_wh[cc][0] = fmaf(hv[cc], d0s[0][0], a_wh[cc][0]);
                a_wh[cc][1] = fmaf(hv[cc], d0s[0][1], a_wh[cc][1]);
                a_wh[cc][2] = fmaf(hv[cc], d0s[0][2], a_wh[cc][2]);
                a_wh[cc][3] = fmaf(hv[cc], d0s[0][3], a_wh[cc][3]);
                a_wh[cc][4] = fmaf(hv[cc], d0s[0][4], a_wh[cc][4]);
            }
            uint32_t phi, plo;
            split2<PREC>(dh[0], dh[1], phi, plo);
            if (PREC == 1) {  // the bf16 workload rounds dh2: the sums take the rounded values
                dh[0] = __uint_as_float(phi << 16);
                dh[1] = __uint_as_float(phi & 0xFFFF0000u);
            }
            a_b2[0] += dh[0];
            a_b2[1] += dh[1];
            if (fullt || r < rows_left) {
                o_hi[r * (H / 2)] = phi;
                if (PREC == 0) o_lo[r * (H / 2)] = plo;
            }
            if (FUSE) {
                // element (k = tile row, n = unit 2 cp) of the MN-major tile: box n/64, byte k*128 + (((n%64)/8) ^ (k%8))*16 +
                // (n%8)*2; rows past the end carry zeros (their h2 was zero-filled)
                const int k = rg * 8 + r;
                unsigned char* tp = s_t + buf * Cfg::OP_TILE + (cp >> 5) * Cfg::BOX + k * 128 + ((((cp & 31) >> 2) ^ (k & 7)) << 4) + (cp & 3) * 4;
                *reinterpret_cast<uint32_t*>(tp) = phi;
                if (PREC == 0) *reinterpret_cast<uint32_t*>(tp + (H / 64) * Cfg::BOX) = plo;
            }
        }
        if (FUSE) tc::fence_proxy_async();  // generic-proxy stores -> visible to the tensor core
        __syncwarp();
        if (lane == 0) {
            tc::mbar_arrive(&empty[buf]);  // the row warp may refill this buffer of output gradients
            if (FUSE) tc::mbar_arrive(&t_ready[buf]);
        }
        // FUSE: after a group's last tile the accumulators go to this CTA's dW2 partial; the next tile's MMAs (which restart
        // the sum) are issued only after every column warp has arrived for that tile, i.e. after its part of the read-out
        if (FUSE && (it + 1) % Cfg::GROUP == 0 && it + 1 < my_its) ok = dw2_out(it) && ok;
    }
    cp_async_wait<0>();
    // ---- per-CTA results: dWh, db2 partials (split index = 4*CTA + row group)
    {
        float* part = a.part_small + (size_t)(4 * blockIdx.x + rg) * a.small_stride;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
#pragma unroll
            for (int c = 0; c < 5; ++c) part[(size_t)(c_base + 2 * cp + cc) * 5 + c] = a_wh[cc][c];
            part[(size_t)H * 5 + c_base + 2 * cp + cc] = a_b2[cc];
        }
    }
    if (FUSE) {
        if (my_its > 0) ok = dw2_out(my_its - 1) && ok;
        else dw2_zero();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(epi_done);
    }
    if (!ok && lane == 0) atomicOr(b.status, DEV_E_WAIT_TIMEOUT);
}

// ----------------------------------------------------------------------------------------------------
// k_heads_bwd_tc: the same step for the bf16 workload with bf16 h2 in HBM (wide layers), with both small products on
// the tensor pipe (mma.sync m16n8k16, bf16 inputs are exact here, fp32 accumulate):
//   dh2 tile [32 rows x 16 cols per warp] = dOut [rows x 16 (5 used)] x Wh^T [16 x cols], then the gate and bf16;
//   dWh [16 cols per warp x 8 (5 used)] += h2^T [cols x 32 rows] x dOut [32 rows x 8]   (accumulators live all kernel).
// A CTA owns a 256-column slab (blockIdx.y) and walks 32-row tiles; the row phase (softmax, loss, dOut) is as in
// k_heads_bwd.  dh2 goes through a shared staging tile and leaves as whole 512-byte row segments.
// ----------------------------------------------------------------------------------------------------
template <int H>
struct HeadsTcCfg {
    static constexpr int TR = 32, HS = 256, NW = 16, NST = 4;
    static constexpr int LD = HS + 8;  // bf16 pitch of the shared tiles (16-byte skew: conflict-free fragment access)
    static constexpr size_t smem_bytes = (size_t)(NST + 2) * TR * LD * 2 + (size_t)2 * TR * 8 * 2 + (size_t)2 * 8 * (TR + 8) * 2 + NW * 8 * 4;
};

template <int H>
__global__ void __launch_bounds__(512, 2) k_heads_bwd_tc(LearnArgs a) {
    using Cfg = HeadsTcCfg<H>;
    constexpr int TR = Cfg::TR, HS = Cfg::HS, NW = Cfg::NW, NST = Cfg::NST, LD = Cfg::LD, LDT = TR + 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* s_h2 = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [NST][TR][LD]
    __nv_bfloat16* s_o = s_h2 + NST * TR * LD;                         // [2][TR][LD] dh2 staging
    __nv_bfloat16* s_dA = s_o + 2 * TR * LD;                           // [2][TR][8]   dOut rows (c fastest)
    __nv_bfloat16* s_dT = s_dA + 2 * TR * 8;                           // [2][8][LDT]  dOut transposed (row fastest)
    float* s_fin = reinterpret_cast<float*>(s_dT + 2 * 8 * LDT);       // [NW][8]
    const int c_base = blockIdx.y * HS;
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const size_t R = (size_t)d.B * a.T;
    const float invR = a.gscale / (float)R;
    const int ntiles = (int)((R + TR - 1) / TR);
    const uint16_t* g_h2 = reinterpret_cast<const uint16_t*>(b.h2);
    uint16_t* g_dh2 = reinterpret_cast<uint16_t*>(b.dh2);
    const int col0 = 16 * wid;  // this warp's 16 columns inside the slab

    // B fragments of Wh^T for the warp's two n8 tiles: k = head index (5 used of 16), n = column
    uint32_t whf[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const float* w = b.theta_c + d.oWh + (size_t)(c_base + col0 + 8 * j + g) * 5;
        const float w0 = 2 * t4 < 5 ? w[2 * t4] : 0.f, w1 = 2 * t4 + 1 < 5 ? w[2 * t4 + 1] : 0.f;
        whf[j] = pack_bf16(__float2bfloat16_rn(w0), __float2bfloat16_rn(w1));
    }
    for (int i = tid; i < 2 * 8 * LDT; i += 512) s_dT[i] = __float2bfloat16_rn(0.f);  // rows 5..7 stay zero
    float acc_wh[4] = {0.f, 0.f, 0.f, 0.f};
    float a_b2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    float a_bh[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
    float l_pg = 0.f, l_v = 0.f, l_ent = 0.f;

    auto load_tile = [&](int tile, int buf) {  // 16-byte chunks, zero-filled past the last row; always commits a group
        __nv_bfloat16* dst = s_h2 + buf * TR * LD;
        for (int c = tid; tile < ntiles && c < TR * (HS / 8); c += 512) {
            const int r = c / (HS / 8), k = 8 * (c - r * (HS / 8));
            const size_t row = (size_t)tile * TR + r;
            const bool ok = row < R;
            cp_async16(dst + r * LD + k, g_h2 + (ok ? row : 0) * H + c_base + k, ok ? 16 : 0);
        }
        cp_async_commit();
    };
    struct RowIn { float4 o4; float v, adv, ret, lpo; int act; bool ok; };
    auto row_load = [&](int tile) {
        RowIn in;
        const size_t i = (size_t)tile * TR + lane;
        in.ok = tile < ntiles && i < R;
        in.o4 = make_float4(0.f, 0.f, 0.f, 0.f);
        in.v = in.adv = in.ret = in.lpo = 0.f;
        in.act = 0;
        if (in.ok) {
            in.o4 = *reinterpret_cast<const float4*>(b.out5 + i * 8);
            in.v = b.out5[i * 8 + 4];
            in.adv = b.adv[i];
            in.lpo = a.ppo_clip > 0.f ? b.tlogp[i] : 0.f;
            in.ret = b.ret[i];
            in.act = b.tact[i];
        }
        return in;
    };
    auto row_finish = [&](const RowIn& in, int buf) {  // lane = row of the tile
        float dO[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
        if (in.ok) {
            const float o[4] = {in.o4.x, in.o4.y, in.o4.z, in.o4.w};
            const float mx = fmaxf(fmaxf(o[0], o[1]), fmaxf(o[2], o[3]));
            float ex[4], Z = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) { ex[c] = expf(o[c] - mx); Z += ex[c]; }
            const float logZ = logf(Z);
            float p[4], lp[4], ent = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) { p[c] = ex[c] / Z; lp[c] = (o[c] - mx) - logZ; ent -= p[c] * lp[c]; }
            const float A = in.adv, err = in.v - in.ret;
            const float pf = policy_term(A, in.act == 0 ? lp[0] : in.act == 1 ? lp[1] : in.act == 2 ? lp[2] : lp[3], in.lpo, a.ppo_clip, l_pg);
#pragma unroll
            for (int c = 0; c < 4; ++c) dO[c] = round_bf16((-A * pf * ((c == in.act ? 1.f : 0.f) - p[c]) + a.c_e * p[c] * (lp[c] + ent)) * invR);
            dO[4] = round_bf16(2.f * a.c_v * err * invR);
            l_v += err * err;
            l_ent += ent;
#pragma unroll
            for (int c = 0; c < 5; ++c) a_bh[c] += dO[c];
        }
        uint4 pk;
        pk.x = pack_bf16(__float2bfloat16_rn(dO[0]), __float2bfloat16_rn(dO[1]));
        pk.y = pack_bf16(__float2bfloat16_rn(dO[2]), __float2bfloat16_rn(dO[3]));
        pk.z = pack_bf16(__float2bfloat16_rn(dO[4]), __float2bfloat16_rn(0.f));
        pk.w = 0u;
        *reinterpret_cast<uint4*>(s_dA + (buf * TR + lane) * 8) = pk;
#pragma unroll
        for (int c = 0; c < 5; ++c) s_dT[(buf * 8 + c) * LDT + lane] = __float2bfloat16_rn(dO[c]);
    };
    // staged dh2 tile -> global: thread = (row, 16-column piece), 32 bytes each, rows in whole 512-byte segments
    auto copy_out = [&](int tile, int buf) {
        const int r = tid >> 4, c16 = (tid & 15) * 16;
        const size_t row = (size_t)tile * TR + r;
        if (row < R) {
            const uint4* src = reinterpret_cast<const uint4*>(s_o + (buf * TR + r) * LD + c16);
            uint4* dst = reinterpret_cast<uint4*>(g_dh2 + row * H + c_base + c16);
            dst[0] = src[0];
            dst[1] = src[1];
        }
    };

    int it = 0, prev_tile = -1;
#pragma unroll
    for (int q = 0; q < NST - 1; ++q) load_tile(blockIdx.x + q * (int)gridDim.x, q);
    __syncthreads();  // the zeroed rows of s_dT are in place before the first row phase writes beside them
    if ((int)blockIdx.x < ntiles && wid == 0) row_finish(row_load(blockIdx.x), 0);
    const int jm = lane >> 3, r8 = lane & 7;  // ldmatrix addressing: matrix index, row inside the matrix
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        const int next = tile + (int)gridDim.x;
        cp_async_wait<NST - 2>();
        __syncthreads();  // this tile's h2 and dOut are in place; the staging tile of the tile before is complete
        load_tile(tile + (NST - 1) * (int)gridDim.x, (it + NST - 1) % NST);
        const bool row_warp = wid == (it + 1) % NW;  // this warp prepares the next tile's output gradients
        RowIn nin;
        if (row_warp) nin = row_load(next);
        if (prev_tile >= 0) copy_out(prev_tile, buf ^ 1);
        const __nv_bfloat16* h2t = s_h2 + (it % NST) * TR * LD;
        __nv_bfloat16* ot = s_o + buf * TR * LD;
        // ---- dh2 = (dOut Wh^T) gated by h2 > 0: A = dOut rows (k = head index; only k < 8 can be non-zero)
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            uint32_t af[4];
            af[0] = *reinterpret_cast<const uint32_t*>(s_dA + (buf * TR + 16 * mt + g) * 8 + 2 * t4);
            af[1] = *reinterpret_cast<const uint32_t*>(s_dA + (buf * TR + 16 * mt + g + 8) * 8 + 2 * t4);
            af[2] = af[3] = 0u;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                mma_bf16(c, af, whf[j], 0u);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int row = 16 * mt + 8 * hh + g, col = col0 + 8 * j + 2 * t4;
                    const uint32_t hv = *reinterpret_cast<const uint32_t*>(h2t + row * LD + col);  // h2 >= 0: any magnitude bit = "> 0"
                    const float v0 = (hv & 0x00007FFFu) ? c[2 * hh] : 0.f, v1 = (hv & 0x7FFF0000u) ? c[2 * hh + 1] : 0.f;
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(v0, v1);
                    const uint32_t pku = *reinterpret_cast<const uint32_t*>(&pk);
                    *reinterpret_cast<uint32_t*>(ot + row * LD + col) = pku;
                    a_b2[j][0] += __uint_as_float(pku << 16);  // the sums take the rounded values
                    a_b2[j][1] += __uint_as_float(pku & 0xFFFF0000u);
                }
            }
        }
        // ---- dWh += h2^T dOut: A[m = column][k = row] comes transposed out of the [row][column] tile
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
            uint32_t af[4];
            ldmatrix_x4_trans(af, h2t + (16 * ks + 8 * (jm >> 1) + r8) * LD + col0 + 8 * (jm & 1));
            const uint32_t b0 = *reinterpret_cast<const uint32_t*>(s_dT + (buf * 8 + g) * LDT + 16 * ks + 2 * t4);
            const uint32_t b1 = *reinterpret_cast<const uint32_t*>(s_dT + (buf * 8 + g) * LDT + 16 * ks + 2 * t4 + 8);
            mma_bf16(acc_wh, af, b0, b1);
        }
        // ---- row phase of the next tile (its inputs were requested before the tensor work)
        if (row_warp && next < ntiles) row_finish(nin, buf ^ 1);
        prev_tile = tile;
    }
    cp_async_wait<0>();
    __syncthreads();
    if (prev_tile >= 0) copy_out(prev_tile, (it - 1) & 1);
    // ---- per-CTA results (split index = CTA): dWh from the accumulator fragments, db2 folded over the 8 row lanes
    float* part = a.part_small + (size_t)(4 * blockIdx.x) * a.small_stride;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int col = c_base + col0 + g + 8 * hh;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc)
            if (2 * t4 + cc < 5) part[(size_t)col * 5 + 2 * t4 + cc] = acc_wh[2 * hh + cc];
    }
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            float v = a_b2[j][cc];
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 4);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 8);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 16);
            if (g == 0) part[(size_t)H * 5 + c_base + col0 + 8 * j + 2 * t4 + cc] = v;
        }
    {   // every warp has taken turns at the row phase: fold its lanes (fixed tree), then the warps in index order
        float vals[8] = {a_bh[0], a_bh[1], a_bh[2], a_bh[3], a_bh[4], l_pg, l_v, l_ent};
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) vals[c] += __shfl_xor_sync(0xFFFFFFFFu, vals[c], off);
        if (lane == 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) s_fin[wid * 8 + c] = vals[c];
        }
    }
    __syncthreads();
    if (tid < 8 && blockIdx.y == 0) {  // dbh and the loss terms come from the first slab only
        float sum = 0.f;
        for (int e = 0; e < NW; ++e) sum += s_fin[e * 8 + tid];
        if (tid < 5) part[(size_t)H * 6 + tid] = sum;
        else b.loss_part[(size_t)blockIdx.x * 4 + (tid - 5)] = sum;
    }
}

// ----------------------------------------------------------------------------------------------------
// k_dh1: dh1 = (dh2 W2^T) gated by h1 > 0 on the tensor pipe, and S = sum over t of dh1.
// A CTA owns 64 envs x BN output columns and walks t = 0..T-1.  Its slice of W2 (BN rows, all K, hi and lo planes)
// stays in shared memory for the whole kernel; the dh2 planes stream through a cp.async ring in 64-wide k chunks
// that runs across the t boundaries without draining.
// ----------------------------------------------------------------------------------------------------
template <int H, int BN, int PREC>
struct Dh1Cfg {
    static constexpr int BM = 64, KC = 64, STAGES = 4;
    static constexpr int PL = PREC == 1 ? 1 : 2;
    static constexpr int LDW = H + 8;     // 16-bit pitch of the resident W2 planes
    static constexpr int LDA = KC + 8;    // 16-bit pitch of an A chunk
    static constexpr int A_STAGE = PL * BM * LDA;
    static constexpr int NCH = H / KC;    // chunks per t
    static constexpr int WM = 32, WN = 16;     // warp tile; 2 x (BN/16) warps
    static constexpr int WARPS_N = BN / WN, THREADS = 2 * WARPS_N * 32;
    static constexpr int MT = WM / 16, NT = WN / 8;
    static constexpr size_t smem_bytes = ((size_t)PL * BN * LDW + (size_t)STAGES * A_STAGE) * 2;
};

template <int H, int BN, int PREC, bool GROUPED = false>
__global__ void __launch_bounds__(Dh1Cfg<H, BN, PREC>::THREADS, 1) k_dh1(LearnArgs a_in) {
    const PolicyArgs<GROUPED, LearnArgs> pa(a_in, blockIdx.z);  // many policies: grid.z = policy
    const LearnArgs& a = pa.a;
    using Cfg = Dh1Cfg<H, BN, PREC>;
    constexpr int NTH = Cfg::THREADS;
    constexpr int BM = Cfg::BM, KC = Cfg::KC, STAGES = Cfg::STAGES, PL = Cfg::PL, LDW = Cfg::LDW, LDA = Cfg::LDA;
    constexpr int NCH = Cfg::NCH, MT = Cfg::MT, NT = Cfg::NT;
    static_assert(NT % 2 == 0, "B fragments are loaded two n-tiles at a time");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint16_t* sW = reinterpret_cast<uint16_t*>(smem_raw);  // [PL][BN][LDW]
    uint16_t* sA = sW + PL * BN * LDW;                      // [STAGES][PL][BM][LDA]
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int wm = wid / Cfg::WARPS_N, wn = wid % Cfg::WARPS_N;
    const int g = lane >> 2, t4 = lane & 3;
    const int B = d.B, T = a.T;
    const int e0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const size_t RH = (size_t)B * d.Tmax * H;
    const uint16_t* g_dh2hi = reinterpret_cast<const uint16_t*>(b.dh2);
    const uint16_t* g_h1hi = reinterpret_cast<const uint16_t*>(b.h1);
    uint16_t* g_dh1hi = reinterpret_cast<uint16_t*>(b.dh1);

    // resident slice of W2: rows n0..n0+BN (output units), all k
    for (int c = tid; c < BN * (H / 8); c += NTH) {
        const int n = c / (H / 8), k = 8 * (c - n * (H / 8));
        cp_async16(sW + n * LDW + k, b.w2p_hi + (size_t)(n0 + n) * H + k, 16);
        if (PL == 2) cp_async16(sW + BN * LDW + n * LDW + k, b.w2p_lo + (size_t)(n0 + n) * H + k, 16);
    }
    cp_async_commit();

    const int nchunks = T * NCH;
    auto issue = [&](int c, int stage) {
        const int t = c / NCH, k0 = (c - t * NCH) * KC;
        uint16_t* a_s = sA + stage * Cfg::A_STAGE;
        for (int q = tid; q < BM * (KC / 8); q += NTH) {
            const int r = q / (KC / 8), k = 8 * (q - r * (KC / 8));
            const bool ok = e0 + r < B;
            const size_t gi = ((size_t)t * B + (ok ? e0 + r : 0)) * H + k0 + k;
            cp_async16(a_s + r * LDA + k, g_dh2hi + gi, ok ? 16 : 0);
            if (PL == 2) cp_async16(a_s + BM * LDA + r * LDA + k, g_dh2hi + RH + gi, ok ? 16 : 0);
        }
    };
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < nchunks) issue(s, s);
        cp_async_commit();
    }

    float acc[MT][NT][4], s_acc[MT][NT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) { acc[i][j][q] = 0.f; s_acc[i][j][q] = 0.f; }
    uint32_t gate1[MT][NT][2];
    const int jm = lane >> 3, r8 = lane & 7;

    for (int c = 0; c < nchunks; ++c) {
        const int t = c / NCH, kc = c - t * NCH;
        cp_async_wait<STAGES - 2>();  // chunk c (and, the first time, the W2 slice) has landed
        __syncthreads();
        {
            const int nxt = c + STAGES - 1;
            if (nxt < nchunks) issue(nxt, nxt % STAGES);
            cp_async_commit();
        }
        if (kc == 0) {  // this step's layer-1 gates, well ahead of the epilogue
#pragma unroll
            for (int i = 0; i < MT; ++i)
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int row = wm * Cfg::WM + 16 * i + 8 * hh + g, col = n0 + wn * Cfg::WN + 8 * j + 2 * t4;
                        gate1[i][j][hh] = (e0 + row < B)
                                              ? __ldg(reinterpret_cast<const uint32_t*>(g_h1hi + ((size_t)t * B + e0 + row) * H + col))
                                              : 0u;
                    }
        }
        const uint16_t* a_s = sA + (c % STAGES) * Cfg::A_STAGE;
#pragma unroll
        for (int k16 = 0; k16 < KC / 16; ++k16) {
            uint32_t ahi[MT][4], alo[MT][4];
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                const uint16_t* p = a_s + (wm * Cfg::WM + 16 * i + (lane & 7) + ((lane >> 3) & 1) * 8) * LDA + 16 * k16 + (lane >> 4) * 8;
                ldmatrix_x4(ahi[i], p);
                if (PL == 2) ldmatrix_x4(alo[i], p + BM * LDA);
            }
#pragma unroll
            for (int j2 = 0; j2 < NT / 2; ++j2) {
                uint32_t bhi[4], blo[4];
                const uint16_t* p = sW + (wn * Cfg::WN + 16 * j2 + 8 * (jm >> 1) + r8) * LDW + kc * KC + 16 * k16 + 8 * (jm & 1);
                ldmatrix_x4(bhi, p);
                if (PL == 2) ldmatrix_x4(blo, p + BN * LDW);
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        if (PL == 2) {
                            mma16816<PREC>(acc[i][2 * j2 + q], alo[i], bhi[2 * q], bhi[2 * q + 1]);
                            mma16816<PREC>(acc[i][2 * j2 + q], ahi[i], blo[2 * q], blo[2 * q + 1]);
                        }
                        mma16816<PREC>(acc[i][2 * j2 + q], ahi[i], bhi[2 * q], bhi[2 * q + 1]);
                    }
            }
        }
        if (kc == NCH - 1) {  // row tile of step t complete: gate, accumulate S, emit dh1 planes
#pragma unroll
            for (int i = 0; i < MT; ++i)
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int row = wm * Cfg::WM + 16 * i + 8 * hh + g, col = n0 + wn * Cfg::WN + 8 * j + 2 * t4;
                        const uint32_t gt = gate1[i][j][hh];
                        // h1 >= 0 always, so "h1 > 0" is "any bit of the 16-bit high part set"
                        const float v0 = rnd<PREC>((gt & 0x0000FFFFu) ? acc[i][j][2 * hh] : 0.f);
                        const float v1 = rnd<PREC>((gt & 0xFFFF0000u) ? acc[i][j][2 * hh + 1] : 0.f);
                        s_acc[i][j][2 * hh] += v0;
                        s_acc[i][j][2 * hh + 1] += v1;
                        acc[i][j][2 * hh] = 0.f;
                        acc[i][j][2 * hh + 1] = 0.f;
                        if (e0 + row < B) {
                            uint32_t phi, plo;
                            split2<PREC>(v0, v1, phi, plo);
                            const size_t gi = ((size_t)t * B + e0 + row) * H + col;
                            *reinterpret_cast<uint32_t*>(g_dh1hi + gi) = phi;
                            if (PL == 2) *reinterpret_cast<uint32_t*>(g_dh1hi + RH + gi) = plo;
                        }
                    }
        }
    }
    cp_async_wait<0>();
    // S (sum over t of dh1) as two 16-bit planes [B][H]: S is an fp32 sum, so it keeps two terms in either workload
    uint16_t* S_hi = reinterpret_cast<uint16_t*>(b.S);
    uint16_t* S_lo = S_hi + (size_t)B * H;
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int row = wm * Cfg::WM + 16 * i + 8 * hh + g, col = n0 + wn * Cfg::WN + 8 * j + 2 * t4;
                if (e0 + row < B) {
                    uint32_t phi, plo;
                    if (PREC == 1) {
                        __nv_bfloat16 h0, l0, h1v, l1;
                        split_bf16(s_acc[i][j][2 * hh], h0, l0);
                        split_bf16(s_acc[i][j][2 * hh + 1], h1v, l1);
                        phi = pack_bf16(h0, h1v);
                        plo = pack_bf16(l0, l1);
                    } else {
                        split2<0>(s_acc[i][j][2 * hh], s_acc[i][j][2 * hh + 1], phi, plo);
                    }
                    const size_t gi = (size_t)(e0 + row) * H + col;
                    *reinterpret_cast<uint32_t*>(S_hi + gi) = phi;
                    *reinterpret_cast<uint32_t*>(S_lo + gi) = plo;
                }
            }
}

// ----------------------------------------------------------------------------------------------------
// k_gemm_tn: C[m][n] = sum_k A[k][m] B[k][n], split-K partial outputs.
// ----------------------------------------------------------------------------------------------------
template <int BM, int BN, int AMODE, int APL, int BPL, int PREC>
struct GemmTnCfg {
    static constexpr int BK = 32, STAGES = 3, THREADS = 256;
    static constexpr int LDA = BM + 8, LDB = BN + 8;  // bf16 pitches
    static constexpr int A_STAGE = APL * BK * LDA, B_STAGE = BPL * BK * LDB;  // elements
    static constexpr size_t smem_bytes = (size_t)STAGES * (A_STAGE + B_STAGE) * 2;
    static constexpr int WM = BM / 2, WN = BN / 4;   // warp tile (2 x 4 warps)
    static constexpr int MT = WM / 16, NT = WN / 8;
};

template <int BM, int BN, int AMODE, int APL, int BPL, int PREC, bool GROUPED = false>
__global__ void __launch_bounds__(256) k_gemm_tn(GemmTnArgs g_in) {
    // many policies: grid.z = policy * nsplit + split
    const PolicyArgs<GROUPED, GemmTnArgs> pa(g_in, GROUPED ? (int)blockIdx.z / g_in.nsplit : 0);
    const GemmTnArgs& g = pa.a;
    using Cfg = GemmTnCfg<BM, BN, AMODE, APL, BPL, PREC>;
    constexpr int BK = Cfg::BK, STAGES = Cfg::STAGES, LDA = Cfg::LDA, LDB = Cfg::LDB, MT = Cfg::MT, NT = Cfg::NT;
    static_assert(NT % 2 == 0, "B fragments are loaded two n-tiles at a time");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* sA = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* sB = sA + STAGES * Cfg::A_STAGE;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int wm = wid >> 2, wn = wid & 3;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN, split = GROUPED ? (int)blockIdx.z % g.nsplit : (int)blockIdx.z;
    const int kbeg = split * g.klen, kend = min(g.K, kbeg + g.klen);
    const int ntiles = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;

    auto issue = [&](int tile, int stage) {
        const int k0 = kbeg + tile * BK;
        __nv_bfloat16* a_s = sA + stage * Cfg::A_STAGE;
        __nv_bfloat16* b_s = sB + stage * Cfg::B_STAGE;
        // B planes: BK rows of BN bf16 -> 16-byte chunks
        for (int c = tid; c < BK * (BN / 8); c += 256) {
            const int kk = c / (BN / 8), nn = 8 * (c - kk * (BN / 8));
            const bool ok = k0 + kk < kend && n0 + nn < g.N;
            const size_t gi = (size_t)(ok ? k0 + kk : 0) * g.ldb + (ok ? n0 + nn : 0);
            cp_async16(b_s + kk * LDB + nn, g.Bhi + gi, ok ? 16 : 0);
            if (BPL == 2) cp_async16(b_s + BK * LDB + kk * LDB + nn, g.Blo + gi, ok ? 16 : 0);
        }
        if (AMODE == A_PLANES) {
            for (int c = tid; c < BK * (BM / 8); c += 256) {
                const int kk = c / (BM / 8), mm = 8 * (c - kk * (BM / 8));
                const bool ok = k0 + kk < kend && m0 + mm < g.M;
                const size_t gi = (size_t)(ok ? k0 + kk : 0) * g.lda + (ok ? m0 + mm : 0);
                cp_async16(a_s + kk * LDA + mm, g.Ahi + gi, ok ? 16 : 0);
                if (APL == 2) cp_async16(a_s + BK * LDA + kk * LDA + mm, g.Alo + gi, ok ? 16 : 0);
            }
        } else if (AMODE == A_ONEHOT) {
            // one 16-byte chunk per thread: zeros, except the chunk that holds this k's single 1.0
            for (int c = tid; c < BK * (BM / 8); c += 256) {
                const int kk = c / (BM / 8), mm = 8 * (c - kk * (BM / 8));
                const int k = k0 + kk;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (k < kend) {
                    const int rel = (int)g.idx[g.kmod ? k % g.kmod : k] - (m0 + mm);
                    if (rel >= 0 && rel < 8) {
                        const uint32_t one = (rel & 1) ? (one16<PREC>() << 16) : one16<PREC>();
                        if ((rel >> 1) == 0) v.x = one; else if ((rel >> 1) == 1) v.y = one; else if ((rel >> 1) == 2) v.z = one; else v.w = one;
                    }
                }
                *reinterpret_cast<uint4*>(a_s + kk * LDA + mm) = v;
            }
        } else {  // A_WALLS
            for (int c = tid; c < BK * (BM / 8); c += 256) {
                const int kk = c / (BM / 8), mm = 8 * (c - kk * (BM / 8));
                const int k = k0 + kk;
                uint32_t w[4] = {0u, 0u, 0u, 0u};
                if (k < kend) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int m = m0 + mm + q;
                        bool on = false;
                        if (m < g.ones_row) on = (g.walls[(size_t)(g.kmod ? k % g.kmod : k) * g.W + (m >> 5)] >> (m & 31)) & 1u;
                        else if (m == g.ones_row) on = true;
                        if (on) w[q >> 1] |= (q & 1) ? (one16<PREC>() << 16) : one16<PREC>();
                    }
                }
                *reinterpret_cast<uint4*>(a_s + kk * LDA + mm) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    };

    float acc[MT][NT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[i][j][q] = 0.f;

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < ntiles) issue(s, s);
        cp_async_commit();
    }
    const int jm = lane >> 3, r8 = lane & 7;
    for (int tile = 0; tile < ntiles; ++tile) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {   // refill the stage consumed in the previous iteration
            const int nxt = tile + STAGES - 1;
            if (nxt < ntiles) issue(nxt, nxt % STAGES);
            cp_async_commit();
        }
        const int stage = tile % STAGES;
        const __nv_bfloat16* a_s = sA + stage * Cfg::A_STAGE;
        const __nv_bfloat16* b_s = sB + stage * Cfg::B_STAGE;
#pragma unroll
        for (int k16 = 0; k16 < BK / 16; ++k16) {
            uint32_t ahi[MT][4], alo[MT][4];
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                const __nv_bfloat16* p = a_s + (16 * k16 + 8 * (jm >> 1) + r8) * LDA + wm * Cfg::WM + 16 * i + 8 * (jm & 1);
                ldmatrix_x4_trans(ahi[i], p);
                if (APL == 2) ldmatrix_x4_trans(alo[i], p + BK * LDA);
            }
#pragma unroll
            for (int j2 = 0; j2 < NT / 2; ++j2) {
                uint32_t bhi[4], blo[4];
                const __nv_bfloat16* p = b_s + (16 * k16 + 8 * (jm & 1) + r8) * LDB + wn * Cfg::WN + 16 * j2 + 8 * (jm >> 1);
                ldmatrix_x4_trans(bhi, p);
                if (BPL == 2) ldmatrix_x4_trans(blo, p + BK * LDB);
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        if (APL == 2) mma16816<PREC>(acc[i][2 * j2 + q], alo[i], bhi[2 * q], bhi[2 * q + 1]);
                        if (BPL == 2) mma16816<PREC>(acc[i][2 * j2 + q], ahi[i], blo[2 * q], blo[2 * q + 1]);
                        mma16816<PREC>(acc[i][2 * j2 + q], ahi[i], bhi[2 * q], bhi[2 * q + 1]);
                    }
            }
        }
    }
    cp_async_wait<0>();
    // ---- split-K partial out
    const int gq = lane >> 2, t4 = lane & 3;
    float* part = g.part + (size_t)split * g.stride;
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int m = m0 + wm * Cfg::WM + 16 * i + 8 * hh + gq;
                const int n = n0 + wn * Cfg::WN + 8 * j + 2 * t4;
                if (n < g.N) {
                    const float2 v = make_float2(acc[i][j][2 * hh], acc[i][j][2 * hh + 1]);
                    if (AMODE == A_WALLS && m == g.ones_row) *reinterpret_cast<float2*>(part + g.off_ones + n) = v;
                    else if (m < g.M && !(AMODE == A_WALLS && m > g.ones_row)) *reinterpret_cast<float2*>(part + g.off + (size_t)m * g.ldc + n) = v;
                }
            }
}

template <int BM, int BN, int AMODE, int APL, int BPL, int PREC>
static cudaError_t launch_gemm_tn(const GemmTnArgs& g, int rows_m, int splits, cudaStream_t s) {
    using Cfg = GemmTnCfg<BM, BN, AMODE, APL, BPL, PREC>;
    dim3 grid((rows_m + BM - 1) / BM, (g.N + BN - 1) / BN, splits);
    if (g.npol > 1) {  // many policies: grid.z = policy * splits + split
        if constexpr (PREC == 0) {
            cudaError_t e = cudaFuncSetAttribute(k_gemm_tn<BM, BN, AMODE, APL, BPL, PREC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
            if (e != cudaSuccess) return e;
            if ((size_t)g.npol * splits > 65535) return cudaErrorNotSupported;
            grid.z = g.npol * splits;
            GemmTnArgs gg = g;
            gg.nsplit = splits;
            k_gemm_tn<BM, BN, AMODE, APL, BPL, PREC, true><<<grid, 256, Cfg::smem_bytes, s>>>(gg);
            return cudaGetLastError();
        }
        return cudaErrorNotSupported;
    }
    cudaError_t e = cudaFuncSetAttribute(k_gemm_tn<BM, BN, AMODE, APL, BPL, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
    if (e != cudaSuccess) return e;
    k_gemm_tn<BM, BN, AMODE, APL, BPL, PREC><<<grid, 256, Cfg::smem_bytes, s>>>(g);
    return cudaGetLastError();
}

// One Adam step of parameter i with gradient g (Kingma & Ba, Algorithm 1), plus the refreshed 16-bit copies.
// (a parameter's state is loaded ahead of its gradient sum: one memory round trip less)
__device__ __forceinline__ AdamIn adam_load(const LearnArgs& a, size_t i) {
    return AdamIn{a.b.adam_m[i], a.b.adam_v[i], a.b.theta[i]};
}
template <int PREC>
__device__ __forceinline__ void adam_step(const LearnArgs& a, size_t i, float g, const AdamIn& in) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const AdamIn o = adam_arith(a, in, g);
    b.adam_m[i] = o.m;
    b.adam_v[i] = o.v;
    const float th = o.theta;
    b.theta[i] = th;
    float thc = th;
    if (PREC == 1) {
        const bool is_bias = (i >= d.ob1 && i < d.oW2) || (i >= d.ob2 && i < d.oWh) || i >= d.obh;
        thc = is_bias ? th : round_bf16(th);
        b.theta_c[i] = thc;
    }
    // refresh the tensor-pipe copies of W2 in place (fragment layouts as in k_pack_w2, and the row-major planes)
    if (b.w2p_hi && i >= d.oW2 && i < d.ob2) {
        const int H = d.H;
        const int k = (int)((i - d.oW2) / H), n = (int)((i - d.oW2) % H);
        uint16_t hi, lo;
        split1<PREC>(thc, hi, lo);
        if (b.w2f_hi) {
            const size_t ef = ((size_t)((k >> 4) * (H / 8) + (n >> 3)) * 32 + (n & 7) * 4 + ((k & 7) >> 1)) * 4 + ((k & 15) >> 3) * 2 + (k & 1);
            reinterpret_cast<uint16_t*>(b.w2f_hi)[ef] = hi;
            reinterpret_cast<uint16_t*>(b.w2f_lo)[ef] = lo;
        }
        b.w2p_hi[i - d.oW2] = hi;
        if (b.w2p_lo) b.w2p_lo[i - d.oW2] = lo;
    }
}

// Adam from the GRADS blob as it stands (the second half of an update whose gradient was averaged over replicas).
template <int PREC, bool GROUPED>
__global__ void __launch_bounds__(256) k_adam_only(LearnArgs a_in) {
    const PolicyArgs<GROUPED, LearnArgs> pa(a_in, blockIdx.y);  // many policies: grid.y = policy
    const LearnArgs& a = pa.a;
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i < a.d.P) {
        float g = a.b.grads[i];
        if (a.grad_div > 1.f) {  // the mean over the replicas (Section 3.1), taken where the sum is consumed
            g = g / a.grad_div;
            a.b.grads[i] = g;
        }
        adam_step<PREC>(a, i, g, adam_load(a, i));
    }
}

// ----------------------------------------------------------------------------------------------------
// k_reduce_adam2: fixed-order sums of each parameter region's partials, then Adam (Kingma & Ba, Algorithm 1).
// ----------------------------------------------------------------------------------------------------
template <int PREC, bool GROUPED>
__global__ void __launch_bounds__(256) k_reduce_adam2(LearnArgs a_in, size_t R_in, int loss_blocks) {
    const PolicyArgs<GROUPED, LearnArgs> pa(a_in, blockIdx.y);  // many policies: grid.y = policy
    const LearnArgs& a = pa.a;
    const size_t R = GROUPED ? (size_t)a.d.B * a.T : R_in;  // rows of THIS policy
    const size_t poff = GROUPED ? (size_t)blockIdx.y * a_in.d.pstride : 0;  // byte offset of this policy's partials
    __shared__ float s_tail[32][8];
    const Dims& d = a.d;
    const Buffers& b = a.b;
    // Batch-mean gradient of parameter i, then (phase 0) its Adam step.
    // (the parameter's Adam state is fetched before its partials, so that the two do not queue up behind one another)
    auto state_of = [&](size_t i) { return a.phase == 0 ? adam_load(a, i) : AdamIn{0.f, 0.f, 0.f}; };
    auto apply = [&](size_t i, float gsum, const AdamIn& in) {
        gsum *= a.inv_gscale;  // exact: a power of two
        b.grads[i] = gsum;
        if (a.phase == 0) adam_step<PREC>(a, i, gsum, in);
    };
    auto region_of = [&](size_t i) {
        int r = 0;
#pragma unroll
        for (int q = 1; q < LearnArgs::NREG; ++q)
            if (i >= a_in.reg[q].start) r = q;
        return r;
    };
    // Parameters before b2 (W1, b1, W2) have at most ~128 partials: one thread each, partials added in index order,
    // thirty-two loads in flight.  The tail (b2 | Wh | bh) has two partials per CTA of the heads kernel: one warp per
    // parameter group, see below.
    // The work is cut into nb_total block-sized pieces; a launch with fewer CTAs per policy (many policies: a handful of
    // fat CTAs each instead of tens of thousands of tiny ones) walks them in a stride loop.
    const int nb_main = (int)((d.ob2 + 255) / 256);
    const int nb_total = nb_main + (int)(GROUPED ? (d.P - d.ob2 + 255) / 256 : (d.P - d.ob2 + 7) / 8);
    for (int bx = blockIdx.x; bx < nb_total; bx += gridDim.x) {
        if (bx < nb_main || GROUPED) {
            // (many policies: few partials everywhere, so the tail is cut into pieces of 256 parameters like the rest)
            const size_t i = bx < nb_main ? (size_t)bx * 256 + threadIdx.x : d.ob2 + (size_t)(bx - nb_main) * 256 + threadIdx.x;
            if (i < (bx < nb_main ? d.ob2 : d.P)) {
                const PartRegion& rg = a_in.reg[region_of(i)];
                const float* p = reinterpret_cast<const float*>(reinterpret_cast<const unsigned char*>(rg.part) + poff) + (i - rg.start);
                const AdamIn in = state_of(i);
                float gsum = 0.f;
                // NF loads in flight per memory round trip (the ragged last batch is predicated, not split up); the
                // additions stay in index order.  Many policies: a region has a handful of partials, and the registers
                // a wide batch costs would halve the CTAs per SM.
                constexpr int NF = GROUPED ? 8 : 32;
                for (int s = 0; s < rg.ns; s += NF) {
                    float v[NF];
#pragma unroll
                    for (int q = 0; q < NF; ++q) v[q] = s + q < rg.ns ? p[(size_t)(s + q) * rg.stride] : 0.f;
#pragma unroll
                    for (int q = 0; q < NF; ++q)
                        if (s + q < rg.ns) gsum += v[q];
                }
                apply(i, gsum, in);
            }
        } else {
            // eight consecutive parameters per CTA: thread = (parameter tid % 8, partial group tid / 8); a group's eight
            // threads read one 32-byte sector per partial.  Group g adds partials g, g+32, ... in order; then one thread
            // per parameter adds the 32 group sums in group order (shared memory).
            const int pi = threadIdx.x & 7, grp = threadIdx.x >> 3;
            const size_t i = d.ob2 + (size_t)(bx - nb_main) * 8 + pi;
            float gsum = 0.f;
            AdamIn in{0.f, 0.f, 0.f};
            if (i < d.P) {
                if (grp == 0) in = state_of(i);
                const PartRegion& rg = a_in.reg[region_of(i)];
                const float* p = reinterpret_cast<const float*>(reinterpret_cast<const unsigned char*>(rg.part) + poff) + (i - rg.start);
                int s = grp;
                for (; s + 32 * 7 < rg.ns; s += 32 * 8) {  // eight loads in flight per thread
                    float v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = p[(size_t)(s + 32 * q) * rg.stride];
#pragma unroll
                    for (int q = 0; q < 8; ++q) gsum += v[q];
                }
                for (; s < rg.ns; s += 32) gsum += p[(size_t)s * rg.stride];
            }
            __syncthreads();  // (the previous piece's readers of s_tail are done)
            s_tail[grp][pi] = gsum;
            __syncthreads();
            if (grp == 0 && i < d.P) {
                float tot = 0.f;
#pragma unroll
                for (int g2 = 0; g2 < 32; ++g2) tot += s_tail[g2][pi];
                apply(i, tot, in);
            }
        }
        // Loss statistics: the first warp of the last CTA (the one with the least other work) adds the per-CTA partials of
        // the heads kernel, lane l taking partials l, l+32, ... in order, then a fixed shuffle tree joins the lanes.
        if (bx == nb_total - 1 && threadIdx.x < 32) {
            const int lane = threadIdx.x;
            float l[3];
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                float s = 0.f;
                int q = lane;
                for (; q + 32 * 3 < loss_blocks; q += 32 * 4) {  // four loads in flight per lane
                    float v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = b.loss_part[(size_t)(q + 32 * u) * 4 + c];
#pragma unroll
                    for (int u = 0; u < 4; ++u) s += v[u];
                }
                for (; q < loss_blocks; q += 32) s += b.loss_part[(size_t)q * 4 + c];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
                l[c] = s / (float)R;
            }
            if (lane == 0) {
                b.stats->loss_pg = l[0];
                b.stats->loss_value = l[1];
                b.stats->entropy = l[2];
                b.stats->loss_total = l[0] + a.c_v * l[1] - a.c_e * l[2];
            }
        }
    }
}

// Debug record of the ReLU gates from the saved activations (h1 hi plane, h2).
template <bool GROUPED>
__global__ void __launch_bounds__(256) k_pack_gates2(DimsBuffers in, size_t R_in, int h2_bf16) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);  // many policies: grid.y = policy
    const Dims& d = pa.a.d;
    const Buffers& b = pa.a.b;
    const size_t R = GROUPED ? R_in / in.d.B * d.B : R_in;  // rows of THIS policy (R_in = B * T of a full one)
    const int lane = threadIdx.x & 31;
    const size_t words = R * (size_t)(d.H / 32);
    const __nv_bfloat16* h1hi = reinterpret_cast<const __nv_bfloat16*>(b.h1);
    for (size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5); w < 2 * words; w += (size_t)gridDim.x * 8) {
        bool on;
        if (w < words) on = (__bfloat16_as_ushort(h1hi[w * 32 + lane]) & 0x7FFFu) != 0;  // h1 >= 0: any magnitude bit
        else if (h2_bf16) on = (reinterpret_cast<const uint16_t*>(b.h2)[(w - words) * 32 + lane] & 0x7FFFu) != 0;
        else on = b.h2[(w - words) * 32 + lane] > 0.f;
        const uint32_t bits = __ballot_sync(0xFFFFFFFFu, on);
        if (lane == 0) b.dbg_gates[w] = bits;
    }
}

// ----------------------------------------------------------------------------------------------------
// host side
// ----------------------------------------------------------------------------------------------------
constexpr int HEADS_GRID = 2 * 148;  // persistent CTAs of k_heads_bwd (two per SM)

static int splits_for(int K, int tiles, int min_k) {
    int ns = (2 * 148 + tiles - 1) / tiles;
    const int cap = K / min_k > 0 ? K / min_k : 1;
    if (ns > cap) ns = cap;
    if (ns > 128) ns = 128;
    return ns < 1 ? 1 : ns;
}

// Launch shape of the fused dh1 + agent-plane kernel: one CTA per SM.  Few env tiles: slice the steps; many: let a CTA
// walk several tiles, so that the number of agent-plane partials stays at most one per CTA row.
static void dh1a_shape(const Dims& d, int T, int* grid_x, int* ts) {
    const int m_tiles = (d.B + 127) / 128, n_tiles = d.H / DH1A_UNITS;
    *grid_x = m_tiles;
    *ts = 1;
    if (m_tiles * n_tiles >= 148) {
        *grid_x = 148 / n_tiles > 0 ? 148 / n_tiles : 1;
    } else {
        int t = 148 / (m_tiles * n_tiles);
        if (t > 4) t = 4;
        if (t > T) t = T;
        if (t >= 2) *ts = t;
    }
}

// dW2 inside the heads kernel: hidden width 128 or 256, one policy.
static bool heads_fuse_dw2(const Dims& d, size_t R, int heads_grid, int prec) {
    (void)R; (void)prec;
    return (d.H == 128 || d.H == 256) && d.npol <= 1 && heads_grid >= 1;
}

void learn_mma_plan(const Dims& d, LearnPlan* p) {
    const int H = d.H, C = d.C;
    const size_t R = (size_t)d.B * d.Tmax;
    const int bt = H >= 128 ? 128 : 64;  // gemm tile side
    int tiles_hh = ((H + bt - 1) / bt) * ((H + bt - 1) / bt);
    const int tiles_ch = ((C + 1 + bt - 1) / bt) * ((H + bt - 1) / bt);
    int tiles_agent = tiles_ch;
    if (H > 256) {  // wide path: 128 x 256 output tiles in the tcgen05 GEMMs
        tiles_hh = (H / 128) * (H / 256);
        tiles_agent = ((C + 127) / 128) * (H / 256);
    }
    p->ns_w2 = splits_for((int)R, tiles_hh, 256);
    p->ns_agent = splits_for((int)R, tiles_agent, 256);
    if (H > 256) {  // the bf16 GEMM CTAs of the wide path take a whole SM each (four 48 KB stages): one wave
        p->ns_w2 = 148 / tiles_hh > 0 ? 148 / tiles_hh : 1;
    }
    if (dh1_agent_tc_supported(d)) {  // the fused kernel writes one agent-plane partial per (CTA row, t slice)
        int gx, ts;
        dh1a_shape(d, d.Tmax, &gx, &ts);
        if (gx * ts > p->ns_agent) p->ns_agent = gx * ts;
    }
    p->ns_env = splits_for(d.B, tiles_ch, 128);
    const size_t tiles32 = (R + 31) / 32;
    size_t hg = H == 256 ? HEADS_GRID / 2 : HEADS_GRID;  // (the H = 256 kernel takes a whole SM)
    if (d.npol > 1) hg = (size_t)(2 * HEADS_GRID / d.npol > 0 ? 2 * HEADS_GRID / d.npol : 1);  // many policies: the CTAs of all policies fill the GPU together
    p->heads_grid = (int)(tiles32 < hg ? tiles32 : hg);
    // (the fused heads + dW2 kernel writes one dW2 partial per CTA: room for the larger of the two partial counts)
    const int w2_slots = heads_fuse_dw2(d, R, p->heads_grid, 1) && p->heads_grid > p->ns_w2 ? p->heads_grid : p->ns_w2;
    p->ns_small = 4 * p->heads_grid;
    p->small_stride = (size_t)6 * H + 8;
    size_t off = 0;
    p->off_w2 = off; off += (size_t)w2_slots * H * H;
    p->off_agent = off; off += (size_t)p->ns_agent * C * H;
    p->off_walls = off; off += (size_t)p->ns_env * (C + 1) * H;
    p->off_goal = off; off += (size_t)p->ns_env * C * H;
    p->off_small = off; off += (size_t)p->ns_small * p->small_stride;
    p->part_floats = off;
    p->loss_blocks = p->heads_grid;
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

template <int H, int NW, int PREC, int HS = H, bool H2BF = false>
static cudaError_t launch_heads_t(const LearnArgs& a, int grid, cudaStream_t s, bool fuse = false) {
    using Cfg = HeadsCfg<H, NW, PREC, HS, H2BF>;
    HeadsMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (a.d.npol > 1) {
        if constexpr (PREC == 0 && HS == H && !H2BF) {
            CK(cudaFuncSetAttribute(k_heads_bwd<H, NW, PREC, HS, H2BF, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes));
            k_heads_bwd<H, NW, PREC, HS, H2BF, true><<<dim3(grid, 1, a.d.npol), Cfg::THREADS, Cfg::smem_bytes, s>>>(a, maps);
            return cudaGetLastError();
        }
        return cudaErrorNotSupported;
    }
    if constexpr ((H == 128 || H == 256) && HS == H && !H2BF) {
        if (fuse) {  // also dW2 = h1^T dh2 for the CTA's rows (tcgen05; the h1 tiles by TMA)
            using FCfg = HeadsCfg<H, NW, PREC, HS, H2BF, true>;
            const size_t R = (size_t)a.d.B * a.T, RH = (size_t)a.d.B * a.d.Tmax * H;
            const uint16_t* h1hi = reinterpret_cast<const uint16_t*>(a.b.h1);
            if (!make_tensor_map_2d(&maps.h1_hi, h1hi, R, H, FCfg::TR, PREC == 1)) return cudaErrorNotSupported;
            if (PREC == 0 && !make_tensor_map_2d(&maps.h1_lo, h1hi + RH, R, H, FCfg::TR, false)) return cudaErrorNotSupported;
            CK(cudaFuncSetAttribute(k_heads_bwd<H, NW, PREC, HS, H2BF, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FCfg::smem_bytes));
            k_heads_bwd<H, NW, PREC, HS, H2BF, false, true><<<dim3(grid, 1), FCfg::THREADS, FCfg::smem_bytes, s>>>(a, maps);
            return cudaGetLastError();
        }
    }
    CK(cudaFuncSetAttribute(k_heads_bwd<H, NW, PREC, HS, H2BF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes));
    k_heads_bwd<H, NW, PREC, HS, H2BF><<<dim3(grid, H / HS), Cfg::THREADS, Cfg::smem_bytes, s>>>(a, maps);
    return cudaGetLastError();
}

template <int H>
static cudaError_t launch_heads_tc_t(const LearnArgs& a, int grid, cudaStream_t s) {
    using Cfg = HeadsTcCfg<H>;
    CK(cudaFuncSetAttribute(k_heads_bwd_tc<H>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes));
    k_heads_bwd_tc<H><<<dim3(grid, H / Cfg::HS), 512, Cfg::smem_bytes, s>>>(a);
    return cudaGetLastError();
}

template <int H, int BN, int PREC>
static cudaError_t launch_dh1_t(const LearnArgs& a, cudaStream_t s) {
    using Cfg = Dh1Cfg<H, BN, PREC>;
    dim3 grid((a.d.B + Cfg::BM - 1) / Cfg::BM, H / BN);
    if (a.d.npol > 1) {
        if constexpr (PREC == 0) {
            CK(cudaFuncSetAttribute(k_dh1<H, BN, PREC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes));
            grid.z = a.d.npol;
            k_dh1<H, BN, PREC, true><<<grid, Cfg::THREADS, Cfg::smem_bytes, s>>>(a);
            return cudaGetLastError();
        }
        return cudaErrorNotSupported;
    }
    CK(cudaFuncSetAttribute(k_dh1<H, BN, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes));
    k_dh1<H, BN, PREC><<<grid, Cfg::THREADS, Cfg::smem_bytes, s>>>(a);
    return cudaGetLastError();
}

template <int PREC>
static cudaError_t launch_learn_mma_p(LearnArgs a, const Ctx& c) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const int H = d.H, C = d.C, B = d.B, T = a.T;
    const size_t R = (size_t)B * T, RH = (size_t)B * d.Tmax * H;
    cudaStream_t s = c.s;
    const bool wide = wide_supported(H, PREC);  // bf16 activations in HBM, layer-2 products as large tcgen05 GEMMs
    // many policies: every kernel gets one grid slice per policy and moves its workspace pointers there; the tcgen05
    // kernels bake addresses into tensor maps, so this path stays on the warp-level kernels
    const bool grouped = d.npol > 1;
    LearnPlan pl;
    learn_mma_plan(d, &pl);
    a.part_small = b.part + pl.off_small;
    a.small_stride = pl.small_stride;
    // parameter regions in flat order: W1 walls | W1 agent | W1 goal | b1 | W2 | b2 | Wh | bh
    const size_t CH = (size_t)C * H;
    a.reg[0] = PartRegion{b.part + pl.off_walls, pl.ns_env, (size_t)(C + 1) * H, d.oW1};
    a.reg[1] = PartRegion{b.part + pl.off_agent, pl.ns_agent, CH, d.oW1 + CH};
    a.reg[2] = PartRegion{b.part + pl.off_goal, pl.ns_env, CH, d.oW1 + 2 * CH};
    a.reg[3] = PartRegion{b.part + pl.off_walls + CH, pl.ns_env, (size_t)(C + 1) * H, d.ob1};  // the all-ones row
    a.reg[4] = PartRegion{b.part + pl.off_w2, pl.ns_w2, (size_t)H * H, d.oW2};
    a.reg[5] = PartRegion{b.part + pl.off_small + (size_t)5 * H, pl.ns_small, pl.small_stride, d.ob2};
    a.reg[6] = PartRegion{b.part + pl.off_small, pl.ns_small, pl.small_stride, d.oWh};
    a.reg[7] = PartRegion{b.part + pl.off_small + (size_t)6 * H, pl.ns_small, pl.small_stride, d.obh};

    // dW2 = h1^T dh2 rides in the heads kernel where its rows per CTA allow (it then has one partial per heads CTA)
    const bool fuse_dw2 = !wide && !grouped && b.w2p_hi != nullptr && heads_fuse_dw2(d, R, pl.heads_grid, PREC);
    if (fuse_dw2) a.reg[4].ns = pl.heads_grid;
    {
        Scope sc(c, K_HEADS_BWD);
        switch (H) {
            case 64: CK((launch_heads_t<64, 4, PREC>(a, pl.heads_grid, s))); break;
            case 128: CK((launch_heads_t<128, 8, PREC>(a, pl.heads_grid, s, fuse_dw2))); break;
            case 256: CK((launch_heads_t<256, 16, PREC>(a, pl.heads_grid, s, fuse_dw2))); break;
            default:
                if constexpr (PREC == 1) {
                    if (wide) {  // tensor-pipe version: one partial slot per CTA (slot 4 * CTA of the small region)
                        for (int q = 5; q <= 7; ++q) { a.reg[q].ns = pl.heads_grid; a.reg[q].stride = 4 * pl.small_stride; }
                        if (H == 512) { CK((launch_heads_tc_t<512>(a, pl.heads_grid, s))); break; }
                        if (H == 1024) { CK((launch_heads_tc_t<1024>(a, pl.heads_grid, s))); break; }
                        if (H == 2048) { CK((launch_heads_tc_t<2048>(a, pl.heads_grid, s))); break; }
                    }
                }
                return cudaErrorNotSupported;
        }
    }
    // t-slices: the tcgen05 dh1 kernel has ceil(B/128)*(H/128) CTAs per slice; slice the T steps so that one wave of
    // CTAs covers the SMs.  The mma.sync fall-back keeps one slice.
    a.ts = 1;
    bool fused_agent = false;  // dh1, S and the agent plane of dW1 in one kernel (dh1 stays on chip)
    if (!wide && !grouped && dh1_agent_tc_supported(d)) {
        int gx, ts;
        dh1a_shape(d, T, &gx, &ts);
        a.ts = ts;
        Scope sc(c, K_DH1);
        const cudaError_t ef = launch_dh1_agent_tc(a, PREC, gx, b.part + pl.off_agent, CH, s);
        if (ef == cudaSuccess) {
            fused_agent = true;
            a.reg[1].ns = gx * ts;
        } else if (ef != cudaErrorNotSupported) {
            return ef;
        } else {
            a.ts = 1;
        }
    }
    if (!fused_agent && !grouped && (H == 128 || H == 256)) {  // (the warp-level dh1 kernel walks all steps itself)
        const int per_slice = ((B + 127) / 128) * (H / 128);
        int ts = 148 / per_slice;
        if (ts > 4) ts = 4;
        if (ts > T) ts = T;
        if (ts >= 2) a.ts = ts;
    }
    if (fused_agent) {
    } else if (wide) {
        CK(launch_dh1_wide(a, c));
    } else {
        Scope sc(c, K_DH1);
        const cudaError_t etc = grouped ? cudaErrorNotSupported : launch_dh1_tc(a, PREC, s);  // tcgen05 where covered, else the mma.sync kernel
        if (etc != cudaErrorNotSupported) CK(etc);
        else a.ts = 1;
        if (etc == cudaErrorNotSupported) switch (H) {
            case 64: CK((launch_dh1_t<64, 64, PREC>(a, s))); break;
            case 128: CK((launch_dh1_t<128, 128, PREC>(a, s))); break;
            case 256: CK((launch_dh1_t<256, 128, PREC>(a, s))); break;
            default: return cudaErrorNotSupported;
        }
    }
    const __nv_bfloat16* h1hi = reinterpret_cast<const __nv_bfloat16*>(b.h1);
    const __nv_bfloat16* dh2hi = reinterpret_cast<const __nv_bfloat16*>(b.dh2);
    const __nv_bfloat16* dh1hi = reinterpret_cast<const __nv_bfloat16*>(b.dh1);
    const __nv_bfloat16* Shi = reinterpret_cast<const __nv_bfloat16*>(b.S);
    constexpr int PL = PREC == 1 ? 1 : 2;
    auto klen_of = [](int K, int ns) { return ((K + ns - 1) / ns + 63) / 64 * 64; };
    GemmTnArgs g;
    memset(&g, 0, sizeof(g));
    const size_t RH_last = (size_t)d.B_last * d.Tmax * H;  // plane offset inside the last policy's (more compact) buffers
    if (grouped) { g.npol = d.npol; g.pstride = d.pstride; }
    auto tc_gemm = [&](int amode, int apl, int bpl, int splits) {
        return grouped ? cudaErrorNotSupported : launch_gemm_tn_tc(g, amode, apl, bpl, PREC, splits, b.status, s);
    };
    // dW2 = h1^T dh2
    g.M = H; g.N = H; g.K = (int)R; g.klen = klen_of(g.K, pl.ns_w2);
    g.Ahi = h1hi; g.Alo = h1hi + RH; g.lda = H;
    g.Bhi = dh2hi; g.Blo = dh2hi + RH; g.ldb = H;
    g.part = b.part + pl.off_w2; g.stride = (size_t)H * H; g.off = 0; g.ldc = H; g.ones_row = -1;
    g.K_last = d.B_last * T; g.kmod_last = 0; g.alo_off_last = g.blo_off_last = RH_last;
    if (!fuse_dw2) {
        Scope sc(c, K_DW2);
        cudaError_t e = tc_gemm(A_PLANES, PL, PL, pl.ns_w2);  // tcgen05 where covered
        if (e == cudaErrorNotSupported) {
            if (H >= 128) e = launch_gemm_tn<128, 128, A_PLANES, PL, PL, PREC>(g, H, pl.ns_w2, s);
            else e = launch_gemm_tn<64, 64, A_PLANES, PL, PL, PREC>(g, H, pl.ns_w2, s);
        }
        CK(e);
    }
    // dW1, agent plane = onehot(pos)^T dh1
    g.M = C; g.K = (int)R; g.klen = klen_of(g.K, pl.ns_agent);
    g.idx = b.tpos;
    g.Bhi = dh1hi; g.Blo = dh1hi + RH;
    g.part = b.part + pl.off_agent; g.stride = CH; g.off = 0;
    if (!fused_agent) {
        Scope sc(c, K_DW1_AGENT);
        cudaError_t e = tc_gemm(A_ONEHOT, 1, PL, pl.ns_agent);
        if (e == cudaErrorNotSupported) {
            if (H >= 128) e = launch_gemm_tn<128, 128, A_ONEHOT, 1, PL, PREC>(g, C, pl.ns_agent, s);
            else e = launch_gemm_tn<64, 64, A_ONEHOT, 1, PL, PREC>(g, C, pl.ns_agent, s);
        }
        CK(e);
    }
    // dW1, wall plane (+ db1 through the all-ones row) = walls^T S; goal plane = onehot(goal)^T S
    g.K = a.ts * B; g.kmod = B; g.klen = klen_of(g.K, pl.ns_env);
    g.K_last = a.ts * d.B_last; g.kmod_last = d.B_last; g.blo_off_last = (size_t)a.ts * d.B_last * H;
    g.Bhi = Shi; g.Blo = Shi + (size_t)a.ts * B * H;
    g.walls = b.walls; g.W = d.W; g.ones_row = C; g.M = C + 1;
    g.part = b.part + pl.off_walls; g.stride = (size_t)(C + 1) * H; g.off = 0; g.off_ones = CH;
    bool env_planes_done = false;
    if (PREC == 0) {  // both planes in one launch: row tile 0 = wall bits + ones row, row tile 1 = one-hot of the goal cell
        g.idx2 = b.goal; g.M2 = C; g.part2 = b.part + pl.off_goal; g.stride2 = CH;
        Scope sc(c, K_DW1_WALLS);
        const cudaError_t e = tc_gemm(A_ENV, 1, 2, pl.ns_env);
        if (e == cudaSuccess) env_planes_done = true;
        else if (e != cudaErrorNotSupported) return e;
    }
    if (!env_planes_done) {
        {
            Scope sc(c, K_DW1_WALLS);
            cudaError_t e = tc_gemm(A_WALLS, 1, 2, pl.ns_env);
            if (e == cudaErrorNotSupported) {
                if (H >= 128) e = launch_gemm_tn<128, 128, A_WALLS, 1, 2, PREC>(g, C + 1, pl.ns_env, s);
                else e = launch_gemm_tn<64, 64, A_WALLS, 1, 2, PREC>(g, C + 1, pl.ns_env, s);
            }
            CK(e);
        }
        g.M = C; g.ones_row = -1; g.idx = b.goal;
        g.part = b.part + pl.off_goal; g.stride = CH;
        {
            Scope sc(c, K_DW1_GOAL);
            cudaError_t e = tc_gemm(A_ONEHOT, 1, 2, pl.ns_env);
            if (e == cudaErrorNotSupported) {
                if (H >= 128) e = launch_gemm_tn<128, 128, A_ONEHOT, 1, 2, PREC>(g, C, pl.ns_env, s);
                else e = launch_gemm_tn<64, 64, A_ONEHOT, 1, 2, PREC>(g, C, pl.ns_env, s);
            }
            CK(e);
        }
    }
    {
        Scope sc(c, K_REDUCE_ADAM);
        const unsigned nb = (unsigned)((d.ob2 + 255) / 256 + (d.P - d.ob2 + 7) / 8);
        if (d.npol > 1) {
            const unsigned per_policy = d.npol >= 74 ? 8u : (nb < 592u / d.npol ? nb : 592u / d.npol);  // at least four CTAs per SM in all, at most eight per policy
            if constexpr (PREC == 0) k_reduce_adam2<PREC, true><<<dim3(per_policy, d.npol), 256, 0, s>>>(a, R, pl.loss_blocks);
            else return cudaErrorNotSupported;
        } else {
            k_reduce_adam2<PREC, false><<<nb, 256, 0, s>>>(a, R, pl.loss_blocks);
        }
        CK(cudaGetLastError());
    }
    if (b.dbg_gates) {
        Scope sc(c, K_PACK_GATES);
        if (d.npol > 1) k_pack_gates2<true><<<dim3(64, d.npol), 256, 0, s>>>(DimsBuffers{d, b}, R, 0);
        else k_pack_gates2<false><<<148 * 8, 256, 0, s>>>(DimsBuffers{d, b}, R, wide ? 1 : 0);
        CK(cudaGetLastError());
    }
    return cudaSuccess;
}

cudaError_t launch_adam_only(const LearnArgs& a, int prec, const Ctx& c) {
    Scope sc(c, K_REDUCE_ADAM);
    const unsigned nb = (unsigned)((a.d.P + 255) / 256);
    if (a.d.npol > 1) {
        if (prec == 1) return cudaErrorNotSupported;
        k_adam_only<0, true><<<dim3(nb, a.d.npol), 256, 0, c.s>>>(a);
    } else if (prec == 1) k_adam_only<1, false><<<nb, 256, 0, c.s>>>(a);
    else k_adam_only<0, false><<<nb, 256, 0, c.s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_learn_mma(const LearnArgs& a, int prec, const Ctx& c) {
    return prec == 1 ? launch_learn_mma_p<1>(a, c) : launch_learn_mma_p<0>(a, c);
}

}  // namespace anakin
