// Weight-gradient GEMMs on the 5th-generation tensor cores:  C[m][n] = sum_k A[k][m] B[k][n],  K = B*T rows.
//
// These are the batch-mean reductions of the update (the single-device form of the paper's cross-core gradient average,
// Podracer paper, Section 3.1): dW2 = h1^T dh2 and the agent plane of dW1 = onehot(pos)^T dh1.  Both operands have the
// contraction index as their slow (row) index, i.e. they are "MN-major" for the MMA.
//
// One CTA owns a 128 x BN output tile (BN = the hidden width up to 256, else column tiles of 256; the accumulator
// columns live in tensor memory) and a
// K range (split-K; partials are summed later in a fixed order).  Per 64-row K chunk:
//   warp 0 (one lane)  issues TMA loads of the operand planes (64 x 64 boxes, 128-byte swizzle) into a 2-stage ring,
//   warps 2-5          for the one-hot A operand: write the 0/1 tile straight into the swizzled layout instead of loading it,
//   warp 1 (one lane)  issues tcgen05.mma: for fp32 workloads three MMAs per k16 (lo*hi, hi*lo, hi*hi fp16 terms) into one
//                      fp32 accumulator; commits free the stage,
//   warps 2-5          after the last chunk: tcgen05.ld the accumulator and store the partial tile.
// Long K ranges (plane operands): the tensor core's fp32 accumulation rounds toward zero, which biases a sum of many
// thousand MMAs by more than the fp32 workloads' 1e-4 bound (measured: -2e-4 after 65,536 rows; fp32 workloads only).  The K range of a CTA
// is therefore cut into groups of GROUP chunks; the groups alternate between two accumulators in tensor memory, and
// while the MMAs of one group run, warps 2-5 add the previous group's accumulator into the partial tile in global
// memory with ordinary (round-to-nearest) fp32 additions, in group order.
// Every wait is bounded; a timeout raises DEV_E_WAIT_TIMEOUT in the status word and the CTA unwinds (tensor memory freed).
#include <cstdio>
#include <cstring>

#include "tc_common.cuh"

namespace anakin {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

bool make_tensor_map_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool bf16) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same over a row-major byte matrix [rows][cols] (cols a multiple of 16) with a box of box_cols x box_rows bytes, not swizzled.
bool make_tensor_map_u8(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn enc = encode_fn();
    if (!enc || cols % 16 != 0 || box_cols % 16 != 0) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// DEEP: as many stages as fit (plane operands, TMA-latency-bound); otherwise two, so that two CTAs share an SM (the
// synthesized-A modes are bound by their builder threads, and a second CTA hides them).
template <int BN, int APL, int BPL, bool DEEP, int PREC = 0>
struct GemmTcCfg {
    static constexpr int BM = 128, KC = 64, THREADS = 192;
    static constexpr int BOX = 64 * 64 * 2;                  // one 64 x 64 box of 16-bit elements
    static constexpr int A_PLANE = (BM / 64) * BOX;          // 16 KB
    static constexpr int B_PLANE = (BN / 64) * BOX;
    static constexpr int STAGE = APL * A_PLANE + BPL * B_PLANE;
    // as many stages as fit beside the slack (the loads are latency-bound: bytes in flight set the rate), at most 4
    static constexpr int FIT = (232448 - 1024 - 128) / STAGE;
    static constexpr int STAGES = !DEEP ? 2 : (FIT >= 4 ? 4 : (FIT >= 2 ? FIT : 2));
    static constexpr size_t smem_bytes = (size_t)STAGES * STAGE + 1024 /*alignment slack*/ + 128 /*barriers, tmem slot*/;
    // plane operands of the fp32 workloads: two accumulators, a group of GROUP 64-row chunks (4096 rows, 768 MMAs) each.
    // The bf16 workload's 2e-2 bound does not need it.
    static constexpr bool FLUSH = DEEP && PREC == 0;
    static constexpr int GROUP = 64;
    static constexpr int TMEM_COLS = FLUSH ? 2 * BN : BN;
};

struct GemmTcMaps {
    CUtensorMap a_hi, a_lo, b_hi, b_lo;
};

template <int BN, int AMODE, int APL, int BPL, int PREC>
__global__ void __launch_bounds__(192, 1) k_gemm_tn_tc(const __grid_constant__ GemmTcMaps maps, GemmTnArgs g, int* status) {
    using Cfg = GemmTcCfg<BN, APL, BPL, AMODE == A_PLANES, PREC>;
    constexpr int BM = Cfg::BM, KC = Cfg::KC, STAGES = Cfg::STAGES;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // the swizzle needs 1024-byte alignment
    uint64_t* bars = (uint64_t*)(base + STAGES * Cfg::STAGE);  // full[STAGES], empty[STAGES], accfull[2], accempty[2]
    uint64_t* accfull = bars + 2 * STAGES;
    uint64_t* accempty = accfull + 2;
    uint32_t* tmem_slot = (uint32_t*)(accempty + 2);
    constexpr bool FLUSH = Cfg::FLUSH;
    constexpr int GROUP = Cfg::GROUP;
    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    // A_ENV: two row tiles with different synthesized A operands (wall bits + ones row; one-hot of idx2), each with its own M space
    const int amode = AMODE == A_ENV ? (blockIdx.x == 0 ? A_WALLS : A_ONEHOT) : AMODE;
    const int m0 = AMODE == A_ENV ? 0 : blockIdx.x * BM, n0 = blockIdx.y * BN, split = blockIdx.z;
    const uint8_t* oh_idx = (AMODE == A_ENV) ? g.idx2 : g.idx;
    const int kbeg = split * g.klen, kend = min(g.K, kbeg + g.klen);
    const int nchunks = kend > kbeg ? (kend - kbeg + KC - 1) / KC : 0;
    const int ngroups = FLUSH ? (nchunks + GROUP - 1) / GROUP : (nchunks > 0 ? 1 : 0);
    constexpr uint32_t NBUILD = AMODE == A_PLANES ? 0u : 128u;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&bars[s], 1 + NBUILD); tc::mbar_init(&bars[STAGES + s], 1); }
        for (int q = 0; q < 2; ++q) { tc::mbar_init(&accfull[q], 1); tc::mbar_init(&accempty[q], 128); }
        tc::mbar_fence_init();
    }
    if (wid == 2) tc::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (wid == 0) {
        if (lane == 0) {  // ---- TMA producer
            for (int c = 0; c < nchunks && ok; ++c) {
                const int s = c % STAGES, k0 = kbeg + c * KC;
                if (c >= STAGES) ok = tc::mbar_wait(&bars[STAGES + s], ((c / STAGES) - 1) & 1);
                if (!ok) break;
                unsigned char* st = base + s * Cfg::STAGE;
                constexpr uint32_t tx = (AMODE == A_PLANES ? APL * Cfg::A_PLANE : 0) + BPL * Cfg::B_PLANE;
                tc::mbar_expect_tx(&bars[s], tx);
                if (AMODE == A_PLANES) {
#pragma unroll
                    for (int bx = 0; bx < BM / 64; ++bx) {
                        tc::tma_load_2d(st + bx * Cfg::BOX, &maps.a_hi, &bars[s], m0 + 64 * bx, k0);
                        if (APL == 2) tc::tma_load_2d(st + Cfg::A_PLANE + bx * Cfg::BOX, &maps.a_lo, &bars[s], m0 + 64 * bx, k0);
                    }
                }
                unsigned char* sb = st + APL * Cfg::A_PLANE;
#pragma unroll
                for (int bx = 0; bx < BN / 64; ++bx) {
                    tc::tma_load_2d(sb + bx * Cfg::BOX, &maps.b_hi, &bars[s], n0 + 64 * bx, k0);
                    if (BPL == 2) tc::tma_load_2d(sb + Cfg::B_PLANE + bx * Cfg::BOX, &maps.b_lo, &bars[s], n0 + 64 * bx, k0);
                }
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else if (wid == 1) {
        if (lane == 0) {  // ---- MMA issuer
            const uint32_t idesc = tc::umma_idesc<PREC>(BM, BN, true, true);
            for (int c = 0; c < nchunks && ok; ++c) {
                const int s = c % STAGES;
                const int grp = FLUSH ? c / GROUP : 0, cg = FLUSH ? c - grp * GROUP : c;  // accumulator group, chunk within it
                const uint32_t acc = tmem + (uint32_t)((grp & 1) * BN);
                // the third and later groups reuse an accumulator: wait until the epilogue warps have read it out
                if (FLUSH && cg == 0 && grp >= 2) ok = tc::mbar_wait(&accempty[grp & 1], ((grp >> 1) - 1) & 1);
                if (ok) ok = tc::mbar_wait(&bars[s], (c / STAGES) & 1);
                if (!ok) break;
                tc::tc_fence_after();
                unsigned char* sa = base + s * Cfg::STAGE;
                unsigned char* sb = sa + APL * Cfg::A_PLANE;
#pragma unroll
                for (int k16 = 0; k16 < KC / 16; ++k16) {
                    // 16 k rows = two 8-row groups = 2048 bytes further into every box
                    const uint64_t a_hi = tc::umma_desc(sa + k16 * 2048, Cfg::BOX, 1024);
                    const uint64_t b_hi = tc::umma_desc(sb + k16 * 2048, Cfg::BOX, 1024);
                    uint32_t accum = (cg > 0 || k16 > 0) ? 1u : 0u;
                    if (APL == 2) { tc::umma(acc, tc::umma_desc(sa + Cfg::A_PLANE + k16 * 2048, Cfg::BOX, 1024), b_hi, idesc, accum); accum = 1u; }
                    if (BPL == 2) { tc::umma(acc, a_hi, tc::umma_desc(sb + Cfg::B_PLANE + k16 * 2048, Cfg::BOX, 1024), idesc, accum); accum = 1u; }
                    tc::umma(acc, a_hi, b_hi, idesc, accum);
                }
                tc::umma_commit(&bars[STAGES + s]);  // frees the stage when these MMAs are done
                if (c == nchunks - 1 || (FLUSH && cg == GROUP - 1)) tc::umma_commit(&accfull[grp & 1]);  // this group's sum is complete
            }
            if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
    } else {
        // ---- warps 2-5: builders of a synthesized A tile, then the epilogue
        const int bt = tid - 64;  // 0..127
        if (AMODE != A_PLANES) {
            // (after a timeout the loop keeps going without waiting, so that every thread still meets every bar.sync)
            for (int c = 0; c < nchunks; ++c) {
                const int s = c % STAGES, k0 = kbeg + c * KC;
                if (ok && c >= STAGES) ok = tc::mbar_wait(&bars[STAGES + s], ((c / STAGES) - 1) & 1);
                unsigned char* sa = base + s * Cfg::STAGE;
                // element (k, m) of the tile lives in box m/64 at byte  k*128 + (((m%64)/8) ^ (k%8))*16 + (m%8)*2
                if (amode == A_ONEHOT) {
                    uint4* z = reinterpret_cast<uint4*>(sa);
                    for (int i = bt; i < Cfg::A_PLANE / 16; i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
                    asm volatile("bar.sync 1, 128;" ::: "memory");  // zeros before ones
                    if (bt < KC && k0 + bt < kend) {
                        const int m = (int)oh_idx[g.kmod ? (k0 + bt) % g.kmod : (k0 + bt)] - m0;
                        if (m >= 0 && m < BM) {
                            const int k = bt;
                            const uint32_t off = (m >> 6) * Cfg::BOX + k * 128 + ((((m & 63) >> 3) ^ (k & 7)) << 4) + (m & 7) * 2;
                            *reinterpret_cast<uint16_t*>(sa + off) = (uint16_t)one16<PREC>();
                        }
                    }
                } else {  // A_WALLS: thread = (k row, 64-wide box); it writes all eight 16-byte chunks of its row segment
                    const int k = bt >> 1, bx = bt & 1;
                    const int kk = k0 + k;
                    // the 64 cells m = mb .. mb + 63 of this box as one bit mask: wall bits below ones_row, the ones row itself
                    const int mb = m0 + 64 * bx;  // a multiple of 64: two whole words of the env's wall mask
                    unsigned long long bits = 0ull;
                    if (kk < kend) {
                        const uint32_t* wrow = g.walls + (size_t)(g.kmod ? kk % g.kmod : kk) * g.W;
                        const int w0 = mb >> 5;
                        const uint32_t lo32 = w0 < g.W ? wrow[w0] : 0u, hi32 = w0 + 1 < g.W ? wrow[w0 + 1] : 0u;
                        bits = (unsigned long long)lo32 | ((unsigned long long)hi32 << 32);
                        const int r1 = g.ones_row - mb;  // position of the ones row in this box
                        if (r1 <= 0) bits = 0ull;
                        else if (r1 < 64) bits &= (1ull << r1) - 1ull;
                        if (r1 >= 0 && r1 < 64) bits |= 1ull << r1;
                    }
                    const uint32_t one = one16<PREC>();
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) {
                        const uint32_t by = (uint32_t)(bits >> (8 * c8)) & 0xFFu;
                        uint32_t w[4];
#pragma unroll
                        for (int q2 = 0; q2 < 4; ++q2) w[q2] = ((by >> (2 * q2)) & 1u) * one | ((by >> (2 * q2 + 1)) & 1u) * (one << 16);
                        *reinterpret_cast<uint4*>(sa + bx * Cfg::BOX + k * 128 + ((c8 ^ (k & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
                tc::fence_proxy_async();  // generic-proxy stores -> visible to the tensor core
                tc::mbar_arrive(&bars[s]);
            }
            if (!ok && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
        }
        // epilogue: warp w reads accumulator lanes 32*(w%4)..+31 = output rows.  Group 0 writes the partial tile, every
        // later group adds to what this same thread wrote (program order; round-to-nearest additions in group order).
        const int q = wid & 3;
        const int m = m0 + 32 * q + lane;
        const bool second = AMODE == A_ENV && blockIdx.x == 1;
        const int Mrows = second ? g.M2 : g.M;
        float* part = second ? g.part2 + (size_t)split * g.stride2 : g.part + (size_t)split * g.stride + g.off;
        bool got = true;
        for (int grp = 0; grp < (ngroups > 0 ? ngroups : 1); ++grp) {
            if (ngroups > 0 && got) got = tc::mbar_wait(&accfull[grp & 1], (grp >> 1) & 1);
            tc::tc_fence_after();
            __syncwarp();
            const uint32_t acc = tmem + (uint32_t)((grp & 1) * BN) + ((uint32_t)(32 * q) << 16);
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                if (ngroups > 0 && got) {
                    tc::tmem_ld32(acc + (uint32_t)c0, r);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;  // an empty K range contributes zeros
                }
                if (m < Mrows && n0 + c0 < g.N) {
                    float4* dst = reinterpret_cast<float4*>(part + (size_t)m * g.ldc + n0 + c0);
                    if (amode == A_WALLS && m == g.ones_row) dst = reinterpret_cast<float4*>(part - g.off + g.off_ones + n0 + c0);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                               __uint_as_float(r[4 * j + 3]));
                        if (grp > 0) {
                            const float4 o = dst[j];
                            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                        }
                        dst[j] = v;
                    }
                }
            }
            if (FLUSH && grp + 2 < ngroups) {  // hand the accumulator back to the issuer
                tc::tc_fence_before();
                tc::mbar_arrive(&accempty[grp & 1]);
            }
        }
        if (!got && lane == 0) atomicOr(status, DEV_E_WAIT_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (wid == 2) tc::tmem_dealloc(tmem, Cfg::TMEM_COLS);
}

template <int BN, int AMODE, int APL, int BPL, int PREC>
static cudaError_t launch_t(const GemmTnArgs& g, int splits, int* status, cudaStream_t s) {
    using Cfg = GemmTcCfg<BN, APL, BPL, AMODE == A_PLANES, PREC>;
    GemmTcMaps maps;
    memset(&maps, 0, sizeof(maps));
    const bool bf = PREC == 1;
    if (AMODE == A_PLANES) {
        if (!make_tensor_map_2d(&maps.a_hi, g.Ahi, (uint64_t)g.K, (uint64_t)g.lda, 64, bf)) return cudaErrorNotSupported;
        if (APL == 2 && !make_tensor_map_2d(&maps.a_lo, g.Alo, (uint64_t)g.K, (uint64_t)g.lda, 64, bf)) return cudaErrorNotSupported;
    }
    if (!make_tensor_map_2d(&maps.b_hi, g.Bhi, (uint64_t)g.K, (uint64_t)g.ldb, 64, bf)) return cudaErrorNotSupported;
    if (BPL == 2 && !make_tensor_map_2d(&maps.b_lo, g.Blo, (uint64_t)g.K, (uint64_t)g.ldb, 64, bf)) return cudaErrorNotSupported;
    cudaError_t e = cudaFuncSetAttribute(k_gemm_tn_tc<BN, AMODE, APL, BPL, PREC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::smem_bytes);
    if (e != cudaSuccess) return e;
    dim3 grid(AMODE == A_ENV ? 2 : (g.M + Cfg::BM - 1) / Cfg::BM, (g.N + BN - 1) / BN, splits);
    k_gemm_tn_tc<BN, AMODE, APL, BPL, PREC><<<grid, Cfg::THREADS, Cfg::smem_bytes, s>>>(maps, g, status);
    return cudaGetLastError();
}

template <int BN, int PREC>
static cudaError_t launch_bn(const GemmTnArgs& g, int amode, int bpl, int splits, int* status, cudaStream_t s) {
    constexpr int PL = PREC == 1 ? 1 : 2;
    if (PREC == 1 && bpl == 2) {  // bf16 workload with a two-term B (the sum over t of dh1): synthesized A only
        if (amode == A_ONEHOT) return launch_t<BN, A_ONEHOT, 1, 2, PREC>(g, splits, status, s);
        if (amode == A_WALLS) return launch_t<BN, A_WALLS, 1, 2, PREC>(g, splits, status, s);
        return cudaErrorNotSupported;
    }
    if (amode == A_PLANES) return launch_t<BN, A_PLANES, PL, PL, PREC>(g, splits, status, s);
    if (amode == A_ONEHOT) return launch_t<BN, A_ONEHOT, 1, PL, PREC>(g, splits, status, s);
    if (amode == A_WALLS) return launch_t<BN, A_WALLS, 1, PL, PREC>(g, splits, status, s);
    if (amode == A_ENV && g.M <= 128 && g.M2 <= 128) return launch_t<BN, A_ENV, 1, PL, PREC>(g, splits, status, s);
    return cudaErrorNotSupported;
}

// Covered: N = ldb = 64, 128, 256 or a multiple of 256 (column tiles of 256 on grid.y), klen a multiple of 64, A planes or one-hot A,
// operand planes as the fp32 workloads (hi+lo fp16) or the bf16 workload (one plane) use them.
cudaError_t launch_gemm_tn_tc(const GemmTnArgs& g, int amode, int apl, int bpl, int prec, int splits, int* status, cudaStream_t s) {
    const int pl = prec == 1 ? 1 : 2;
    if (g.N != g.ldb || g.klen % 64 != 0 || (bpl != pl && !(prec == 1 && bpl == 2 && amode != A_PLANES)) ||
        (amode == A_PLANES && (apl != pl || g.lda % 64 != 0)))
        return cudaErrorNotSupported;
    if (amode != A_PLANES && apl != 1) return cudaErrorNotSupported;
    const int bn = g.N > 256 && g.N % 256 == 0 ? 256 : g.N;
    if (prec == 1) {
        switch (bn) {
            case 64: return launch_bn<64, 1>(g, amode, bpl, splits, status, s);
            case 128: return launch_bn<128, 1>(g, amode, bpl, splits, status, s);
            case 256: return launch_bn<256, 1>(g, amode, bpl, splits, status, s);
        }
    } else {
        switch (bn) {
            case 64: return launch_bn<64, 0>(g, amode, bpl, splits, status, s);
            case 128: return launch_bn<128, 0>(g, amode, bpl, splits, status, s);
            case 256: return launch_bn<256, 0>(g, amode, bpl, splits, status, s);
        }
    }
    return cudaErrorNotSupported;
}

}  // namespace anakin
