// Shared pieces of the wide-path GEMM kernels  C[m][n] = sum_k A[m][k] Bop[k][n]  (bf16 operands, fp32 accumulators in
// tensor memory): argument block, tensor maps, and the per-row epilogue that both the one-CTA and the CTA-pair kernel use.
#pragma once
#include "tc_common.cuh"

namespace anakin {
namespace widegemm {

enum : int { EPI_FWD = 0, EPI_GATE = 1, EPI_BASE = 2 };

struct NtArgs {
    int M, N, K;           // C is M x N; M rows starting at row0 of A, out and gate
    int row0;
    uint16_t* out;         // bf16 [rows][N]
    const float* bias;     // EPI_FWD, EPI_BASE: [N]
    const uint16_t* gate;  // EPI_GATE: bf16 [rows][N], non-negative; out = gate > 0 ? acc : 0
    float* outf;           // EPI_BASE: fp32 [rows][N] = acc + bias[n] + addrows[(addrow0 + addidx[m])*N + n]
    const float* addrows;
    const uint8_t* addidx;
    int addrow0;
    int* status;
};

struct NtMaps {
    CUtensorMap a, b;
};

constexpr int NT_BN = 256;    // accumulator columns of an output tile
constexpr int NT_MAXN = 2048;  // bias staging in shared memory

// Pulls the gate bytes of one output row's tile (512 B) towards L2; called before the accumulator is waited for.
__device__ __forceinline__ void nt_prefetch_gate(const NtArgs& g, size_t gi) {
#pragma unroll
    for (int l = 0; l < 4; ++l) asm volatile("prefetch.global.L2 [%0];" ::"l"(g.gate + gi + 64 * l));
}

constexpr int NT_STAGE_BYTES = 4096;  // per epilogue warp: 32 rows x 64 bf16 columns
constexpr int NT_EPI_WARPS = 8;       // warps 2..9: lane quarter (wid % 4) x column half ((wid - 2) / 4)

// A warp's 32 output rows (accumulator lanes) and columns [c_begin, c_end) of a 256-column tile, 64 columns at a time:
//   EPI_FWD   bf16(relu(acc + bias))                       EPI_GATE  bf16(gate > 0 ? acc : 0)
//   EPI_BASE  fp32: acc + bias + the row's extra weight row
// The memory system takes one request per 16-byte piece a lane touches, and a lane = row mapping touches 32 different
// lines per instruction, so the bf16 tiles go through a warp-private staging buffer (16-byte chunks XOR-swizzled by the
// row to stay conflict-free): gates are LOADED and results STORED with 8 lanes per row, i.e. whole 128-byte lines.
// taddr = tensor-memory address of the warp's first lane and the tile's first column; mb = output row of lane 0.
template <int EPI>
__device__ __forceinline__ void nt_epilogue_warp(const NtArgs& g, const float* s_bias, unsigned char* stage, uint32_t taddr, int mb, int n0,
                                                 int lane, int c_begin, int c_end) {
    const int m = mb + lane;
    const bool valid = m < g.M;
    const size_t gi = ((size_t)g.row0 + (valid ? m : 0)) * g.N + n0;  // this lane's own row (EPI_BASE)
    const int crow = lane >> 3, cch = lane & 7;                       // coalesced phase: row 4i + crow, 16-byte chunk cch
#pragma unroll 1
    for (int c0 = c_begin; c0 < c_end; c0 += 64) {
        uint32_t r0[32], r1[32];
        if (EPI == EPI_BASE) {
            tc::tmem_ld32(taddr + (uint32_t)c0, r0);
            tc::tmem_ld32(taddr + (uint32_t)(c0 + 32), r1);
            if (valid) {
                const float4* add = reinterpret_cast<const float4*>(g.addrows + ((size_t)g.addrow0 + g.addidx[m]) * g.N + n0 + c0);
                float4* dst = reinterpret_cast<float4*>(g.outf + gi + c0);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float4 w = __ldg(add + j);
                    const float* bs = s_bias + n0 + c0 + 4 * j;
                    const uint32_t* r = j < 8 ? r0 + 4 * j : r1 + 4 * (j - 8);
                    dst[j] = make_float4(__uint_as_float(r[0]) + bs[0] + w.x, __uint_as_float(r[1]) + bs[1] + w.y,
                                         __uint_as_float(r[2]) + bs[2] + w.z, __uint_as_float(r[3]) + bs[3] + w.w);
                }
            }
            continue;
        }
        uint4 gt[8];
        if (EPI == EPI_GATE) {  // gates of the 32 rows x 64 columns: whole lines in, then every lane picks up its row
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int row = 4 * i + crow;
                const bool rv = mb + row < g.M;
                const uint4 v = rv ? __ldg(reinterpret_cast<const uint4*>(g.gate + ((size_t)g.row0 + mb + row) * g.N + n0 + c0) + cch)
                                   : make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(stage + row * 128 + ((cch ^ (row & 7)) << 4)) = v;
            }
            __syncwarp();
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) gt[ch] = *reinterpret_cast<const uint4*>(stage + lane * 128 + ((ch ^ (lane & 7)) << 4));
            __syncwarp();
        }
        tc::tmem_ld32(taddr + (uint32_t)c0, r0);
        tc::tmem_ld32(taddr + (uint32_t)(c0 + 32), r1);
        const uint32_t* gw = reinterpret_cast<const uint32_t*>(gt);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {  // 8 columns = one 16-byte chunk of bf16
            uint32_t pk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int col = 8 * ch + 2 * j;
                float x0 = __uint_as_float(col < 32 ? r0[col] : r1[col - 32]);
                float x1 = __uint_as_float(col < 32 ? r0[col + 1] : r1[col - 31]);
                if (EPI == EPI_FWD) {
                    x0 = fmaxf(x0 + s_bias[n0 + c0 + col], 0.f);
                    x1 = fmaxf(x1 + s_bias[n0 + c0 + col + 1], 0.f);
                } else {
                    const uint32_t gv = gw[4 * ch + j];
                    x0 = (gv & 0x00007FFFu) ? x0 : 0.f;  // gate >= 0: "> 0" is "any magnitude bit set"
                    x1 = (gv & 0x7FFF0000u) ? x1 : 0.f;
                }
                pk[j] = pack_bf16(__float2bfloat16_rn(x0), __float2bfloat16_rn(x1));
            }
            *reinterpret_cast<uint4*>(stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 8; ++i) {  // whole lines out
            const int row = 4 * i + crow;
            if (mb + row < g.M)
                reinterpret_cast<uint4*>(g.out + ((size_t)g.row0 + mb + row) * g.N + n0 + c0)[cch] =
                    *reinterpret_cast<const uint4*>(stage + row * 128 + ((cch ^ (row & 7)) << 4));
        }
        __syncwarp();
    }
}

// CTA-pair kernel (wide2.cu): cudaErrorNotSupported when the shape is not covered.
cudaError_t launch_nt_pair(int epi, bool b_mn, const NtMaps& maps, const NtArgs& g, cudaStream_t s);

}  // namespace widegemm
}  // namespace anakin
