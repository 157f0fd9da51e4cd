// Learning half of the Anakin minimal unit (Podracer paper, Section 3.1; Figure 2, top): the parameter update
// computed from the T recorded interactions.  The forward pass is recomputed on all R = B*T rows (the paper
// notes the update may reuse the policy's forward pass; parameters do not change between acting and
// learning, so recomputing gives the same function), the A2C loss gradient is formed per row, back-propagated
// through the MLP, averaged over the whole batch (the single-device form of the paper's cross-core average,
// done here as fixed-order split-K partial sums so that results are run-to-run identical), and applied by Adam.
#include "common.cuh"

namespace anakin {

// h1[i][j] = relu(base[b][j] + W1[C+pos_i][j]),  b = i % B
template <int PREC>
__global__ void __launch_bounds__(256) k_h1(Dims d, Buffers b, size_t R) {
    const size_t total = R * (size_t)d.H;
    const float* W1 = b.theta_c + d.oW1;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const size_t i = idx / d.H;
        const int j = (int)(idx - i * d.H);
        const int e = (int)(i % (size_t)d.B);
        const float z = b.base[(size_t)e * d.H + j] + W1[(size_t)(d.C + b.tpos[i]) * d.H + j];
        b.h1[idx] = rnd<PREC>(fmaxf(z, 0.f));
    }
}

// ----------------------------------------------------------------------------------------------------
// Generic FFMA GEMM, 64x64x16 tiles, 256 threads, 4x4 outputs per thread, optional split-K over blockIdx.z.
// AL(m,k) / BL(k,n) are element loaders (with a flag saying which index is contiguous in memory so that the
// cooperative tile load is coalesced); EP(m,n,acc,split) consumes a finished element.
// ----------------------------------------------------------------------------------------------------
template <class AL, class BL, class EP>
__global__ void __launch_bounds__(256) k_sgemm(int M, int N, int K, int klen, AL al, BL bl, EP ep) {
    __shared__ __align__(16) float As[16][68];
    __shared__ __align__(16) float Bs[16][68];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * 64, n0 = blockIdx.y * 64;
    const int split = blockIdx.z;
    const int kbeg = split * klen;
    const int kend = min(K, kbeg + klen);
    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = kbeg; k0 < kend; k0 += 16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = tid + 256 * i;
            int mm, kk;
            if (AL::kfast) { kk = idx & 15; mm = idx >> 4; } else { mm = idx & 63; kk = idx >> 6; }
            As[kk][mm] = (m0 + mm < M && k0 + kk < kend) ? al(m0 + mm, k0 + kk) : 0.f;
            int nn, kb;
            if (BL::kfast) { kb = idx & 15; nn = idx >> 4; } else { nn = idx & 63; kb = idx >> 6; }
            Bs[kb][nn] = (n0 + nn < N && k0 + kb < kend) ? bl(k0 + kb, n0 + nn) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float a4[4] = {av.x, av.y, av.z, av.w};
            const float b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a4[i], b4[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (m < M && n < N) ep(m, n, acc[i][j], split);
        }
}

// loaders ---------------------------------------------------------------------------------------------
struct LdRowMajorA {  // A(m,k) = p[m*ld + k]
    static constexpr bool kfast = true;
    const float* p; int ld;
    __device__ float operator()(int m, int k) const { return p[(size_t)m * ld + k]; }
};
struct LdTransA {  // A(m,k) = p[k*ld + m]
    static constexpr bool kfast = false;
    const float* p; int ld;
    __device__ float operator()(int m, int k) const { return p[(size_t)k * ld + m]; }
};
struct LdRowMajorB {  // B(k,n) = p[k*ld + n]
    static constexpr bool kfast = false;
    const float* p; int ld;
    __device__ float operator()(int k, int n) const { return p[(size_t)k * ld + n]; }
};
struct LdTransB {  // B(k,n) = p[n*ld + k]
    static constexpr bool kfast = true;
    const float* p; int ld;
    __device__ float operator()(int k, int n) const { return p[(size_t)n * ld + k]; }
};
// one-hot observation planes, transposed: A(m = cell, k = row or env)
struct LdAgentPlane {
    static constexpr bool kfast = false;
    const uint8_t* tpos;
    __device__ float operator()(int m, int k) const { return tpos[k] == m ? 1.f : 0.f; }
};
struct LdWallPlane {
    static constexpr bool kfast = false;
    const uint32_t* walls; int W;
    __device__ float operator()(int m, int k) const { return (float)((walls[(size_t)k * W + (m >> 5)] >> (m & 31)) & 1u); }
};
struct LdGoalPlane {
    static constexpr bool kfast = false;
    const uint8_t* goal;
    __device__ float operator()(int m, int k) const { return goal[k] == m ? 1.f : 0.f; }
};

// epilogues -------------------------------------------------------------------------------------------
template <int PREC>
struct EpBiasRelu {  // h2 = relu(acc + bias)
    float* out; const float* bias; int ld;
    __device__ void operator()(int m, int n, float acc, int) const { out[(size_t)m * ld + n] = rnd<PREC>(fmaxf(acc + bias[n], 0.f)); }
};
template <int PREC>
struct EpReluMask {  // dh1 = acc where the forward activation was positive
    float* out; const float* act; int ld;
    __device__ void operator()(int m, int n, float acc, int) const {
        const size_t i = (size_t)m * ld + n;
        out[i] = rnd<PREC>(act[i] > 0.f ? acc : 0.f);
    }
};
struct EpPartial {  // split-K partial of a weight gradient, in flat parameter layout
    float* part; size_t P; size_t off; int ld;
    __device__ void operator()(int m, int n, float acc, int split) const { part[(size_t)split * P + off + (size_t)m * ld + n] = acc; }
};

// ----------------------------------------------------------------------------------------------------
// Heads, loss and output gradients, one warp per row:
//   out = h2 Wh + bh;  p = softmax(logits);  H = -sum p log p
//   dz_k = [-A (1{k=a} - p_k) + c_e p_k (log p_k + H)] / R;   dV = 2 c_v (V - ret) / R
//   dh2 = (dOut Wh^T) masked by h2 > 0
// ----------------------------------------------------------------------------------------------------
template <int PREC>
__global__ void __launch_bounds__(256) k_heads_loss(Dims d, Buffers b, size_t R, float c_v, float c_e, float ppo_clip) {
    __shared__ float s_loss[8][3];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int H = d.H;
    const float* Wh = b.theta_c + d.oWh;
    const float* bh = b.theta_c + d.obh;
    const float invR = 1.0f / (float)R;
    float l_pg = 0.f, l_v = 0.f, l_ent = 0.f;
    for (size_t i = (size_t)blockIdx.x * 8 + wid; i < R; i += (size_t)gridDim.x * 8) {
        const float* h2 = b.h2 + i * H;
        float o[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
        for (int k = lane; k < H; k += 32) {
            const float x = h2[k];
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c] = fmaf(x, __ldg(Wh + k * 5 + c), o[c]);
        }
#pragma unroll
        for (int c = 0; c < 5; ++c) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) o[c] += __shfl_xor_sync(0xFFFFFFFFu, o[c], off);
            o[c] += __ldg(bh + c);
        }
        const float mx = fmaxf(fmaxf(o[0], o[1]), fmaxf(o[2], o[3]));
        float ex[4], Z = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) { ex[c] = expf(o[c] - mx); Z += ex[c]; }
        const float logZ = logf(Z);
        float p[4], lp[4], ent = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) { p[c] = ex[c] / Z; lp[c] = (o[c] - mx) - logZ; ent -= p[c] * lp[c]; }
        const int act = b.tact[i];
        const float A = b.adv[i];
        const float err = o[4] - b.ret[i];
        float dO[5];
        float lpg_row = 0.f;
        const float pf = policy_term(A, act == 0 ? lp[0] : act == 1 ? lp[1] : act == 2 ? lp[2] : lp[3], ppo_clip > 0.f ? b.tlogp[i] : 0.f, ppo_clip, lpg_row);
#pragma unroll
        for (int c = 0; c < 4; ++c) dO[c] = rnd<PREC>((-A * pf * ((c == act ? 1.f : 0.f) - p[c]) + c_e * p[c] * (lp[c] + ent)) * invR);
        dO[4] = rnd<PREC>(2.f * c_v * err * invR);
        if (lane == 0) {
            float4* o4 = reinterpret_cast<float4*>(b.dout + i * 8);
            o4[0] = make_float4(dO[0], dO[1], dO[2], dO[3]);
            o4[1] = make_float4(dO[4], 0.f, 0.f, 0.f);
            l_pg += lpg_row;
            l_v += err * err;
            l_ent += ent;
        }
        float* dh2 = b.dh2 + i * H;
        for (int k = lane; k < H; k += 32) {
            float back = 0.f;
#pragma unroll
            for (int c = 0; c < 5; ++c) back = fmaf(dO[c], __ldg(Wh + k * 5 + c), back);
            dh2[k] = rnd<PREC>(h2[k] > 0.f ? back : 0.f);
        }
    }
    if (lane == 0) { s_loss[wid][0] = l_pg; s_loss[wid][1] = l_v; s_loss[wid][2] = l_ent; }
    __syncthreads();
    if (threadIdx.x < 3) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += s_loss[w][threadIdx.x];
        b.loss_part[blockIdx.x * 4 + threadIdx.x] = s;
    }
}

// Column sums over a row range (one split per blockIdx.y), 32 columns x 8 row phases per block:
//   dWh[j][c] = sum_i h2[i][j] dOut[i][c];  db2[j] = sum_i dh2[i][j];  db1[j] = sum_i dh1[i][j];  dbh[c] = sum_i dOut[i][c]
__global__ void __launch_bounds__(256) k_colsums(Dims d, Buffers b, size_t R, int NS) {
    __shared__ float red[8][32][7];
    const int lane = threadIdx.x & 31, ph = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + lane;
    const int split = blockIdx.y;
    const size_t rlen = (R + NS - 1) / NS;
    const size_t rbeg = (size_t)split * rlen, rend = min(R, rbeg + rlen);
    const int H = d.H;
    float s[7] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float sbh = 0.f;  // dbh: column `lane` (< 5) of dOut, only in the first column block
    for (size_t i = rbeg + ph; i < rend; i += 8) {
        const float4 d0 = *reinterpret_cast<const float4*>(b.dout + i * 8);
        const float d4 = b.dout[i * 8 + 4];
        if (j < H) {
            const float x = b.h2[i * H + j];
            s[0] = fmaf(x, d0.x, s[0]);
            s[1] = fmaf(x, d0.y, s[1]);
            s[2] = fmaf(x, d0.z, s[2]);
            s[3] = fmaf(x, d0.w, s[3]);
            s[4] = fmaf(x, d4, s[4]);
            s[5] += b.dh2[i * H + j];
            s[6] += b.dh1[i * H + j];
        }
        if (blockIdx.x == 0 && lane < 5) sbh += lane == 0 ? d0.x : lane == 1 ? d0.y : lane == 2 ? d0.z : lane == 3 ? d0.w : d4;
    }
#pragma unroll
    for (int c = 0; c < 7; ++c) red[ph][lane][c] = s[c];
    __syncthreads();
    float* part = b.part + (size_t)split * d.P;
    if (ph == 0 && j < H) {
        float t[7];
#pragma unroll
        for (int c = 0; c < 7; ++c) {
            t[c] = 0.f;
            for (int q = 0; q < 8; ++q) t[c] += red[q][lane][c];
        }
#pragma unroll
        for (int c = 0; c < 5; ++c) part[d.oWh + (size_t)j * 5 + c] = t[c];
        part[d.ob2 + j] = t[5];
        part[d.ob1 + j] = t[6];
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        if (lane < 5) red[ph][lane][0] = sbh;
        __syncthreads();
        if (ph == 0 && lane < 5) {
            float t = 0.f;
            for (int q = 0; q < 8; ++q) t += red[q][lane][0];
            part[d.obh + lane] = t;
        }
    }
}

// S[b][j] = sum over t (ascending) of dh1[t*B+b][j]
__global__ void __launch_bounds__(256) k_sum_over_t(Dims d, Buffers b, int T) {
    const size_t total = (size_t)d.B * d.H;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int t = 0; t < T; ++t) s += b.dh1[(size_t)t * total + idx];
        b.S[idx] = s;
    }
}

// Fixed-order sum of the split-K partials = batch-mean gradient, then Adam (Kingma & Ba, Algorithm 1):
//   m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;  theta -= lr (m/(1-b1^k)) / (sqrt(v/(1-b2^k)) + eps)
// Block 0 also folds the loss partials into the statistics.
template <int PREC>
__global__ void __launch_bounds__(256) k_reduce_adam(LearnArgs a, size_t R, int loss_blocks) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < d.P) {
        float g = 0.f;
        for (int s = 0; s < a.NS; ++s) g += b.part[(size_t)s * d.P + i];
        b.grads[i] = g;
        if (a.phase == 0) {  // phase 1 stops at the gradient
            const AdamIn o = adam_arith(a, AdamIn{b.adam_m[i], b.adam_v[i], b.theta[i]}, g);
            b.adam_m[i] = o.m;
            b.adam_v[i] = o.v;
            const float th = o.theta;
            b.theta[i] = th;
            if (PREC == 1) {
                const bool is_bias = (i >= d.ob1 && i < d.oW2) || (i >= d.ob2 && i < d.oWh) || i >= d.obh;
                b.theta_c[i] = is_bias ? th : round_bf16(th);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < 3) {
        float s = 0.f;
        for (int q = 0; q < loss_blocks; ++q) s += b.loss_part[q * 4 + threadIdx.x];
        s /= (float)R;
        float* dst = threadIdx.x == 0 ? &b.stats->loss_pg : threadIdx.x == 1 ? &b.stats->loss_value : &b.stats->entropy;
        *dst = s;
    }
}

// Debug record: one warp packs the gates (h > 0) of 32 consecutive units of one row into a word.
__global__ void __launch_bounds__(256) k_pack_gates(Dims d, Buffers b, size_t R) {
    const int lane = threadIdx.x & 31;
    const size_t words = R * (size_t)(d.H / 32);
    for (size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5); w < 2 * words; w += (size_t)gridDim.x * 8) {
        const float* h = w < words ? b.h1 : b.h2;
        const size_t wi = w < words ? w : w - words;
        const uint32_t bits = __ballot_sync(0xFFFFFFFFu, h[wi * 32 + lane] > 0.f);
        if (lane == 0) b.dbg_gates[w] = bits;
    }
}

__global__ void k_loss_total(Buffers b, float c_v, float c_e) {
    b.stats->loss_total = b.stats->loss_pg + c_v * b.stats->loss_value - c_e * b.stats->entropy;
}

template <class AL, class BL, class EP>
static cudaError_t gemm(int id, int M, int N, int K, int splits, AL al, BL bl, EP ep, const Ctx& c) {
    const int klen = ((K + splits - 1) / splits + 15) / 16 * 16;
    dim3 grid((M + 63) / 64, (N + 63) / 64, splits);
    Scope sc(c, id);
    k_sgemm<AL, BL, EP><<<grid, 256, 0, c.s>>>(M, N, K, klen, al, bl, ep);
    return cudaGetLastError();
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

template <int PREC>
static cudaError_t launch_learn_p(const LearnArgs& a, const Ctx& c) {
    const Dims& d = a.d;
    const Buffers& b = a.b;
    const size_t R = (size_t)d.B * a.T;
    const int H = d.H, C = d.C, NS = a.NS;
    const float* W2 = b.theta_c + d.oW2;
    cudaStream_t s = c.s;
    const size_t ew = (R * (size_t)H + 255) / 256;
    const int ew_blocks = (int)(ew < 148 * 16 ? ew : 148 * 16);

    // forward (recomputed)
    {
        Scope sc(c, K_H1);
        k_h1<PREC><<<ew_blocks, 256, 0, s>>>(d, b, R);
        CK(cudaGetLastError());
    }
    CK(gemm(K_FWD2, (int)R, H, H, 1, LdRowMajorA{b.h1, H}, LdRowMajorB{W2, H}, EpBiasRelu<PREC>{b.h2, b.theta_c + d.ob2, H}, c));
    // heads + loss + output gradients + dh2
    const int lb = (int)((R + 7) / 8 < (size_t)LOSS_BLOCKS ? (R + 7) / 8 : LOSS_BLOCKS);
    {
        Scope sc(c, K_HEADS_LOSS);
        k_heads_loss<PREC><<<lb, 256, 0, s>>>(d, b, R, a.c_v, a.c_e, a.ppo_clip);
        CK(cudaGetLastError());
    }
    // dh1 = (dh2 W2^T) masked
    CK(gemm(K_DH1, (int)R, H, H, 1, LdRowMajorA{b.dh2, H}, LdTransB{W2, H}, EpReluMask<PREC>{b.dh1, b.h1, H}, c));
    // weight gradients as split-K partials in the flat parameter layout
    CK(gemm(K_DW2, H, H, (int)R, NS, LdTransA{b.h1, H}, LdRowMajorB{b.dh2, H}, EpPartial{b.part, d.P, d.oW2, H}, c));
    {
        Scope sc(c, K_COLSUMS);
        k_colsums<<<dim3((H + 31) / 32, NS), 256, 0, s>>>(d, b, R, NS);
        CK(cudaGetLastError());
    }
    // first layer: the agent plane sees every row; the wall and goal planes are constant over t, so they
    // contract S = sum_t dh1 over envs instead
    const size_t sbn = ((size_t)d.B * H + 255) / 256;
    {
        Scope sc(c, K_SUM_OVER_T);
        k_sum_over_t<<<(int)(sbn < 148 * 8 ? sbn : 148 * 8), 256, 0, s>>>(d, b, a.T);
        CK(cudaGetLastError());
    }
    CK(gemm(K_DW1_AGENT, C, H, (int)R, NS, LdAgentPlane{b.tpos}, LdRowMajorB{b.dh1, H}, EpPartial{b.part, d.P, d.oW1 + (size_t)C * H, H}, c));
    CK(gemm(K_DW1_WALLS, C, H, d.B, NS, LdWallPlane{b.walls, d.W}, LdRowMajorB{b.S, H}, EpPartial{b.part, d.P, d.oW1, H}, c));
    CK(gemm(K_DW1_GOAL, C, H, d.B, NS, LdGoalPlane{b.goal}, LdRowMajorB{b.S, H}, EpPartial{b.part, d.P, d.oW1 + (size_t)2 * C * H, H}, c));
    // batch mean (fixed order) + Adam + loss statistics
    {
        Scope sc(c, K_REDUCE_ADAM);
        k_reduce_adam<PREC><<<(unsigned)((d.P + 255) / 256), 256, 0, s>>>(a, R, lb);
        CK(cudaGetLastError());
    }
    if (b.dbg_gates) {
        Scope sc(c, K_PACK_GATES);
        k_pack_gates<<<148 * 8, 256, 0, s>>>(d, b, R);
        CK(cudaGetLastError());
    }
    Scope sc(c, K_LOSS_TOTAL);
    k_loss_total<<<1, 1, 0, s>>>(b, a.c_v, a.c_e);
    return cudaGetLastError();
}

cudaError_t launch_learn(const LearnArgs& a, int prec, const Ctx& c) {
    return prec == 1 ? launch_learn_p<1>(a, c) : launch_learn_p<0>(a, c);
}

}  // namespace anakin
