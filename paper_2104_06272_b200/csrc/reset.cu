// Reset kernels: the env's `initial_state` for every env (Podracer paper, Section 3.1) and the agent's
// parameter initialisation.  Everything is drawn from Philox4x32-10 counters, so the result is a pure
// function of the seed.
#include "common.cuh"

namespace anakin {

// One thread per env.  Stream ENV: counter (b,0,0) -> start (word 0) and goal (word 1, among the other C-1
// cells); counter (b,1+c/4,0) word (c%4) below floor(density*2^32) makes cell c a wall; start and goal stay free.
template <bool GROUPED>
__global__ void __launch_bounds__(128) k_reset_env(DimsBuffers in, uint32_t k0, uint32_t k1, uint32_t thr) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);  // many policies: grid.y = policy
    const Dims& d = pa.a.d;
    const Buffers& b = pa.a.b;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= d.B) return;
    const uint32_t ge = (uint32_t)(d.env0 + e);  // global env index
    const U4 x = philox4x32_10(ge, 0, 0, STREAM_ENV, k0, k1);
    const uint32_t s = (uint32_t)(((uint64_t)x.x * (uint32_t)d.C) >> 32);
    uint32_t g = (uint32_t)(((uint64_t)x.y * (uint32_t)(d.C - 1)) >> 32);
    if (g >= s) g += 1;
    uint32_t word = 0;
    for (int c4 = 0; c4 * 4 < d.C; ++c4) {
        const U4 y = philox4x32_10(ge, (uint32_t)(1 + c4), 0, STREAM_ENV, k0, k1);
        const uint32_t ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = c4 * 4 + i;
            if (c < d.C && ys[i] < thr && (uint32_t)c != s && (uint32_t)c != g) word |= 1u << (c & 31);
        }
        // 4 cells per counter and 32 cells per word: a word is complete after every 8th counter
        if ((c4 & 7) == 7 || (c4 + 1) * 4 >= d.C) {
            b.walls[(size_t)e * d.W + (c4 >> 3)] = word;
            word = 0;
        }
    }
    b.start[e] = (uint8_t)s;
    b.goal[e] = (uint8_t)g;
    b.pos[e] = (uint8_t)s;
    b.tep[e] = 0;
}

// One thread per parameter.  Stream PARAM: u = uniform24(word 0 of counter (i,0,0));
// w = (2u-1)*sqrt(6/(fan_in+fan_out)) evaluated in double, rounded once.  Biases are zero.  With many policies, policy p
// draws counter (i,p,0): its own, independent initialisation (policy 0 = the single-policy one).
template <bool GROUPED>
__global__ void __launch_bounds__(256) k_reset_params(DimsBuffers in, uint32_t k0, uint32_t k1) {
    const PolicyArgs<GROUPED, DimsBuffers> pa(in, blockIdx.y);
    const Dims& d = pa.a.d;
    const Buffers& b = pa.a.b;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        anakin_stats z;
        z.frames = z.episodes = z.goals = z.episode_steps = 0;
        z.loss_total = z.loss_pg = z.loss_value = z.entropy = 0.f;
        *b.stats = z;
        if (blockIdx.y == 0) *b.status = 0;
    }
    if (i >= d.P) return;
    double bound = 0.0;
    if (i < d.ob1) bound = sqrt(6.0 / (double)(d.D + d.H));
    else if (i < d.oW2) bound = 0.0;
    else if (i < d.ob2) bound = sqrt(6.0 / (double)(d.H + d.H));
    else if (i < d.oWh) bound = 0.0;
    else if (i < d.obh) bound = sqrt(6.0 / (double)(d.H + (((i - d.oWh) % 5) < 4 ? 4 : 1)));
    float w = 0.f;
    if (bound != 0.0) {
        const U4 x = philox4x32_10((uint32_t)i, GROUPED ? blockIdx.y : 0u, 0, STREAM_PARAM, k0, k1);
        const double u = (double)(x.x >> 8) * (1.0 / 16777216.0);
        w = (float)((2.0 * u - 1.0) * bound);
    }
    b.theta[i] = w;
    b.adam_m[i] = 0.f;
    b.adam_v[i] = 0.f;
    b.grads[i] = 0.f;
}

// bf16 mode: the network computes with bf16-rounded weight matrices and unrounded biases.
__global__ void __launch_bounds__(256) k_refresh_compute_params(Dims d, Buffers b) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d.P) return;
    const bool is_bias = (i >= d.ob1 && i < d.oW2) || (i >= d.ob2 && i < d.oWh) || i >= d.obh;
    const float w = b.theta[i];
    b.theta_c[i] = is_bias ? w : round_bf16(w);
}

cudaError_t launch_refresh_compute_params(const Dims& d, const Buffers& b, int prec, const Ctx& c) {
    if (prec != 1) return cudaSuccess;
    Scope sc(c, K_REFRESH_PARAMS);
    k_refresh_compute_params<<<(unsigned)((d.P + 255) / 256), 256, 0, c.s>>>(d, b);
    return cudaGetLastError();
}

cudaError_t launch_reset(const Dims& d, const Buffers& b, uint64_t seed, double density, int prec, const Ctx& c) {
    const uint32_t k0 = (uint32_t)(seed & 0xFFFFFFFFu), k1 = (uint32_t)(seed >> 32);
    const uint32_t thr = (uint32_t)floor(density * 4294967296.0);
    cudaError_t e;
    {
        Scope sc(c, K_RESET_ENV);
        if (d.npol > 1) k_reset_env<true><<<dim3((d.B + 127) / 128, d.npol), 128, 0, c.s>>>(DimsBuffers{d, b}, k0, k1, thr);
        else k_reset_env<false><<<(d.B + 127) / 128, 128, 0, c.s>>>(DimsBuffers{d, b}, k0, k1, thr);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return e;
    {
        Scope sc(c, K_RESET_PARAMS);
        const unsigned nb = (unsigned)((d.P + 255) / 256);
        if (d.npol > 1) k_reset_params<true><<<dim3(nb, d.npol), 256, 0, c.s>>>(DimsBuffers{d, b}, k0, k1);
        else k_reset_params<false><<<nb, 256, 0, c.s>>>(DimsBuffers{d, b}, k0, k1);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return e;
    return launch_refresh_compute_params(d, b, prec, c);
}

}  // namespace anakin
