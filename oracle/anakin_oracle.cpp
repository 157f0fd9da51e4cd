// Anakin hot-path ORACLE  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-file CPU restatement of the co-located act+learn loop of the Anakin
// architecture (Podracer paper, Section 3.1 "Online Learning with Anakin"; Figure 2, top): a batch
// of environments written as array code is stepped next to the agent for T interactions, then one
// parameter update is computed from those interactions and averaged over the batch.
//
// Only the tests, the smoke check and the benchmark's CPU-baseline leg may load this file.  It shares
// no code, header, table or constant generator with the CUDA library; the two were written separately
// from the same written definitions.
//
// The paper fixes the structure of the loop (env `initial_state` / `step` as pure functions of an
// explicit state, Section 3.1; update averaged over all participants, Section 3.1; determinism,
// Section 3.1) but none of its numerics.  The concrete rules below (gridworld, MLP, Philox sampling,
// GAE, A2C loss, Adam) are the workload definition this repository builds to; each function states the
// rule it implements.
//
// Precision model: values are STORED in the scalar type S (float for the fp32/bf16 workloads, double
// for the finite-difference self-check); every dot product and reduction is ACCUMULATED in double and
// rounded to S once.  The bf16 workload adds round-to-nearest-even bf16 rounding at the stated points.
//
// Parity pins (tests/, CPU only): Philox against cuRAND's host generator and an independent
// big-integer restatement; env invariants and a hand-traced episode; forward pass against a library
// fp64 matmul; GAE against the direct discounted sum and closed forms; gradients against central
// finite differences in fp64; entropy of uniform logits = ln 4; Adam closed forms.
// Parity unpinned: the action-direction convention, plane order, parameter order, time-outs treated
// as terminal in GAE, the value-loss constant and the Adam epsilon placement are conventions chosen
// here; the paper fixes none of them.

#include <algorithm>
#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ----------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11).
// Counter c[0..3], key k[0..1]; ten rounds; the key is bumped by the Weyl constants between rounds.
// ----------------------------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = M0 * (uint64_t)c0;
        const uint64_t p1 = M1 * (uint64_t)c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n1 = lo1;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        const uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum : uint32_t { STREAM_ENV = 1, STREAM_PARAM = 2, STREAM_ACT = 3 };

void philox_at(uint64_t seed, uint32_t i0, uint32_t i1, uint32_t i2, uint32_t stream, uint32_t out[4]) {
    const uint32_t ctr[4] = {i0, i1, i2, stream};
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    philox4x32_10(ctr, key, out);
}

// uniform in [0,1): top 24 bits of the word, scaled by 2^-24 (exact in fp32).
double uniform24(uint32_t x) { return (double)(x >> 8) * (1.0 / 16777216.0); }

// integer in [0, n): high half of the 64-bit product.
uint32_t mulhi_range(uint32_t x, uint32_t n) { return (uint32_t)(((uint64_t)x * (uint64_t)n) >> 32); }

// ----------------------------------------------------------------------------------------------
// Sizes and the flat parameter order  W1[D][H], b1[H], W2[H][H], b2[H], Wh[H][5], bh[5]
// (head columns 0..3 = action logits, column 4 = value).
// ----------------------------------------------------------------------------------------------
struct Dims {
    int N, C, D, H, W;  // grid side, cells, obs features, hidden units, 32-bit wall words per env
    size_t oW1, ob1, oW2, ob2, oWh, obh, P;
};

Dims make_dims(int N, int H) {
    Dims d;
    d.N = N; d.C = N * N; d.D = 3 * d.C; d.H = H; d.W = (d.C + 31) / 32;
    d.oW1 = 0;
    d.ob1 = d.oW1 + (size_t)d.D * H;
    d.oW2 = d.ob1 + H;
    d.ob2 = d.oW2 + (size_t)H * H;
    d.oWh = d.ob2 + H;
    d.obh = d.oWh + (size_t)H * 5;
    d.P = d.obh + 5;
    return d;
}

bool wall_at(const uint32_t* walls, int cell) { return (walls[cell >> 5] >> (cell & 31)) & 1u; }

// round-to-nearest-even to bfloat16, returned as float.
float round_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return f;  // inf / nan unchanged
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    float r;
    std::memcpy(&r, &u, 4);
    return r;
}
template <typename S> S maybe_bf16(S v, int prec) { return v; }
template <> float maybe_bf16<float>(float v, int prec) { return prec == 1 ? round_bf16(v) : v; }

// ----------------------------------------------------------------------------------------------
// Environment: `initial_state` (Section 3.1).  Per env b, everything is drawn from Philox stream ENV:
//   counter (b,0,0): word0 -> start cell, word1 -> goal cell among the other C-1 cells;
//   counter (b,1+c/4,0): word (c%4) < floor(density*2^32)  <=>  cell c is a wall;
//   start and goal are forced free.  Reachability is not enforced.
// ----------------------------------------------------------------------------------------------
void env_init(uint64_t seed, int B, int N, double density, uint32_t* walls, uint8_t* start, uint8_t* goal) {
    const Dims d = make_dims(N, 16);
    const uint32_t thr = (uint32_t)std::floor(density * 4294967296.0);
    for (int b = 0; b < B; ++b) {
        uint32_t x[4];
        philox_at(seed, (uint32_t)b, 0, 0, STREAM_ENV, x);
        uint32_t s = mulhi_range(x[0], (uint32_t)d.C);
        uint32_t g = mulhi_range(x[1], (uint32_t)(d.C - 1));
        if (g >= s) g += 1;
        uint32_t* w = walls + (size_t)b * d.W;
        for (int i = 0; i < d.W; ++i) w[i] = 0;
        for (int c = 0; c < d.C; ++c) {
            uint32_t y[4];
            philox_at(seed, (uint32_t)b, (uint32_t)(1 + c / 4), 0, STREAM_ENV, y);
            const bool is_wall = y[c % 4] < thr;
            if (is_wall && (uint32_t)c != s && (uint32_t)c != g) w[c >> 5] |= (1u << (c & 31));
        }
        start[b] = (uint8_t)s;
        goal[b] = (uint8_t)g;
    }
}

// Environment: `step(state, action) -> (state, reward)` (Section 3.1).  Actions: 0 up (row-1),
// 1 right (col+1), 2 down (row+1), 3 left (col-1).  A move into a wall or off the grid leaves the agent
// in place.  Reaching the goal pays 1 and ends the episode; the step cap ends it with reward 0.  On
// episode end the env resets itself to its seeded start inside the same step.
// The paper's env interface is generic (any `initial_state` / `step` written as array code); `kind` selects a
// second env with the same state and observation: kind 1 = torus, where a move off an edge re-enters at the
// opposite edge (walls still block).
void env_step(const Dims& d, const uint32_t* walls, uint8_t start, uint8_t goal, int cap,
              uint8_t* pos, uint8_t* tep, int action, float* reward, uint8_t* done, int kind = 0) {
    const int N = d.N;
    const int row = *pos / N, col = *pos % N;
    int nr = row, nc = col;
    if (action == 0) nr = row - 1;
    else if (action == 1) nc = col + 1;
    else if (action == 2) nr = row + 1;
    else nc = col - 1;
    if (kind == 1) {
        nr = (nr + N) % N;
        nc = (nc + N) % N;
    }
    int np = *pos;
    if (nr >= 0 && nr < N && nc >= 0 && nc < N) {
        const int cand = nr * N + nc;
        if (!wall_at(walls, cand)) np = cand;
    }
    const int t = (int)*tep + 1;
    float r = 0.0f;
    uint8_t dn = 0;
    if (np == (int)goal) { r = 1.0f; dn = 1; }
    else if (t >= cap) { r = 0.0f; dn = 1; }
    if (dn) { *pos = start; *tep = 0; }
    else { *pos = (uint8_t)np; *tep = (uint8_t)t; }
    *reward = r;
    *done = dn;
}

// Observation: three one-hot planes flattened, x[plane*C + row*N + col]; plane 0 walls, 1 agent, 2 goal.
template <typename S>
void observe(const Dims& d, const uint32_t* walls, uint8_t pos, uint8_t goal, S* x) {
    for (int k = 0; k < d.D; ++k) x[k] = (S)0;
    for (int c = 0; c < d.C; ++c)
        if (wall_at(walls, c)) x[c] = (S)1;
    x[d.C + pos] = (S)1;
    x[2 * d.C + goal] = (S)1;
}

// Parameter init: Xavier-uniform from Philox stream PARAM.  Flat index i draws
// u = uniform24(word0 of counter (i,0,0)); w = (2u-1)*sqrt(6/(fan_in+fan_out)) evaluated in double and
// rounded once.  Policy head columns use fan_out 4, the value column fan_out 1.  Biases are zero.
// With many policies (independent networks trained side by side), policy p draws word 0 of counter (i,p,0): policy 0
// is the single-policy initialisation.
template <typename S>
void param_init(uint64_t seed, const Dims& d, S* theta, uint32_t policy = 0) {
    for (size_t i = 0; i < d.P; ++i) {
        double bound = 0.0;
        if (i < d.ob1) bound = std::sqrt(6.0 / (double)(d.D + d.H));
        else if (i < d.oW2) bound = 0.0;
        else if (i < d.ob2) bound = std::sqrt(6.0 / (double)(d.H + d.H));
        else if (i < d.oWh) bound = 0.0;
        else if (i < d.obh) {
            const size_t col = (i - d.oWh) % 5;
            bound = std::sqrt(6.0 / (double)(d.H + (col < 4 ? 4 : 1)));
        } else bound = 0.0;
        if (bound == 0.0) { theta[i] = (S)0; continue; }
        uint32_t x[4];
        philox_at(seed, (uint32_t)i, policy, 0, STREAM_PARAM, x);
        const double u = uniform24(x[0]);
        theta[i] = (S)((2.0 * u - 1.0) * bound);
    }
}

// The parameters the network computes with: the master copy, except that in the bf16 workload the
// three weight matrices are rounded to bf16 (biases stay as stored).
template <typename S>
std::vector<S> compute_params(const Dims& d, const S* theta, int prec) {
    std::vector<S> c(theta, theta + d.P);
    if (prec == 1) {
        for (size_t i = d.oW1; i < d.ob1; ++i) c[i] = maybe_bf16(c[i], 1);
        for (size_t i = d.oW2; i < d.ob2; ++i) c[i] = maybe_bf16(c[i], 1);
        for (size_t i = d.oWh; i < d.obh; ++i) c[i] = maybe_bf16(c[i], 1);
    }
    return c;
}

// Policy/value network on one row: h1 = relu(x W1 + b1); h2 = relu(h1 W2 + b2); out = h2 Wh + bh.
// In the bf16 workload h1 and h2 are rounded to bf16 after the ReLU; out stays in S.
template <typename S>
void forward_row(const Dims& d, const S* cp, int prec, const S* x, S* h1, S* h2, S* out5,
                 std::vector<double>& acc, S* z1 = nullptr, S* z2 = nullptr) {
    const int H = d.H, D = d.D;
    acc.assign((size_t)H, 0.0);
    for (int k = 0; k < D; ++k) {
        const double xk = (double)x[k];
        const S* wrow = cp + d.oW1 + (size_t)k * H;
        for (int j = 0; j < H; ++j) acc[j] += xk * (double)wrow[j];
    }
    for (int j = 0; j < H; ++j) {
        S z = (S)(acc[j] + (double)cp[d.ob1 + j]);
        if (z1) z1[j] = z;
        z = z > (S)0 ? z : (S)0;
        h1[j] = maybe_bf16(z, prec);
    }
    acc.assign((size_t)H, 0.0);
    for (int k = 0; k < H; ++k) {
        const double hk = (double)h1[k];
        const S* wrow = cp + d.oW2 + (size_t)k * H;
        for (int j = 0; j < H; ++j) acc[j] += hk * (double)wrow[j];
    }
    for (int j = 0; j < H; ++j) {
        S z = (S)(acc[j] + (double)cp[d.ob2 + j]);
        if (z2) z2[j] = z;
        z = z > (S)0 ? z : (S)0;
        h2[j] = maybe_bf16(z, prec);
    }
    double o[5] = {0, 0, 0, 0, 0};
    for (int k = 0; k < H; ++k) {
        const double hk = (double)h2[k];
        const S* wrow = cp + d.oWh + (size_t)k * 5;
        for (int c = 0; c < 5; ++c) o[c] += hk * (double)wrow[c];
    }
    for (int c = 0; c < 5; ++c) out5[c] = (S)(o[c] + (double)cp[d.obh + c]);
}

// softmax over 4 logits in double, max-subtracted; also log-probabilities and entropy.
struct Soft {
    double p[4], logp[4], entropy;
};
template <typename S>
Soft softmax4(const S* l) {
    Soft s;
    double m = (double)l[0];
    for (int k = 1; k < 4; ++k) m = std::max(m, (double)l[k]);
    double e[4], Z = 0.0;
    for (int k = 0; k < 4; ++k) { e[k] = std::exp((double)l[k] - m); Z += e[k]; }
    const double logZ = std::log(Z);
    s.entropy = 0.0;
    for (int k = 0; k < 4; ++k) {
        s.p[k] = e[k] / Z;
        s.logp[k] = ((double)l[k] - m) - logZ;
        s.entropy -= s.p[k] * s.logp[k];
    }
    return s;
}

// Categorical sample by inverse CDF: c0=p0, c1=c0+p1, c2=c1+p2; a = [u>=c0]+[u>=c1]+[u>=c2].
// `near` flags a uniform within 1e-5 of any CDF boundary (where an fp32 implementation may differ).
void sample4(const float* logits, double u, int* a, float* logp, uint8_t* near) {
    const Soft s = softmax4(logits);
    const double c0 = s.p[0], c1 = c0 + s.p[1], c2 = c1 + s.p[2];
    const int act = (u >= c0) + (u >= c1) + (u >= c2);
    *a = act;
    *logp = (float)s.logp[act];
    *near = (std::fabs(u - c0) < 1e-5 || std::fabs(u - c1) < 1e-5 || std::fabs(u - c2) < 1e-5) ? 1 : 0;
}

double act_uniform(uint64_t seed, uint32_t b, uint32_t gstep) {
    uint32_t x[4];
    philox_at(seed, b, gstep, 0, STREAM_ACT, x);
    return uniform24(x[0]);
}

// ----------------------------------------------------------------------------------------------
// Loss and gradient over R = B*T recorded rows (row i: env b = i % B, time t = i / B).
//   L = -(1/R) sum A_i log pi(a_i|s_i) + c_v (1/R) sum (V_i - ret_i)^2 - c_e (1/R) sum H_i
// Advantages and returns are constants.  Gradients are the mean over all rows: this batch mean is the
// single-device form of the paper's cross-core average of updates (Section 3.1).
//
// ReLU gates.  The derivative of ReLU is a floating-point comparison that decides a bit.  When the
// caller passes gate bitmaps (bit j%32 of word [row][j/32]; recorded by the implementation under test),
// the BACKWARD pass uses those gates instead of the oracle's own h > 0, so that both sides take the
// decision in the same (the kernel's) precision; the forward pass is unchanged.  gate_info reports, per
// layer, how many given gates differ from the oracle's own, the largest |pre-activation| among those,
// and the rms pre-activation: a differing gate is legitimate only where the pre-activation is within
// rounding of zero, which the caller checks.
// ----------------------------------------------------------------------------------------------
template <typename S>
void loss_and_grad(const Dims& d, int prec, int B, int T, const S* theta, const uint32_t* walls,
                   const uint8_t* goal, const uint8_t* tpos, const int8_t* tact, const S* adv,
                   const S* ret, double c_v, double c_e, S* grads /*nullable*/, double loss4[4],
                   const uint32_t* gate1 = nullptr, const uint32_t* gate2 = nullptr, double* gate_info /*[6]*/ = nullptr,
                   const S* logp_old = nullptr, double clip = 0.0) {
    // logp_old != nullptr selects the clipped-surrogate policy term (PPO, Schulman et al. 2017, Eq. 7) in place of the
    // plain policy-gradient term:  -min(r A, clip(r, 1-eps, 1+eps) A),  r = pi(a|s) / pi_old(a|s) = exp(logp - logp_old).
    // Its gradient is that of -r A where the unclipped product is the smaller one (ties included) and zero elsewhere.
    const size_t R = (size_t)B * T;
    const int GW = (d.H + 31) / 32;
    const std::vector<S> cp = compute_params(d, theta, prec);
    const int H = d.H, D = d.D;
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    std::vector<std::vector<double>> gpart(nthreads);
    std::vector<double> lpart((size_t)nthreads * 3, 0.0);
    std::vector<double> kpart((size_t)nthreads * 6, 0.0);
#pragma omp parallel num_threads(nthreads)
    {
        int tid = 0;
#ifdef _OPENMP
        tid = omp_get_thread_num();
#endif
        std::vector<double>& g = gpart[tid];
        if (grads) g.assign(d.P, 0.0);
        std::vector<S> x(D), h1(H), h2(H), dh2(H), dh1(H), z1(H), z2(H);
        std::vector<double> acc;
        S out[5];
        double l_pg = 0.0, l_v = 0.0, l_ent = 0.0;
        double* kp = kpart.data() + (size_t)tid * 6;  // mismatches, max|z| among them, sum z^2 (per layer)
        // static contiguous split of the rows over threads
        const size_t lo = R * (size_t)tid / nthreads, hi = R * (size_t)(tid + 1) / nthreads;
        for (size_t i = lo; i < hi; ++i) {
            const size_t b = i % (size_t)B;
            observe(d, walls + b * d.W, tpos[i], goal[b], x.data());
            forward_row(d, cp.data(), prec, x.data(), h1.data(), h2.data(), out, acc, z1.data(), z2.data());
            // gate of unit j in each layer: the caller's bit if given, else the oracle's own h > 0
            auto gate = [&](const uint32_t* g, const std::vector<S>& h, const std::vector<S>& z, int j, double* k3) -> bool {
                const bool own = h[j] > (S)0;
                k3[2] += (double)z[j] * (double)z[j];
                if (!g) return own;
                const bool given = (g[i * GW + (j >> 5)] >> (j & 31)) & 1u;
                if (given != own) { k3[0] += 1.0; k3[1] = std::max(k3[1], std::fabs((double)z[j])); }
                return given;
            };
            const Soft s = softmax4(out);
            const int a = (int)tact[i];
            const double A = (double)adv[i];
            const double V = (double)out[4];
            const double err = V - (double)ret[i];
            double pg_coef = 1.0;  // d(policy term)/d(logp[a]) = -A * pg_coef
            if (logp_old) {
                const double r = std::exp(s.logp[a] - (double)logp_old[i]);
                const double rc = std::min(std::max(r, 1.0 - clip), 1.0 + clip);
                const bool unclipped = r * A <= rc * A;
                l_pg += -std::min(r * A, rc * A);
                pg_coef = unclipped ? r : 0.0;
            } else {
                l_pg += -A * s.logp[a];
            }
            l_v += err * err;
            l_ent += s.entropy;
            if (!grads) continue;
            // output gradients (already divided by R)
            S dOut[5];
            for (int k = 0; k < 4; ++k) {
                const double dz = (-A * pg_coef * ((k == a ? 1.0 : 0.0) - s.p[k]) + c_e * s.p[k] * (s.logp[k] + s.entropy)) / (double)R;
                dOut[k] = maybe_bf16((S)dz, prec);
            }
            dOut[4] = maybe_bf16((S)(2.0 * c_v * err / (double)R), prec);
            // head
            for (int j = 0; j < H; ++j) {
                const double hj = (double)h2[j];
                double back = 0.0;
                for (int k = 0; k < 5; ++k) {
                    g[d.oWh + (size_t)j * 5 + k] += hj * (double)dOut[k];
                    back += (double)dOut[k] * (double)cp[d.oWh + (size_t)j * 5 + k];
                }
                S v = gate(gate2, h2, z2, j, kp + 3) ? (S)back : (S)0;
                dh2[j] = maybe_bf16(v, prec);
            }
            for (int k = 0; k < 5; ++k) g[d.obh + k] += (double)dOut[k];
            // layer 2
            for (int i1 = 0; i1 < H; ++i1) {
                const double hi1 = (double)h1[i1];
                const S* wrow = cp.data() + d.oW2 + (size_t)i1 * H;
                double* grow = g.data() + d.oW2 + (size_t)i1 * H;
                double back = 0.0;
                for (int j = 0; j < H; ++j) {
                    grow[j] += hi1 * (double)dh2[j];
                    back += (double)dh2[j] * (double)wrow[j];
                }
                S v = gate(gate1, h1, z1, i1, kp) ? (S)back : (S)0;
                dh1[i1] = maybe_bf16(v, prec);
            }
            for (int j = 0; j < H; ++j) g[d.ob2 + j] += (double)dh2[j];
            // layer 1 (no gradient with respect to the observation is needed)
            for (int k = 0; k < D; ++k) {
                const double xk = (double)x[k];
                double* grow = g.data() + d.oW1 + (size_t)k * H;
                for (int j = 0; j < H; ++j) grow[j] += xk * (double)dh1[j];
            }
            for (int j = 0; j < H; ++j) g[d.ob1 + j] += (double)dh1[j];
        }
        lpart[(size_t)tid * 3 + 0] = l_pg;
        lpart[(size_t)tid * 3 + 1] = l_v;
        lpart[(size_t)tid * 3 + 2] = l_ent;
    }
    double l_pg = 0.0, l_v = 0.0, l_ent = 0.0;
    for (int t = 0; t < nthreads; ++t) {
        l_pg += lpart[(size_t)t * 3 + 0];
        l_v += lpart[(size_t)t * 3 + 1];
        l_ent += lpart[(size_t)t * 3 + 2];
    }
    l_pg /= (double)R; l_v /= (double)R; l_ent /= (double)R;
    loss4[0] = l_pg + c_v * l_v - c_e * l_ent;
    loss4[1] = l_pg;
    loss4[2] = l_v;
    loss4[3] = l_ent;
    if (gate_info) {
        for (int l = 0; l < 2; ++l) {
            double n = 0.0, mx = 0.0, ss = 0.0;
            for (int t = 0; t < nthreads; ++t) {
                n += kpart[(size_t)t * 6 + 3 * l + 0];
                mx = std::max(mx, kpart[(size_t)t * 6 + 3 * l + 1]);
                ss += kpart[(size_t)t * 6 + 3 * l + 2];
            }
            gate_info[3 * l + 0] = n;
            gate_info[3 * l + 1] = mx;
            gate_info[3 * l + 2] = std::sqrt(ss / ((double)R * H));
        }
    }
    if (grads) {
        for (size_t i = 0; i < d.P; ++i) {
            double s = 0.0;
            for (int t = 0; t < nthreads; ++t) s += gpart[t][i];  // thread order
            grads[i] = (S)s;
        }
    }
}

}  // namespace

// ================================================================================================
// C ABI (host pointers only).  Loaded with ctypes by oracle/binding.py.
// ================================================================================================
extern "C" {

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

void orc_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }

double orc_uniform24(uint32_t x) { return uniform24(x); }

uint64_t orc_param_count(int N, int H) { return (uint64_t)make_dims(N, H).P; }

void orc_env_init(uint64_t seed, int B, int N, double density, uint32_t* walls, uint8_t* start, uint8_t* goal) {
    env_init(seed, B, N, density, walls, start, goal);
}

void orc_param_init(uint64_t seed, int N, int H, float* theta) { param_init(seed, make_dims(N, H), theta); }

// one env, one step; pos/tep updated in place
void orc_env_step(int N, const uint32_t* walls, uint8_t start, uint8_t goal, int cap, uint8_t* pos,
                  uint8_t* tep, int action, float* reward, uint8_t* done) {
    env_step(make_dims(N, 16), walls, start, goal, cap, pos, tep, action, reward, done);
}

void orc_env_step_kind(int kind, int N, const uint32_t* walls, uint8_t start, uint8_t goal, int cap, uint8_t* pos,
                       uint8_t* tep, int action, float* reward, uint8_t* done) {
    env_step(make_dims(N, 16), walls, start, goal, cap, pos, tep, action, reward, done, kind);
}

void orc_observe(int N, const uint32_t* walls, uint8_t pos, uint8_t goal, float* x) {
    observe(make_dims(N, 16), walls, pos, goal, x);
}

void orc_round_bf16(size_t n, const float* in, float* out) {
    for (size_t i = 0; i < n; ++i) out[i] = round_bf16(in[i]);
}

// forward on n dense rows x[n][D]; h1/h2 may be null
void orc_forward(int N, int H, int prec, const float* theta, size_t n, const float* x, float* h1o,
                 float* h2o, float* out5) {
    const Dims d = make_dims(N, H);
    const std::vector<float> cp = compute_params(d, theta, prec);
#pragma omp parallel
    {
        std::vector<float> h1(H), h2(H);
        std::vector<double> acc;
#pragma omp for schedule(static)
        for (long long i = 0; i < (long long)n; ++i) {
            forward_row(d, cp.data(), prec, x + (size_t)i * d.D, h1.data(), h2.data(), out5 + (size_t)i * 5, acc);
            if (h1o) std::copy(h1.begin(), h1.end(), h1o + (size_t)i * H);
            if (h2o) std::copy(h2.begin(), h2.end(), h2o + (size_t)i * H);
        }
    }
}

void orc_forward_f64(int N, int H, const double* theta, size_t n, const double* x, double* out5) {
    const Dims d = make_dims(N, H);
    std::vector<double> h1(H), h2(H), acc;
    for (size_t i = 0; i < n; ++i) forward_row(d, theta, 0, x + i * d.D, h1.data(), h2.data(), out5 + i * 5, acc);
}

void orc_sample_one(const float* logits4, double u, int* a, float* logp, uint8_t* near) {
    sample4(logits4, u, a, logp, near);
}

double orc_act_uniform(uint64_t seed, uint32_t b, uint32_t gstep) { return act_uniform(seed, b, gstep); }

// Sample every (t,b) from GIVEN logits[T][B][4] with the ACT-stream uniform of (b, gstep0+t).
void orc_sample_from_logits(uint64_t seed, uint32_t gstep0, int T, int B, const float* logits, int8_t* act,
                            float* logp, uint8_t* near) {
    for (int t = 0; t < T; ++t)
        for (int b = 0; b < B; ++b) {
            const size_t i = (size_t)t * B + b;
            int a;
            sample4(logits + i * 4, act_uniform(seed, (uint32_t)b, gstep0 + (uint32_t)t), &a, logp + i, near + i);
            act[i] = (int8_t)a;
        }
}

// T interactions of every env with the agent (Figure 2, top: "a sequence of interactions").
// Per step t and env b: observe -> network -> sample (or take forced[t][b]) -> env step; record the
// state the action was taken in, the action, reward, done, value and log-probability.  After the last
// step the value of the current state is stored in value[T][b] (the bootstrap).
// Env dynamic state (pos, tep) is updated in place; the global step counter advances by T (caller).
// env0: global index of env 0 of this batch (the action uniform of env b is keyed by env0 + b), so that a slice of a
// larger job (a replica's shard, one policy's envs) draws what the whole job would draw for those envs.
void orc_rollout_env0(int kind, int N, int H, int prec, int B, int T, int cap, const float* theta, const uint32_t* walls,
                      const uint8_t* start, const uint8_t* goal, uint8_t* pos, uint8_t* tep, uint64_t seed,
                      uint32_t gstep0, const int8_t* forced /*nullable [T][B]*/, uint8_t* tpos, int8_t* tact,
                      uint8_t* tdone, float* trew, float* tval /*[T+1][B]*/, float* tlogp,
                      float* tlogits /*nullable [T][B][4]*/, uint8_t* tnear /*nullable*/, uint32_t env0) {
    const Dims d = make_dims(N, H);
    const std::vector<float> cp = compute_params(d, theta, prec);
#pragma omp parallel
    {
        std::vector<float> x(d.D), h1(H), h2(H);
        std::vector<double> acc;
        float out[5];
#pragma omp for schedule(static)
        for (int b = 0; b < B; ++b) {
            const uint32_t* w = walls + (size_t)b * d.W;
            for (int t = 0; t <= T; ++t) {
                const size_t i = (size_t)t * B + b;
                observe(d, w, pos[b], goal[b], x.data());
                forward_row(d, cp.data(), prec, x.data(), h1.data(), h2.data(), out, acc);
                tval[i] = out[4];
                if (t == T) break;
                if (tlogits) for (int k = 0; k < 4; ++k) tlogits[i * 4 + k] = out[k];
                int a;
                float lp;
                uint8_t nr;
                sample4(out, act_uniform(seed, env0 + (uint32_t)b, gstep0 + (uint32_t)t), &a, &lp, &nr);
                if (forced) {
                    a = (int)forced[i];
                    lp = (float)softmax4(out).logp[a];
                }
                tpos[i] = pos[b];
                tact[i] = (int8_t)a;
                tlogp[i] = lp;
                if (tnear) tnear[i] = nr;
                env_step(d, w, start[b], goal[b], cap, &pos[b], &tep[b], a, &trew[i], &tdone[i], kind);
            }
        }
    }
}

void orc_rollout_kind(int kind, int N, int H, int prec, int B, int T, int cap, const float* theta, const uint32_t* walls,
                      const uint8_t* start, const uint8_t* goal, uint8_t* pos, uint8_t* tep, uint64_t seed,
                      uint32_t gstep0, const int8_t* forced /*nullable [T][B]*/, uint8_t* tpos, int8_t* tact,
                      uint8_t* tdone, float* trew, float* tval /*[T+1][B]*/, float* tlogp,
                      float* tlogits /*nullable [T][B][4]*/, uint8_t* tnear /*nullable*/) {
    orc_rollout_env0(kind, N, H, prec, B, T, cap, theta, walls, start, goal, pos, tep, seed, gstep0, forced, tpos, tact, tdone,
                     trew, tval, tlogp, tlogits, tnear, 0u);
}

void orc_rollout(int N, int H, int prec, int B, int T, int cap, const float* theta, const uint32_t* walls,
                 const uint8_t* start, const uint8_t* goal, uint8_t* pos, uint8_t* tep, uint64_t seed,
                 uint32_t gstep0, const int8_t* forced, uint8_t* tpos, int8_t* tact, uint8_t* tdone, float* trew,
                 float* tval, float* tlogp, float* tlogits, uint8_t* tnear) {
    orc_rollout_kind(0, N, H, prec, B, T, cap, theta, walls, start, goal, pos, tep, seed, gstep0, forced, tpos, tact, tdone,
                     trew, tval, tlogp, tlogits, tnear);
}

// Generalised advantage estimation, reverse scan over t for each env:
//   d_t = 1 - done_t;  delta_t = r_t + gamma d_t V_{t+1} - V_t;  A_t = delta_t + gamma lambda d_t A_{t+1}
//   (A_T = 0);  ret_t = A_t + V_t.  Both goal and time-out ends cut the bootstrap.
void orc_gae(int T, int B, double gamma, double lambda, const float* rew, const float* val /*[T+1][B]*/,
             const uint8_t* done, float* adv, float* ret) {
    for (int b = 0; b < B; ++b) {
        double A = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            const size_t i = (size_t)t * B + b;
            const double dt = 1.0 - (double)done[i];
            const double delta = (double)rew[i] + gamma * dt * (double)val[i + B] - (double)val[i];
            A = delta + gamma * lambda * dt * A;
            adv[i] = (float)A;
            ret[i] = (float)(A + (double)val[i]);
        }
    }
}

// V-trace targets (Espeholt et al. 2018, "IMPALA", Eq. 1 and Remark 1 in its recursive form), reverse scan over t for
// each env.  The trajectory was generated by a behaviour policy mu (its log-probabilities logp_mu were recorded when the
// actions were taken); pi is the policy being updated (logp_pi, and the values V, come from the current parameters):
//   w_t = exp(logp_pi_t - logp_mu_t);  rho_t = min(rho_bar, w_t);  c_t = min(c_bar, w_t);  d_t = 1 - done_t
//   delta_t = rho_t (r_t + gamma d_t V_{t+1} - V_t)
//   e_t = delta_t + gamma d_t c_t e_{t+1},  e_T = 0          (e_t = v_t - V_t)
//   ret_t = v_t = V_t + e_t                                   value target
//   adv_t = rho_t (r_t + gamma d_t v_{t+1} - V_t),  v_T = V_T  policy-gradient advantage
// An episode end (goal or time-out) cuts both the bootstrap and the trace, as in the GAE scan.
void orc_vtrace(int T, int B, double gamma, double rho_bar, double c_bar, const float* rew, const float* val /*[T+1][B]*/,
                const uint8_t* done, const float* logp_pi, const float* logp_mu, float* adv, float* ret) {
    for (int b = 0; b < B; ++b) {
        double e_next = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            const size_t i = (size_t)t * B + b;
            const double w = std::exp((double)logp_pi[i] - (double)logp_mu[i]);
            const double rho = std::min(rho_bar, w), c = std::min(c_bar, w);
            const double dt = 1.0 - (double)done[i];
            const double v_next = (double)val[i + B] + e_next;
            const double delta = rho * ((double)rew[i] + gamma * dt * (double)val[i + B] - (double)val[i]);
            const double e = delta + gamma * dt * c * e_next;
            adv[i] = (float)(rho * ((double)rew[i] + gamma * dt * v_next - (double)val[i]));
            ret[i] = (float)((double)val[i] + e);
            e_next = e;
        }
    }
}

void orc_learn_f32(int N, int H, int prec, int B, int T, const float* theta, const uint32_t* walls,
                   const uint8_t* goal, const uint8_t* tpos, const int8_t* tact, const float* adv,
                   const float* ret, double c_v, double c_e, float* grads, double* loss4,
                   const uint32_t* gate1 /*nullable*/, const uint32_t* gate2 /*nullable*/, double* gate_info /*nullable [6]*/) {
    loss_and_grad<float>(make_dims(N, H), prec, B, T, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e, grads, loss4,
                         gate1, gate2, gate_info);
}

// fp64 instantiation (storage in double): used only to pin the gradient against finite differences.
void orc_learn_f64(int N, int H, int B, int T, const double* theta, const uint32_t* walls, const uint8_t* goal,
                   const uint8_t* tpos, const int8_t* tact, const double* adv, const double* ret, double c_v,
                   double c_e, double* grads /*nullable*/, double* loss4) {
    loss_and_grad<double>(make_dims(N, H), 0, B, T, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e, grads, loss4);
}

// The same with the clipped-surrogate policy term (logp_old = log-probabilities recorded when the actions were taken).
void orc_learn_ppo_f32(int N, int H, int prec, int B, int T, const float* theta, const uint32_t* walls,
                       const uint8_t* goal, const uint8_t* tpos, const int8_t* tact, const float* adv,
                       const float* ret, const float* logp_old, double clip, double c_v, double c_e, float* grads,
                       double* loss4, const uint32_t* gate1, const uint32_t* gate2, double* gate_info) {
    loss_and_grad<float>(make_dims(N, H), prec, B, T, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e, grads, loss4,
                         gate1, gate2, gate_info, logp_old, clip);
}

void orc_learn_ppo_f64(int N, int H, int B, int T, const double* theta, const uint32_t* walls, const uint8_t* goal,
                       const uint8_t* tpos, const int8_t* tact, const double* adv, const double* ret,
                       const double* logp_old, double clip, double c_v, double c_e, double* grads, double* loss4) {
    loss_and_grad<double>(make_dims(N, H), 0, B, T, theta, walls, goal, tpos, tact, adv, ret, c_v, c_e, grads, loss4,
                          nullptr, nullptr, nullptr, logp_old, clip);
}

// ----------------------------------------------------------------------------------------------
// Many policies: K independent networks, policy p acting in and learning from its own envs
// [p*Bp, min(B, (p+1)*Bp)), Bp = ceil(B/K) (the shape of the paper's meta-learning use case, Section 4.1: many
// small policies trained side by side on one accelerator).  Nothing couples the policies, so every function here
// is literally a loop of K single-policy calls.  Layout: parameters and gradients [K][P]; per-env arrays [B] in
// global env order; per-step arrays as K consecutive blocks, block p = [T][B_p] (values [T+1][B_p]) of policy p.
// ----------------------------------------------------------------------------------------------
static int policy_envs(int B, int K, int p, int* first) {
    const int Bp = (B + K - 1) / K;
    *first = p * Bp;
    return std::min(Bp, B - p * Bp);
}

void orc_param_init_policy(uint64_t seed, int N, int H, uint32_t policy, float* theta) {
    param_init(seed, make_dims(N, H), theta, policy);
}

void orc_rollout_policies(int kind, int N, int H, int prec, int B, int K, int T, int cap, const float* theta /*[K][P]*/,
                          const uint32_t* walls, const uint8_t* start, const uint8_t* goal, uint8_t* pos, uint8_t* tep,
                          uint64_t seed, uint32_t gstep0, uint8_t* tpos, int8_t* tact, uint8_t* tdone, float* trew,
                          float* tval, float* tlogp, float* tlogits /*nullable*/, uint8_t* tnear /*nullable*/) {
    const Dims d = make_dims(N, H);
    for (int p = 0; p < K; ++p) {
        int e0;
        const int Bk = policy_envs(B, K, p, &e0);
        const size_t o = (size_t)T * e0, ov = (size_t)(T + 1) * e0;  // every earlier block is a full one
        orc_rollout_env0(kind, N, H, prec, Bk, T, cap, theta + (size_t)p * d.P, walls + (size_t)e0 * d.W, start + e0, goal + e0,
                         pos + e0, tep + e0, seed, gstep0, nullptr, tpos + o, tact + o, tdone + o, trew + o, tval + ov, tlogp + o,
                         tlogits ? tlogits + 4 * o : nullptr, tnear ? tnear + o : nullptr, (uint32_t)e0);
    }
}

void orc_gae_policies(int T, int B, int K, double gamma, double lambda, const float* rew, const float* val,
                      const uint8_t* done, float* adv, float* ret) {
    for (int p = 0; p < K; ++p) {
        int e0;
        const int Bk = policy_envs(B, K, p, &e0);
        const size_t o = (size_t)T * e0, ov = (size_t)(T + 1) * e0;
        orc_gae(T, Bk, gamma, lambda, rew + o, val + ov, done + o, adv + o, ret + o);
    }
}

// Each policy's gradient is the mean over ITS OWN B_p*T rows.  gates / gate_info as in orc_learn_f32, per policy:
// gate bitmaps as K blocks [T*B_p][ceil(H/32)], gate_info [K][6].
void orc_learn_policies(int N, int H, int prec, int B, int K, int T, const float* theta /*[K][P]*/, const uint32_t* walls,
                        const uint8_t* goal, const uint8_t* tpos, const int8_t* tact, const float* adv, const float* ret,
                        double c_v, double c_e, float* grads /*[K][P]*/, double* loss4 /*[K][4]*/,
                        const uint32_t* gate1 /*nullable*/, const uint32_t* gate2 /*nullable*/, double* gate_info /*nullable*/) {
    const Dims d = make_dims(N, H);
    const size_t GW = (size_t)(H + 31) / 32;
    for (int p = 0; p < K; ++p) {
        int e0;
        const int Bk = policy_envs(B, K, p, &e0);
        const size_t o = (size_t)T * e0;
        loss_and_grad<float>(d, prec, Bk, T, theta + (size_t)p * d.P, walls + (size_t)e0 * d.W, goal + e0, tpos + o, tact + o,
                             adv + o, ret + o, c_v, c_e, grads + (size_t)p * d.P, loss4 + 4 * p, gate1 ? gate1 + o * GW : nullptr,
                             gate2 ? gate2 + o * GW : nullptr, gate_info ? gate_info + 6 * p : nullptr);
    }
}

// Adam (Kingma & Ba, Algorithm 1), k = step index AFTER the increment (first call: k = 1):
//   m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2;  theta -= lr * (m/(1-b1^k)) / (sqrt(v/(1-b2^k)) + eps)
void orc_adam(size_t P, float* theta, const float* g, float* m, float* v, int k, double lr, double b1,
              double b2, double eps) {
    const double c1 = 1.0 - std::pow(b1, (double)k), c2 = 1.0 - std::pow(b2, (double)k);
    for (size_t i = 0; i < P; ++i) {
        const double gi = (double)g[i];
        const double mi = b1 * (double)m[i] + (1.0 - b1) * gi;
        const double vi = b2 * (double)v[i] + (1.0 - b2) * gi * gi;
        m[i] = (float)mi;
        v[i] = (float)vi;
        const double mhat = (double)m[i] / c1, vhat = (double)v[i] / c2;
        theta[i] = (float)((double)theta[i] - lr * mhat / (std::sqrt(vhat) + eps));
    }
}

}  // extern "C"
