// Host side of the C ABI declared in include/anakin.h: configuration checks, workspace carving, state
// tracking and kernel enqueueing.  The host only schedules (Podracer paper, Section 3.1): no call in the
// rollout/learn/run path copies data or synchronises.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

using namespace anakin;

struct anakin_handle {
    anakin_cfg cfg;
    Dims d;
    Buffers b;
    unsigned char* ws;
    size_t ws_bytes;
    cudaStream_t stream;
    bool is_reset;
    bool rollout_pending;
    bool base_valid;  // `base` matches the current parameters
    bool frags_valid; // the tensor-pipe fragment copies of W2 match the current parameters
    bool adv_valid;   // ADV/RET were computed from the pending trajectory (by the rollout's fused GAE scan)
    bool acts_valid;  // the saved h1/h2 belong to the pending trajectory and the current parameters
    int last_T;
    int NS;
    int K;             // policies (>= 1)
    size_t sub_bytes;  // size of one policy's sub-workspace
    uint64_t seed;
    int64_t gstep;
    int64_t adam_k;
    uint64_t launches;
    Profiler prof;
    char cuda_err[256];
    Ctx ctx() { return Ctx{stream, &launches, &prof}; }
};

namespace {

int validate(const anakin_cfg* c) {
    if (!c) return ANAKIN_E_INVALID_ARG;
    if (c->struct_size != sizeof(anakin_cfg)) return ANAKIN_E_INVALID_ARG;
    if (c->B < 1 || c->T_max < 1 || c->episode_cap < 1 || c->episode_cap > 255) return ANAKIN_E_INVALID_ARG;
    if (!(c->wall_density >= 0.0 && c->wall_density < 1.0)) return ANAKIN_E_INVALID_ARG;
    if (c->precision != ANAKIN_PRECISION_FP32 && c->precision != ANAKIN_PRECISION_BF16) return ANAKIN_E_INVALID_ARG;
    if (c->n_policies < 0) return ANAKIN_E_INVALID_ARG;
    if (c->env_kind != ANAKIN_ENV_GRID && c->env_kind != ANAKIN_ENV_TORUS) return ANAKIN_E_UNSUPPORTED_CFG;
    if (c->env_offset < 0 || (double)c->env_offset + (double)c->B > 2147483647.0) return ANAKIN_E_INVALID_ARG;
    if (c->N < 2 || c->N > 16) return ANAKIN_E_UNSUPPORTED_CFG;
    const int hj = c->H / 32;
    if (c->H % 32 != 0) return ANAKIN_E_UNSUPPORTED_CFG;
    switch (hj) {
        case 1: case 2: case 3: case 4: case 6: case 8: case 12: case 16: case 24: case 32: break;
        default: return ANAKIN_E_UNSUPPORTED_CFG;
    }
    if ((double)c->B * (double)c->T_max > 2.0e9) return ANAKIN_E_UNSUPPORTED_CFG;
    if (c->n_policies >= 2) {  // many policies: fp32 on the warp-level tensor path, every policy with at least one env
        const int K = c->n_policies, Bp = (c->B + K - 1) / K;
        if (K > c->B || (long long)(K - 1) * Bp >= c->B) return ANAKIN_E_INVALID_ARG;
        if (K > 65535 || c->precision != ANAKIN_PRECISION_FP32 || (c->H != 64 && c->H != 128)) return ANAKIN_E_UNSUPPORTED_CFG;
    }
    return ANAKIN_OK;
}

int policies_of(const anakin_cfg& c) { return c.n_policies >= 2 ? c.n_policies : 1; }
int envs_per_policy(const anakin_cfg& c) { const int K = policies_of(c); return (c.B + K - 1) / K; }

int choose_splits(const Dims& d) {
    const int tiles = ((d.H + 63) / 64) * ((d.H + 63) / 64);
    int ns = (4 * 148 + tiles - 1) / tiles;
    if (ns > 64) ns = 64;
    const size_t R = (size_t)d.B * d.Tmax;
    const size_t cap = R / 64 > 0 ? R / 64 : 1;
    if ((size_t)ns > cap) ns = (int)cap;
    if (ns < 1) ns = 1;
    return ns;
}

// Carves the workspace; with base == nullptr only sizes it.
size_t carve(const anakin_cfg& c, const Dims& d, int NS, unsigned char* base, Buffers* out) {
    size_t off = 0;
    auto take = [&](size_t bytes) -> void* {
        void* p = base ? base + off : nullptr;
        off += (bytes + 255) / 256 * 256;
        return p;
    };
    Buffers b;
    memset(&b, 0, sizeof(b));
    const size_t P = d.P, B = d.B, T = d.Tmax, R = B * T, H = d.H;
    b.theta = (float*)take(P * 4);
    b.theta_c = c.precision == ANAKIN_PRECISION_BF16 ? (float*)take(P * 4) : b.theta;
    b.grads = (float*)take(P * 4);
    b.adam_m = (float*)take(P * 4);
    b.adam_v = (float*)take(P * 4);
    b.walls = (uint32_t*)take(B * d.W * 4);
    b.start = (uint8_t*)take(B);
    b.goal = (uint8_t*)take(B);
    b.pos = (uint8_t*)take(B);
    b.tep = (uint8_t*)take(B);
    b.tpos = (uint8_t*)take(R);
    b.tact = (int8_t*)take(R);
    b.tdone = (uint8_t*)take(R);
    b.trew = (float*)take(R * 4);
    b.tval = (float*)take((R + B) * 4);
    b.tlogp = (float*)take(R * 4);
    b.adv = (float*)take(R * 4);
    b.ret = (float*)take(R * 4);
    b.dbg_logits = c.debug_logits ? (float*)take(R * 16) : nullptr;
    b.dbg_gates = c.debug_logits ? (uint32_t*)take(2 * R * (H / 32) * 4) : nullptr;
    b.base = (float*)take(B * H * 4);
    const bool mma = rollout_mma_supported(d.H), tensor = tensor_path_supported(d.H, c.precision);
    const bool frags = mma && rollout_uses_fragments(d.H, c.precision);
    b.w2f_hi = frags ? (uint2*)take(H * H * 2) : nullptr;
    b.w2f_lo = frags ? (uint2*)take(H * H * 2) : nullptr;
    b.w2p_hi = tensor ? (uint16_t*)take(H * H * 2) : nullptr;
    b.w2p_lo = mma ? (uint16_t*)take(H * H * 2) : nullptr;
    b.h1 = (float*)take(R * H * 4);
    b.gate1 = (dh1_agent_tc_supported(d) && policies_of(c) <= 1) ? (uint8_t*)take(R * (H / 8)) : nullptr;  // what the fused dh1 kernel gates with
    b.h2 = (float*)take(R * H * 4);
    b.out5 = tensor ? (float*)take(R * 8 * 4) : nullptr;
    b.vboot = tensor ? (float*)take(B * 4) : nullptr;
    b.dh2 = (float*)take(R * H * 4);
    b.dh1 = (float*)take(R * H * 4);
    b.dout = (float*)take(R * 8 * 4);
    b.S = (float*)take(4 * B * H * 4);  // up to four t-slices of two 16-bit planes
    size_t part_floats = (size_t)NS * P, loss_blocks = LOSS_BLOCKS;
    if (tensor) {
        LearnPlan pl;
        learn_mma_plan(d, &pl);
        if (pl.part_floats > part_floats) part_floats = pl.part_floats;
        if ((size_t)pl.loss_blocks > loss_blocks) loss_blocks = pl.loss_blocks;
    }
    b.part = (float*)take(part_floats * 4);
    b.loss_part = (float*)take(loss_blocks * 4 * 4);
    b.stats = (anakin_stats*)take(sizeof(anakin_stats));
    b.status = (int*)take(sizeof(int));
    if (out) *out = b;
    return off;
}

int fail_cuda(anakin_t* h, cudaError_t e) {
    snprintf(h->cuda_err, sizeof(h->cuda_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return ANAKIN_E_CUDA;
}

struct Blob {
    void* ptr;
    size_t bytes;
    bool writable;
    bool host_only;
    bool is_traj;
};

// The blob of ONE policy with `envs` envs (the handle's Buffers are the first policy's).
Blob blob_of(anakin_t* h, int which, int envs) {
    const Dims& d = h->d;
    const Buffers& b = h->b;
    const size_t B = (size_t)envs, T = h->last_T > 0 ? h->last_T : d.Tmax, R = B * T, P = d.P;
    switch (which) {
        case ANAKIN_PARAMS: return {b.theta, P * 4, true, false, false};
        case ANAKIN_GRADS: return {b.grads, P * 4, true, false, false};
        case ANAKIN_ADAM_M: return {b.adam_m, P * 4, true, false, false};
        case ANAKIN_ADAM_V: return {b.adam_v, P * 4, true, false, false};
        case ANAKIN_ADAM_STEP: return {&h->adam_k, 8, true, true, false};
        case ANAKIN_ENV_WALLS: return {b.walls, B * d.W * 4, true, false, false};
        case ANAKIN_ENV_START: return {b.start, B, true, false, false};
        case ANAKIN_ENV_GOAL: return {b.goal, B, true, false, false};
        case ANAKIN_ENV_POS: return {b.pos, B, true, false, false};
        case ANAKIN_ENV_TEP: return {b.tep, B, true, false, false};
        case ANAKIN_GLOBAL_STEP: return {&h->gstep, 8, true, true, false};
        case ANAKIN_TRAJ_POS: return {b.tpos, R, true, false, true};
        case ANAKIN_TRAJ_ACTION: return {b.tact, R, true, false, true};
        case ANAKIN_TRAJ_DONE: return {b.tdone, R, true, false, true};
        case ANAKIN_TRAJ_REWARD: return {b.trew, R * 4, true, false, true};
        case ANAKIN_TRAJ_VALUE: return {b.tval, (R + B) * 4, true, false, true};
        case ANAKIN_TRAJ_LOGP: return {b.tlogp, R * 4, true, false, true};
        case ANAKIN_ADV: return {b.adv, R * 4, true, false, true};
        case ANAKIN_RET: return {b.ret, R * 4, true, false, true};
        case ANAKIN_STATS: return {b.stats, sizeof(anakin_stats), false, false, false};
        case ANAKIN_DEBUG_LOGITS: return {b.dbg_logits, b.dbg_logits ? R * 16 : 0, false, false, false};
        case ANAKIN_DEBUG_GATES: return {b.dbg_gates, b.dbg_gates ? 2 * R * (size_t)(d.H / 32) * 4 : 0, false, false, false};
        default: return {nullptr, 0, false, false, false};
    }
}

// Size of a blob over all policies (K consecutive single-policy blobs).
size_t blob_total(anakin_t* h, int which) {
    const Blob b0 = blob_of(h, which, h->d.B);
    if (b0.host_only || h->K == 1) return b0.bytes;
    return b0.bytes * (size_t)(h->K - 1) + blob_of(h, which, h->d.B_last).bytes;
}

// 16-bit copies of W2 in the layouts the tensor-core kernels read.
cudaError_t pack_w2(anakin_t* h) {
    if (wide_supported(h->d.H, h->cfg.precision)) return launch_pack_w2_wide(h->d, h->b, h->ctx());
    return launch_pack_w2(h->d, h->b, h->cfg.precision, h->ctx());
}

int do_rollout(anakin_t* h, int T, const int8_t* forced) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset) return ANAKIN_E_BAD_STATE;
    if (T < 1 || T > h->cfg.T_max) return ANAKIN_E_INVALID_ARG;
    cudaError_t e;
    if (!h->base_valid) {
        e = launch_env_base(h->d, h->b, h->ctx());
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->base_valid = true;
    }
    if (!h->frags_valid) {
        e = pack_w2(h);
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->frags_valid = true;
    }
    RolloutArgs a;
    a.d = h->d;
    a.b = h->b;
    a.T = T;
    a.cap = h->cfg.episode_cap;
    a.gstep0 = (uint32_t)h->gstep;
    a.key0 = (uint32_t)(h->seed & 0xFFFFFFFFu);
    a.key1 = (uint32_t)(h->seed >> 32);
    a.env_kind = h->cfg.env_kind;
    a.forced = forced;
    a.replay = 0;
    a.fuse_gae = rollout_mma_supported(h->d.H) ? 1 : 0;
    a.gamma = h->cfg.gamma;
    a.lambda = h->cfg.gae_lambda;
    e = launch_rollout(a, h->cfg.precision, h->ctx());
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->gstep += T;
    h->last_T = T;
    h->rollout_pending = true;
    h->acts_valid = tensor_path_supported(h->d.H, h->cfg.precision);  // the tensor-core rollouts save h1 and h2 of every row
    h->adv_valid = a.fuse_gae != 0;
    return ANAKIN_OK;
}

// Recomputes and saves the activations of the pending trajectory's rows (positions from TRAJ_POS); with_boot: also the
// value of the current env state (the state after the last recorded step) under the current parameters, into vboot.
int replay_activations(anakin_t* h, bool with_boot = false) {
    cudaError_t e;
    if (!h->base_valid) {
        e = launch_env_base(h->d, h->b, h->ctx());
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->base_valid = true;
    }
    if (!h->frags_valid) {
        e = pack_w2(h);
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->frags_valid = true;
    }
    RolloutArgs a;
    a.d = h->d;
    a.b = h->b;
    a.T = h->last_T;
    a.cap = h->cfg.episode_cap;
    a.gstep0 = 0;
    a.key0 = a.key1 = 0;
    a.env_kind = h->cfg.env_kind;
    a.forced = nullptr;
    a.replay = with_boot ? 2 : 1;
    a.fuse_gae = 0;
    a.gamma = a.lambda = 0.f;
    if (wide_supported(h->d.H, h->cfg.precision)) {
        e = launch_rollout_wide(a, h->ctx());
    } else {
        Scope sc(h->ctx(), K_REPLAY);
        e = launch_rollout_mma(a, h->cfg.precision, h->stream);
    }
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->acts_valid = true;
    return ANAKIN_OK;
}

}  // namespace

extern "C" {

int anakin_workspace_bytes(const anakin_cfg* cfg, size_t* bytes) {
    if (!bytes) return ANAKIN_E_INVALID_ARG;
    const int rc = validate(cfg);
    if (rc != ANAKIN_OK) return rc;
    Dims d = make_dims(envs_per_policy(*cfg), cfg->N, cfg->H, cfg->T_max);
    d.npol = policies_of(*cfg);  // (the update's launch plan, and with it the partial buffers, depend on it)
    *bytes = carve(*cfg, d, choose_splits(d), nullptr, nullptr) * (size_t)policies_of(*cfg);  // one sub-workspace per policy
    return ANAKIN_OK;
}

int anakin_create(const anakin_cfg* cfg, void* dev_workspace, size_t bytes, void* cuda_stream, anakin_t** out) {
    if (!out) return ANAKIN_E_INVALID_ARG;
    *out = nullptr;
    const int rc = validate(cfg);
    if (rc != ANAKIN_OK) return rc;
    if (!dev_workspace || ((uintptr_t)dev_workspace & 255u)) return ANAKIN_E_INVALID_ARG;
    const int K = policies_of(*cfg), Bp = envs_per_policy(*cfg);
    Dims d = make_dims(Bp, cfg->N, cfg->H, cfg->T_max);
    d.env0 = cfg->env_offset;
    d.npol = K;
    const int NS = choose_splits(d);
    const size_t sub = carve(*cfg, d, NS, nullptr, nullptr), need = sub * (size_t)K;
    d.B_last = cfg->B - (K - 1) * Bp;
    d.pstride = sub;
    if (bytes < need) return ANAKIN_E_WORKSPACE_TOO_SMALL;
    anakin_t* h = new (std::nothrow) anakin_t();
    if (!h) return ANAKIN_E_INVALID_ARG;
    h->is_reset = h->rollout_pending = h->base_valid = h->frags_valid = h->acts_valid = h->adv_valid = false;
    h->last_T = 0;
    h->seed = 0;
    h->gstep = h->adam_k = 0;
    h->launches = 0;
    h->cuda_err[0] = 0;
    h->cfg = *cfg;
    h->d = d;
    h->NS = NS;
    h->K = K;
    h->sub_bytes = sub;
    h->ws = (unsigned char*)dev_workspace;
    h->ws_bytes = bytes;
    h->stream = (cudaStream_t)cuda_stream;
    carve(*cfg, d, NS, h->ws, &h->b);
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e == cudaSuccess && cur != cfg->device) e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) {
        delete h;
        return ANAKIN_E_CUDA;
    }
    *out = h;
    return ANAKIN_OK;
}

int anakin_destroy(anakin_t* h) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    for (const Profiler::Rec& r : h->prof.recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : h->prof.pool) cudaEventDestroy(e);
    delete h;
    return ANAKIN_OK;
}

int anakin_reset(anakin_t* h, uint64_t seed) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    cudaError_t e = launch_reset(h->d, h->b, seed, h->cfg.wall_density, h->cfg.precision, h->ctx());
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->seed = seed;
    h->gstep = 0;
    h->adam_k = 0;
    h->is_reset = true;
    h->rollout_pending = false;
    h->base_valid = false;
    h->frags_valid = false;
    h->acts_valid = false;
    h->adv_valid = false;
    h->last_T = 0;
    return ANAKIN_OK;
}

int anakin_rollout(anakin_t* h, int T) { return do_rollout(h, T, nullptr); }

int anakin_rollout_forced(anakin_t* h, int T, const int8_t* dev_actions) {
    if (!dev_actions) return ANAKIN_E_INVALID_ARG;
    return do_rollout(h, T, dev_actions);
}

int anakin_gae(anakin_t* h) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    cudaError_t e = launch_gae(h->d, h->b, h->last_T, h->cfg.gamma, h->cfg.gae_lambda, h->ctx());
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->adv_valid = true;
    return ANAKIN_OK;
}

// The update proper, from ADV/RET as they stand.  phase 0: through Adam; phase 1: stop at the batch-mean gradient.
static int learn_after_gae(anakin_t* h, int phase, float ppo_clip = 0.f, bool consume = true) {
    cudaError_t e;
    if (!h->base_valid) {
        e = launch_env_base(h->d, h->b, h->ctx());
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->base_valid = true;
    }
    if (!h->frags_valid) {
        e = pack_w2(h);
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->frags_valid = true;
    }
    LearnArgs a;
    a.d = h->d;
    a.b = h->b;
    a.T = h->last_T;
    a.NS = h->NS;
    a.c_v = h->cfg.value_coef;
    a.c_e = h->cfg.entropy_coef;
    a.lr = h->cfg.lr;
    a.beta1 = h->cfg.adam_b1;
    a.beta2 = h->cfg.adam_b2;
    a.eps = h->cfg.adam_eps;
    a.adam_k = (int)(h->adam_k + 1);
    a.bc1 = (float)(1.0 - pow((double)a.beta1, (double)a.adam_k));
    a.bc2 = (float)(1.0 - pow((double)a.beta2, (double)a.adam_k));
    a.phase = phase;
    a.grad_div = 1.f;
    a.ppo_clip = ppo_clip;
    {   // smallest power of two >= R: keeps the scaled output gradients O(1) for the fp16 operand format
        const double Rrows = (double)h->d.B * (double)h->last_T;
        int ex = 0;
        while (ldexp(1.0, ex) < Rrows) ++ex;
        a.gscale = (float)ldexp(1.0, ex);
        a.inv_gscale = (float)ldexp(1.0, -ex);
    }
    if (tensor_path_supported(h->d.H, h->cfg.precision)) {
        if (!h->acts_valid) {
            const int rc = replay_activations(h);
            if (rc != ANAKIN_OK) return rc;
        }
        e = launch_learn_mma(a, h->cfg.precision, h->ctx());
    } else {
        e = launch_learn(a, h->cfg.precision, h->ctx());
    }
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->acts_valid = false;  // saved activations belong to the parameters they were computed with
    if (consume) {
        h->adv_valid = false;
        h->rollout_pending = false;
    }
    if (phase == 0) {
        h->adam_k += 1;
        h->base_valid = false;  // parameters changed
        h->frags_valid = tensor_path_supported(h->d.H, h->cfg.precision);  // the tensor-core update refreshes the 16-bit copies itself
    }
    return ANAKIN_OK;
}

int anakin_learn(anakin_t* h) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    if (!h->adv_valid) {  // the tensor-pipe rollout already ran the GAE scan of a trajectory it produced
        const int rc = anakin_gae(h);
        if (rc != ANAKIN_OK) return rc;
    }
    return learn_after_gae(h, 0);
}

int anakin_update(anakin_t* h) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    return learn_after_gae(h, 0);
}

int anakin_learn_ppo(anakin_t* h, int epochs, float clip_eps) {
    if (!h || epochs < 1 || !(clip_eps > 0.f)) return ANAKIN_E_INVALID_ARG;
    if (h->K > 1) return ANAKIN_E_UNSUPPORTED_CFG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    if (!h->adv_valid) {
        const int rc = anakin_gae(h);
        if (rc != ANAKIN_OK) return rc;
    }
    for (int e = 0; e < epochs; ++e) {
        const int rc = learn_after_gae(h, 0, clip_eps, e == epochs - 1);
        if (rc != ANAKIN_OK) return rc;
    }
    return ANAKIN_OK;
}

int anakin_learn_vtrace(anakin_t* h, int epochs, float rho_bar, float c_bar) {
    if (!h || epochs < 1 || !(rho_bar >= 0.f) || !(c_bar >= 0.f)) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    if (h->K > 1 || !tensor_path_supported(h->d.H, h->cfg.precision)) return ANAKIN_E_UNSUPPORTED_CFG;  // needs the saved head outputs
    for (int ep = 0; ep < epochs; ++ep) {
        cudaError_t e;
        if (!h->base_valid) {
            e = launch_env_base(h->d, h->b, h->ctx());
            if (e != cudaSuccess) return fail_cuda(h, e);
            h->base_valid = true;
        }
        if (!h->frags_valid) {
            e = pack_w2(h);
            if (e != cudaSuccess) return fail_cuda(h, e);
            h->frags_valid = true;
        }
        // Head outputs of the recorded rows under the current parameters: the rollout's own when nothing has changed since
        // (then the recorded bootstrap row is the current one too), else a replay that also evaluates the final state.
        const float* boot = h->b.tval + (size_t)h->last_T * h->d.B;
        if (!h->acts_valid) {
            const int rc = replay_activations(h, true);
            if (rc != ANAKIN_OK) return rc;
            boot = h->b.vboot;
        }
        e = launch_vtrace(h->d, h->b, h->last_T, h->cfg.gamma, rho_bar, c_bar, boot, h->ctx());
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->adv_valid = true;
        const int rc = learn_after_gae(h, 0, 0.f, ep == epochs - 1);
        if (rc != ANAKIN_OK) return rc;
    }
    return ANAKIN_OK;
}

int anakin_grads(anakin_t* h) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset || !h->rollout_pending) return ANAKIN_E_BAD_STATE;
    if (!h->adv_valid) {
        const int rc = anakin_gae(h);
        if (rc != ANAKIN_OK) return rc;
    }
    return learn_after_gae(h, 1);
}

int anakin_apply_grads(anakin_t* h) { return anakin_apply_grads_mean(h, 1); }

int anakin_apply_grads_mean(anakin_t* h, int n_replicas) {
    if (!h || n_replicas < 1) return ANAKIN_E_INVALID_ARG;
    if (!h->is_reset) return ANAKIN_E_BAD_STATE;
    LearnArgs a;
    memset(&a, 0, sizeof(a));
    a.d = h->d;
    a.b = h->b;
    a.lr = h->cfg.lr;
    a.beta1 = h->cfg.adam_b1;
    a.beta2 = h->cfg.adam_b2;
    a.eps = h->cfg.adam_eps;
    a.adam_k = (int)(h->adam_k + 1);
    a.bc1 = (float)(1.0 - pow((double)a.beta1, (double)a.adam_k));
    a.bc2 = (float)(1.0 - pow((double)a.beta2, (double)a.adam_k));
    a.grad_div = (float)n_replicas;
    const cudaError_t e = launch_adam_only(a, h->cfg.precision, h->ctx());
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->adam_k += 1;
    h->base_valid = false;  // parameters changed
    h->frags_valid = tensor_path_supported(h->d.H, h->cfg.precision);  // every element of the 16-bit copies of W2 was rewritten
    return ANAKIN_OK;
}

int anakin_run(anakin_t* h, int iters) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    if (iters < 0) return ANAKIN_E_INVALID_ARG;
    for (int it = 0; it < iters; ++it) {
        int rc = do_rollout(h, h->cfg.T_max, nullptr);
        if (rc != ANAKIN_OK) return rc;
        rc = anakin_learn(h);
        if (rc != ANAKIN_OK) return rc;
    }
    return ANAKIN_OK;
}

size_t anakin_blob_bytes(anakin_t* h, int which) {
    if (!h) return 0;
    return blob_total(h, which);
}

static int copy_blob(anakin_t* h, int which, void* ptr, size_t bytes, int ptr_is_device, bool to_lib) {
    if (!h || !ptr) return ANAKIN_E_INVALID_ARG;
    const Blob bl = blob_of(h, which, h->d.B);
    if (!bl.ptr || bl.bytes == 0 || bytes != blob_total(h, which)) return ANAKIN_E_INVALID_ARG;
    if (to_lib && !bl.writable) return ANAKIN_E_INVALID_ARG;
    if (bl.host_only) {
        if (ptr_is_device) return ANAKIN_E_INVALID_ARG;
        if (to_lib) memcpy(bl.ptr, ptr, bytes); else memcpy(ptr, bl.ptr, bytes);
        return ANAKIN_OK;
    }
    if (ptr_is_device < 0 || ptr_is_device > 2) return ANAKIN_E_INVALID_ARG;
    // 2 = page-locked host memory, asynchronous: the runtime infers the direction from the (unified) addresses
    const cudaMemcpyKind kind = ptr_is_device == 1 ? cudaMemcpyDeviceToDevice
                              : ptr_is_device == 2 ? cudaMemcpyDefault
                              : (to_lib ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost);
    cudaError_t e = cudaSuccess;
    {   // one copy per policy: its blob sits at the same offset inside its sub-workspace
        unsigned char* user = static_cast<unsigned char*>(ptr);
        for (int p = 0; p < h->K && e == cudaSuccess; ++p) {
            const size_t n = p == h->K - 1 ? blob_of(h, which, h->d.B_last).bytes : bl.bytes;
            unsigned char* mine = static_cast<unsigned char*>(bl.ptr) + (size_t)p * h->sub_bytes;
            e = to_lib ? cudaMemcpyAsync(mine, user, n, kind, h->stream) : cudaMemcpyAsync(user, mine, n, kind, h->stream);
            user += n;
        }
    }
    if (e != cudaSuccess) return fail_cuda(h, e);
    if (to_lib) {
        if (which == ANAKIN_PARAMS) {
            e = launch_refresh_compute_params(h->d, h->b, h->cfg.precision, h->ctx());
            if (e != cudaSuccess) return fail_cuda(h, e);
            h->base_valid = false;
            h->frags_valid = false;
            h->acts_valid = false;
        }
        if (which == ANAKIN_ENV_WALLS || which == ANAKIN_ENV_GOAL) h->base_valid = h->acts_valid = false;
        if (which == ANAKIN_TRAJ_POS) h->acts_valid = false;
        if (bl.is_traj) h->adv_valid = false;  // includes ADV and RET: anakin_learn recomputes them, anakin_update uses them
        if (bl.is_traj && h->is_reset) {
            if (h->last_T == 0) h->last_T = h->cfg.T_max;
            h->rollout_pending = true;
        }
    }
    // A read into host memory must have landed when the call returns.  A write from host memory is stream-ordered like
    // everything else: the runtime stages pageable memory before cudaMemcpyAsync returns, and a page-locked source is the
    // caller's to keep unchanged until the stream has run the copy.
    if (!ptr_is_device && !to_lib) {
        e = cudaStreamSynchronize(h->stream);
        if (e != cudaSuccess) return fail_cuda(h, e);
    }
    return ANAKIN_OK;
}

int anakin_get(anakin_t* h, int which, void* ptr, size_t bytes, int ptr_is_device) {
    return copy_blob(h, which, ptr, bytes, ptr_is_device, false);
}

int anakin_set(anakin_t* h, int which, const void* ptr, size_t bytes, int ptr_is_device) {
    return copy_blob(h, which, const_cast<void*>(ptr), bytes, ptr_is_device, true);
}

int anakin_status(anakin_t* h, int* device_status) {
    if (!h || !device_status) return ANAKIN_E_INVALID_ARG;
    int st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, h->b.status, sizeof(int), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e);
    *device_status = st;
    return st == 0 ? ANAKIN_OK : ANAKIN_E_DEVICE_STATUS;
}

int anakin_selftest_wait_timeout(anakin_t* h, int64_t limit_clocks) {
    if (!h || limit_clocks < 1 || limit_clocks > 2000000000LL) return ANAKIN_E_INVALID_ARG;
    const cudaError_t e = launch_selftest_wait(h->b.status, (long long)limit_clocks, nullptr, h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e);
    ++h->launches;
    return ANAKIN_OK;
}

uint64_t anakin_launch_count(anakin_t* h) { return h ? h->launches : 0; }

int anakin_kernel_count(void) { return K_COUNT; }

const char* anakin_kernel_name(int id) {
    static const char* names[K_COUNT] = {"reset_env", "reset_params", "refresh_params", "env_base", "rollout", "gae", "h1",
                                         "fwd2", "heads_loss", "dh1", "dw2", "colsums", "sum_over_t", "dw1_agent",
                                         "dw1_walls", "dw1_goal", "reduce_adam", "loss_total", "pack_gates", "pack_w2", "heads_bwd", "replay", "vtrace"};
    return (id >= 0 && id < K_COUNT) ? names[id] : "";
}

int anakin_profile_enable(anakin_t* h, int on) {
    if (!h) return ANAKIN_E_INVALID_ARG;
    h->prof.on = on != 0;
    return ANAKIN_OK;
}

int anakin_profile_read(anakin_t* h, int n_ids, double* total_ms, uint64_t* counts) {
    if (!h || !total_ms || !counts || n_ids < K_COUNT) return ANAKIN_E_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return fail_cuda(h, e);
    for (int i = 0; i < n_ids; ++i) { total_ms[i] = 0.0; counts[i] = 0; }
    for (const Profiler::Rec& r : h->prof.recs) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, r.a, r.b);
        if (e != cudaSuccess) return fail_cuda(h, e);
        total_ms[r.id] += ms;
        counts[r.id] += 1;
        h->prof.pool.push_back(r.a);
        h->prof.pool.push_back(r.b);
    }
    h->prof.recs.clear();
    return ANAKIN_OK;
}

const char* anakin_strerror(int code) {
    switch (code) {
        case ANAKIN_OK: return "ok";
        case ANAKIN_E_INVALID_ARG: return "invalid argument";
        case ANAKIN_E_BAD_STATE: return "call not valid in the handle's current state";
        case ANAKIN_E_WORKSPACE_TOO_SMALL: return "workspace too small";
        case ANAKIN_E_UNSUPPORTED_CFG: return "unsupported configuration";
        case ANAKIN_E_CUDA: return "CUDA runtime error";
        case ANAKIN_E_DEVICE_STATUS: return "device status word is non-zero";
        default: return "unknown error code";
    }
}

const char* anakin_last_cuda_error(anakin_t* h) { return h ? h->cuda_err : ""; }

}  // extern "C"
