// anakin_rollout_noalloc: the rollout for callers that cannot allocate device memory.
//
// Who cannot allocate: code that runs where cudaMalloc is forbidden or unaffordable -- a control loop with a
// fixed memory budget handed out at start-up, a plug-in inside a host application that owns the allocator, a
// process that must not synchronise the device (cudaMalloc and cudaFree may) -- and that therefore cannot size
// and provide the library's workspace either.  Such a caller passes only the rollout's inputs and outputs; the
// scratch the rollout needs (the per-env first-layer constant `base`, B*H floats, and two repacked copies of the
// second-layer weights) lives in a file-scope device array of fixed size inside this library.
//
// The array below is device memory reserved in every CUDA context that loads the library, from load to exit,
// whether or not this entry point is ever called.  Its name is a host-side stand-in in host code: the device
// address is obtained once per device with cudaGetSymbolAddress and only that pointer is handed to kernels.
#include <cstdio>
#include <cstring>

#include "common.cuh"

using namespace anakin;

namespace {

constexpr size_t kMaxBaseFloats = ANAKIN_NOALLOC_MAX_BH;  // B*H limit (floats)
constexpr size_t kW2FragBytes = 2 * 256 * 256 * 2;          // W2 as tensor-pipe fragments, hi and lo planes (H <= 256)
constexpr size_t kW2PlaneBytes = 2 * 256 * 256 * 2;         // W2 row-major as 16-bit hi and lo planes (H <= 256)
constexpr size_t kTailBytes = 256;                          // statistics block + status word
constexpr int kMaxDevices = 64;

// [ base: kMaxBaseFloats floats | W2 fragments hi, lo | W2 planes hi, lo | anakin_stats | status word ]
static __device__ __align__(256) unsigned char g_noalloc_scratch[kMaxBaseFloats * sizeof(float) + kW2FragBytes + kW2PlaneBytes + kTailBytes];

unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};  // device address of the array, per device ordinal

// First call on a device: resolve the array's device address (with that device current).
cudaError_t scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int anakin_rollout_noalloc(const anakin_cfg* cfg, uint64_t seed, int64_t global_step, int T,
                                      const float* dev_params, const uint32_t* dev_walls, const uint8_t* dev_start,
                                      const uint8_t* dev_goal, uint8_t* dev_pos, uint8_t* dev_tep,
                                      uint8_t* dev_traj_pos, int8_t* dev_traj_action, uint8_t* dev_traj_done,
                                      float* dev_traj_reward, float* dev_traj_value, float* dev_traj_logp,
                                      void* cuda_stream) {
    size_t unused = 0;
    const int rc = anakin_workspace_bytes(cfg, &unused);  // validates cfg; computes sizes only
    if (rc != ANAKIN_OK) return rc;
    if (cfg->n_policies >= 2) return ANAKIN_E_UNSUPPORTED_CFG;  // one policy only
    if (!dev_params || !dev_walls || !dev_start || !dev_goal || !dev_pos || !dev_tep || !dev_traj_pos || !dev_traj_action ||
        !dev_traj_done || !dev_traj_reward || !dev_traj_value || !dev_traj_logp)
        return ANAKIN_E_INVALID_ARG;
    if (T < 1 || T > cfg->T_max || global_step < 0) return ANAKIN_E_INVALID_ARG;
    if (cfg->precision != ANAKIN_PRECISION_FP32) return ANAKIN_E_UNSUPPORTED_CFG;  // bf16 needs a second scratch copy
    if ((size_t)cfg->B * (size_t)cfg->H > kMaxBaseFloats) {
        fprintf(stderr, "anakin_rollout_noalloc: B*H = %zu exceeds the built-in scratch of %zu floats\n",
                (size_t)cfg->B * (size_t)cfg->H, kMaxBaseFloats);
        return ANAKIN_E_WORKSPACE_TOO_SMALL;
    }
    unsigned char* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) return ANAKIN_E_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;

    RolloutArgs a;
    memset(&a, 0, sizeof(a));
    a.d = make_dims(cfg->B, cfg->N, cfg->H, cfg->T_max);
    a.d.env0 = cfg->env_offset;
    Buffers& b = a.b;
    b.theta = b.theta_c = const_cast<float*>(dev_params);
    b.walls = const_cast<uint32_t*>(dev_walls);
    b.start = const_cast<uint8_t*>(dev_start);
    b.goal = const_cast<uint8_t*>(dev_goal);
    b.pos = dev_pos;
    b.tep = dev_tep;
    b.tpos = dev_traj_pos;
    b.tact = dev_traj_action;
    b.tdone = dev_traj_done;
    b.trew = dev_traj_reward;
    b.tval = dev_traj_value;
    b.tlogp = dev_traj_logp;
    b.base = reinterpret_cast<float*>(scratch);
    unsigned char* frag = scratch + kMaxBaseFloats * sizeof(float);
    if (rollout_mma_supported(cfg->H)) {  // same kernel choice as the handle-based rollout
        if (rollout_uses_fragments(cfg->H, cfg->precision)) {
            b.w2f_hi = reinterpret_cast<uint2*>(frag);
            b.w2f_lo = reinterpret_cast<uint2*>(frag + kW2FragBytes / 2);
        }
        b.w2p_hi = reinterpret_cast<uint16_t*>(frag + kW2FragBytes);
        b.w2p_lo = reinterpret_cast<uint16_t*>(frag + kW2FragBytes + kW2PlaneBytes / 2);
    }
    unsigned char* tail = frag + kW2FragBytes + kW2PlaneBytes;
    b.stats = reinterpret_cast<anakin_stats*>(tail);
    b.status = reinterpret_cast<int*>(tail + 128);
    // the tail holds accumulators and a sticky status word left by the previous call: start them at zero
    if (cudaMemsetAsync(tail, 0, kTailBytes, s) != cudaSuccess) return ANAKIN_E_CUDA;
    a.T = T;
    a.cap = cfg->episode_cap;
    a.gstep0 = (uint32_t)global_step;
    a.key0 = (uint32_t)(seed & 0xFFFFFFFFu);
    a.key1 = (uint32_t)(seed >> 32);
    a.env_kind = cfg->env_kind;
    a.forced = nullptr;
    a.replay = 0;
    a.fuse_gae = 0;  // the caller gets the trajectory only
    uint64_t launches = 0;
    const Ctx ctx{s, &launches, nullptr};
    if (launch_env_base(a.d, b, ctx) != cudaSuccess) return ANAKIN_E_CUDA;  // fills `base`: nothing of the last call survives
    if (launch_pack_w2(a.d, b, cfg->precision, ctx) != cudaSuccess) return ANAKIN_E_CUDA;   // likewise the weight fragments
    if (launch_rollout(a, cfg->precision, ctx) != cudaSuccess) return ANAKIN_E_CUDA;
    return ANAKIN_OK;
}

// The sticky status word of the last anakin_rollout_noalloc call on the current device lives in the array's tail, where
// no caller can see it; this call brings it out (a 4-byte stream-ordered copy, then a stream synchronisation).
extern "C" int anakin_noalloc_status(void* cuda_stream, int* device_status) {
    if (!device_status) return ANAKIN_E_INVALID_ARG;
    unsigned char* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) return ANAKIN_E_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const unsigned char* tail = scratch + kMaxBaseFloats * sizeof(float) + kW2FragBytes + kW2PlaneBytes;
    int st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, tail + 128, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return ANAKIN_E_CUDA;
    *device_status = st;
    return st == 0 ? ANAKIN_OK : ANAKIN_E_DEVICE_STATUS;
}
