// arl2_commit_static_scratch: the state commit for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a region being
// captured or replayed by someone else's framework, in a plugin whose host hands it finished
// buffers and forbids allocation, or in a process whose memory pool is owned by another
// component.  Such a caller has the tensors of the layer (state, K, V, logits) but no
// spare buffer for the partial sums the commit reduction needs, and arl2_create wants a workspace.
// Here the partial sums live in a fixed array that is part of the library image itself.
#include <cuda_runtime.h>

#include <mutex>

#include "arl2_internal.h"

namespace {

constexpr size_t kScratchBytes = ARL2_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Partial sums [B, H, ceil(L/512), D, D] fp32 of one commit.  Every GPU that loads the library
// carries this array until the process exits.  In host code this name is only a handle for the
// runtime, not a device address: the address a kernel may use comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_commit_scratch[kScratchBytes];

std::mutex g_mutex;
float* g_scratch_ptr[kMaxDevices] = {};   // per device, filled on that device's first call

// Device address of the array on the current device; looked up once per device.
int scratch_for_current_device(float** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        arl2::set_error("commit_static_scratch: cannot identify the current device (%s)",
                        cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_commit_scratch);   // needs `dev` current: it is
        if (e != cudaSuccess || p == nullptr) {
            arl2::set_error("commit_static_scratch: cudaGetSymbolAddress failed on device %d: %s", dev,
                            cudaGetErrorString(e));
            return ARL2_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_ptr[dev];
    return ARL2_OK;
}

}  // namespace

extern "C" int arl2_commit_static_scratch(const arl2_config* cfg, void* d_state, const void* d_k_clean,
                                          const void* d_v_clean, const float* d_decay_logits,
                                          const void* d_wphi_k, const void* d_wphi_v,
                                          const float* d_rope_cos, const float* d_rope_sin, void* stream)
{
    using namespace arl2;
    if (cfg == nullptr || cfg->struct_size != sizeof(arl2_config)) {
        set_error("commit_static_scratch: config is NULL or has the wrong struct_size");
        return ARL2_ERR_INVALID_ARG;
    }
    if (cfg->B < 1 || cfg->H < 1 || cfg->L < 1 || (cfg->D != 64 && cfg->D != 128) ||
        (cfg->io_dtype != ARL2_BF16 && cfg->io_dtype != ARL2_FP32) || cfg->commit_rule != 0 ||
        !(cfg->l2_eps >= 0.0f)) {
        set_error("commit_static_scratch: unsupported configuration (B=%d H=%d L=%d D=%d dtype=%d rule=%d)",
                  cfg->B, cfg->H, cfg->L, cfg->D, cfg->io_dtype, cfg->commit_rule);
        return ARL2_ERR_INVALID_ARG;
    }
    if (!d_state || !d_k_clean || !d_v_clean || !d_decay_logits) {
        set_error("commit_static_scratch: state, k_clean, v_clean and decay_logits must not be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    if ((d_rope_cos == nullptr) != (d_rope_sin == nullptr)) {
        set_error("commit_static_scratch: rope_cos and rope_sin must both be given or both be NULL");
        return ARL2_ERR_INVALID_ARG;
    }
    // the kernels read and write these with 16-byte (state, K, V), 8-byte (tables) and element-wide
    // (maps) accesses: a misaligned slice must be refused here, before anything is launched
    const size_t esz = cfg->io_dtype == ARL2_FP32 ? 4 : 2;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(d_state, 16) || misaligned(d_k_clean, 16) || misaligned(d_v_clean, 16) ||
        misaligned(d_rope_cos, 16) || misaligned(d_rope_sin, 16) || misaligned(d_decay_logits, 4) ||
        misaligned(d_wphi_k, esz) || misaligned(d_wphi_v, esz)) {
        set_error("commit_static_scratch: state, k_clean, v_clean and the rope tables must be 16-byte "
                  "aligned, decay_logits 4-byte and the feature maps element aligned");
        return ARL2_ERR_INVALID_ARG;
    }
    const int nsplit = (cfg->L + kCommitChunk - 1) / kCommitChunk;
    const unsigned long long need =
        (unsigned long long)cfg->B * cfg->H * nsplit * cfg->D * cfg->D * sizeof(float);
    if (need > kScratchBytes) {
        set_error("commit_static_scratch: this shape needs %llu bytes of partial sums "
                  "(B*H*ceil(L/512)*D*D*4); the built-in scratch holds %zu.  Use arl2_create / "
                  "arl2_commit with a caller-provided workspace instead.", need, kScratchBytes);
        return ARL2_ERR_WORKSPACE;
    }
    float* scratch = nullptr;
    if (int r = scratch_for_current_device(&scratch)) return r;

    CommitArgs a;
    a.s.B = cfg->B; a.s.H = cfg->H; a.s.L = cfg->L; a.s.D = cfg->D;
    a.s.scale_log2 = 0.0f;   // the commit has no softmax
    a.s.eps = cfg->l2_eps > 0.0f ? cfg->l2_eps : 1e-6f;
    a.k = d_k_clean; a.v = d_v_clean; a.decay = d_decay_logits;
    a.wk = d_wphi_k; a.wv = d_wphi_v;
    a.rope_cos = d_rope_cos; a.rope_sin = d_rope_sin;
    a.state = static_cast<float*>(d_state);
    a.partials = scratch;        // every slot the reduce reads is written by the partial kernel
    a.state_bf16 = nullptr;
    a.nsplit = nsplit;
    a.rope_h = nullptr;
    a.status = nullptr;          // the plain-FMA kernels have no waits and report nothing
    int n = simt_commit(a, cfg->io_dtype, static_cast<cudaStream_t>(stream));
    return n < 0 ? n : ARL2_OK;
}
