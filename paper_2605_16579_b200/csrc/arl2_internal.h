// Internal declarations shared by the host API and the kernel translation units.
// Nothing here is part of the public ABI (see include/arl2.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "arl2.h"

namespace arl2 {

// Words of the device status block at the start of the workspace.
enum StatusWord : int {
    kStatusError = 0,    // first error code a kernel recorded (0 = none)
    kStatusWhere = 1,    // which wait gave up (kernel-specific tag)
    kStatusSched = 2,    // two item counters of the persistent step kernel (words 2 and 3)
    kStatusWords = 64
};

constexpr int kCommitChunk = 512;  // tokens per partial sum of the commit reduction
// Key-range split of the step kernel's last wave: at most kMaxSplit parts per item, and room for
// the partial rows of 2 x 148 parts of two query tiles each (more SMs: the launcher splits less)
constexpr int kMaxSplit = 4;
constexpr int kSplitTileParts = 4 * 148;

struct Shape {
    int B, H, L, D;
    float scale_log2;  // softmax scale * log2(e): scores are exponentiated in base 2
    float eps;
};

// Everything a step launch needs; plain pointers only.
struct StepArgs {
    Shape s;
    const void* q;
    const void* k_rot;      // K after RoPE (or the caller's K when there is no rotation)
    const void* v;
    const float* gate;      // [B, L, H]
    const float* state;     // [B, H, D, D] fp32, read only
    const void* wq;         // [H, D, D] (in, out) io dtype, or nullptr
    const float* rope_cos;  // [L, D/2] or nullptr
    const float* rope_sin;
    void* out;
    uint32_t* status;
    int launch_parity;      // step launches so far on this context, mod 2 (scheduler counters)
    const void* rope_h;     // [L, D/2] half2 (cos, sin) copy of the tables (tensor-core path), or nullptr
    int Lk = 0;             // > 0: K and V hold Lk tokens (a cache), [B, Lk, H, D]; 0: L
    int gate_mode = 0;      // 0: gate [B, L, H]; 1: [B, L]; 2: [B, L, H, D]
    uint32_t wait_limit = 0;  // 0: default; n > 0: bounded waits give up after n - 1 polls (test hook)
    // key-range split of the last wave of work items (tensor-core path), or nullptr: never split
    float* split_o = nullptr;            // [split_tile_parts][128][128] fp32
    float* split_ml = nullptr;           // [split_tile_parts][128][2] fp32
    int split_tile_parts = 0;
};

struct CommitArgs {
    Shape s;
    const void* k;
    const void* v;
    const float* decay;     // [B, H]
    const void* wk;
    const void* wv;
    const float* rope_cos;
    const float* rope_sin;
    float* state;           // [B, H, D, D] fp32, read-modify-write by the reduce kernel
    float* partials;        // [B, H, nsplit, D, D] fp32
    __nv_bfloat16* state_bf16;  // operand copy refreshed by the reduce kernel, or nullptr
    int nsplit;
    const void* rope_h;     // half2 (cos, sin) copy of the tables (tensor-core path), or nullptr
    uint32_t* status;
    // 0: value rows V'; 1: Eq. 4 as printed, diag(sigmoid(beta)) (V' - K' S_old); 2: diag(beta) V'
    // with beta given directly (per-token decay weights)
    int mode = 0;
    const float* beta = nullptr;   // [B, L, H]: logits (mode 1) or weights (mode 2); nullptr = 1
    bool decay_direct = false;     // `decay` holds the factors themselves, not logits
    // How the partial sums of a head are laid out for the reduce kernel: nsplit slots of fixed
    // 512-token chunks (run_share == 0), or the tensor-core kernel's runs of run_share tiles over
    // the flattened tile sequence (a head's slots are the CTAs its run_ntile tiles fall into)
    int run_share = 0;
    int run_ntile = 0;
    int nslot = 0;                 // slots per head in `partials` (0: nsplit)
    uint32_t wait_limit = 0;       // as in StepArgs
    // tensor-core path only
    float* partials_g = nullptr;              // second accumulator of the delta rule, shaped like `partials`
    __nv_bfloat16* state_bf16_next = nullptr; // the mirror buffer the finishing kernel writes
    void* k_rot_out = nullptr;                // when set (and there is a rotation): RoPE(k) is written here too
};

// Eq. 4 token by token with per-token gates (chunkwise form): the two launches share these.
struct TokenCommitArgs {
    Shape s;
    const void* k;
    const void* v;
    const float* alpha;     // [B, L, H] forget-gate logits, or nullptr = 1
    const float* beta;      // [B, L, H] learning-rate logits, or nullptr = 1
    const void* wk;
    const void* wv;
    const float* rope_cos;
    const float* rope_sin;
    float* state;           // [B, H, D, D] fp32, updated in place
    __nv_bfloat16* state_bf16;  // operand copy to refresh, or nullptr
    float* w;               // [B, H, nchunk * 64, D] fp32 scratch
    float* u1;              // same shape
    float* kh;              // same shape
    float* gc;              // [B, H, nchunk] decay of a whole chunk
    int nchunk;             // ceil(L / 64)
    bool decayed = false;   // each token predicts against alpha_j S_{j-1} instead of S_{j-1}
    uint32_t wait_limit = 0;   // as in StepArgs
};
constexpr int kTokenChunk = 64;

// ---- plain-FMA kernels (arl2_simt.cu) -------------------------------------------------
// Each returns the number of kernels it launched (>= 0) or a negative arl2_status.
int simt_rope_k(const Shape& s, int dtype, const void* k, const float* cos_t, const float* sin_t,
                void* k_rot, cudaStream_t st);
int simt_step(const StepArgs& a, int dtype, cudaStream_t st);
int simt_commit(const CommitArgs& a, int dtype, cudaStream_t st);
int commit_reduce(const CommitArgs& a, cudaStream_t st);  // fixed-order sum + gated decay
// w[b,l,h] = prod_{i>l} sigmoid(alpha[b,i,h]), total[b,h] = prod_l sigmoid(alpha[b,l,h])
int decay_weights(const Shape& s, const float* alpha_logits, float* w, float* total, cudaStream_t st);
int simt_commit_tokens(const TokenCommitArgs& a, int dtype, cudaStream_t st);
int fill_zero(void* p, size_t bytes, cudaStream_t st);
int state_to_bf16(const float* state, __nv_bfloat16* dst, size_t n, cudaStream_t st);

// ---- tensor-core kernels (arl2_tc.cu) ---------------------------------------------------
bool tc_supported(const arl2_config& c);
// w: [H, 128, 128] (in, out) bf16 or nullptr (identity) -> w_op: [H, out, in] bf16
int tc_prepare_map(const void* w, __nv_bfloat16* w_op, int H, cudaStream_t st);
// cos, sin [L, 64] fp32 -> out [L, 64] half2 (cos, sin): one 256-byte row per token
int tc_prepare_rope(const float* cos_t, const float* sin_t, void* out, int L, cudaStream_t st);
// k_rot = RoPE(k), bf16 [B, L, H, 128], from the packed table tc_prepare_rope wrote
int tc_rope_k(const Shape& s, const void* k, const void* rope_h, void* k_rot, cudaStream_t st);
int tc_step(const StepArgs& a, const __nv_bfloat16* wq_op, const __nv_bfloat16* state_bf16,
            cudaStream_t st);
// partial sums on tensor cores (fills a.run_share / a.run_ntile for the finishing kernel) ...
int tc_commit_partials(CommitArgs& a, const __nv_bfloat16* wk_op, cudaStream_t st);
// ... then S <- alpha S + (sum of slots) W_phi_v [- (sum of G slots) S_old], mirror written to state_bf16_next
int tc_commit_finish(const CommitArgs& a, cudaStream_t st);

// out += sigmoid(g) Q' S^(i): token-level state access (a.k_rot holds the RAW K here; a.out already holds the
// softmax branch); alpha_logits [B, L, H] or nullptr
int tc_token_readout(const StepArgs& a, const float* alpha_logits, const __nv_bfloat16* wq_op,
                     const __nv_bfloat16* wk_op, const __nv_bfloat16* wv_op, cudaStream_t st);

int tc_commit_tokens(const TokenCommitArgs& a, const __nv_bfloat16* wk_op, const __nv_bfloat16* wv_op,
                     const void* rope_h, uint32_t* status, cudaStream_t st);   // prepare + ordered scan

// C[M, N] = A[M, K] B[K, N] on tensor cores (bf16 operands, row-major); the columns of C are routed to up to
// four bf16 tensors of seg_cols columns each (row stride ld_out) and, after them, one fp32 tensor.
struct GemmArgs {
    const void* a;        // [M, K] bf16
    const void* b;        // [K, N] bf16
    int M, N, K;
    void* out[4] = {nullptr, nullptr, nullptr, nullptr};
    int seg_cols = 0, ld_out = 0, n_bf16_seg = 0;
    float* out_f32 = nullptr;
    int f32_cols = 0, ld_f32 = 0;
    uint32_t* status = nullptr;
    uint32_t wait_limit = 0;
};
int tc_gemm(const GemmArgs& a, cudaStream_t st);

void set_error(const char* fmt, ...);

}  // namespace arl2
