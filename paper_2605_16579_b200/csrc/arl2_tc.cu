// Tensor-core (tcgen05 / TMEM / TMA) kernels of the ARL^2 layer for bf16 I/O, D = 128.
//
// Step kernel: one CTA per (stream b, head h, pair of 128-row query tiles).   (Eq. 2, 3, 5-8)
//   warps 0-3 / 4-7  softmax group of query tile 0 / 1 (one thread per query row)
//   warp 8           TMA producer: Q tiles, then K_j, V_j tiles through a 3-slot ring, then the
//                    head's feature map W_phi_q^T and the bf16 copy of the state S as the
//                    last two "tiles" of the ring
//   warp 9           MMA issuer (one thread): S_t = Q~_t K_j^T and O_t += P_t V_j into TMEM
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1, 128 fp32 columns each; the bf16 probabilities P_t
// overwrite the first 64 columns of S_t and feed the second MMA straight from TMEM.
// The inter branch reuses the loop as one more iteration: "S" = Q W_phi_q (A = raw Q tile),
// the group turns each row into sigmoid(g) * l * L2Norm(RoPE(.)) (l = softmax row sum) and
// the "PV" MMA multiplies it by the state, accumulating into O_t, so the final O_t / l is
// O_intra + sigmoid(g) O_inter.  The state is only read.
//
// Every wait is bounded: when a limit expires the thread records ARL2_ERR_TIMEOUT in the
// device status block, raises the CTA's abort flag and every role falls through to the exit.
#include <cuda.h>

#include "arl2_internal.h"
#include "tc_ptx.cuh"

namespace arl2 {

namespace {

using namespace ptx;

constexpr int kTile = 128;               // query rows per tile = keys per tile = head dim
constexpr int kTileBytes = kTile * kTile * 2;
constexpr int kHalfBytes = kTileBytes / 2;  // one 64-column TMA box of a tile
constexpr int kStages = 3;
constexpr int kThreads = 320;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr float kRescaleThreshold = 8.0f;   // log2 units of slack before O is rescaled

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQRaw = 0;                              // 2 tiles, as loaded
constexpr int kOffQRot = kOffQRaw + 2 * kTileBytes;      // 2 tiles, after RoPE
constexpr int kOffRing = kOffQRot + 2 * kTileBytes;      // kStages tiles
constexpr int kOffBars = kOffRing + kStages * kTileBytes;
constexpr int kSmemBytes = kOffBars + 256 + 1024;        // barriers + alignment slack

enum Bar : int {
    kBarQFull = 0,
    kBarQRot0, kBarQRot1,
    kBarFull0,                                  // kStages of them
    kBarEmpty0 = kBarFull0 + kStages,           // kStages of them
    kBarSFull0 = kBarEmpty0 + kStages, kBarSFull1,
    kBarPFull0, kBarPFull1,
    kBarOFinal,
    kNumBars
};
static_assert(kNumBars * 8 + 16 <= 256, "barrier block");

struct TcStepParams {
    Shape s;
    const float* gate;
    const float* rope_cos;
    const float* rope_sin;
    __nv_bfloat16* out;
    uint32_t* status;
    int n_kv;      // key tiles per head
};

struct Abort {
    volatile int* flag;   // in shared memory
    uint32_t* status;     // device status block
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Abort& ab, int site)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *ab.flag) return false;
    }
    *ab.flag = 1;
    if (atomicCAS(ab.status + kStatusError, 0u, (uint32_t)(-ARL2_ERR_TIMEOUT)) == 0u)
        ab.status[kStatusWhere] = (uint32_t)site;
    return false;
}

// Bounded wait that ignores the abort flag: used on the way out, for copies still in flight.
__device__ __forceinline__ void drain_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it)
        if (mbar_try_wait(bar, parity)) return;
}

__device__ __forceinline__ float sigmoid_fast(float x) { return 1.0f / (1.0f + __expf(-x)); }

// One softmax group thread: owns query row `r` of tile `t`.
__device__ __forceinline__ void softmax_role(const TcStepParams& p, uint8_t* smem, uint32_t bars,
                                             uint32_t tmem_base, const Abort& ab, int t, int r,
                                             int warp_in_group, int b, int h, int q_row0,
                                             bool tile_active)
{
    const int L = p.s.L, H = p.s.H;
    const int row = q_row0 + r;
    const bool valid_row = row < L;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp_in_group * 32) << 16);
    const uint32_t s_addr = lane_base + (uint32_t)(t * kTile);
    const uint32_t o_addr = lane_base + (uint32_t)(2 * kTile + t * kTile);
    const uint32_t bar_s = bars + 8 * (kBarSFull0 + t);
    const uint32_t bar_p = bars + 8 * (kBarPFull0 + t);

    // ---- Q~ = RoPE(Q): rotate this thread's row from the raw tile into the MMA operand tile
    if (!wait_bar(bars + 8 * kBarQFull, 0, ab, 10)) return;
    if (!tile_active) return;
    if (p.rope_cos != nullptr) {
        const uint8_t* src = smem + kOffQRaw + t * kTileBytes;
        uint8_t* dst = smem + kOffQRot + t * kTileBytes;
        const float* cs = p.rope_cos + (size_t)(valid_row ? row : 0) * (kTile / 2);
        const float* sn = p.rope_sin + (size_t)(valid_row ? row : 0) * (kTile / 2);
#pragma unroll 4
        for (int c = 0; c < 16; ++c) {
            int off = (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
            uint4 raw = *reinterpret_cast<const uint4*>(src + off);
            float4 cv = *reinterpret_cast<const float4*>(cs + c * 4);
            float4 sv = *reinterpret_cast<const float4*>(sn + c * 4);
            uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            float cc[4] = {cv.x, cv.y, cv.z, cv.w}, ss[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                float x0 = __uint_as_float(w[m] << 16);
                float x1 = __uint_as_float(w[m] & 0xFFFF0000u);
                w[m] = pack_bf16(x0 * cc[m] - x1 * ss[m], x0 * ss[m] + x1 * cc[m]);
            }
            *reinterpret_cast<uint4*>(dst + off) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        fence_proxy_async_smem();
    }
    mbar_arrive(bars + 8 * (kBarQRot0 + t));

    float m_ref = -INFINITY;   // reference maximum (scaled, base 2) the probabilities use
    float l_sum = 0.0f;        // running row sum relative to m_ref
    const float c2 = p.s.scale_log2;
    const int n_kv = p.n_kv;
    uint32_t sreg[128];

    for (int j = 0; j < n_kv; ++j) {
        if (!wait_bar(bar_s, (uint32_t)(j & 1), ab, 20 + t)) return;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c)
            tmem_ld32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
        tmem_wait_ld();

        const int n_valid = L - j * kTile;  // keys of this tile that exist
        if (n_valid < kTile) {   // ragged last tile: zero-filled key rows must not count
#pragma unroll
            for (int c = 0; c < 128; ++c)
                if (c >= n_valid) sreg[c] = __float_as_uint(-INFINITY);
        }
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sreg[c]));
        float m_new = fmaxf(m_ref, mx * c2);
        bool need = (m_new - m_ref) > kRescaleThreshold;   // first tile: inf > threshold
        if (__any_sync(0xffffffffu, need)) {
            float alpha = 1.0f;
            if (need) {
                alpha = ex2_approx(m_ref - m_new);
                m_ref = m_new;
                l_sum *= alpha;
            }
            if (j > 0) {
                // the MMA that last accumulated into O_t finished before S_t(j) was signalled,
                // and the next one waits for this group's arrival below: O_t is ours for now
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(o_addr + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    tmem_st32(o_addr + c * 32, o);
                }
            }
        }
        const float neg_m = -m_ref;
#pragma unroll
        for (int c = 0; c < 64; ++c) {
            float p0 = ex2_approx(fmaf(__uint_as_float(sreg[2 * c]), c2, neg_m));
            float p1 = ex2_approx(fmaf(__uint_as_float(sreg[2 * c + 1]), c2, neg_m));
            l_sum += p0 + p1;
            sreg[c] = pack_bf16(p0, p1);
        }
        tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
        tmem_st32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p);
    }

    // ---- inter branch: U = Q W_phi_q arrives in the S columns                       (Eq. 3)
    if (!wait_bar(bar_s, (uint32_t)(n_kv & 1), ab, 30 + t)) return;
    tc_fence_after();
#pragma unroll
    for (int c = 0; c < 4; ++c)
        tmem_ld32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
    tmem_wait_ld();
    {
        float ss = 0.0f;
        if (p.rope_cos != nullptr && valid_row) {
            const float* cs = p.rope_cos + (size_t)row * (kTile / 2);
            const float* sn = p.rope_sin + (size_t)row * (kTile / 2);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                float4 cv = *reinterpret_cast<const float4*>(cs + c * 4);
                float4 sv = *reinterpret_cast<const float4*>(sn + c * 4);
                float cc[4] = {cv.x, cv.y, cv.z, cv.w}, s4[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    float x0 = __uint_as_float(sreg[c * 8 + 2 * m]);
                    float x1 = __uint_as_float(sreg[c * 8 + 2 * m + 1]);
                    sreg[c * 8 + 2 * m] = __float_as_uint(x0 * cc[m] - x1 * s4[m]);
                    sreg[c * 8 + 2 * m + 1] = __float_as_uint(x0 * s4[m] + x1 * cc[m]);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < 128; ++c) ss = fmaf(__uint_as_float(sreg[c]), __uint_as_float(sreg[c]), ss);
        float gate = valid_row ? sigmoid_fast(p.gate[((size_t)b * L + row) * H + h]) : 0.0f;
        // scaled by the row sum so that the common 1/l of the epilogue leaves gate * Q' S
        float f = rsqrtf(ss + p.s.eps) * gate * l_sum;
#pragma unroll
        for (int c = 0; c < 64; ++c)
            sreg[c] = pack_bf16(__uint_as_float(sreg[2 * c]) * f, __uint_as_float(sreg[2 * c + 1]) * f);
    }
    tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
    tmem_st32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(bar_p);

    // ---- epilogue: O_t / l -> bf16 -> global                                   (Eq. 6-7)
    if (!wait_bar(bars + 8 * kBarOFinal, 0, ab, 40 + t)) return;
    tc_fence_after();
    const float inv_l = 1.0f / l_sum;
    __nv_bfloat16* orow = p.out + (((size_t)b * L + (valid_row ? row : 0)) * H + h) * kTile;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(o_addr + c * 32, o);
        tmem_wait_ld();
        if (valid_row) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(o[e * 8 + 0]) * inv_l, __uint_as_float(o[e * 8 + 1]) * inv_l);
                v.y = pack_bf16(__uint_as_float(o[e * 8 + 2]) * inv_l, __uint_as_float(o[e * 8 + 3]) * inv_l);
                v.z = pack_bf16(__uint_as_float(o[e * 8 + 4]) * inv_l, __uint_as_float(o[e * 8 + 5]) * inv_l);
                v.w = pack_bf16(__uint_as_float(o[e * 8 + 6]) * inv_l, __uint_as_float(o[e * 8 + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + c * 32 + e * 8) = v;
            }
        }
    }
    tc_fence_before();
}

__global__ void __launch_bounds__(kThreads, 1)
tc_step_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_w,
               const __grid_constant__ CUtensorMap tm_s, const TcStepParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kOffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBars + kNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBars + kNumBars * 8 + 4);
    const Abort ab{abort_flag, p.status};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int L = p.s.L, H = p.s.H;
    const int q_row0 = pair * 2 * kTile;
    const bool two = q_row0 + kTile < L;   // the pair's second tile exists
    const int n_kv = p.n_kv;
    const int n_it = n_kv + 1;             // key tiles + the inter-branch iteration

    if (threadIdx.x == 0) {
        mbar_init(bars + 8 * kBarQFull, 1);
        mbar_init(bars + 8 * kBarQRot0, 128);
        mbar_init(bars + 8 * kBarQRot1, 128);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bars + 8 * (kBarFull0 + s), 1);
            mbar_init(bars + 8 * (kBarEmpty0 + s), 1);
        }
        mbar_init(bars + 8 * kBarSFull0, 1);
        mbar_init(bars + 8 * kBarSFull1, 1);
        mbar_init(bars + 8 * kBarPFull0, 128);
        mbar_init(bars + 8 * kBarPFull1, 128);
        mbar_init(bars + 8 * kBarOFinal, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 8) {
        const int t = warp >> 2;
        softmax_role(p, smem, bars, tmem_base, ab, t, (warp & 3) * 32 + lane, warp & 3, b, h,
                     q_row0 + t * kTile, t == 0 || two);
    } else if (warp == 8) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_v);
            const uint32_t bar_q = bars + 8 * kBarQFull;
            mbar_expect_tx(bar_q, two ? 2 * kTileBytes : kTileBytes);
            for (int t = 0; t < (two ? 2 : 1); ++t) {
                uint32_t dst = smem_base + kOffQRaw + t * kTileBytes;
                tma_load_4d(dst, &tm_q, bar_q, 0, h, q_row0 + t * kTile, b);
                tma_load_4d(dst + kHalfBytes, &tm_q, bar_q, 64, h, q_row0 + t * kTile, b);
            }
            const int n_loads = 2 * n_kv + 2;
            int n = 0;
            bool ok = true;
            for (; n < n_loads && ok; ++n) {
                const int slot = n % kStages;
                if (n >= kStages)
                    ok = wait_bar(bars + 8 * (kBarEmpty0 + slot), (uint32_t)(((n / kStages) - 1) & 1), ab, 50);
                if (!ok) break;
                const uint32_t bar = bars + 8 * (kBarFull0 + slot);
                const uint32_t dst = smem_base + kOffRing + slot * kTileBytes;
                mbar_expect_tx(bar, kTileBytes);
                if (n < 2 * n_kv) {
                    const CUtensorMap* tm = (n & 1) ? &tm_v : &tm_k;
                    const int row0 = (n >> 1) * kTile;
                    tma_load_4d(dst, tm, bar, 0, h, row0, b);
                    tma_load_4d(dst + kHalfBytes, tm, bar, 64, h, row0, b);
                } else if (n == 2 * n_kv) {
                    tma_load_2d(dst, &tm_w, bar, 0, h * kTile);
                    tma_load_2d(dst + kHalfBytes, &tm_w, bar, 64, h * kTile);
                } else {
                    tma_load_2d(dst, &tm_s, bar, 0, (b * H + h) * kTile);
                    tma_load_2d(dst + kHalfBytes, &tm_s, bar, 64, (b * H + h) * kTile);
                }
            }
            if (!ok || *abort_flag) {
                // do not leave the CTA while bulk copies into its shared memory are in flight
                drain_bar(bar_q, 0);
                for (int m = (n > kStages ? n - kStages : 0); m < n; ++m)
                    drain_bar(bars + 8 * (kBarFull0 + m % kStages), (uint32_t)((m / kStages) & 1));
            }
        }
    } else {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(kTile, kTile, 0, 0);  // A, B K-major
            constexpr uint32_t idesc_pv = idesc_bf16(kTile, kTile, 0, 1);  // A in TMEM, B N-contiguous
            const bool rotated = p.rope_cos != nullptr;
            const uint32_t q_op = smem_base + (rotated ? kOffQRot : kOffQRaw);
            const uint32_t q_raw = smem_base + kOffQRaw;
            const uint32_t s_col[2] = {tmem_base, tmem_base + kTile};
            const uint32_t o_col[2] = {tmem_base + 2 * kTile, tmem_base + 3 * kTile};
            const int ntile = two ? 2 : 1;

            // S_t (or U_t) = A_t * B^T with both operands K-major, 8 k-steps of 16
            auto issue_qk = [&](int t, uint32_t a_tile, uint32_t b_tile) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_ss(s_col[t], smem_desc_sw128(a_tile + koff, 16), smem_desc_sw128(b_tile + koff, 16),
                           idesc_qk, ks > 0);
                }
            };
            // O_t (+)= P_t * V with P in TMEM and V rows = contraction index, 8 k-steps of 16
            auto issue_pv = [&](int t, uint32_t v_tile, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(o_col[t], s_col[t] + ks * 8, smem_desc_sw128(v_tile + ks * 2048, kHalfBytes),
                           idesc_pv, (accumulate || ks > 0) ? 1u : 0u);
            };

            bool ok = wait_bar(bars + 8 * kBarQFull, 0, ab, 60);
            for (int t = 0; t < ntile && ok; ++t) ok = wait_bar(bars + 8 * (kBarQRot0 + t), 0, ab, 61);
            tc_fence_after();
            int cons = 0;   // ring entries consumed so far
            if (ok) ok = wait_bar(bars + 8 * (kBarFull0 + 0), 0, ab, 62);
            if (ok) {
                tc_fence_after();
                const uint32_t k_tile = smem_base + kOffRing;
                for (int t = 0; t < ntile; ++t) {
                    issue_qk(t, (n_kv > 0 ? q_op : q_raw) + t * kTileBytes, k_tile);
                    mma_commit(bars + 8 * (kBarSFull0 + t));
                }
                mma_commit(bars + 8 * (kBarEmpty0 + 0));
                cons = 1;
            }
            for (int j = 0; j < n_it && ok; ++j) {
                const int vslot = cons % kStages;
                const uint32_t v_tile = smem_base + kOffRing + vslot * kTileBytes;
                ok = wait_bar(bars + 8 * (kBarFull0 + vslot), (uint32_t)((cons / kStages) & 1), ab, 63);
                if (!ok) break;
                const bool has_next = j + 1 < n_it;
                const int kslot = (cons + 1) % kStages;
                const uint32_t k_tile = smem_base + kOffRing + kslot * kTileBytes;
                const uint32_t a_next = (j + 1 == n_kv) ? q_raw : q_op;   // the last "S" is Q W
                for (int t = 0; t < ntile && ok; ++t) {
                    ok = wait_bar(bars + 8 * (kBarPFull0 + t), (uint32_t)(j & 1), ab, 64 + t);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(t, v_tile, j > 0);
                    if (has_next) {
                        if (t == 0) {
                            ok = wait_bar(bars + 8 * (kBarFull0 + kslot),
                                          (uint32_t)(((cons + 1) / kStages) & 1), ab, 66);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        issue_qk(t, a_next + t * kTileBytes, k_tile);
                        mma_commit(bars + 8 * (kBarSFull0 + t));
                    }
                }
                if (!ok) break;
                mma_commit(bars + 8 * (kBarEmpty0 + vslot));
                if (has_next) mma_commit(bars + 8 * (kBarEmpty0 + kslot));
                cons += has_next ? 2 : 1;
            }
            if (ok) mma_commit(bars + 8 * kBarOFinal);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// out[h][o][i] = w[h][i][o] (bf16), or the identity when w is null: the K-major B operand of
// U = Q W_phi (B[n][k] = W[k][n]).
__global__ void transpose_map_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ out,
                                     int D, size_t total)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    int i = (int)(t % D);
    int o = (int)((t / D) % D);
    size_t hh = t / ((size_t)D * D);
    __nv_bfloat16 v;
    if (w != nullptr) v = w[(hh * D + i) * D + o];
    else v = __float2bfloat16_rn(i == o ? 1.0f : 0.0f);
    out[t] = v;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [B, L, H, 128] bf16 viewed as a 4-D tensor (d, h, l, b); box = 64 columns x 128 rows of one head.
int make_map_blhd(CUtensorMap* m, const void* base, const Shape& s)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return ARL2_ERR_CUDA; }
    cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)s.H, (cuuint64_t)s.L, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)s.D * 2, (cuuint64_t)s.H * s.D * 2, (cuuint64_t)s.L * s.H * s.D * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled([B,L,H,D]) failed with %d", (int)r); return ARL2_ERR_CUDA; }
    return 0;
}

// [rows, 128] bf16 row-major; box = 64 columns x 128 rows.
int make_map_rows(CUtensorMap* m, const void* base, size_t rows)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return ARL2_ERR_CUDA; }
    cuuint64_t dims[2] = {(cuuint64_t)kTile, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kTile * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled([rows,128]) failed with %d", (int)r); return ARL2_ERR_CUDA; }
    return 0;
}

}  // namespace

bool tc_supported(const arl2_config& c)
{
    return c.io_dtype == ARL2_BF16 && c.D == kTile && !(c.flags & ARL2_FLAG_FORCE_SIMT);
}

int tc_prepare_map(const void* w, __nv_bfloat16* w_op, int H, cudaStream_t st)
{
    size_t total = (size_t)H * kTile * kTile;
    transpose_map_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(w), w_op, kTile, total);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of transpose_map_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

int tc_step(const StepArgs& a, const __nv_bfloat16* wq_op, const __nv_bfloat16* state_bf16, cudaStream_t st)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute(tc_step_kernel, %d): %s", kSmemBytes, cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
        attr_set = true;
    }
    CUtensorMap tm_q, tm_k, tm_v, tm_w, tm_s;
    if (int r = make_map_blhd(&tm_q, a.q, a.s)) return r;
    if (int r = make_map_blhd(&tm_k, a.k_rot, a.s)) return r;
    if (int r = make_map_blhd(&tm_v, a.v, a.s)) return r;
    if (int r = make_map_rows(&tm_w, wq_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_s, state_bf16, (size_t)a.s.B * a.s.H * kTile)) return r;
    TcStepParams p;
    p.s = a.s;
    p.gate = a.gate;
    p.rope_cos = a.rope_cos;
    p.rope_sin = a.rope_sin;
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.status = a.status;
    p.n_kv = (a.s.L + kTile - 1) / kTile;
    const int n_qtiles = p.n_kv;
    dim3 grid((n_qtiles + 1) / 2, a.s.H, a.s.B);
    tc_step_kernel<<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_w, tm_s, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_step_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

}  // namespace arl2
