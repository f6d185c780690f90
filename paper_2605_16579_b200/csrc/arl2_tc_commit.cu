// State commit on tensor cores (bf16 I/O, D = 128): Eq. 3 and Eq. 4 (gated-linear form, the
// block-level delta rule, per-token decay weights), once per block from the clean pass's K and V.
//
// The value map is taken out of the token loop: sum_l K'_l^T (V_l W_phi_v) = (sum_l K'_l^T V_l) W_phi_v,
// so a V tile goes from TMA straight into the state MMA and the D x D map is applied once per
// head when the partial sums are added up.  The delta rule splits the same way,
//   sum_l beta_l K'_l^T (V'_l - K'_l S_old) = (sum_l beta_l K'_l^T V_l) W_phi_v - (sum_l beta_l K'_l^T K'_l) S_old,
// into two accumulators that share the A operand diag(beta) K'.
//
// tc_commit_kernel: the 128-token tiles of all (stream, head) units form one flattened sequence
// cut into equal runs, one CTA (one per SM) per run; a run may cross from one head into the next.
//   warp 0      TMA producer: W_phi_k^T of the head, then (K tile, V tile) pairs through a ring
//   warp 1      MMA issuer:   U = K_c W_phi_k into one of two TMEM buffers
//   warp 10     MMA issuer:   dS += K'^T V_c (and G += (beta K')^T K' for the delta rule) into TMEM
//                             accumulators
//   warps 2-9   token threads, two per token (64 of the 128 columns each):
//                             K' = L2Norm(RoPE(U)) -> bf16, written over the raw K tile in the
//                             swizzled operand layout; optionally RoPE(K_c) to global memory for
//                             the softmax branch of a fused clean pass
// When a head's tiles end inside a run (or the run ends) the token threads store the accumulators
// to that (head, CTA) slot of the partial-sum buffer: the assignment of tiles to CTAs and slots is
// static, so the fixed-order sum of the finishing kernel is bitwise reproducible.
//
// tc_commit_finish_kernel: S <- alpha S + (sum of slots) W_phi_v [- (sum of G slots) S_old], fp32
// FMA arithmetic, 16 state rows per CTA; also writes the bf16 operand copy of the new state into
// the OTHER of two mirror buffers (the delta rule reads S_old from the current one while rows
// are being replaced, so the mirrors alternate from commit to commit).
//
// Every wait is bounded (see wait_bar); a CTA that gives up records ARL2_ERR_TIMEOUT, drains its
// copies and MMAs in flight and frees its tensor memory; the finishing kernel then leaves S alone.
#include "tc_common.cuh"

namespace arl2 {

namespace {

constexpr int kCThreads = 352;        // producer, U issuer, 8 token warps, accumulator issuer
constexpr int kCTokenThreads = 256;
constexpr int kCMaxStages = 3;
// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kCOffWk = 0;                                  // W_phi_k^T of the current head
constexpr int kCOffStage = kTileBytes;                      // stages of (K tile, V tile)
constexpr int kCOffBars = kCOffStage + 2 * kCMaxStages * kTileBytes;
constexpr int kCommitSmemBytes = kCOffBars + 256 + 1024;    // barriers + alignment slack
// The delta rule keeps two stages and uses the third stage's two tiles for diag(beta) K'.

enum CBar : int {
    kCBarWFull = 0, kCBarWFree,
    kCBarStageFull0,                                        // kCMaxStages of each
    kCBarStageFree0 = kCBarStageFull0 + kCMaxStages,
    kCBarKpFull0 = kCBarStageFree0 + kCMaxStages,           // token threads -> MMA: K' of the stage written
    kCBarUFull0 = kCBarKpFull0 + kCMaxStages, kCBarUFull1,  // MMA -> token threads: U in buffer 0 / 1
    kCBarUFree0, kCBarUFree1,                               // token threads -> MMA: buffer read
    kCBarAccDone, kCBarAccFree,                             // accumulators complete: store them / stored
    kCBarDrain0, kCBarDrain1,
    kCNumBars
};
static_assert(kCNumBars * 8 + 16 <= 256, "barrier block");

struct TcCommitParams {
    Shape s;
    const uint4* rope_h;   // warp-interleaved half2 (cos, sin) table, or nullptr
    const float* beta;     // [B, L, H]: learning-rate logits (delta rule) or weights (mode 2), or nullptr = 1
    float* partials;       // [B * H, nslot, 128, 128] fp32: sum_l (w_l K'_l)^T V_l
    float* partials_g;     // same shape: sum_l beta_l K'_l^T K'_l (delta rule)
    __nv_bfloat16* k_rot;  // [B, L, H, 128]: RoPE(K_c) written on the way, or nullptr
    uint32_t* status;
    uint32_t spin_limit;
    int ntile;             // 128-token tiles per (stream, head)
    int total_tiles;       // B * H * ntile
    int share;             // tiles per CTA: CTA c takes tiles [c * share, (c + 1) * share) of the flattened order
    int nslot;             // partial-sum slots per (stream, head)
};

// kMode 0: S-increment K'^T V'; 1: Eq. 4 at block level (two accumulators); 2: per-token weights on K'.
template <int kMode>
__global__ void __launch_bounds__(kCThreads, 1)
tc_commit_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const __grid_constant__ CUtensorMap tm_wk, const TcCommitParams p)
{
    constexpr int kS = kMode == 1 ? 2 : 3;   // ring stages
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kCOffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kCOffBars + kCNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kCOffBars + kCNumBars * 8 + 4);
    const Abort ab{abort_flag, p.status, p.spin_limit};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.s.L, H = p.s.H;
    const int g_begin = (int)blockIdx.x * p.share;
    const int n_my = min(p.total_tiles, g_begin + p.share) - g_begin;
    auto tile_of = [&](int k, int& bh, int& tl) {
        const int g = g_begin + k;
        bh = g / p.ntile;
        tl = g - bh * p.ntile;
    };
    auto seg_first = [&](int k) { return k == 0 || (g_begin + k) % p.ntile == 0; };
    auto seg_last = [&](int k) { return k + 1 == n_my || (g_begin + k + 1) % p.ntile == 0; };
    auto stage_k = [&](int s) { return (uint32_t)(kCOffStage + s * 2 * kTileBytes); };          // K tile, then V tile
    auto extra_tile = [&](int s) { return (uint32_t)(kCOffStage + (2 * 2 + s) * kTileBytes); };  // delta rule: beta K'

    if (tid == 0) {
        mbar_init(bars + 8 * kCBarWFull, 1);
        mbar_init(bars + 8 * kCBarWFree, 1);
        for (int s = 0; s < kCMaxStages; ++s) {
            mbar_init(bars + 8 * (kCBarStageFull0 + s), 1);
            mbar_init(bars + 8 * (kCBarStageFree0 + s), 1);
            mbar_init(bars + 8 * (kCBarKpFull0 + s), kCTokenThreads);
        }
        mbar_init(bars + 8 * kCBarUFull0, 1);
        mbar_init(bars + 8 * kCBarUFull1, 1);
        mbar_init(bars + 8 * kCBarUFree0, kCTokenThreads);
        mbar_init(bars + 8 * kCBarUFree1, kCTokenThreads);
        mbar_init(bars + 8 * kCBarAccDone, 1);
        mbar_init(bars + 8 * kCBarAccFree, kCTokenThreads);
        mbar_init(bars + 8 * kCBarDrain0, 1);
        mbar_init(bars + 8 * kCBarDrain1, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        // this thread is the TMA producer: the run's first map and first tile are requested now, while
        // tensor memory is still being allocated (nothing else can start before they land)
        if (n_my > 0) {
            int bh, tl;
            tile_of(0, bh, tl);
            const int hb = bh / H, hh = bh - hb * H;
            mbar_expect_tx(bars + 8 * kCBarWFull, kTileBytes);
            tma_load_2d(smem_base + kCOffWk, &tm_wk, bars + 8 * kCBarWFull, 0, hh * kTile);
            tma_load_2d(smem_base + kCOffWk + kHalfBytes, &tm_wk, bars + 8 * kCBarWFull, 64, hh * kTile);
            const uint32_t bar = bars + 8 * (kCBarStageFull0 + 0);
            const uint32_t dst = smem_base + stage_k(0);
            mbar_expect_tx(bar, 2 * kTileBytes);
            tma_load_4d(dst, &tm_k, bar, 0, hh, tl * kTile, hb);
            tma_load_4d(dst + kHalfBytes, &tm_k, bar, 64, hh, tl * kTile, hb);
            tma_load_4d(dst + kTileBytes, &tm_v, bar, 0, hh, tl * kTile, hb);
            tma_load_4d(dst + kTileBytes + kHalfBytes, &tm_v, bar, 64, hh, tl * kTile, hb);
        }
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // TMEM columns: U buffer 0 | U buffer 1 | dS | G
    constexpr uint32_t kColDS = 2 * kTile, kColG = 3 * kTile;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && n_my > 0) {
            bool ok = true;
            int n_w = 1, issued = 1;   // tile 0 and its map went out in the prologue
            for (int k = 0; k < n_my && ok; ++k) {
                int bh, tl;
                tile_of(k, bh, tl);
                const int hb = bh / H, hh = bh - hb * H;
                const int s = k % kS;
                if (k >= kS) ok = wait_bar(bars + 8 * (kCBarStageFree0 + s), (uint32_t)((k / kS) - 1) & 1u, ab, 80);
                if (!ok) break;
                if (k > 0) {
                    const uint32_t bar = bars + 8 * (kCBarStageFull0 + s);
                    const uint32_t dst = smem_base + stage_k(s);
                    mbar_expect_tx(bar, 2 * kTileBytes);
                    tma_load_4d(dst, &tm_k, bar, 0, hh, tl * kTile, hb);
                    tma_load_4d(dst + kHalfBytes, &tm_k, bar, 64, hh, tl * kTile, hb);
                    tma_load_4d(dst + kTileBytes, &tm_v, bar, 0, hh, tl * kTile, hb);
                    tma_load_4d(dst + kTileBytes + kHalfBytes, &tm_v, bar, 64, hh, tl * kTile, hb);
                    ++issued;
                }
                if (k > 0 && seg_first(k)) {
                    // the map of this head: once the MMAs that read the previous head's are done
                    if (n_w > 0) ok = wait_bar(bars + 8 * kCBarWFree, (uint32_t)(n_w - 1) & 1u, ab, 81);
                    if (!ok) break;
                    mbar_expect_tx(bars + 8 * kCBarWFull, kTileBytes);
                    tma_load_2d(smem_base + kCOffWk, &tm_wk, bars + 8 * kCBarWFull, 0, hh * kTile);
                    tma_load_2d(smem_base + kCOffWk + kHalfBytes, &tm_wk, bars + 8 * kCBarWFull, 64, hh * kTile);
                    ++n_w;
                }
                // the first tile alone first: with every CTA of the grid asking for its whole ring at
                // once the first stage would land only after a third of that burst
                if (k == 0 && n_my > 1) ok = wait_bar(bars + 8 * (kCBarStageFull0 + 0), 0u, ab, 79);
            }
            if (!ok || *abort_flag) {
                // do not leave the CTA while bulk copies into its shared memory are in flight
                if (n_w > 0) drain_bar(bars + 8 * kCBarWFull, (uint32_t)(n_w - 1) & 1u);
                for (int m = (issued > kS ? issued - kS : 0); m < issued; ++m)
                    drain_bar(bars + 8 * (kCBarStageFull0 + m % kS), (uint32_t)(m / kS) & 1u);
            }
        }
    } else if (warp == 1 || warp == kCThreads / 32 - 1) {
        // ---------------- two MMA issuers ----------------
        // warp 1: U(k) = K_c W_phi_k for each tile whose K has landed, into the TMEM buffer k & 1 once the
        // token threads have read U(k - 2) out of it.  Last warp: the accumulator MMAs of each tile whose
        // K' has been written.  One thread each: a thread that has MMAs in flight is held at its next
        // tcgen05 fence until they are done, so with a single issuer the two queues ran one after the other.
        if (lane == 0 && n_my > 0) {
            const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
            constexpr uint32_t kLboK = 1u << 16;
            constexpr uint32_t kLboMN = (uint32_t)(kHalfBytes >> 4) << 16;
            auto desc64 = [&](uint32_t lo) {
                uint64_t d;
                asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
                return d;
            };
            bool ok = true;
            if (warp == 1) {
                constexpr uint32_t idesc_u = idesc_bf16(kTile, kTile, 0, 0);    // tile x map: both K-major
                uint32_t w_seen = 0;                                             // maps consumed
                for (int k = 0; k < n_my && ok; ++k) {
                    const int s = k % kS, u = k & 1;
                    if (seg_first(k)) {
                        ok = wait_bar(bars + 8 * kCBarWFull, w_seen & 1u, ab, 82);
                        ++w_seen;
                    }
                    if (ok) ok = wait_bar(bars + 8 * (kCBarStageFull0 + s), (uint32_t)(k / kS) & 1u, ab, 83);
                    if (ok && k >= 2) ok = wait_bar(bars + 8 * (kCBarUFree0 + u), (uint32_t)((k >> 1) - 1) & 1u, ab, 84);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_lo = ((smem_base + stage_k(s)) >> 4) | kLboK;
                    const uint32_t b_lo = ((smem_base + kCOffWk) >> 4) | kLboK;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t koff = (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                        mma_ss(tmem_base + u * kTile, desc64(a_lo + koff), desc64(b_lo + koff), idesc_u, ks > 0);
                    }
                    mma_commit(bars + 8 * (kCBarUFull0 + u));
                    // the next tile belongs to another head: its map may replace this one
                    if (k + 1 < n_my && seg_first(k + 1)) mma_commit(bars + 8 * kCBarWFree);
                }
            } else {
                constexpr uint32_t idesc_tt = idesc_bf16(kTile, kTile, 1, 1);   // both operands token-major
                uint32_t n_seg = 0;             // segments whose accumulators were handed over
                for (int k = 0; k < n_my && ok; ++k) {
                    const int s = k % kS;
                    const bool first = seg_first(k);
                    ok = wait_bar(bars + 8 * (kCBarKpFull0 + s), (uint32_t)(k / kS) & 1u, ab, 85);
                    if (ok && first && n_seg > 0) ok = wait_bar(bars + 8 * kCBarAccFree, (n_seg - 1) & 1u, ab, 86);
                    if (!ok) break;
                    // accumulators += (w K')^T V_c  [and (beta K')^T K']
                    tc_fence_after();
                    const uint32_t k_lo = ((smem_base + stage_k(s)) >> 4) | kLboMN;
                    const uint32_t v_lo = ((smem_base + stage_k(s) + kTileBytes) >> 4) | kLboMN;
                    const uint32_t a_lo = kMode == 1 ? (((smem_base + extra_tile(s)) >> 4) | kLboMN) : k_lo;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)   // 16 tokens per step
                        mma_ss(tmem_base + kColDS, desc64(a_lo + (uint32_t)(ks * (2048 >> 4))),
                               desc64(v_lo + (uint32_t)(ks * (2048 >> 4))), idesc_tt, (!first || ks > 0) ? 1u : 0u);
                    if (kMode == 1) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            mma_ss(tmem_base + kColG, desc64(a_lo + (uint32_t)(ks * (2048 >> 4))),
                                   desc64(k_lo + (uint32_t)(ks * (2048 >> 4))), idesc_tt, (!first || ks > 0) ? 1u : 0u);
                    }
                    mma_commit(bars + 8 * (kCBarStageFree0 + s));
                    if (seg_last(k)) {
                        mma_commit(bars + 8 * kCBarAccDone);
                        ++n_seg;
                    }
                }
            }
            if (!ok || *abort_flag) {
                // tensor memory is freed below: none of this thread's MMAs may still be running
                const uint32_t bar_drain = bars + 8 * (warp == 1 ? kCBarDrain0 : kCBarDrain1);
                mma_commit(bar_drain);
                drain_bar(bar_drain, 0);
            }
        }
    } else {
        // ---------------- token threads: (row r, half hf) of every tile of the run ----------------
        const int hf = (warp - 2) >> 2;             // which 64 of the 128 columns
        const int q = warp & 3;                     // TMEM lane quarter this warp may access
        const int r = q * 32 + lane;                // token row of the tile = TMEM lane
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const bool rotate = p.rope_h != nullptr;
        uint32_t n_seg = 0;                         // accumulator hand-overs so far
        bool ok = true;
        for (int k = 0; k < n_my && ok; ++k) {
            int bh, tl;
            tile_of(k, bh, tl);
            const int b = bh / H, h = bh - b * H;
            const int s = k % kS;
            const int row = tl * kTile + r;
            uint8_t* ktile = smem + stage_k(s);
            const uint32_t u_addr = lane_base + (uint32_t)((k & 1) * kTile);
            // my half of the row of the rotation table (32 pairs as half2, 8 vectors): requested before
            // any wait, so its latency hides behind the wait for the tile
            uint4 cs[8];
            if (rotate) {
                const uint4* tab = p.rope_h + ((size_t)(row >> 5) * 16 + hf * 8) * 32 + (row & 31);
#pragma unroll
                for (int c = 0; c < 8; ++c) cs[c] = __ldg(tab + c * 32);
            }
            // per-token factor on K': the decay weight (mode 2) or the learning rate (delta rule)
            float wtok = 1.0f;
            if (kMode != 0 && p.beta != nullptr && row < L) {
                const float x = __ldg(p.beta + ((size_t)b * L + row) * H + h);
                wtok = kMode == 1 ? sigmoid_fast(x) : x;
            }
            if (p.k_rot != nullptr) {
                // ---- RoPE(K_c) for the softmax branch: the raw tile is in shared memory
                ok = wait_bar(bars + 8 * (kCBarStageFull0 + s), (uint32_t)(k / kS) & 1u, ab, 87);
                if (!ok) break;
                if (row < L) {
                    __nv_bfloat16* dst = p.k_rot + (((size_t)b * L + row) * H + h) * kTile + hf * 64;
#pragma unroll
                    for (int c2 = 0; c2 < 4; ++c2) {
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int c = c2 * 2 + e;
                            const uint4 raw = *reinterpret_cast<const uint4*>(ktile + hf * kHalfBytes + r * 128 + ((c ^ (r & 7)) << 4));
                            const uint32_t x[4] = {raw.x, raw.y, raw.z, raw.w};
                            const uint32_t h2[4] = {cs[c].x, cs[c].y, cs[c].z, cs[c].w};
#pragma unroll
                            for (int m = 0; m < 4; ++m) {
                                float cc, ss;
                                unpack_cs(h2[m], cc, ss);
                                const float x0 = __uint_as_float(x[m] << 16);
                                const float x1 = __uint_as_float(x[m] & 0xFFFF0000u);
                                w[e * 4 + m] = pack_bf16(x0 * cc - x1 * ss, x0 * ss + x1 * cc);
                            }
                        }
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + c2 * 16),
                                     "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                     : "memory");
                    }
                }
            }
            // ---- K' = L2Norm(RoPE(U)).  Both threads of a row read the whole row for its norm (a
            // rotation leaves the norm as it is, so the unrotated values serve), the other half first;
            // each keeps, rotates, rounds and stores its own half.
            ok = wait_bar(bars + 8 * (kCBarUFull0 + (k & 1)), (uint32_t)(k >> 1) & 1u, ab, 88);
            if (!ok) break;
            tc_fence_after();
            uint32_t x[64];
            float ss4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const int col = (part == 0 ? (hf ^ 1) : hf) * 64;
                tmem_ld32(u_addr + col, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
                tmem_ld32(u_addr + col + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) ss4[e] = fmaf(__uint_as_float(x[c + e]), __uint_as_float(x[c + e]), ss4[e]);
                }
            }
            tc_fence_before();
            mbar_arrive(bars + 8 * (kCBarUFree0 + (k & 1)));      // the buffer may receive U(k + 2)
            const float f = rsqrtf((ss4[0] + ss4[1]) + (ss4[2] + ss4[3]) + p.s.eps);
            if (rotate) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t h2[4] = {cs[c].x, cs[c].y, cs[c].z, cs[c].w};
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        float cc, s1;
                        unpack_cs(h2[m], cc, s1);
                        const int i = c * 8 + 2 * m;
                        const float x0 = __uint_as_float(x[i]), x1 = __uint_as_float(x[i + 1]);
                        x[i] = __float_as_uint(x0 * cc - x1 * s1);
                        x[i + 1] = __float_as_uint(x0 * s1 + x1 * cc);
                    }
                }
            }
            // rows past L are zero (TMA fills them, the table's padding rows are zero): K' = 0 there
            if (kMode == 1) {
                store_half_row_bf16_swizzled(ktile, r, hf, x, f);                       // K'      (B of G)
                store_half_row_bf16_swizzled(smem + extra_tile(s), r, hf, x, f * wtok); // beta K' (A of both)
            } else {
                store_half_row_bf16_swizzled(ktile, r, hf, x, f * wtok);
            }
            fence_proxy_async_smem();
            mbar_arrive(bars + 8 * (kCBarKpFull0 + s));
            if (seg_last(k)) {
                // ---- this head's share of the accumulators (row d_k = r, my 64 columns) -> its slot
                ok = wait_bar(bars + 8 * kCBarAccDone, n_seg & 1u, ab, 89);
                if (!ok) break;
                tc_fence_after();
                const int part = (int)blockIdx.x - (bh * p.ntile) / p.share;
                // inside a slot the 128 x 128 sums are stored in groups of 8 columns, rows running fastest
                // (element (row, col) at ((col / 8) * 128 + row) * 8 + col % 8): the 32 rows of a warp
                // then write 1 KB in one piece with every store instruction
                const size_t at = ((size_t)bh * p.nslot + part) * kTile * kTile + ((size_t)(hf * 8) * kTile + r) * 8;
#pragma unroll 1
                for (int acc = 0; acc < (kMode == 1 ? 2 : 1); ++acc) {
                    float* dst = (acc == 0 ? p.partials : p.partials_g) + at;
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
                        tmem_ld32(lane_base + kColDS + acc * kTile + hf * 64 + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 4; ++e)   // 32-byte stores: whole sectors, the warp's 32 side by side
                            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + (size_t)(c * 4 + e) * kTile * 8),
                                         "r"(o[e * 8]), "r"(o[e * 8 + 1]), "r"(o[e * 8 + 2]), "r"(o[e * 8 + 3]), "r"(o[e * 8 + 4]),
                                         "r"(o[e * 8 + 5]), "r"(o[e * 8 + 6]), "r"(o[e * 8 + 7])
                                         : "memory");
                    }
                }
                tc_fence_before();
                mbar_arrive(bars + 8 * kCBarAccFree);
                ++n_seg;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// S <- alpha S + (sum_s A_s) W_phi_v [- (sum_s G_s) S_old]; one CTA per 16 state rows of a head, 128
// threads.  The slots of a head are added in index order (each thread a 4 x 4 block) into shared
// memory; the products with the right-hand matrices (the head's value map, then S_old; both bf16)
// run on the warp-level tensor-core instruction, one 16 x 32 block of the output per warp, with the
// fp32 sums split into a bf16 head and a bf16 remainder (two MMAs, relative error 2^-17: far below
// the bf16 rounding of the matrices themselves).  Every global load the CTA needs is requested
// before the first result is used.
constexpr int kFinRows = 16;
constexpr int kFinThreads = 128;
constexpr int kFinMaxParts = 6;     // slots of one head the unrolled loads cover; more fall back to a loop
constexpr int kFinLdM = kTile + 8;  // bf16 row stride of a right-hand matrix: 272 bytes, conflict-free 8 x 8 loads
constexpr int kFinLdA = kTile + 8;  // fp32 row stride of the summed rows: a fragment's 8-byte reads spread over the banks
constexpr int kFinMatBytes = kTile * kFinLdM * 2;
// shared memory: value map | A rows | delta rule only: S_old | G rows
constexpr int kFinRowBytes = kFinRows * kFinLdA * 4;
constexpr int fin_smem_bytes(int mode) { return (mode == 1 ? 2 : 1) * (kFinMatBytes + kFinRowBytes); }

// a [128][128] bf16 matrix from global memory into padded rows of shared memory, as asynchronous
// 16-byte copies (no registers, and the thread goes on to request its other loads at once);
// fin_matrices_landed() before the matrix is read
__device__ __forceinline__ void fin_load_matrix(__nv_bfloat16* dst, const __nv_bfloat16* __restrict__ src, int tid)
{
    constexpr int kPer = kTile * kTile / 8 / kFinThreads;   // 16-byte pieces per thread
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int c = tid + i * kFinThreads;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst + (c >> 4) * kFinLdM + (c & 15) * 8)),
                     "l"(src + (size_t)c * 8)
                     : "memory");
    }
}
__device__ __forceinline__ void fin_matrices_landed() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// x = head + remainder, both bf16 (two values at a time)
__device__ __forceinline__ void fin_split(float x0, float x1, uint32_t& head, uint32_t& rem)
{
    head = pack_bf16(x0, x1);
    rem = pack_bf16(x0 - __uint_as_float(head << 16), x1 - __uint_as_float(head & 0xFFFF0000u));
}

__device__ __forceinline__ void fin_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// acc[j] (+/-)= X[16 x 128] * M[128 x 8 columns of block j], j = 0..3: this warp's 32 columns.
// X: fp32 rows in shared memory (stride kFinLdA); M: bf16 [m][e] in shared memory (stride kFinLdM).
// Fragment layout of the instruction (g = lane / 4, t = lane % 4): A rows g, g + 8, columns 2t, 2t + 1
// (+ 8); B rows 2t, 2t + 1 (+ 8), column g -- the 8 x 8 blocks of M come transposed from ldmatrix.
template <bool kSubtract>
__device__ __forceinline__ void fin_multiply(float (&acc)[4][4], const float* __restrict__ X,
                                             const __nv_bfloat16* __restrict__ M, int warp, int lane)
{
    constexpr uint32_t kSign = kSubtract ? 0x80008000u : 0u;
    const int g = lane >> 2, t = lane & 3;
    const int mat = lane >> 3;
    const uint32_t m_base = smem_u32(M + ((lane & 7) + (mat & 1) * 8) * kFinLdM + warp * 32 + (mat >> 1) * 8);
#pragma unroll
    for (int ks = 0; ks < kTile / 16; ++ks) {
        const float2 x0 = *reinterpret_cast<const float2*>(X + g * kFinLdA + ks * 16 + 2 * t);
        const float2 x1 = *reinterpret_cast<const float2*>(X + (g + 8) * kFinLdA + ks * 16 + 2 * t);
        const float2 x2 = *reinterpret_cast<const float2*>(X + g * kFinLdA + ks * 16 + 2 * t + 8);
        const float2 x3 = *reinterpret_cast<const float2*>(X + (g + 8) * kFinLdA + ks * 16 + 2 * t + 8);
        uint32_t ah[4], al[4];
        fin_split(x0.x, x0.y, ah[0], al[0]);
        fin_split(x1.x, x1.y, ah[1], al[1]);
        fin_split(x2.x, x2.y, ah[2], al[2]);
        fin_split(x3.x, x3.y, ah[3], al[3]);
#pragma unroll
        for (int i = 0; i < 4; ++i) { ah[i] ^= kSign; al[i] ^= kSign; }
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
            uint32_t b[4];   // blocks j = 2 jj (b[0], b[1]) and 2 jj + 1 (b[2], b[3])
            const uint32_t addr = m_base + (uint32_t)((ks * 16 * kFinLdM + jj * 16) * 2);
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3])
                         : "r"(addr));
            // the two accumulators alternate, so that no instruction waits for the one before it
            fin_mma(acc[2 * jj], al, b[0], b[1]);
            fin_mma(acc[2 * jj + 1], al, b[2], b[3]);
            fin_mma(acc[2 * jj], ah, b[0], b[1]);
            fin_mma(acc[2 * jj + 1], ah, b[2], b[3]);
        }
    }
}

template <int kMode>
__global__ void __launch_bounds__(kFinThreads)
tc_commit_finish_kernel(float* __restrict__ state, const float* __restrict__ partials,
                        const float* __restrict__ partials_g, const __nv_bfloat16* __restrict__ wv,
                        const float* __restrict__ decay, int decay_direct,
                        const __nv_bfloat16* __restrict__ mirror_cur, __nv_bfloat16* __restrict__ mirror_next,
                        int H, int share, int ntile, int nslot, const uint32_t* __restrict__ status)
{
    extern __shared__ __align__(16) uint8_t fin_smem[];
    __nv_bfloat16* Ws = reinterpret_cast<__nv_bfloat16*>(fin_smem);                  // value map [m][e]
    float* As = reinterpret_cast<float*>(fin_smem + kFinMatBytes);                   // [16][128] summed rows
    __nv_bfloat16* Ss = reinterpret_cast<__nv_bfloat16*>(fin_smem + kFinMatBytes + kFinRowBytes);   // S_old [m][e] (delta rule)
    float* Gs = reinterpret_cast<float*>(fin_smem + 2 * kFinMatBytes + kFinRowBytes);               // its rows
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // what this thread sums: row lane / 2 of the CTA's 16, four columns (lane % 2) * 4 .. of each of
    // the column groups 4 warp .. 4 warp + 3 -- a warp then reads 512 contiguous bytes of a slot at a time
    const int srow = lane >> 1, shalf = lane & 1;
    const int bh = (int)(blockIdx.x / (kTile / kFinRows)), h = bh % H;
    const int cta_row0 = (int)(blockIdx.x % (kTile / kFinRows)) * kFinRows;
    const size_t head = (size_t)bh * kTile * kTile;
    // Launched with programmatic stream serialisation: the CTA may start while the partial-sum kernel
    // is still draining.  What does not depend on that kernel (the value map, the current mirror) is
    // fetched first; the wait below returns once the whole preceding kernel has finished and its
    // writes are visible.
    if (wv != nullptr) fin_load_matrix(Ws, wv + (size_t)h * kTile * kTile, tid);
    if (kMode == 1) fin_load_matrix(Ss, mirror_cur + head, tid);
    const float decay_v = decay[bh];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t err = status != nullptr ? status[kStatusError] : 0u;
    const int first = (bh * ntile) / share, last = (bh * ntile + ntile - 1) / share;
    const int nparts = last - first + 1;
    // slots hold their sums in groups of 8 columns, rows running fastest (see the write-out); from one
    // of this thread's column groups to the next: 128 rows x 8
    const size_t slot0 = (size_t)bh * nslot * kTile * kTile + ((size_t)(warp * 4) * kTile + cta_row0 + srow) * 8 + shalf * 4;
    // ---- all loads first: the slots, the old state at the positions of this thread's output fragment
    float4 pa[kFinMaxParts][4];
#pragma unroll
    for (int s = 0; s < kFinMaxParts; ++s) {
        if (s < nparts) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                pa[s][i] = *reinterpret_cast<const float4*>(partials + slot0 + (size_t)s * kTile * kTile + (size_t)i * kTile * 8);
        }
    }
    const int g = lane >> 2, t = lane & 3;
    // output fragment: rows g and g + 8 of the CTA's 16, columns warp * 32 + 8 j + 2 t (+ 1), j = 0..3
    const size_t out0 = head + (size_t)(cta_row0 + g) * kTile + warp * 32 + 2 * t;
    float2 old[4][2];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        old[j][0] = *reinterpret_cast<const float2*>(state + out0 + j * 8);
        old[j][1] = *reinterpret_cast<const float2*>(state + out0 + j * 8 + 8 * kTile);
    }
    if (err != 0u) {
        // a partial-sum CTA gave up on a bounded wait: S stays as it was, and so does its mirror
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            *reinterpret_cast<uint32_t*>(mirror_next + out0 + j * 8) = *reinterpret_cast<const uint32_t*>(mirror_cur + out0 + j * 8);
            *reinterpret_cast<uint32_t*>(mirror_next + out0 + j * 8 + 8 * kTile) =
                *reinterpret_cast<const uint32_t*>(mirror_cur + out0 + j * 8 + 8 * kTile);
        }
        fin_matrices_landed();   // no copy into this CTA's shared memory outlives it
        return;
    }
    auto add4 = [](float4& d, const float4& v) { d.x += v.x; d.y += v.y; d.z += v.z; d.w += v.w; };
    float4 a[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s = 0; s < kFinMaxParts; ++s) {
        if (s < nparts) {
#pragma unroll
            for (int i = 0; i < 4; ++i) add4(a[i], pa[s][i]);
        }
    }
    for (int s = kFinMaxParts; s < nparts; ++s) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            add4(a[i], *reinterpret_cast<const float4*>(partials + slot0 + (size_t)s * kTile * kTile + (size_t)i * kTile * 8));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<float4*>(As + srow * kFinLdA + (warp * 4 + i) * 8 + shalf * 4) = a[i];
    if (kMode == 1) {
        float4 gs[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) gs[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < nparts; ++s) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                add4(gs[i], *reinterpret_cast<const float4*>(partials_g + slot0 + (size_t)s * kTile * kTile + (size_t)i * kTile * 8));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<float4*>(Gs + srow * kFinLdA + (warp * 4 + i) * 8 + shalf * 4) = gs[i];
    }
    fin_matrices_landed();
    __syncthreads();
    float out[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (wv == nullptr) {   // identity value map: the sums themselves
            const float2 lo = *reinterpret_cast<const float2*>(As + g * kFinLdA + warp * 32 + j * 8 + 2 * t);
            const float2 hi = *reinterpret_cast<const float2*>(As + (g + 8) * kFinLdA + warp * 32 + j * 8 + 2 * t);
            out[j][0] = lo.x; out[j][1] = lo.y; out[j][2] = hi.x; out[j][3] = hi.y;
        } else {
            out[j][0] = out[j][1] = out[j][2] = out[j][3] = 0.0f;
        }
    }
    if (wv != nullptr) fin_multiply<false>(out, As, Ws, warp, lane);
    if (kMode == 1) fin_multiply<true>(out, Gs, Ss, warp, lane);
    const float alpha = decay_direct ? decay_v : 1.0f / (1.0f + __expf(-decay_v));
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const float2 o = old[j][half];
            const float2 nw = make_float2(alpha * o.x + out[j][2 * half], alpha * o.y + out[j][2 * half + 1]);
            const size_t at = out0 + j * 8 + (size_t)half * 8 * kTile;
            *reinterpret_cast<float2*>(state + at) = nw;
            *reinterpret_cast<uint32_t*>(mirror_next + at) = pack_bf16(nw.x, nw.y);
        }
    }
}

std::mutex g_setup_mutex;
DeviceSetup g_setup[kMaxDevices];

int device_setup(int* num_sms)
{
    return device_setup_once(g_setup_mutex, g_setup, [] {
        cudaError_t e = opt_in_smem(tc_commit_kernel<0>, kCommitSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_commit_kernel<1>, kCommitSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_commit_kernel<2>, kCommitSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_commit_finish_kernel<0>, fin_smem_bytes(0));
        if (e == cudaSuccess) e = opt_in_smem(tc_commit_finish_kernel<1>, fin_smem_bytes(1));
        return e;
    }, num_sms);
}

}  // namespace

int tc_commit_partials(CommitArgs& a, const __nv_bfloat16* wk_op, cudaStream_t st)
{
    int num_sms = 0;
    if (int r = device_setup(&num_sms)) return r;
    if (a.mode == 1 && (a.partials_g == nullptr || a.state_bf16 == nullptr)) {
        set_error("tc_commit: the delta rule needs the second accumulator and the bf16 copy of the state");
        return ARL2_ERR_INVALID_ARG;
    }
    CUtensorMap tm_k, tm_v, tm_wk;
    if (int r = make_map_blhd(&tm_k, a.k, a.s)) return r;
    if (int r = make_map_blhd(&tm_v, a.v, a.s)) return r;
    if (int r = make_map_rows(&tm_wk, wk_op, (size_t)a.s.H * kTile)) return r;
    TcCommitParams p;
    p.s = a.s;
    p.rope_h = static_cast<const uint4*>(a.rope_h);
    p.beta = a.beta;
    p.partials = a.partials;
    p.partials_g = a.partials_g;
    p.k_rot = a.rope_h != nullptr ? static_cast<__nv_bfloat16*>(a.k_rot_out) : nullptr;
    p.status = a.status;
    p.spin_limit = a.wait_limit ? a.wait_limit - 1 : kSpinLimit;
    // equal runs of the flattened tile sequence, at least 2 tiles each and long enough for a head's
    // partial sums (one per run it falls into, at most ceil(ntile / share) + 1) to fit the slots
    p.ntile = (a.s.L + kTile - 1) / kTile;
    p.total_tiles = a.s.B * a.s.H * p.ntile;
    p.share = (p.total_tiles + num_sms - 1) / num_sms;
    if (p.share < 2) p.share = 2;
    p.nslot = a.nslot;
    if (p.nslot < 2) {
        set_error("tc_commit: needs at least two partial-sum slots per head (got %d)", p.nslot);
        return ARL2_ERR_WORKSPACE;
    }
    if ((p.ntile + p.share - 1) / p.share + 1 > p.nslot) p.share = (p.ntile + p.nslot - 2) / (p.nslot - 1);
    const unsigned grid = (unsigned)((p.total_tiles + p.share - 1) / p.share);
    if (a.mode == 1)
        tc_commit_kernel<1><<<grid, kCThreads, kCommitSmemBytes, st>>>(tm_k, tm_v, tm_wk, p);
    else if (a.mode == 2)
        tc_commit_kernel<2><<<grid, kCThreads, kCommitSmemBytes, st>>>(tm_k, tm_v, tm_wk, p);
    else
        tc_commit_kernel<0><<<grid, kCThreads, kCommitSmemBytes, st>>>(tm_k, tm_v, tm_wk, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_commit_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    a.run_share = p.share;
    a.run_ntile = p.ntile;
    return 1;
}

int tc_commit_finish(const CommitArgs& a, cudaStream_t st)
{
    // programmatic stream serialisation: the grid is staged while the kernel before it in the stream
    // (the partial sums) is still running; the kernel itself waits for that kernel where it must
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.s.B * a.s.H) * (kTile / kFinRows));
    cfg.blockDim = dim3(kFinThreads);
    cfg.dynamicSmemBytes = (size_t)fin_smem_bytes(a.mode == 1 ? 1 : 0);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const __nv_bfloat16* wv = static_cast<const __nv_bfloat16*>(a.wv);
    const float* partials = a.partials;
    const float* partials_g = a.partials_g;
    const __nv_bfloat16* cur = a.state_bf16;
    const uint32_t* status = a.status;
    const int direct = a.decay_direct ? 1 : 0;
    cudaError_t e;
    if (a.mode == 1)
        e = cudaLaunchKernelEx(&cfg, tc_commit_finish_kernel<1>, a.state, partials, partials_g, wv, a.decay, direct, cur,
                               a.state_bf16_next, a.s.H, a.run_share, a.run_ntile, a.nslot, status);
    else
        e = cudaLaunchKernelEx(&cfg, tc_commit_finish_kernel<0>, a.state, partials, partials_g, wv, a.decay, direct, cur,
                               a.state_bf16_next, a.s.H, a.run_share, a.run_ntile, a.nslot, status);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_commit_finish_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

}  // namespace arl2
