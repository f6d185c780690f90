// Token-level state access on tensor cores (bf16 I/O, D = 128): the comparison mode of the paper's
// "State access granularity" ablation (Sec. 4.3).  Token i of the block reads the state advanced by the
// block's tokens before it,
//   S^(0) = S,  S^(i+1) = alpha_i S^(i) + K'_i^T V'_i,   X_i = Q'_i S^(i),
// which is a causal linear attention over the block on top of the carried state.  This kernel ADDS
// sigmoid(g_i) X_i to an output that already holds the intra-block softmax branch; S is only read.
//
// Chunkwise form (own derivation), chunks of C = 128 tokens, inside a chunk that enters with state
// S_c:  lg_j = sum_{m <= j} log alpha_m,  la_i = lg_{i-1} (la_0 = 0),  w_j = exp(lg_last - lg_j) <= 1,
//   Khat_j = w_j K'_j,   Shat = exp(lg_last) S_c,
//   X_i = exp(la_i - lg_last) [ Q'_i Shat + sum_{j < i} (Q'_i . Khat_j) V'_j ],
//   S_{c+1} = Shat + Khat^T V'.
// Every factor that multiplies an operand is <= 1; only the final row factor exp(la_i - lg_last) is
// >= 1 (bounded by 1 / prod of the chunk's gates: gates that stay below about 0.5 for a whole chunk
// would leave the fp32 range, which a forget gate of a model that remembers anything never does).
//
// One CTA (256 threads, two per token row) per (stream, head) walks the chunks in order; the fp32
// state lives in TMEM for the whole walk.  Per chunk:
//   U_q, U_k, U_v = Q W_q, K W_k, V W_v                      3 MMAs into TMEM
//   pass 1: gates (log-space scan), Q' , Khat, V' as bf16 over the raw tiles; Shat into TMEM and as a
//           bf16 operand copy
//   SC = Q' Khat^T,  O = Q' Shat                             2 MMAs
//   pass 2: P = strictly lower triangle of SC as bf16 into TMEM
//   O += P V',  S += Khat^T V'                               2 MMAs
//   epilogue: out_i += sigmoid(g_i) exp(la_i - lg_last) O_i
// Every wait is bounded; on expiry the CTA records ARL2_ERR_TIMEOUT and leaves through the common exit.
#include "tc_common.cuh"

namespace arl2 {

namespace {

constexpr int kTRThreads = 256;
constexpr int kTROffWq = 0, kTROffWk = kTileBytes, kTROffWv = 2 * kTileBytes;
constexpr int kTROffQ = 3 * kTileBytes, kTROffK = 4 * kTileBytes, kTROffV = 5 * kTileBytes;
constexpr int kTROffS = 6 * kTileBytes;                 // bf16 copy of Shat, [d][e]
constexpr int kTROffBars = 7 * kTileBytes;
constexpr int kTROffGates = kTROffBars + 128;           // lg[128], then warp totals
constexpr int kTRSmemBytes = kTROffGates + 128 * 4 + 64 + 1024;

enum TRBar : int { kTRBarW = 0, kTRBarLoad, kTRBarU, kTRBarA, kTRBarB, kTRBarDrain, kTRNumBars };

struct TcReadoutParams {
    Shape s;
    const uint4* rope_h;
    const float* alpha;        // [B, L, H] forget-gate logits, or nullptr = 1
    const float* gate;         // [B, L, H] combine-gate logits
    const float* state;        // [B, H, 128, 128] fp32, read only
    __nv_bfloat16* out;        // [B, L, H, 128]: receives += sigmoid(g) X
    uint32_t* status;
    uint32_t spin_limit;
    int ntile;
};

__global__ void __launch_bounds__(kTRThreads, 1)
tc_token_readout_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_wq,
                        const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                        const TcReadoutParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kTROffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kTROffBars + kTRNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kTROffBars + kTRNumBars * 8 + 4);
    float* lg_s = reinterpret_cast<float*>(smem + kTROffGates);          // [128] inclusive log products
    float* wsum = lg_s + 128;                                            // [4] warp totals
    const Abort ab{abort_flag, p.status, p.spin_limit};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, b = blockIdx.y;
    const int L = p.s.L, H = p.s.H;
    const size_t bh = (size_t)b * H + h;

    if (tid == 0) {
        for (int i = 0; i < kTRNumBars; ++i) mbar_init(bars + 8 * i, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // two threads per row: warps w and w + 4 own the same 32 TMEM lanes and split the 128 columns
    const int r = (warp & 3) * 32 + lane;
    const int hf = warp >> 2;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    // TMEM columns: U_q, later SC | U_k, later O | U_v, later P | S
    constexpr uint32_t kColQ = 0, kColK = kTile, kColV = 2 * kTile, kColS = 3 * kTile;

    bool ok = true;
    if (tid == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        const uint32_t bar = bars + 8 * kTRBarW;
        mbar_expect_tx(bar, 3 * kTileBytes);
        const CUtensorMap* maps[3] = {&tm_wq, &tm_wk, &tm_wv};
        for (int i = 0; i < 3; ++i) {
            tma_load_2d(smem_base + i * kTileBytes, maps[i], bar, 0, h * kTile);
            tma_load_2d(smem_base + i * kTileBytes + kHalfBytes, maps[i], bar, 64, h * kTile);
        }
    }
    // the carried state S (fp32) into TMEM: row d = r, this thread's 64 columns
    {
        const float* srow = p.state + (bh * kTile + r) * kTile + hf * 64;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t x[32];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float4 v = *reinterpret_cast<const float4*>(srow + c * 32 + e * 4);
                x[e * 4 + 0] = __float_as_uint(v.x); x[e * 4 + 1] = __float_as_uint(v.y);
                x[e * 4 + 2] = __float_as_uint(v.z); x[e * 4 + 3] = __float_as_uint(v.w);
            }
            tmem_st32(lane_base + kColS + hf * 64 + c * 32, x);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();

    constexpr uint32_t kLboK = 1u << 16;
    constexpr uint32_t kLboMN = (uint32_t)(kHalfBytes >> 4) << 16;
    const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
    auto desc64 = [&](uint32_t lo) {
        uint64_t d;
        asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
        return d;
    };
    constexpr uint32_t idesc_kk = idesc_bf16(kTile, kTile, 0, 0);   // both operands contraction-contiguous
    constexpr uint32_t idesc_kn = idesc_bf16(kTile, kTile, 0, 1);   // B rows = contraction index
    constexpr uint32_t idesc_nn = idesc_bf16(kTile, kTile, 1, 1);   // both operands row = contraction index
    auto koff_k = [](int ks) { return (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4); };
    auto koff_n = [](int ks) { return (uint32_t)(ks * (2048 >> 4)); };
    auto lo_of = [&](int off, uint32_t lbo) { return ((smem_base + (uint32_t)off) >> 4) | lbo; };

    bool alive = true;
    int loads = 0;
    for (int c = 0; c < p.ntile; ++c) {
        const uint32_t par = (uint32_t)c & 1u;
        const int row = c * kTile + r;                 // this thread's token
        // ---- tiles of the chunk, then U_q, U_k, U_v
        if (tid == 0) {
            const uint32_t bar = bars + 8 * kTRBarLoad;
            mbar_expect_tx(bar, 3 * kTileBytes);
            const CUtensorMap* maps[3] = {&tm_q, &tm_k, &tm_v};
            for (int i = 0; i < 3; ++i) {
                tma_load_4d(smem_base + kTROffQ + i * kTileBytes, maps[i], bar, 0, h, c * kTile, b);
                tma_load_4d(smem_base + kTROffQ + i * kTileBytes + kHalfBytes, maps[i], bar, 64, h, c * kTile, b);
            }
            ++loads;
            if (c == 0) ok = wait_bar(bars + 8 * kTRBarW, 0, ab, 110);
            if (ok) ok = wait_bar(bar, par, ab, 111);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int u = 0; u < 3; ++u) {
                    const uint32_t a_lo = lo_of(kTROffQ + u * kTileBytes, kLboK), b_lo = lo_of(u * kTileBytes, kLboK);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ss(tmem_base + u * kTile, desc64(a_lo + koff_k(ks)), desc64(b_lo + koff_k(ks)), idesc_kk, ks > 0);
                }
                mma_commit(bars + 8 * kTRBarU);
            }
        }
        // ---- gates of the chunk: lg_j = sum_{m <= j} log alpha_m (tokens past L: alpha = 1)
        float la_log = 0.0f;   // log alpha of this thread's token
        if (hf == 0) {
            if (row < L && p.alpha != nullptr) {
                const float x = __ldg(p.alpha + ((size_t)b * L + row) * H + h);
                la_log = x >= 0.0f ? -log1pf(expf(-x)) : x - log1pf(expf(x));
            }
            float cl = la_log;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float up = __shfl_up_sync(0xffffffffu, cl, off);
                if (lane >= off) cl += up;
            }
            if (lane == 31) wsum[warp] = cl;
            lg_s[r] = cl;              // within the warp so far
        }
        __syncthreads();
        if (hf == 0) {
            float add = 0.0f;
            for (int w = 0; w < (warp & 3); ++w) add += wsum[w];
            lg_s[r] += add;
        }
        const float gate_logit = (row < L) ? __ldg(p.gate + ((size_t)b * L + row) * H + h) : 0.0f;
        uint4 cs[8];
        if (p.rope_h != nullptr) {
            const uint4* tab = p.rope_h + ((size_t)(row >> 5) * 16 + hf * 8) * 32 + (row & 31);
#pragma unroll
            for (int i = 0; i < 8; ++i) cs[i] = __ldg(tab + i * 32);
        }
        __syncthreads();
        const float lg_last = lg_s[kTile - 1];
        const float lg_r = lg_s[r];
        const float la_r = r > 0 ? lg_s[r - 1] : 0.0f;

        alive = wait_bar(bars + 8 * kTRBarU, par, ab, 112);
        if (alive) {
            tc_fence_after();
            // ---- pass 1: Q' and Khat (norm over the whole row, this thread keeps its half), V'
            uint32_t x[64];
#pragma unroll
            for (int t = 0; t < 2; ++t) {   // t = 0: Q, t = 1: K
                float ss4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    const int col = (part == 0 ? (hf ^ 1) : hf) * 64;
                    tmem_ld32(lane_base + t * kTile + col, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
                    tmem_ld32(lane_base + t * kTile + col + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 64; i += 4) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) ss4[e] = fmaf(__uint_as_float(x[i + e]), __uint_as_float(x[i + e]), ss4[e]);
                    }
                }
                float f = rsqrtf((ss4[0] + ss4[1]) + (ss4[2] + ss4[3]) + p.s.eps);
                if (t == 1) f *= __expf(lg_last - lg_r);          // Khat_j = w_j K'_j
                if (p.rope_h != nullptr) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t h2[4] = {cs[i].x, cs[i].y, cs[i].z, cs[i].w};
#pragma unroll
                        for (int m = 0; m < 4; ++m) {
                            float cc, s1;
                            unpack_cs(h2[m], cc, s1);
                            const int at = i * 8 + 2 * m;
                            const float x0 = __uint_as_float(x[at]), x1 = __uint_as_float(x[at + 1]);
                            x[at] = __float_as_uint(x0 * cc - x1 * s1);
                            x[at + 1] = __float_as_uint(x0 * s1 + x1 * cc);
                        }
                    }
                }
                store_half_row_bf16_swizzled(smem + kTROffQ + t * kTileBytes, r, hf, x, f);
            }
            tmem_ld32(lane_base + kColV + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
            tmem_ld32(lane_base + kColV + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
            tmem_wait_ld();
            store_half_row_bf16_swizzled(smem + kTROffV, r, hf, x, 1.0f);
            // ---- Shat = exp(lg_last) S: back into TMEM (row d = r) and as a bf16 operand copy
            const float g_last = __expf(lg_last);
            tmem_ld32(lane_base + kColS + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
            tmem_ld32(lane_base + kColS + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 64; ++i) x[i] = __float_as_uint(__uint_as_float(x[i]) * g_last);
            tmem_st32(lane_base + kColS + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
            tmem_st32(lane_base + kColS + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
            store_half_row_bf16_swizzled(smem + kTROffS, r, hf, x, 1.0f);
            tmem_wait_st();
        }
        fence_proxy_async_smem();
        tc_fence_before();
        if (__syncthreads_or(!alive)) break;   // every thread leaves together
        // ---- SC = Q' Khat^T (columns of U_q), O = Q' Shat (columns of U_k)
        if (tid == 0 && ok) {
            tc_fence_after();
            const uint32_t q_lo = lo_of(kTROffQ, kLboK), k_lo = lo_of(kTROffK, kLboK), s_lo = lo_of(kTROffS, kLboMN);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(tmem_base + kColQ, desc64(q_lo + koff_k(ks)), desc64(k_lo + koff_k(ks)), idesc_kk, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(tmem_base + kColK, desc64(q_lo + koff_k(ks)), desc64(s_lo + koff_n(ks)), idesc_kn, ks > 0);
            mma_commit(bars + 8 * kTRBarA);
        }
        alive = wait_bar(bars + 8 * kTRBarA, par, ab, 113);
        if (alive) {
            tc_fence_after();
            // ---- pass 2: P = strictly lower triangle of SC (keys hf * 64 ..), bf16 pairs into the U_v columns
            uint32_t sc[64], pk[32];
            tmem_ld32(lane_base + kColQ + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
            tmem_ld32(lane_base + kColQ + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int j0 = hf * 64 + 2 * i;
                pk[i] = pack_bf16(j0 < r ? __uint_as_float(sc[2 * i]) : 0.0f, j0 + 1 < r ? __uint_as_float(sc[2 * i + 1]) : 0.0f);
            }
            tmem_st32(lane_base + kColV + hf * 32, pk);
            tmem_wait_st();
        }
        tc_fence_before();
        if (__syncthreads_or(!alive)) break;
        // ---- O += P V',  S += Khat^T V'
        if (tid == 0 && ok) {
            tc_fence_after();
            const uint32_t v_lo = lo_of(kTROffV, kLboMN), k_lo = lo_of(kTROffK, kLboMN);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ts(tmem_base + kColK, tmem_base + kColV + ks * 8, desc64(v_lo + koff_n(ks)), idesc_kn, 1u);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(tmem_base + kColS, desc64(k_lo + koff_n(ks)), desc64(v_lo + koff_n(ks)), idesc_nn, 1u);
            mma_commit(bars + 8 * kTRBarB);
        }
        alive = wait_bar(bars + 8 * kTRBarB, par, ab, 114);
        if (alive) {
            tc_fence_after();
            // ---- epilogue: out_i += sigmoid(g_i) exp(la_i - lg_last) O_i
            uint32_t o[64];
            tmem_ld32(lane_base + kColK + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&o[0]));
            tmem_ld32(lane_base + kColK + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&o[32]));
            tmem_wait_ld();
            if (row < L) {
                const float f = sigmoid_fast(gate_logit) * __expf(la_r - lg_last);
                uint4* orow = reinterpret_cast<uint4*>(p.out + (((size_t)b * L + row) * H + h) * kTile + hf * 64);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint4 prev = orow[i];
                    const uint32_t pw[4] = {prev.x, prev.y, prev.z, prev.w};
                    uint32_t nw[4];
#pragma unroll
                    for (int m = 0; m < 4; ++m)
                        nw[m] = pack_bf16(__uint_as_float(pw[m] << 16) + f * __uint_as_float(o[i * 8 + 2 * m]),
                                          __uint_as_float(pw[m] & 0xFFFF0000u) + f * __uint_as_float(o[i * 8 + 2 * m + 1]));
                    orow[i] = make_uint4(nw[0], nw[1], nw[2], nw[3]);
                }
            }
        }
        tc_fence_before();
        if (__syncthreads_or(!alive)) break;   // the tiles and the gate arrays may be overwritten now
    }
    if (tid == 0 && (!ok || *abort_flag)) {
        // leave no bulk copy in flight into this CTA's shared memory, no MMA writing tensor memory
        drain_bar(bars + 8 * kTRBarW, 0);
        if (loads > 0) drain_bar(bars + 8 * kTRBarLoad, (uint32_t)(loads - 1) & 1u);
        mma_commit(bars + 8 * kTRBarDrain);
        drain_bar(bars + 8 * kTRBarDrain, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

std::mutex g_setup_mutex;
DeviceSetup g_setup[kMaxDevices];

}  // namespace

int tc_token_readout(const StepArgs& a, const float* alpha_logits, const __nv_bfloat16* wq_op,
                     const __nv_bfloat16* wk_op, const __nv_bfloat16* wv_op, cudaStream_t st)
{
    int num_sms = 0;
    if (int r = device_setup_once(g_setup_mutex, g_setup,
                                  [] { return opt_in_smem(tc_token_readout_kernel, kTRSmemBytes); }, &num_sms))
        return r;
    CUtensorMap tm_q, tm_k, tm_v, tm_wq, tm_wk, tm_wv;
    if (int r = make_map_blhd(&tm_q, a.q, a.s)) return r;
    if (int r = make_map_blhd(&tm_k, a.k_rot, a.s)) return r;     // raw K: the feature map comes before the rotation
    if (int r = make_map_blhd(&tm_v, a.v, a.s)) return r;
    if (int r = make_map_rows(&tm_wq, wq_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_wk, wk_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_wv, wv_op, (size_t)a.s.H * kTile)) return r;
    TcReadoutParams p;
    p.s = a.s;
    p.rope_h = static_cast<const uint4*>(a.rope_h);
    p.alpha = alpha_logits;
    p.gate = a.gate;
    p.state = a.state;
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.status = a.status;
    p.spin_limit = a.wait_limit ? a.wait_limit - 1 : kSpinLimit;
    p.ntile = (a.s.L + kTile - 1) / kTile;
    dim3 grid(a.s.H, a.s.B);
    tc_token_readout_kernel<<<grid, kTRThreads, kTRSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_wq, tm_wk, tm_wv, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_token_readout_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

}  // namespace arl2
