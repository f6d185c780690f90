// The projections around the core (Sec. 3.1: Q = x W_q, K = x W_k, V = x W_v; Eq. 6-7: gate logits
// x W_g and y = O W_o) as one persistent tcgen05 GEMM kernel: C[M, N] = A[M, K] B[K, N], bf16 operands,
// fp32 accumulation in tensor memory, bf16 (or, for the gate logits, fp32) results.
//
// Tiles of (128 MH) x BN outputs, MH = 1 or 2 row halves of 128, BN = 256, 192 or 128 columns; the
// contraction in blocks of 64; one CTA per SM walks its tiles.
//   warp 0     TMA producer: per k-block the A tile [128 MH x 64] (K-major) and the B tile [64 x BN]
//              (rows = contraction index, as it lies in a row-major (in, out) weight) through a ring
//              of 4 (MH = 1) or 3 (MH = 2) stages
//   warp 1     MMA issuer: per k-block 4 MMAs of 128 x BN x 16 per row half into TMEM accumulators
//   warps 2-5  epilogue, one thread per output row of a half: TMEM -> registers -> bf16 -> global,
//              32-byte stores
// MH = 1 keeps two accumulators (while the epilogue drains one the issuer fills the other).  MH = 2
// uses the whole of tensor memory for one 256 x 256 tile: both halves share every B block, which
// cuts the bytes fetched from L2 per flop by a third -- with 128-row tiles the operand fetch
// (48 KB per 512 MMA clocks) is what the tensor pipe waits for.
// The N axis is a concatenation of column segments (Q | K | V | gate logits): a tile's columns go to
// the segment's own tensor, so the three [B, L, H, D] tensors and the [B, L, H] logits come out of one
// launch in the layouts the attention kernels read.
// Every wait is bounded; on expiry the CTA records ARL2_ERR_TIMEOUT and leaves through the common exit.
#include "tc_common.cuh"

namespace arl2 {

namespace {

constexpr int kGBM = 128, kGBK = 64;   // an MMA covers kGBM x BN outputs; a tile is MH of them on top of each other
constexpr int kGMaxStages = 4;
constexpr int kGABytes = kGBM * kGBK * 2;             // 16 KB per row half
constexpr int kGBBytes = kGBK * 256 * 2;              // up to 32 KB: groups of 64 columns x 64 rows
// 4 stages of one A half + B, or 3 stages of two A halves + B: 192 KB either way
constexpr int kGOffBars = 4 * (kGABytes + kGBBytes);
static_assert(3 * (2 * kGABytes + kGBBytes) == kGOffBars, "ring size");
constexpr int kGemmSmemBytes = kGOffBars + 256 + 1024;
constexpr int kGThreads = 192;

enum GBar : int {
    kGBarFull0 = 0,
    kGBarEmpty0 = kGBarFull0 + kGMaxStages,
    kGBarAccFull0 = kGBarEmpty0 + kGMaxStages, kGBarAccFull1,
    kGBarAccFree0, kGBarAccFree1,
    kGBarDrain,
    kGNumBars
};
static_assert(kGNumBars * 8 + 16 <= 256, "barrier block");

struct GemmParams {
    int M, N, K;
    int m_tiles, n_tiles, bn, tile_rows;   // tile_rows = 128 or 256
    // output routing: column n of the product belongs to segment n / seg_cols; segments
    // 0 .. n_bf16_seg - 1 are bf16 tensors with row stride ld_out, the one after them (if any) is the
    // fp32 tensor out_f32 with f32_cols valid columns and row stride ld_f32
    __nv_bfloat16* out[4];
    int seg_cols, ld_out, n_bf16_seg;
    float* out_f32;
    int f32_cols, ld_f32;
    uint32_t* status;
    uint32_t spin_limit;
};

// Tile order: bands of kGBand row tiles; inside a band the row tile varies fastest, then the column
// tile, so the CTAs running at one time share a few B tiles and a band of A that stays in L2.
constexpr int kGBand = 32;
__device__ __forceinline__ void tile_origin(int t, const GemmParams& p, int& m0, int& n0)
{
    const int per_band = kGBand * p.n_tiles;
    const int band = t / per_band, in_band = t - band * per_band;
    const int rows = min(kGBand, p.m_tiles - band * kGBand);   // the last band may be shorter
    const int nt = in_band / rows;
    m0 = (band * kGBand + in_band - nt * rows) * p.tile_rows;
    n0 = nt * p.bn;
}

template <int BN, int MH>
__global__ void __launch_bounds__(kGThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kGOffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kGOffBars + kGNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kGOffBars + kGNumBars * 8 + 4);
    const Abort ab{abort_flag, p.status, p.spin_limit};
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total = p.m_tiles * p.n_tiles;
    const int n_kb = p.K / kGBK;
    constexpr int kGStages = MH == 2 ? 3 : 4;
    constexpr int kGStageBytes = MH * kGABytes + kGBBytes;

    if (tid == 0) {
        for (int s = 0; s < kGMaxStages; ++s) {
            mbar_init(bars + 8 * (kGBarFull0 + s), 1);
            mbar_init(bars + 8 * (kGBarEmpty0 + s), 1);
        }
        mbar_init(bars + 8 * kGBarAccFull0, 1);
        mbar_init(bars + 8 * kGBarAccFull1, 1);
        mbar_init(bars + 8 * kGBarAccFree0, 128);
        mbar_init(bars + 8 * kGBarAccFree1, 128);
        mbar_init(bars + 8 * kGBarDrain, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            prefetch_tensormap(&tm_a);
            prefetch_tensormap(&tm_b);
            bool ok = true;
            uint32_t n = 0;
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
                int m0, n0;
                tile_origin(t, p, m0, n0);
                for (int kb = 0; kb < n_kb && ok; ++kb, ++n) {
                    const uint32_t s = n % kGStages;
                    if (n >= (uint32_t)kGStages) ok = wait_bar(bars + 8 * (kGBarEmpty0 + s), ((n / kGStages) - 1) & 1u, ab, 120);
                    if (!ok) break;
                    const uint32_t bar = bars + 8 * (kGBarFull0 + s);
                    const uint32_t dst = smem_base + s * kGStageBytes;
                    mbar_expect_tx(bar, MH * kGABytes + kGBK * BN * 2);
#pragma unroll
                    for (int hlf = 0; hlf < MH; ++hlf)   // rows past M are fetched as zeros
                        tma_load_2d(dst + hlf * kGABytes, &tm_a, bar, kb * kGBK, m0 + hlf * kGBM);
#pragma unroll
                    for (int g = 0; g < BN / 64; ++g)
                        tma_load_2d(dst + MH * kGABytes + g * (kGBK * 128), &tm_b, bar, n0 + g * 64, kb * kGBK);
                }
            }
            if (!ok || *abort_flag) {
                for (uint32_t m = (n > (uint32_t)kGStages ? n - kGStages : 0); m < n; ++m)
                    drain_bar(bars + 8 * (kGBarFull0 + m % kGStages), (m / kGStages) & 1u);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
            constexpr uint32_t kLboK = 1u << 16;
            constexpr uint32_t kLboB = (uint32_t)((kGBK * 128) >> 4) << 16;     // 64-column groups of B, 8 KB apart
            auto desc64 = [&](uint32_t lo) {
                uint64_t d;
                asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
                return d;
            };
            constexpr uint32_t idesc = idesc_bf16(kGBM, BN, 0, 1);   // A K-major, B rows = contraction index
            bool ok = true;
            uint32_t n = 0, it = 0;
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
                // MH = 1: two accumulators take turns; MH = 2: the one tile fills tensor memory, and its
                // epilogue must be through before the next tile's first MMA
                const uint32_t buf = MH == 1 ? (it & 1u) : 0u;
                if (MH == 1) {
                    if (it >= 2) ok = wait_bar(bars + 8 * (kGBarAccFree0 + buf), ((it >> 1) - 1) & 1u, ab, 121);
                } else {
                    if (it >= 1) ok = wait_bar(bars + 8 * kGBarAccFree0, (it - 1) & 1u, ab, 121);
                }
                // ordered after the epilogue's reads of this accumulator; inside the k loop the operands
                // come from TMA (an mbarrier wait is all they need), and a tcgen05 fence there would hold
                // the thread until the MMAs already in flight are done
                tc_fence_after();
                for (int kb = 0; kb < n_kb && ok; ++kb, ++n) {
                    const uint32_t s = n % kGStages;
                    ok = wait_bar(bars + 8 * (kGBarFull0 + s), (n / kGStages) & 1u, ab, 122);
                    if (!ok) break;
                    const uint32_t a_lo = ((smem_base + s * kGStageBytes) >> 4) | kLboK;
                    const uint32_t b_lo = ((smem_base + s * kGStageBytes + MH * kGABytes) >> 4) | kLboB;
#pragma unroll
                    for (int ks = 0; ks < kGBK / 16; ++ks) {
#pragma unroll
                        for (int hlf = 0; hlf < MH; ++hlf)
                            mma_ss(tmem_base + (MH == 1 ? buf : (uint32_t)hlf) * 256,
                                   desc64(a_lo + (uint32_t)((hlf * kGABytes + ks * 32) >> 4)),
                                   desc64(b_lo + (uint32_t)(ks * (2048 >> 4))), idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                    }
                    mma_commit(bars + 8 * (kGBarEmpty0 + s));
                }
                if (ok) mma_commit(bars + 8 * (kGBarAccFull0 + buf));
            }
            if (!ok || *abort_flag) {
                mma_commit(bars + 8 * kGBarDrain);
                drain_bar(bars + 8 * kGBarDrain, 0);
            }
        }
    } else {
        // ---------------- epilogue: thread = output row of the tile ----------------
        const int q = warp & 3;
        const int r = q * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        bool ok = true;
        uint32_t it = 0;
        for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
            const uint32_t buf = MH == 1 ? (it & 1u) : 0u;
            int m0, n0;
            tile_origin(t, p, m0, n0);
            ok = wait_bar(bars + 8 * (kGBarAccFull0 + buf), (MH == 1 ? (it >> 1) : it) & 1u, ab, 123);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < MH * (BN / 32); ++c) {
                // (MH = 2: the second half's chunks follow the first's; its rows lie 128 further down)
                const int hlf = c / (BN / 32), cc = c - hlf * (BN / 32);
                const int row = m0 + hlf * kGBM + r;
                uint32_t o[32];
                tmem_ld32(lane_base + (MH == 1 ? buf : (uint32_t)hlf) * 256 + cc * 32, o);
                tmem_wait_ld();
                const int n = n0 + cc * 32;                                 // 32 columns lie inside one segment
                if (row >= p.M || n >= p.N) continue;
                const int seg = n / p.seg_cols, col = n - seg * p.seg_cols;
                if (seg < p.n_bf16_seg) {
                    __nv_bfloat16* dst = p.out[seg] + (size_t)row * p.ld_out + col;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            w[i] = pack_bf16(__uint_as_float(o[e * 16 + 2 * i]), __uint_as_float(o[e * 16 + 2 * i + 1]));
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + e * 16),
                                     "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                     : "memory");
                    }
                } else {
                    float* dst = p.out_f32 + (size_t)row * p.ld_f32;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (col + i < p.f32_cols) dst[col + i] = __uint_as_float(o[i]);
                }
            }
            tc_fence_before();
            mbar_arrive(bars + 8 * (kGBarAccFree0 + buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// [rows, cols] bf16 row-major; box = 64 columns x box_rows rows, 128-byte swizzle
int make_map_2d(CUtensorMap* m, const void* base, size_t rows, size_t cols, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return ARL2_ERR_CUDA; }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled([%zu, %zu]) failed with %d", rows, cols, (int)r); return ARL2_ERR_CUDA; }
    return 0;
}

std::mutex g_setup_mutex;
DeviceSetup g_setup[kMaxDevices];

}  // namespace

int tc_gemm(const GemmArgs& a, cudaStream_t st)
{
    int num_sms = 0;
    if (int r = device_setup_once(g_setup_mutex, g_setup, [] {
            cudaError_t e = opt_in_smem(tc_gemm_kernel<256, 1>, kGemmSmemBytes);
            if (e == cudaSuccess) e = opt_in_smem(tc_gemm_kernel<192, 1>, kGemmSmemBytes);
            if (e == cudaSuccess) e = opt_in_smem(tc_gemm_kernel<128, 1>, kGemmSmemBytes);
            if (e == cudaSuccess) e = opt_in_smem(tc_gemm_kernel<256, 2>, kGemmSmemBytes);
            if (e == cudaSuccess) e = opt_in_smem(tc_gemm_kernel<192, 2>, kGemmSmemBytes);
            return e;
        }, &num_sms))
        return r;
    if (a.K % kGBK != 0 || a.N % 64 != 0 || a.seg_cols % 32 != 0 || a.M < 1) {
        set_error("tc_gemm: K must be a multiple of %d, N of 64 and the segment width of 32 (got M=%d N=%d K=%d)",
                  kGBK, a.M, a.N, a.K);
        return ARL2_ERR_UNSUPPORTED;
    }
    CUtensorMap tm_a, tm_b;
    if (int r = make_map_2d(&tm_a, a.a, (size_t)a.M, (size_t)a.K, kGBM)) return r;
    if (int r = make_map_2d(&tm_b, a.b, (size_t)a.K, (size_t)a.N, kGBK)) return r;
    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    // Tile shape, by a cost in MMA clocks per CTA: (rounds of tiles over the persistent grid) x (time of
    // a tile).  Measured: a 128-row tile's k-block of 512 MMA clocks takes about 740 (its 48 KB of
    // operands come from L2 at about 53 B/clk per SM) with the epilogue hidden behind the next tile; a
    // 256-row tile shares every B block between its halves -- a k-block of 1024 MMA clocks takes about
    // 1200 -- but fills tensor memory, so its epilogue (about 4000 clocks) is not hidden: it pays for long
    // contractions (K = 5120: 1430 against 1230 TFLOP/s) and not for K = 1536.  192 columns instead of 256
    // where that fills the rounds better (the 1536-wide output projection of 4680 tokens: 222 tiles of
    // 128 x 256 are two rounds on 148 SMs, the second half empty; 296 of 128 x 192 are two full ones).
    // The 128-column tile serves N <= 128 only: at 128 x 128 both operands of an MMA come from shared
    // memory at its full rate, measured slower even where it fills the rounds.
    int mh = 1;
    p.bn = a.N <= 128 ? 128 : 256;
    if (p.bn == 256) {
        const int n_kb = a.K / kGBK;
        float best = 0.0f;
        for (int cand_mh = 1; cand_mh <= 2; ++cand_mh) {
            if (cand_mh == 2 && a.M <= kGBM) break;
            for (int cand_bn = 256; cand_bn >= 192; cand_bn -= 64) {
                const long tiles = (long)((a.M + cand_mh * kGBM - 1) / (cand_mh * kGBM)) * ((a.N + cand_bn - 1) / cand_bn);
                const float tile = (cand_mh == 1 ? n_kb * 740.0f : n_kb * 1200.0f + 4000.0f) * cand_bn / 256.0f;
                const float cost = (float)((tiles + num_sms - 1) / num_sms) * tile;
                if (best == 0.0f || cost < best) { best = cost; mh = cand_mh; p.bn = cand_bn; }
            }
        }
    }
    p.tile_rows = mh * kGBM;
    p.m_tiles = (a.M + p.tile_rows - 1) / p.tile_rows;
    p.n_tiles = (a.N + p.bn - 1) / p.bn;   // columns past N are fetched as zeros and not stored
    for (int i = 0; i < 4; ++i) p.out[i] = static_cast<__nv_bfloat16*>(a.out[i]);
    p.seg_cols = a.seg_cols; p.ld_out = a.ld_out; p.n_bf16_seg = a.n_bf16_seg;
    p.out_f32 = a.out_f32; p.f32_cols = a.f32_cols; p.ld_f32 = a.ld_f32;
    p.status = a.status;
    p.spin_limit = a.wait_limit ? a.wait_limit - 1 : kSpinLimit;
    const int total = p.m_tiles * p.n_tiles;
    const int grid = total < num_sms ? total : num_sms;
    if (mh == 2 && p.bn == 256)
        tc_gemm_kernel<256, 2><<<grid, kGThreads, kGemmSmemBytes, st>>>(tm_a, tm_b, p);
    else if (mh == 2)
        tc_gemm_kernel<192, 2><<<grid, kGThreads, kGemmSmemBytes, st>>>(tm_a, tm_b, p);
    else if (p.bn == 256)
        tc_gemm_kernel<256, 1><<<grid, kGThreads, kGemmSmemBytes, st>>>(tm_a, tm_b, p);
    else if (p.bn == 192)
        tc_gemm_kernel<192, 1><<<grid, kGThreads, kGemmSmemBytes, st>>>(tm_a, tm_b, p);
    else
        tc_gemm_kernel<128, 1><<<grid, kGThreads, kGemmSmemBytes, st>>>(tm_a, tm_b, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_gemm_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

}  // namespace arl2
