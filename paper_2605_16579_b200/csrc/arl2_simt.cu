// Plain-FMA (CUDA-core) kernels of the ARL^2 layer: the fp32 mode (Q, K, V, O in fp32, all
// arithmetic in fp32) and a slow bf16-I/O variant used for A/B checks of the tensor-core
// path.  Also the small elementwise kernels every path shares: RoPE of K (once per step),
// the deterministic commit reduction with the gated decay, zero fill, fp32 -> bf16 copy.
//
// Step kernel, per (stream b, head h, 64-query tile):   (Eq. 2, 3, 5-8; Algorithm 1)
//   scores over all L keys with an online softmax (running max / sum in fp32, base-2
//   exponent), O_intra accumulated in registers; then U = Q W_phi_q, RoPE, L2Norm,
//   O_inter = Q' S; out = O_intra / l + sigmoid(g) O_inter.  The state is only read.
// Commit kernel, per (b, h, 512-token chunk):              (Eq. 3, Eq. 4 gated-linear form)
//   K' = L2Norm(RoPE(K W_phi_k)), V' = V W_phi_v, partial = K'^T V'; a second kernel adds the
//   partials in a fixed order and applies S <- sigmoid(a) S + sum.
#include <math.h>

#include "arl2_internal.h"

namespace arl2 {

namespace {

constexpr int BM = 64;       // query rows (or tokens) per tile
constexpr int BN = 64;       // keys per tile / contraction chunk
constexpr int PAD = 4;       // floats of padding per smem row (keeps float4 alignment)
constexpr int NT = 256;      // threads: 16 x 16, each a 4 x 4 (or 4 x D/16) micro-tile

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f(float& d, float x) { d = x; }
__device__ __forceinline__ void from_f(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

__device__ __forceinline__ float sigmoidf_(float x) { return 1.0f / (1.0f + __expf(-x)); }

// acc[i][c*4+e] += sum_kk A[(ty*4+i)*lda + kk] * Bm[kk*D + c*64 + tx*4 + e], kk < 64.
// A: 64 x 64 slice of a row-major smem matrix; Bm: 64 x D smem tile.
template <int D>
__device__ __forceinline__ void tile_gemm(float (&acc)[4][D / 16], const float* __restrict__ A,
                                          int lda, const float* __restrict__ Bm, int tx, int ty)
{
#pragma unroll 4
    for (int k4 = 0; k4 < BN / 4; ++k4) {
        float4 a[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            a[i] = *reinterpret_cast<const float4*>(A + (ty * 4 + i) * lda + k4 * 4);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                float4 b = *reinterpret_cast<const float4*>(Bm + (k4 * 4 + kk) * D + c * 64 + tx * 4);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float av = kk == 0 ? a[i].x : kk == 1 ? a[i].y : kk == 2 ? a[i].z : a[i].w;
                    acc[i][c * 4 + 0] += av * b.x;
                    acc[i][c * 4 + 1] += av * b.y;
                    acc[i][c * 4 + 2] += av * b.z;
                    acc[i][c * 4 + 3] += av * b.w;
                }
            }
        }
    }
}

// Load rows [r0, r0+64) x cols [c0, c0+ncols) of a [B, L, H, D] tensor (head h, stream b) into
// a row-major smem matrix dst[r*ld + c]; rows at or past `row_end` are zero.
template <typename T>
__device__ __forceinline__ void load_rows(float* dst, int ld, const T* __restrict__ src, int b,
                                          int h, int r0, int c0, int ncols, int row_end, int L,
                                          int H, int D, int tid)
{
    for (int idx = tid; idx < BM * ncols; idx += NT) {
        int r = idx / ncols, c = idx % ncols;
        int row = r0 + r;
        float x = 0.0f;
        if (row < row_end) x = to_f(src[(((size_t)b * L + row) * H + h) * D + c0 + c]);
        dst[r * ld + c] = x;
    }
}

// Load 64 rows [k0, k0+64) of a row-major [D, D] matrix (fp32 state or a feature map) into
// smem tile dst[kk*D + n].
template <typename T>
__device__ __forceinline__ void load_mat_rows(float* dst, const T* __restrict__ M, int k0, int D,
                                              int tid)
{
    for (int idx = tid; idx < BN * D; idx += NT) dst[idx] = to_f(M[(size_t)k0 * D + idx]);
}

// Rotate the thread's micro-tile (rows ty*4+i, columns c*64 + tx*4 + e) by the rotary tables
// and scale each row to unit L2 norm.  Rows are shared by the 16 lanes with the same ty.
template <int D>
__device__ __forceinline__ void rope_l2norm(float (&u)[4][D / 16], int row0, int L, int tx,
                                            const float* __restrict__ cos_t,
                                            const float* __restrict__ sin_t, float eps,
                                            bool normalise)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int row = row0 + i;
        if (cos_t != nullptr && row < L) {
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                int m = (c * 64 + tx * 4) / 2;
                float2 cs = *reinterpret_cast<const float2*>(cos_t + (size_t)row * (D / 2) + m);
                float2 sn = *reinterpret_cast<const float2*>(sin_t + (size_t)row * (D / 2) + m);
                float x0 = u[i][c * 4 + 0], x1 = u[i][c * 4 + 1];
                u[i][c * 4 + 0] = x0 * cs.x - x1 * sn.x;
                u[i][c * 4 + 1] = x0 * sn.x + x1 * cs.x;
                x0 = u[i][c * 4 + 2];
                x1 = u[i][c * 4 + 3];
                u[i][c * 4 + 2] = x0 * cs.y - x1 * sn.y;
                u[i][c * 4 + 3] = x0 * sn.y + x1 * cs.y;
            }
        }
        if (normalise) {
            float ss = 0.0f;
#pragma unroll
            for (int e = 0; e < D / 16; ++e) ss += u[i][e] * u[i][e];
#pragma unroll
            for (int off = 8; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            float rn = 1.0f / sqrtf(ss + eps);
#pragma unroll
            for (int e = 0; e < D / 16; ++e) u[i][e] *= rn;
        }
    }
}

// y = L2Norm(RoPE(x W)) (normalise) or y = x W, for the 64-token tile held row-major in
// `xs` (ld = D + PAD); result written back over `xs`.  `ws` is a 64 x D staging tile.
template <int D, typename T>
__device__ __forceinline__ void feature_tile(float* xs, float* ws, const T* __restrict__ W,
                                             int row_glob0, int L, const float* cos_t,
                                             const float* sin_t, float eps, bool normalise,
                                             int tx, int ty, int tid)
{
    constexpr int LD = D + PAD;
    float u[4][D / 16];
    if (W != nullptr) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < D / 16; ++e) u[i][e] = 0.0f;
        for (int c = 0; c < D / BN; ++c) {
            __syncthreads();
            load_mat_rows(ws, W, c * BN, D, tid);
            __syncthreads();
            tile_gemm<D>(u, xs + c * BN, LD, ws, tx, ty);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                float4 x = *reinterpret_cast<const float4*>(xs + (ty * 4 + i) * LD + c * 64 + tx * 4);
                u[i][c * 4 + 0] = x.x; u[i][c * 4 + 1] = x.y;
                u[i][c * 4 + 2] = x.z; u[i][c * 4 + 3] = x.w;
            }
    }
    rope_l2norm<D>(u, row_glob0 + ty * 4, L, tx, normalise ? cos_t : nullptr, sin_t, eps, normalise);
    __syncthreads();  // every read of xs as the GEMM's A operand is done
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < D / 64; ++c)
            *reinterpret_cast<float4*>(xs + (ty * 4 + i) * LD + c * 64 + tx * 4) =
                make_float4(u[i][c * 4 + 0], u[i][c * 4 + 1], u[i][c * 4 + 2], u[i][c * 4 + 3]);
    __syncthreads();
}

template <int D, typename T>
__global__ void __launch_bounds__(NT) simt_step_kernel(StepArgs a)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int LD = D + PAD;       // row-major [64][D] matrices
    constexpr int LT = BM + PAD;      // transposed [D][64] matrices
    float* Qt = smem;                 // [D][LT]  rotated Q, transposed; later [64][LD] raw Q / Q'
    float* Kt = Qt + D * LT;          // [D][LT]  rotated K tile, transposed
    float* Vs = Kt + D * LT;          // [64][D]  V tile; later rows of W_phi_q / S
    float* Ps = Vs + BN * D;          // [64][LT] probabilities
    static_assert(D * LT >= BM * LD, "the Q buffer is reused with both layouts");

    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int L = a.s.L, H = a.s.H;
    const int i0 = blockIdx.x * BM, h = blockIdx.y, b = blockIdx.z;
    const T* q = static_cast<const T*>(a.q);
    const T* k = static_cast<const T*>(a.k_rot);
    const T* v = static_cast<const T*>(a.v);

    // rotated Q tile, transposed so that the score loop reads float4 along the rows
    for (int idx = tid; idx < BM * (D / 2); idx += NT) {
        int r = idx / (D / 2), m = idx % (D / 2);
        int row = i0 + r;
        float x0 = 0.0f, x1 = 0.0f;
        if (row < L) {
            const T* p = q + (((size_t)b * L + row) * H + h) * D + 2 * m;
            x0 = to_f(p[0]);
            x1 = to_f(p[1]);
            if (a.rope_cos != nullptr) {
                float c = a.rope_cos[(size_t)row * (D / 2) + m];
                float s = a.rope_sin[(size_t)row * (D / 2) + m];
                float y0 = x0 * c - x1 * s, y1 = x0 * s + x1 * c;
                // the bf16 path rounds rotated operands to bf16; mirror it so that the two
                // kernel families see the same scores
                if (sizeof(T) == 2) {
                    y0 = __bfloat162float(__float2bfloat16_rn(y0));
                    y1 = __bfloat162float(__float2bfloat16_rn(y1));
                }
                x0 = y0;
                x1 = y1;
            }
        }
        Qt[(2 * m) * LT + r] = x0;
        Qt[(2 * m + 1) * LT + r] = x1;
    }

    float o[4][D / 16];
    float mrun[4], lrun[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        mrun[i] = -INFINITY;
        lrun[i] = 0.0f;
#pragma unroll
        for (int e = 0; e < D / 16; ++e) o[i][e] = 0.0f;
    }

    for (int j0 = 0; j0 < L; j0 += BN) {
        __syncthreads();  // previous tile fully consumed (and Qt written, first time)
        for (int idx = tid; idx < BN * D; idx += NT) {
            int r = idx / D, d = idx % D;
            int row = j0 + r;
            float kv = 0.0f, vv = 0.0f;
            if (row < L) {
                size_t off = (((size_t)b * L + row) * H + h) * D + d;
                kv = to_f(k[off]);
                vv = to_f(v[off]);
            }
            Kt[d * LT + r] = kv;
            Vs[r * D + d] = vv;
        }
        __syncthreads();

        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.0f;
#pragma unroll 8
        for (int d = 0; d < D; ++d) {
            float4 qa = *reinterpret_cast<const float4*>(Qt + d * LT + ty * 4);
            float4 kb = *reinterpret_cast<const float4*>(Kt + d * LT + tx * 4);
            float qv[4] = {qa.x, qa.y, qa.z, qa.w};
            float kv[4] = {kb.x, kb.y, kb.z, kb.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[i][j] += qv[i] * kv[j];
        }

        // online softmax in base 2; keys past L are masked out
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[i][j] = (j0 + tx * 4 + j < L) ? s[i][j] * a.s.scale_log2 : -INFINITY;
                mx = fmaxf(mx, s[i][j]);
            }
#pragma unroll
            for (int off = 8; off >= 1; off >>= 1)
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            float mnew = fmaxf(mrun[i], mx);   // finite: every tile has at least one valid key
            float corr = exp2f(mrun[i] - mnew);
            float sum = 0.0f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[i][j] = exp2f(s[i][j] - mnew);
                sum += s[i][j];
            }
#pragma unroll
            for (int off = 8; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            lrun[i] = lrun[i] * corr + sum;
            mrun[i] = mnew;
#pragma unroll
            for (int e = 0; e < D / 16; ++e) o[i][e] *= corr;
            *reinterpret_cast<float4*>(Ps + (ty * 4 + i) * LT + tx * 4) =
                make_float4(s[i][0], s[i][1], s[i][2], s[i][3]);
        }
        __syncthreads();
        tile_gemm<D>(o, Ps, LT, Vs, tx, ty);
    }
    __syncthreads();

    // inter branch: raw Q tile -> Q' = L2Norm(RoPE(Q W_phi_q)) -> Q' S
    float* Qp = Qt;  // [64][LD]
    load_rows<T>(Qp, LD, q, b, h, i0, 0, D, L, L, H, D, tid);
    __syncthreads();
    feature_tile<D, T>(Qp, Vs, a.wq ? static_cast<const T*>(a.wq) + (size_t)h * D * D : nullptr,
                       i0, L, a.rope_cos, a.rope_sin, a.s.eps, true, tx, ty, tid);

    float x[4][D / 16];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int e = 0; e < D / 16; ++e) x[i][e] = 0.0f;
    const float* Sh = a.state + ((size_t)b * H + h) * D * D;
    for (int c = 0; c < D / BN; ++c) {
        __syncthreads();
        load_mat_rows<float>(Vs, Sh, c * BN, D, tid);
        __syncthreads();
        tile_gemm<D>(x, Qp + c * BN, LD, Vs, tx, ty);
    }

    T* out = static_cast<T*>(a.out);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int row = i0 + ty * 4 + i;
        if (row >= L) continue;
        // combine gate: one per (token, head), one per token, or one per output channel
        const size_t rh = ((size_t)b * L + row) * H + h;
        float gate = a.gate_mode == 2 ? 0.0f : sigmoidf_(a.gate[a.gate_mode == 1 ? (size_t)b * L + row : rh]);
        float inv = 1.0f / lrun[i];
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
            T* p = out + rh * D + c * 64 + tx * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (a.gate_mode == 2) gate = sigmoidf_(a.gate[rh * D + c * 64 + tx * 4 + e]);
                from_f(p[e], o[i][c * 4 + e] * inv + gate * x[i][c * 4 + e]);
            }
        }
    }
}

// partial[b, h, split] = K'^T V' over tokens [split*chunk, min(L, (split+1)*chunk)).
template <int D, typename T>
__global__ void __launch_bounds__(NT) simt_commit_partial_kernel(CommitArgs a)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int LD = D + PAD;
    float* Ks = smem;             // [64][LD]  K tile -> K'
    float* Vs2 = Ks + BM * LD;    // [64][LD]  V tile -> V'
    float* Ws = Vs2 + BM * LD;    // [64][D]   rows of a feature map

    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int L = a.s.L, H = a.s.H;
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int l0 = split * kCommitChunk, l1 = min(L, l0 + kCommitChunk);
    const T* kc = static_cast<const T*>(a.k);
    const T* vc = static_cast<const T*>(a.v);
    const T* wk = a.wk ? static_cast<const T*>(a.wk) + (size_t)h * D * D : nullptr;
    const T* wv = a.wv ? static_cast<const T*>(a.wv) + (size_t)h * D * D : nullptr;

    // thread micro-tile of the D x D partial: rows ty*4 + 64*ci + i, cols tx*4 + 64*cj + e
    float acc[D / 16][D / 16];
#pragma unroll
    for (int i = 0; i < D / 16; ++i)
#pragma unroll
        for (int j = 0; j < D / 16; ++j) acc[i][j] = 0.0f;

    for (int r0 = l0; r0 < l1; r0 += BM) {
        __syncthreads();
        // rows past l1 belong to the next chunk (or do not exist): zero them
        const int lim = l1;
        load_rows<T>(Ks, LD, kc, b, h, r0, 0, D, lim, L, H, D, tid);
        load_rows<T>(Vs2, LD, vc, b, h, r0, 0, D, lim, L, H, D, tid);
        __syncthreads();
        feature_tile<D, T>(Ks, Ws, wk, r0, lim, a.rope_cos, a.rope_sin, a.s.eps, true, tx, ty, tid);
        feature_tile<D, T>(Vs2, Ws, wv, r0, lim, nullptr, nullptr, a.s.eps, false, tx, ty, tid);
        if (a.mode == 2) {
            // per-token decay weights: the value rows are scaled by w_l = prod_{i>l} alpha_i
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = r0 + ty * 4 + i;
                const float wgt = (a.beta != nullptr && row < lim) ? a.beta[((size_t)b * L + row) * H + h]
                                                                   : (row < lim ? 1.0f : 0.0f);
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    float4* pv = reinterpret_cast<float4*>(Vs2 + (ty * 4 + i) * LD + c * 64 + tx * 4);
                    float4 v = *pv;
                    v.x *= wgt; v.y *= wgt; v.z *= wgt; v.w *= wgt;
                    *pv = v;
                }
            }
            __syncthreads();
        }
        if (a.mode == 1) {
            // Eq. 4 as printed: the value rows become beta (V' - K' S_old); S_old is the state as
            // it stands (the reduce kernel, a later launch, is the only writer)
            float x[4][D / 16];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < D / 16; ++e) x[i][e] = 0.0f;
            const float* Sh = a.state + ((size_t)b * H + h) * D * D;
            for (int c = 0; c < D / BN; ++c) {
                __syncthreads();
                load_mat_rows<float>(Ws, Sh, c * BN, D, tid);
                __syncthreads();
                tile_gemm<D>(x, Ks + c * BN, LD, Ws, tx, ty);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = r0 + ty * 4 + i;
                float beta = 1.0f;
                if (a.beta != nullptr)
                    beta = row < lim ? sigmoidf_(a.beta[((size_t)b * L + row) * H + h]) : 0.0f;
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    float4* pv = reinterpret_cast<float4*>(Vs2 + (ty * 4 + i) * LD + c * 64 + tx * 4);
                    float4 v = *pv;   // this thread is the only one to touch these four values
                    v.x = beta * (v.x - x[i][c * 4 + 0]);
                    v.y = beta * (v.y - x[i][c * 4 + 1]);
                    v.z = beta * (v.z - x[i][c * 4 + 2]);
                    v.w = beta * (v.w - x[i][c * 4 + 3]);
                    *pv = v;
                }
            }
            __syncthreads();
        }
#pragma unroll 2
        for (int r = 0; r < BM; ++r) {
            float ka[D / 16], vb[D / 16];
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                float4 t = *reinterpret_cast<const float4*>(Ks + r * LD + c * 64 + ty * 4);
                ka[c * 4 + 0] = t.x; ka[c * 4 + 1] = t.y; ka[c * 4 + 2] = t.z; ka[c * 4 + 3] = t.w;
                float4 u = *reinterpret_cast<const float4*>(Vs2 + r * LD + c * 64 + tx * 4);
                vb[c * 4 + 0] = u.x; vb[c * 4 + 1] = u.y; vb[c * 4 + 2] = u.z; vb[c * 4 + 3] = u.w;
            }
#pragma unroll
            for (int i = 0; i < D / 16; ++i)
#pragma unroll
                for (int j = 0; j < D / 16; ++j) acc[i][j] += ka[i] * vb[j];
        }
    }

    float* dst = a.partials + (((size_t)b * H + h) * a.nsplit + split) * D * D;
#pragma unroll
    for (int i = 0; i < D / 16; ++i) {
        int d = (i / 4) * 64 + ty * 4 + (i % 4);
#pragma unroll
        for (int cj = 0; cj < D / 64; ++cj)
            *reinterpret_cast<float4*>(dst + (size_t)d * D + cj * 64 + tx * 4) =
                make_float4(acc[i][cj * 4 + 0], acc[i][cj * 4 + 1], acc[i][cj * 4 + 2],
                            acc[i][cj * 4 + 3]);
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 4 token by token with per-token gates, in chunkwise form.  For the tokens j = 0..C-1 of a
// chunk (C = 64) entering with state S_0, write g_j = alpha_0 ... alpha_j (g_{-1} = 1) and
// u_j = beta_j (V'_j - K'_j S_{j-1}).  Unrolling S_j = alpha_j S_{j-1} + K'_j^T u_j gives
//   (I + A) U = diag(beta) V' - diag(beta g_{j-1}) K' S_0,
//   A_ji = beta_j (g_{j-1} / g_i) <K'_j, K'_i> for i < j (strictly lower triangular),
//   S_C = g_{C-1} S_0 + Khat^T U,   Khat_i = (g_{C-1} / g_i) K'_i.
// With T = (I + A)^-1:  U = U1 - W S_0,  U1 = T diag(beta) V',  W = T diag(beta g_{j-1}) K'.
// Every ratio of g's is a product of alphas, so at most 1.  token_prepare_kernel computes W, U1,
// Khat and g_{C-1} for every chunk in parallel; token_scan_kernel then walks the chunks in
// order, each CTA owning 16 columns of one head's state (columns never mix).
// ---------------------------------------------------------------------------------------------
constexpr int kTokChunk = kTokenChunk;
constexpr int LA = kTokChunk + 4;   // row stride of the C x C matrices

template <int D, typename T>
__global__ void __launch_bounds__(NT) token_prepare_kernel(TokenCommitArgs a)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int LD = D + PAD;
    float* Ks = smem;                       // [64][LD]  K tile -> K'
    float* Vs2 = Ks + BM * LD;              // [64][LD]  V tile -> V'
    float* Ws = Vs2 + BM * LD;              // [64][D]   feature-map rows, then scaled K' / V'
    float* As = Ws + BN * D;                // [64][LA]  A
    float* Ts = As + kTokChunk * LA;        // [64][LA]  T = (I + A)^-1
    float* cl = Ts + kTokChunk * LA;        // [65]      cl[j+1] = log g_j, cl[0] = 0
    float* bet = cl + kTokChunk + 4;        // [64]      beta_j
    float* lg = bet + kTokChunk;            // [64]      log alpha_j

    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int L = a.s.L, H = a.s.H;
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int r0 = chunk * kTokChunk;
    const T* kc = static_cast<const T*>(a.k);
    const T* vc = static_cast<const T*>(a.v);
    const T* wk = a.wk ? static_cast<const T*>(a.wk) + (size_t)h * D * D : nullptr;
    const T* wv = a.wv ? static_cast<const T*>(a.wv) + (size_t)h * D * D : nullptr;

    const int dec = a.decayed ? 1 : 0;
    load_rows<T>(Ks, LD, kc, b, h, r0, 0, D, L, L, H, D, tid);
    load_rows<T>(Vs2, LD, vc, b, h, r0, 0, D, L, L, H, D, tid);
    if (tid < kTokChunk) {
        // tokens past L: alpha = 1, beta = 0 -- they change nothing
        const int row = r0 + tid;
        float la = 0.0f, be = 0.0f;
        if (row < L) {
            const size_t gi = ((size_t)b * L + row) * H + h;
            if (a.alpha != nullptr) {
                const float x = a.alpha[gi];   // log sigmoid(x) = -log(1 + e^-x), stable on both sides
                la = x >= 0.0f ? -log1pf(expf(-x)) : x - log1pf(expf(x));
            }
            be = a.beta != nullptr ? 1.0f / (1.0f + expf(-a.beta[gi])) : 1.0f;
        }
        lg[tid] = la;
        bet[tid] = be;
    }
    __syncthreads();
    if (tid == 0) {
        float run = 0.0f;
        cl[0] = 0.0f;
        for (int j = 0; j < kTokChunk; ++j) {
            run += lg[j];
            cl[j + 1] = run;
        }
    }
    feature_tile<D, T>(Ks, Ws, wk, r0, L, a.rope_cos, a.rope_sin, a.s.eps, true, tx, ty, tid);
    feature_tile<D, T>(Vs2, Ws, wv, r0, L, nullptr, nullptr, a.s.eps, false, tx, ty, tid);

    // A: Gram matrix of the K' rows, masked and weighted
    {
        float g[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) g[i][e] = 0.0f;
        for (int d4 = 0; d4 < D / 4; ++d4) {
            float4 ar[4], bc[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                ar[i] = *reinterpret_cast<const float4*>(Ks + (ty * 4 + i) * LD + d4 * 4);
                bc[i] = *reinterpret_cast<const float4*>(Ks + (tx * 4 + i) * LD + d4 * 4);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    g[i][e] += ar[i].x * bc[e].x + ar[i].y * bc[e].y + ar[i].z * bc[e].z + ar[i].w * bc[e].w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int row = ty * 4 + i, col = tx * 4 + e;
                // g_{j-1} / g_i as printed; g_j / g_i when the prediction is made against the decayed state
                As[row * LA + col] = col < row ? bet[row] * expf(cl[row + dec] - cl[col + 1]) * g[i][e] : 0.0f;
            }
    }
    __syncthreads();
    // T = (I + A)^-1 by forward substitution: thread c owns column c
    if (tid < kTokChunk) {
        float t[kTokChunk];
#pragma unroll
        for (int j = 0; j < kTokChunk; ++j) {
            float acc = j == tid ? 1.0f : 0.0f;
#pragma unroll
            for (int i = 0; i < j; ++i) acc -= As[j * LA + i] * t[i];
            t[j] = acc;
            Ts[j * LA + tid] = acc;
        }
    }
    __syncthreads();

    const size_t rows_pad = (size_t)a.nchunk * kTokChunk;
    const size_t base = (((size_t)b * H + h) * rows_pad + r0) * D;
    // W = T diag(beta g_{j-1}) K', then U1 = T diag(beta) V'
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        const float* src = pass == 0 ? Ks : Vs2;
        for (int idx = tid; idx < kTokChunk * D; idx += NT) {
            const int j = idx / D, d = idx % D;
            const float sc = pass == 0 ? bet[j] * expf(cl[j + dec]) : bet[j];
            Ws[idx] = src[j * LD + d] * sc;
        }
        __syncthreads();
        float acc[4][D / 16];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < D / 16; ++e) acc[i][e] = 0.0f;
        tile_gemm<D>(acc, Ts, LA, Ws, tx, ty);
        float* dst = (pass == 0 ? a.w : a.u1) + base;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < D / 64; ++c)
                *reinterpret_cast<float4*>(dst + (size_t)(ty * 4 + i) * D + c * 64 + tx * 4) =
                    make_float4(acc[i][c * 4 + 0], acc[i][c * 4 + 1], acc[i][c * 4 + 2], acc[i][c * 4 + 3]);
        __syncthreads();
    }
    // Khat = diag(g_{C-1} / g_j) K'
    for (int idx = tid; idx < kTokChunk * D; idx += NT) {
        const int j = idx / D, d = idx % D;
        a.kh[base + idx] = Ks[j * LD + d] * expf(cl[kTokChunk] - cl[j + 1]);
    }
    if (tid == 0) a.gc[((size_t)b * H + h) * a.nchunk + chunk] = expf(cl[kTokChunk]);
}

// The sequential pass: S <- g S + Khat^T (U1 - W S) chunk after chunk, for kScanCols columns of
// the state of one (stream, head).  Reads and writes the fp32 state in place and refreshes the
// bf16 operand copy when one is kept.  The W tile of the next chunk is fetched (cp.async) while
// the state update of this chunk runs, the Khat tile while the next U is formed.
__device__ __forceinline__ void cp_async16(float* dst_smem, const float* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int D, int kScanCols>
__global__ void __launch_bounds__(NT) token_scan_kernel(TokenCommitArgs a)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int LD = D + PAD;
    constexpr int CG = kScanCols / 4;           // float4 column groups
    constexpr int RPT = kTokChunk * CG / NT;    // U rows per thread: 1 (16 columns) or 2 (32)
    constexpr int CP = D * kScanCols / NT;      // state columns per thread in the update
    constexpr int TPR = kScanCols / CP;         // threads per state row
    static_assert(RPT >= 1 && CP % 4 == 0 && TPR >= 1, "thread mapping");
    float* Wt = smem;                           // [64][LD]
    float* Kt = Wt + kTokChunk * LD;            // [64][LD]
    float* U1t = Kt + kTokChunk * LD;           // [64][kScanCols]
    float* Ut = U1t + kTokChunk * kScanCols;    // [64][kScanCols]
    float* Ss = Ut + kTokChunk * kScanCols;     // [D][kScanCols]

    const int tid = threadIdx.x;
    const int H = a.s.H;
    const int e0 = blockIdx.x * kScanCols, h = blockIdx.y, b = blockIdx.z;
    const size_t bh = (size_t)b * H + h;
    float* Sg = a.state + bh * D * D;
    const size_t rows_pad = (size_t)a.nchunk * kTokChunk;
    const float* wbase = a.w + bh * rows_pad * D;
    const float* kbase = a.kh + bh * rows_pad * D;
    const float* ubase = a.u1 + bh * rows_pad * D;

    auto fetch_tile = [&](float* dst, const float* src) {   // 64 x D floats, row stride LD in smem
        for (int idx = tid; idx < kTokChunk * D / 4; idx += NT) {
            const int j = idx / (D / 4), d4 = idx % (D / 4);
            cp_async16(dst + j * LD + d4 * 4, src + (size_t)j * D + d4 * 4);
        }
    };
    auto fetch_u1 = [&](const float* src) {                 // 64 x kScanCols floats
        for (int idx = tid; idx < kTokChunk * CG; idx += NT) {
            const int j = idx / CG, q = idx % CG;
            cp_async16(U1t + j * kScanCols + q * 4, src + (size_t)j * D + e0 + q * 4);
        }
    };

    // group order per chunk: {W, U1} then {Khat}
    fetch_tile(Wt, wbase);
    fetch_u1(ubase);
    cp_async_commit();
    fetch_tile(Kt, kbase);
    cp_async_commit();
    for (int idx = tid; idx < D * kScanCols; idx += NT)
        Ss[idx] = Sg[(size_t)(idx / kScanCols) * D + e0 + idx % kScanCols];

    const int cg = tid % CG, r_first = tid / CG;            // U phase: rows r_first + k * (NT / CG)
    const int sd = tid / TPR, sc = (tid % TPR) * CP;        // update phase: state row sd, columns sc ..
    for (int chunk = 0; chunk < a.nchunk; ++chunk) {
        const float g = a.gc[bh * a.nchunk + chunk];
        cp_async_wait<1>();     // W and U1 of this chunk have landed (Khat may still be in flight)
        __syncthreads();        // ... for every thread; the previous update's writes of Ss are visible

        // U = U1 - W S
#pragma unroll
        for (int k = 0; k < RPT; ++k) {
            const int r = r_first + k * (NT / CG);
            float4 u = *reinterpret_cast<const float4*>(U1t + r * kScanCols + cg * 4);
#pragma unroll 4
            for (int d4 = 0; d4 < D / 4; ++d4) {
                const float4 w = *reinterpret_cast<const float4*>(Wt + r * LD + d4 * 4);
                const float wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int dd = 0; dd < 4; ++dd) {
                    const float4 s4 = *reinterpret_cast<const float4*>(Ss + (d4 * 4 + dd) * kScanCols + cg * 4);
                    u.x -= wv[dd] * s4.x;
                    u.y -= wv[dd] * s4.y;
                    u.z -= wv[dd] * s4.z;
                    u.w -= wv[dd] * s4.w;
                }
            }
            *reinterpret_cast<float4*>(Ut + r * kScanCols + cg * 4) = u;
        }
        cp_async_wait<0>();     // Khat of this chunk
        __syncthreads();        // U complete; nobody reads W, U1 or (others' rows of) Ss any more
        if (chunk + 1 < a.nchunk) {
            fetch_tile(Wt, wbase + (size_t)(chunk + 1) * kTokChunk * D);
            fetch_u1(ubase + (size_t)(chunk + 1) * kTokChunk * D);
        }
        cp_async_commit();

        // S <- g S + Khat^T U   (this thread's CP elements of row sd)
        float s[CP];
#pragma unroll
        for (int e = 0; e < CP; ++e) s[e] = g * Ss[sd * kScanCols + sc + e];
#pragma unroll 4
        for (int i = 0; i < kTokChunk; ++i) {
            const float kv = Kt[i * LD + sd];
#pragma unroll
            for (int e4 = 0; e4 < CP / 4; ++e4) {
                const float4 uu = *reinterpret_cast<const float4*>(Ut + i * kScanCols + sc + e4 * 4);
                s[e4 * 4 + 0] += kv * uu.x;
                s[e4 * 4 + 1] += kv * uu.y;
                s[e4 * 4 + 2] += kv * uu.z;
                s[e4 * 4 + 3] += kv * uu.w;
            }
        }
#pragma unroll
        for (int e = 0; e < CP; ++e) Ss[sd * kScanCols + sc + e] = s[e];
        __syncthreads();        // every thread is done with Khat and U
        if (chunk + 1 < a.nchunk) fetch_tile(Kt, kbase + (size_t)(chunk + 1) * kTokChunk * D);
        cp_async_commit();
    }
    cp_async_wait<0>();
    __syncthreads();
    for (int idx = tid; idx < D * kScanCols; idx += NT) {
        const size_t at = (size_t)(idx / kScanCols) * D + e0 + idx % kScanCols;
        Sg[at] = Ss[idx];
        if (a.state_bf16 != nullptr) a.state_bf16[bh * D * D + at] = __float2bfloat16_rn(Ss[idx]);
    }
}

}  // namespace

// S[b,h] <- sigmoid(a[b,h]) S[b,h] + sum_split partial[b,h,split], splits added in index
// order so that the result does not depend on scheduling.  Also refreshes the bf16 operand
// copy of S when one is kept.  One thread per 4 state elements.
__global__ void commit_reduce_kernel(float* __restrict__ state, const float* __restrict__ partials,
                                     const float* __restrict__ decay, int decay_direct,
                                     __nv_bfloat16* __restrict__ state_bf16, int nsplit, int DD,
                                     size_t total4, int run_share, int run_ntile, int nslot,
                                     const uint32_t* __restrict__ status)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total4) return;
    // a partial-sum kernel that gave up on a bounded wait left its slots unwritten: S stays as it was
    if (status != nullptr && status[kStatusError] != 0u) return;
    size_t e = t * 4;
    size_t bh = e / DD;
    size_t within = e % DD;
    float alpha = decay_direct ? decay[bh] : 1.0f / (1.0f + __expf(-decay[bh]));
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    int nparts = nsplit, stride = nsplit;
    if (run_share > 0) {   // the slots are the runs this head's tiles fall into
        const int first = (int)((bh * run_ntile) / run_share);
        const int last = (int)((bh * run_ntile + run_ntile - 1) / run_share);
        nparts = last - first + 1;
        stride = nslot;
    }
    const float* p = partials + bh * (size_t)stride * DD + within;
    for (int s = 0; s < nparts; ++s) {
        float4 x = *reinterpret_cast<const float4*>(p + (size_t)s * DD);
        sum.x += x.x; sum.y += x.y; sum.z += x.z; sum.w += x.w;
    }
    float4 old = *reinterpret_cast<const float4*>(state + e);
    float4 nw = make_float4(alpha * old.x + sum.x, alpha * old.y + sum.y, alpha * old.z + sum.z,
                            alpha * old.w + sum.w);
    *reinterpret_cast<float4*>(state + e) = nw;
    if (state_bf16 != nullptr) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(nw.x, nw.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(nw.z, nw.w);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo);
        packed.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(state_bf16 + e) = packed;
    }
}

namespace {

// k_rot = RoPE(k), 8 elements per thread, output in the input's dtype.
template <typename T>
__global__ void rope_k_kernel(const T* __restrict__ k, const float* __restrict__ cos_t,
                              const float* __restrict__ sin_t, T* __restrict__ out, int L, int H,
                              int D, size_t total8)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total8) return;
    size_t e = t * 8;
    int d = (int)(e % D);
    int l = (int)((e / ((size_t)D * H)) % L);
    const float* c = cos_t + (size_t)l * (D / 2) + d / 2;
    const float* s = sin_t + (size_t)l * (D / 2) + d / 2;
    float4 cv = *reinterpret_cast<const float4*>(c);
    float4 sv = *reinterpret_cast<const float4*>(s);
    float cc[4] = {cv.x, cv.y, cv.z, cv.w}, ss[4] = {sv.x, sv.y, sv.z, sv.w};
    __align__(16) T in[8];
    __align__(16) T o[8];
    if (sizeof(T) == 2) {
        *reinterpret_cast<uint4*>(in) = *reinterpret_cast<const uint4*>(k + e);
    } else {
        *reinterpret_cast<float4*>(in) = *reinterpret_cast<const float4*>(k + e);
        *reinterpret_cast<float4*>(in + 4) = *reinterpret_cast<const float4*>(k + e + 4);
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        float x0 = to_f(in[2 * m]), x1 = to_f(in[2 * m + 1]);
        from_f(o[2 * m], x0 * cc[m] - x1 * ss[m]);
        from_f(o[2 * m + 1], x0 * ss[m] + x1 * cc[m]);
    }
    if (sizeof(T) == 2) {
        *reinterpret_cast<uint4*>(out + e) = *reinterpret_cast<uint4*>(o);
    } else {
        *reinterpret_cast<float4*>(out + e) = *reinterpret_cast<float4*>(o);
        *reinterpret_cast<float4*>(out + e + 4) = *reinterpret_cast<float4*>(o + 4);
    }
}

__global__ void fill_zero_kernel(uint4* __restrict__ p, size_t n16)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n16) p[t] = make_uint4(0, 0, 0, 0);
}

__global__ void state_to_bf16_kernel(const float* __restrict__ s, __nv_bfloat16* __restrict__ d,
                                     size_t n4)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n4) return;
    float4 x = *reinterpret_cast<const float4*>(s + t * 4);
    __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(x.z, x.w);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(d + t * 4) = packed;
}

template <typename K>
int set_smem(K kernel, size_t bytes)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)bytes);
    if (e != cudaSuccess) {
        set_error("cudaFuncSetAttribute(%zu bytes of shared memory): %s", bytes,
                  cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    return 0;
}

int check_launch(const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("launch of %s failed: %s", what, cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    return 0;
}

template <int D, typename T>
int launch_step(const StepArgs& a, cudaStream_t st)
{
    size_t smem = sizeof(float) * (2 * D * (BM + PAD) + BN * D + BM * (BM + PAD));
    if (int r = set_smem(simt_step_kernel<D, T>, smem)) return r;
    dim3 grid((a.s.L + BM - 1) / BM, a.s.H, a.s.B);
    simt_step_kernel<D, T><<<grid, NT, smem, st>>>(a);
    if (int r = check_launch("simt_step_kernel")) return r;
    return 1;
}

template <int D, typename T>
int launch_commit(const CommitArgs& a, cudaStream_t st)
{
    size_t smem = sizeof(float) * (2 * BM * (D + PAD) + BN * D);
    if (int r = set_smem(simt_commit_partial_kernel<D, T>, smem)) return r;
    dim3 grid(a.nsplit, a.s.H, a.s.B);
    simt_commit_partial_kernel<D, T><<<grid, NT, smem, st>>>(a);
    if (int r = check_launch("simt_commit_partial_kernel")) return r;
    return 1;
}

}  // namespace

// Suffix products of the per-token forget gates of one (stream, head), in log space.  The block
// (1024 threads) walks the tokens from the end of the sequence in tiles of 1024 x seg, seg chosen
// by the host so that a block of up to 8192 tokens is a single tile with every thread busy; inside
// a tile every thread owns seg consecutive tokens, the threads' sums are combined by a suffix scan
// (warp shuffles, then the 32 warp totals through shared memory), and `carry` holds the
// log-product of all later tiles.
__global__ void __launch_bounds__(1024) decay_weights_kernel(const float* __restrict__ alpha,
                                                             float* __restrict__ w, float* __restrict__ total,
                                                             int L, int H, int seg)
{
    constexpr int kMaxSeg = 8;
    __shared__ float warp_tot[32];
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const size_t base = (size_t)b * L * H + h;
    const int tile_tokens = 1024 * seg;
    float carry = 0.0f;
    const int ntile = (L + tile_tokens - 1) / tile_tokens;
    for (int tile = ntile - 1; tile >= 0; --tile) {
        const int l0 = tile * tile_tokens + tid * seg;
        float la[kMaxSeg];
        float mine = 0.0f;
        // every load goes out before the first logarithm
#pragma unroll
        for (int i = 0; i < kMaxSeg; ++i)
            la[i] = (i < seg && l0 + i < L) ? alpha[base + (size_t)(l0 + i) * H] : INFINITY;   // past L: alpha = 1
#pragma unroll
        for (int i = 0; i < kMaxSeg; ++i) {
            const float x = la[i];
            const float v = x >= 0.0f ? -log1pf(expf(-x)) : x - log1pf(expf(x));   // log sigmoid(x)
            la[i] = v;
            mine += v;
        }
        // exclusive suffix sum of `mine` over the threads of the block (later threads = later tokens)
        float incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float dn = __shfl_down_sync(0xffffffffu, incl, off);
            if (lane + off < 32) incl += dn;
        }
        if (lane == 0) warp_tot[wid] = incl;
        __syncthreads();
        float later_warps = 0.0f, tile_total = 0.0f;
        for (int q = 31; q >= 0; --q) {
            if (q == wid) later_warps = tile_total;
            tile_total += warp_tot[q];
        }
        float run = carry + later_warps + (incl - mine);   // log-product of every token after mine
#pragma unroll
        for (int i = kMaxSeg - 1; i >= 0; --i) {
            if (i < seg && l0 + i < L) w[base + (size_t)(l0 + i) * H] = expf(run);
            run += la[i];
        }
        carry += tile_total;
        __syncthreads();   // warp_tot is rewritten by the next tile
    }
    if (tid == 0) total[(size_t)b * H + h] = expf(carry);
}

int decay_weights(const Shape& s, const float* alpha_logits, float* w, float* total, cudaStream_t st)
{
    int seg = (s.L + 1023) / 1024;
    seg = seg < 1 ? 1 : seg > 8 ? 8 : seg;
    decay_weights_kernel<<<dim3(s.H, s.B), 1024, 0, st>>>(alpha_logits, w, total, s.L, s.H, seg);
    if (int r = check_launch("decay_weights_kernel")) return r;
    return 1;
}

int commit_reduce(const CommitArgs& a, cudaStream_t st)
{
    int DD = a.s.D * a.s.D;
    size_t total4 = (size_t)a.s.B * a.s.H * DD / 4;
    commit_reduce_kernel<<<(unsigned)((total4 + 255) / 256), 256, 0, st>>>(
        a.state, a.partials, a.decay, a.decay_direct ? 1 : 0, a.state_bf16, a.nsplit, DD, total4,
        a.run_share, a.run_ntile, a.nslot, a.status);
    if (int r = check_launch("commit_reduce_kernel")) return r;
    return 1;
}

int simt_rope_k(const Shape& s, int dtype, const void* k, const float* cos_t, const float* sin_t,
                void* k_rot, cudaStream_t st)
{
    size_t total8 = (size_t)s.B * s.L * s.H * s.D / 8;
    unsigned blocks = (unsigned)((total8 + 255) / 256);
    if (dtype == ARL2_FP32)
        rope_k_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(k), cos_t, sin_t,
                                                     static_cast<float*>(k_rot), s.L, s.H, s.D, total8);
    else
        rope_k_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(
            static_cast<const __nv_bfloat16*>(k), cos_t, sin_t, static_cast<__nv_bfloat16*>(k_rot),
            s.L, s.H, s.D, total8);
    if (int r = check_launch("rope_k_kernel")) return r;
    return 1;
}

int simt_step(const StepArgs& a, int dtype, cudaStream_t st)
{
    if (a.s.D == 64 && dtype == ARL2_FP32) return launch_step<64, float>(a, st);
    if (a.s.D == 128 && dtype == ARL2_FP32) return launch_step<128, float>(a, st);
    if (a.s.D == 64 && dtype == ARL2_BF16) return launch_step<64, __nv_bfloat16>(a, st);
    if (a.s.D == 128 && dtype == ARL2_BF16) return launch_step<128, __nv_bfloat16>(a, st);
    set_error("no plain-FMA step kernel for D=%d dtype=%d", a.s.D, dtype);
    return ARL2_ERR_UNSUPPORTED;
}

template <int D, typename T>
int launch_commit_tokens(const TokenCommitArgs& a, cudaStream_t st)
{
    size_t smem1 = sizeof(float) * (2 * BM * (D + PAD) + BN * D + 2 * kTokChunk * LA + 3 * kTokChunk + 8);
    if (int r = set_smem(token_prepare_kernel<D, T>, smem1)) return r;
    dim3 grid1(a.nchunk, a.s.H, a.s.B);
    token_prepare_kernel<D, T><<<grid1, NT, smem1, st>>>(a);
    if (int r = check_launch("token_prepare_kernel")) return r;
    constexpr int kScanCols = D / 4;   // 4 CTAs per (stream, head)
    size_t smem2 = sizeof(float) * (2 * kTokChunk * (D + PAD) + 2 * kTokChunk * kScanCols + D * kScanCols);
    if (int r = set_smem(token_scan_kernel<D, kScanCols>, smem2)) return r;
    dim3 grid2(D / kScanCols, a.s.H, a.s.B);
    token_scan_kernel<D, kScanCols><<<grid2, NT, smem2, st>>>(a);
    if (int r = check_launch("token_scan_kernel")) return r;
    return 2;
}

int simt_commit_tokens(const TokenCommitArgs& a, int dtype, cudaStream_t st)
{
    if (a.s.D == 64 && dtype == ARL2_FP32) return launch_commit_tokens<64, float>(a, st);
    if (a.s.D == 128 && dtype == ARL2_FP32) return launch_commit_tokens<128, float>(a, st);
    if (a.s.D == 64 && dtype == ARL2_BF16) return launch_commit_tokens<64, __nv_bfloat16>(a, st);
    if (a.s.D == 128 && dtype == ARL2_BF16) return launch_commit_tokens<128, __nv_bfloat16>(a, st);
    set_error("no token-gate commit kernel for D=%d dtype=%d", a.s.D, dtype);
    return ARL2_ERR_UNSUPPORTED;
}

int simt_commit(const CommitArgs& a, int dtype, cudaStream_t st)
{
    int n;
    if (a.s.D == 64 && dtype == ARL2_FP32) n = launch_commit<64, float>(a, st);
    else if (a.s.D == 128 && dtype == ARL2_FP32) n = launch_commit<128, float>(a, st);
    else if (a.s.D == 64 && dtype == ARL2_BF16) n = launch_commit<64, __nv_bfloat16>(a, st);
    else if (a.s.D == 128 && dtype == ARL2_BF16) n = launch_commit<128, __nv_bfloat16>(a, st);
    else {
        set_error("no plain-FMA commit kernel for D=%d dtype=%d", a.s.D, dtype);
        return ARL2_ERR_UNSUPPORTED;
    }
    if (n < 0) return n;
    int m = commit_reduce(a, st);
    if (m < 0) return m;
    return n + m;
}

int fill_zero(void* p, size_t bytes, cudaStream_t st)
{
    size_t n16 = bytes / 16;  // callers pass multiples of 16 bytes
    if (n16 == 0) return 0;
    fill_zero_kernel<<<(unsigned)((n16 + 255) / 256), 256, 0, st>>>(static_cast<uint4*>(p), n16);
    if (int r = check_launch("fill_zero_kernel")) return r;
    return 1;
}

int state_to_bf16(const float* state, __nv_bfloat16* dst, size_t n, cudaStream_t st)
{
    size_t n4 = n / 4;
    state_to_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(state, dst, n4);
    if (int r = check_launch("state_to_bf16_kernel")) return r;
    return 1;
}

}  // namespace arl2
