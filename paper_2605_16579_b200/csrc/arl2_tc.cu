// Tensor-core (tcgen05 / TMEM / TMA) kernels of the ARL^2 layer for bf16 I/O, D = 128.
//
// Step kernel (Eq. 2, 3, 5-8): persistent, one CTA per SM.  A work item drives two 128-row query
// tiles: two consecutive tiles of one (stream, head), or the ragged last tiles of two different
// (stream, head) units.  Items are handed out by an atomic counter, the pairs first.
//   warps 0-3 / 4-7  softmax group of query tile 0 / 1 (one thread per query row)
//   warp 8           TMA producer and scheduler: the Q tiles, then through a 5-slot ring K_j, V_j
//                    for every key tile, then W_phi_q^T, the raw Q tiles again and the bf16
//                    copy of the state S
//   warp 9 / 10      MMA issuer of tile 0 / 1 (one thread each): S_t = Q~_t K_j^T and
//                    O_t += P_t V_j into TMEM
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1, 128 fp32 columns each; the bf16 probabilities P_t
// overwrite the first 64 columns of S_t and feed the second MMA straight from TMEM.
// RoPE(Q) is applied in place in shared memory by the softmax groups; K arrives rotated.
// The inter branch reuses the loop as one more iteration: "S" = Q W_phi_q (A = the raw Q tile
// from the ring), the group turns each row into sigmoid(g) * l * L2Norm(RoPE(.)) (l = softmax
// row sum) and the "PV" MMA multiplies it by the state, accumulating into O_t, so that the
// final O_t / l is O_intra + sigmoid(g) O_inter.  The state is only read.
//
// Every wait is bounded: when a limit expires the thread records ARL2_ERR_TIMEOUT in the
// device status block, raises the CTA's abort flag and every role falls through to the exit.
#include "tc_common.cuh"

namespace arl2 {

namespace {

constexpr int kStages = 5;
constexpr int kThreads = 384;              // 3 warpgroups: softmax 0, softmax 1, {TMA, MMA, 2 idle}
constexpr int kRegsSoftmax = 232;          // per-thread registers after the warpgroups rebalance
constexpr int kRegsOther = 40;
// setmaxnreg.inc waits (without a bound) for registers of the CTA's own launch allocation
// (threads x the launch register count): the rebalanced total must fit in it
constexpr int kLaunchRegs = (65536 / kThreads) / 8 * 8;
static_assert(256 * kRegsSoftmax + (kThreads - 256) * kRegsOther <= kThreads * kLaunchRegs, "register pool");
constexpr float kRescaleThreshold = 8.0f;   // log2 units of slack before O is rescaled

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;                                 // 2 query tiles (rotated in place)
constexpr int kOffRing = kOffQ + 2 * kTileBytes;         // kStages tiles
constexpr int kOffBars = kOffRing + kStages * kTileBytes;
constexpr int kSmemBytes = kOffBars + 256 + 1024;        // barriers + alignment slack

enum Bar : int {
    kBarQFull = 0,                              // producer -> all: Q tiles (and the item id) landed
    kBarQFree,                                  // MMA -> producer: last MMA reading Q~ is done
    kBarQRot0, kBarQRot1,                       // softmax group t -> MMA: Q~_t rotated
    kBarFull0,                                  // kStages of them
    kBarEmpty0 = kBarFull0 + kStages,           // kStages of them
    kBarSFull0 = kBarEmpty0 + kStages, kBarSFull1,
    kBarPFull0, kBarPFull1,
    kBarOFinal0, kBarOFinal1,
    kBarTok0, kBarTok1,                         // softmax groups take turns in the exponential phase
    kBarDrain0, kBarDrain1,                     // an MMA issuer that gives up waits here for its MMAs in flight
    kNumBars
};
// after the barriers: TMEM base (4 B), abort flag (4 B), two item-id slots (8 B)
static_assert(kNumBars * 8 + 16 <= 256, "barrier block");

struct TcStepParams {
    Shape s;
    const float* gate;
    const float* rope_cos;
    const float* rope_sin;
    const uint4* rope_h;       // half2 (cos, sin) table, warp-interleaved (see pack_rope_kernel), or nullptr
    __nv_bfloat16* out;
    uint32_t* status;
    uint32_t spin_limit;       // polls a bounded wait makes before it gives up
    uint32_t* sched_counter;   // this launch's item counter (zero on entry)
    uint32_t* sched_next;      // the next launch's counter: cleared by this launch
    int gate_mode;             // 0: gate logits [B, L, H]; 1: [B, L] (one per token); 2: [B, L, H, D] (per channel)
    int Lk;                    // keys per head: L, or the length of a key/value cache (Eq. 1)
    int n_q;                   // query tiles per head
    int n_kv;                  // key tiles per head
    int n_pair_items;          // B * H * (n_q / 2): items with two query tiles
    int n_items;               // + ceil(B * H / 2) items of ragged last tiles when n_q is odd
    // Key-range split of the last wave: items [0, n_whole) run whole; item n_whole + s (s = "slot")
    // runs as k_split parts over consecutive ranges of key tiles, scheduled as ids n_whole +
    // s * k_split + part.  Every part leaves its unnormalised rows, reference maxima and row sums in
    // the split buffers; tc_split_merge_kernel then combines the parts of a row in index order.
    int n_whole;
    int k_split;               // 1: nothing is split
    int n_sched;               // ids the scheduler hands out: n_whole + (n_items - n_whole) * k_split
    float* split_o;            // [slot][tile][part][128 rows][128] unnormalised output rows
    float* split_ml;           // [slot][tile][part][128 rows][2] reference maximum (log2 units), row sum
};

// A work item drives up to two 128-row query tiles.  A "pair" item holds two consecutive tiles of
// one (stream, head): they share every K/V tile.  A "ragged" item holds the last, partial tiles
// of two different (stream, head) units (or of one, when the number of units is odd): each tile
// then streams its own K/V, W_phi_q and state through the ring.
struct Item {
    int b[2], h[2], row0[2];
    int ntile;    // active tiles: 1 or 2
    bool shared;  // both tiles read the same K, V, W_phi_q and state
    int j0, nj;   // key tiles [j0, j0 + nj) of the head
    int part;     // -1: the whole key range; else index of this part
    int slot;     // split items only: index among the split items
};

// Items [0, n_pair_items) are pairs of full tiles, (b, h)-major so that neighbours share K and V
// in L2; the rest pack the ragged last tiles two by two.
template <bool kSplit>
__device__ __forceinline__ Item decode_item(int id, const TcStepParams& p)
{
    Item it;
    it.j0 = 0;
    it.nj = p.n_kv;
    it.part = -1;
    it.slot = 0;
    if (kSplit && id >= p.n_whole) {
        const int x = id - p.n_whole;
        it.slot = x / p.k_split;
        it.part = x - it.slot * p.k_split;
        id = p.n_whole + it.slot;
        it.j0 = (it.part * p.n_kv) / p.k_split;
        it.nj = ((it.part + 1) * p.n_kv) / p.k_split - it.j0;
    }
    const int full_pairs = p.n_q >> 1;
    const int units = p.s.B * p.s.H;
    if (id < p.n_pair_items) {
        const int bh = id / full_pairs;
        const int pair = id - bh * full_pairs;
        it.b[0] = it.b[1] = bh / p.s.H;
        it.h[0] = it.h[1] = bh - it.b[0] * p.s.H;
        it.row0[0] = pair * 2 * kTile;
        it.row0[1] = it.row0[0] + kTile;
        it.ntile = 2;
        it.shared = true;
    } else {
        const int u = id - p.n_pair_items;
        it.ntile = (2 * u + 1 < units) ? 2 : 1;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int bh = min(2 * u + t, units - 1);
            it.b[t] = bh / p.s.H;
            it.h[t] = bh - it.b[t] * p.s.H;
            it.row0[t] = full_pairs * 2 * kTile;
        }
        it.shared = false;
    }
    return it;
}

// The ring entries of an item, in the order both MMA issuers walk them.
enum EntryKind : int { kEntK = 0, kEntV, kEntW, kEntQRaw, kEntState };
struct Entry {
    int kind, tile, j;   // j: key tile index for K / V
};
// pair item:   K_0 | V_0 K_1 | V_1 K_2 | ... | V_{n-1} W Qraw_0 Qraw_1 | S
// ragged item: K^0_0 K^1_0 | V^0_0 K^0_1 V^1_0 K^1_1 | ... | V^0_{n-1} W^0 Qraw_0 V^1_{n-1} W^1 Qraw_1 | S^0 S^1
__device__ __forceinline__ int item_entries(const Item& it, int n_kv)
{
    return it.shared ? 2 * n_kv + 2 + it.ntile : it.ntile * (2 * n_kv + 3);
}
__device__ __forceinline__ Entry item_entry(const Item& it, int n_kv, int e)
{
    Entry en;
    if (it.shared) {
        en.tile = 0;
        if (e == 0) { en.kind = kEntK; en.j = 0; }
        else if (e < 2 * n_kv) { en.kind = (e & 1) ? kEntV : kEntK; en.j = (e & 1) ? (e - 1) >> 1 : e >> 1; }
        else if (e == 2 * n_kv) { en.kind = kEntW; en.j = 0; }
        else if (e < 2 * n_kv + 1 + it.ntile) { en.kind = kEntQRaw; en.tile = e - (2 * n_kv + 1); en.j = 0; }
        else { en.kind = kEntState; en.j = 0; }
    } else {
        const int nt = it.ntile;
        const int body = nt + 2 * nt * (n_kv - 1);   // entries before the last key iteration
        if (e < nt) { en.kind = kEntK; en.tile = e; en.j = 0; }
        else if (e < body) {
            const int x = e - nt, jj = x / (2 * nt), y = x - jj * 2 * nt;
            en.tile = y >> 1;
            en.kind = (y & 1) ? kEntK : kEntV;
            en.j = (y & 1) ? jj + 1 : jj;
        } else if (e < body + 3 * nt) {
            const int y = e - body;
            en.tile = y / 3;
            const int z = y - en.tile * 3;
            en.kind = z == 0 ? kEntV : z == 1 ? kEntW : kEntQRaw;
            en.j = n_kv - 1;
        } else { en.kind = kEntState; en.tile = e - (body + 3 * nt); en.j = 0; }
    }
    return en;
}

// One softmax group thread: owns query row `r` of tile `t` of every item.  kElemGate compiles the
// per-channel gate variant in (a separate kernel instantiation, so the default path is unchanged).
template <bool kElemGate, bool kSplit>
__device__ __forceinline__ void softmax_role(const TcStepParams& p, uint8_t* smem, uint32_t bars,
                                             uint32_t tmem_base, const Abort& ab,
                                             const volatile int* item_slots, int t, int r,
                                             int warp_in_group)
{
    const int L = p.s.L, H = p.s.H;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp_in_group * 32) << 16);
    const uint32_t s_addr = lane_base + (uint32_t)(t * kTile);
    const uint32_t o_addr = lane_base + (uint32_t)(2 * kTile + t * kTile);
    const uint32_t bar_s = bars + 8 * (kBarSFull0 + t);
    const uint32_t bar_p = bars + 8 * (kBarPFull0 + t);
    const float c2 = p.s.scale_log2;
    const uint64_t c2x2 = pack2(c2, c2);
    const int n_kv = p.n_kv;
    uint32_t s_cnt = 0;   // phases of bar_s consumed so far
    uint32_t of_cnt = 0;  // phases of this tile's final-O barrier consumed so far
    uint32_t tok_cnt = 0; // turns taken in the exponential phase
    uint32_t sreg[128];

    for (uint32_t item = 0;; ++item) {
        if (!wait_bar(bars + 8 * kBarQFull, item & 1, ab, 10)) return;
        const int id = item_slots[item & 1];
        if (id < 0) return;
        const Item it = decode_item<kSplit>(id, p);
        const int j0 = kSplit ? it.j0 : 0, nj = kSplit ? it.nj : n_kv;
        const int b = it.b[t], h = it.h[t];
        const int row = it.row0[t] + r;
        const bool valid_row = row < L;
        const bool active = t < it.ntile;

        if (active) {
            // ---- Q~ = RoPE(Q): rotate this thread's row of the tile in place          (Eq. 2)
            if (p.rope_h != nullptr) {
                uint8_t* tile = smem + kOffQ + t * kTileBytes;
                // all 16 table loads of the row go out before the first one is used
                const uint4* tab = p.rope_h + ((size_t)(row >> 5) * 16) * 32 + (row & 31);
                uint4 cs[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) cs[c] = __ldg(tab + c * 32);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    int off = (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
                    uint4 raw = *reinterpret_cast<const uint4*>(tile + off);
                    uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                    const uint32_t h2[4] = {cs[c].x, cs[c].y, cs[c].z, cs[c].w};
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        float cc, ss;
                        unpack_cs(h2[m], cc, ss);
                        float x0 = __uint_as_float(w[m] << 16);
                        float x1 = __uint_as_float(w[m] & 0xFFFF0000u);
                        w[m] = pack_bf16(x0 * cc - x1 * ss, x0 * ss + x1 * cc);
                    }
                    *reinterpret_cast<uint4*>(tile + off) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                fence_proxy_async_smem();
            }
            mbar_arrive(bars + 8 * (kBarQRot0 + t));

            float m_ref = -INFINITY;   // reference maximum (scaled, base 2) of the probabilities
            uint64_t l2 = pack2(0.0f, 0.0f);   // running row sum relative to m_ref, two lanes

            for (int jj = 0; jj < nj; ++jj) {
                const int j = j0 + jj;
                if (!wait_bar(bar_s, s_cnt & 1, ab, 20 + t)) return;
                ++s_cnt;
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    tmem_ld32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
                tmem_wait_ld();

                const int n_valid = p.Lk - j * kTile;  // keys of this tile that exist
                if (n_valid < kTile) {   // ragged last tile: zero-filled key rows must not count
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= n_valid) sreg[c] = __float_as_uint(-INFINITY);
                }
                float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int c = 0; c < 128; c += 8) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        m4[k] = max3(m4[k], __uint_as_float(sreg[c + 2 * k]), __uint_as_float(sreg[c + 2 * k + 1]));
                }
                const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                const float m_new = fmaxf(m_ref, mx * c2);
                const bool need = (m_new - m_ref) > kRescaleThreshold;   // first tile: inf > threshold
                if (__any_sync(0xffffffffu, need)) {
                    float alpha = 1.0f;
                    if (need) {
                        alpha = ex2_approx(m_ref - m_new);
                        m_ref = m_new;
                        l2 = fma2(l2, pack2(alpha, alpha), pack2(0.0f, 0.0f));
                    }
                    if (jj > 0) {
                        // the MMA that last accumulated into O_t finished before S_t(j) was
                        // signalled, and the next one waits for this group's arrival below
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
                const uint64_t neg_m2 = pack2(-m_ref, -m_ref);
                if (it.ntile == 2) {
                    // the two groups alternate in the exponential phase, so that one group's
                    // exponentials overlap the other tile's MMAs instead of its exponentials
                    const uint32_t par = (t == 0) ? ((tok_cnt + 1) & 1) : (tok_cnt & 1);
                    if (!wait_bar(bars + 8 * (kBarTok0 + t), par, ab, 24 + t)) return;
                    ++tok_cnt;
                }
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    float x0, x1, p0, p1;
                    unpack2(fma2(pack2(__uint_as_float(sreg[2 * c]), __uint_as_float(sreg[2 * c + 1])), c2x2, neg_m2),
                            x0, x1);
                    p0 = ex2_approx(x0);
                    p1 = ex2_approx(x1);
                    l2 = add2(l2, pack2(p0, p1));
                    sreg[c] = pack_bf16(p0, p1);
                }
                if (it.ntile == 2) mbar_arrive(bars + 8 * (kBarTok0 + (t ^ 1)));
                tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
                tmem_st32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar_p);
            }
            float l_lo, l_hi;
            unpack2(l2, l_lo, l_hi);
            const float l_sum = l_lo + l_hi;

            // ---- inter branch: U = Q W_phi_q arrives in the S columns                  (Eq. 3)
            // the row's rotation table is fetched while the MMA is still running
            uint4 cs[16];
            // fetched early too; no gate tensor = closed gate (plain softmax attention, Eq. 1)
            const bool elem_gate = kElemGate && p.gate_mode == 2 && p.gate != nullptr;   // one gate per output channel
            const float gate_logit = (valid_row && p.gate != nullptr && !elem_gate)
                                         ? __ldg(p.gate + (p.gate_mode == 1 ? (size_t)b * L + row : ((size_t)b * L + row) * H + h))
                                         : -INFINITY;
            const bool rotate_u = p.rope_h != nullptr && valid_row;
            if (rotate_u) {
                const uint4* tab = p.rope_h + ((size_t)(row >> 5) * 16) * 32 + (row & 31);
#pragma unroll
                for (int c = 0; c < 16; ++c) cs[c] = __ldg(tab + c * 32);
            }
            if (!wait_bar(bar_s, s_cnt & 1, ab, 30 + t)) return;
            ++s_cnt;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c)
                tmem_ld32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
            tmem_wait_ld();
            {
                if (rotate_u) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const uint32_t h2[4] = {cs[c].x, cs[c].y, cs[c].z, cs[c].w};
#pragma unroll
                        for (int m = 0; m < 4; ++m) {
                            float cc, s1;
                            unpack_cs(h2[m], cc, s1);
                            float x0 = __uint_as_float(sreg[c * 8 + 2 * m]);
                            float x1 = __uint_as_float(sreg[c * 8 + 2 * m + 1]);
                            sreg[c * 8 + 2 * m] = __float_as_uint(x0 * cc - x1 * s1);
                            sreg[c * 8 + 2 * m + 1] = __float_as_uint(x0 * s1 + x1 * cc);
                        }
                    }
                }
                float ss4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int c = 0; c < 128; c += 4) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        ss4[k] = fmaf(__uint_as_float(sreg[c + k]), __uint_as_float(sreg[c + k]), ss4[k]);
                }
                const float ss = (ss4[0] + ss4[1]) + (ss4[2] + ss4[3]);
                const float gate = valid_row ? sigmoid_fast(gate_logit) : 0.0f;
                // scaled by the row sum so that the common 1/l of the epilogue leaves gate * Q' S;
                // with per-channel gates the readout is kept apart and gated in the epilogue
                const float f = elem_gate ? rsqrtf(ss + p.s.eps) : rsqrtf(ss + p.s.eps) * gate * l_sum;
#pragma unroll
                for (int c = 0; c < 64; ++c)
                    sreg[c] = pack_bf16(__uint_as_float(sreg[2 * c]) * f, __uint_as_float(sreg[2 * c + 1]) * f);
            }
            tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
            tmem_st32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p);

            if (elem_gate) {
                // ---- per-channel gates: X = Q' S arrives 64 channels at a time in columns 64-127 of
                // S_t; out = O_t / l + sigmoid(G) X.  O_t is final: its last MMA preceded U's.
                const float inv_l = 1.0f / l_sum;
                const size_t rbase = ((size_t)b * L + (valid_row ? row : 0)) * H + h;
                __nv_bfloat16* orow = p.out + rbase * kTile;
                const float* grow = p.gate + rbase * kTile;
#pragma unroll 1
                for (int hv = 0; hv < 2; ++hv) {
                    if (!wait_bar(bar_s, s_cnt & 1, ab, 32 + t)) return;
                    ++s_cnt;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t x[32], o[32];
                        tmem_ld32(s_addr + 64 + c * 32, x);
                        tmem_ld32(o_addr + hv * 64 + c * 32, o);
                        tmem_wait_ld();
                        if (valid_row) {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                uint32_t w[8];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const float4 gl = __ldg(reinterpret_cast<const float4*>(grow + hv * 64 + c * 32 + e * 16 + i * 4));
                                    const float gv[4] = {gl.x, gl.y, gl.z, gl.w};
                                    float y[4];
#pragma unroll
                                    for (int u = 0; u < 4; ++u) {
                                        const int n = e * 16 + i * 4 + u;
                                        y[u] = __uint_as_float(o[n]) * inv_l + sigmoid_fast(gv[u]) * __uint_as_float(x[n]);
                                    }
                                    w[i * 2] = pack_bf16(y[0], y[1]);
                                    w[i * 2 + 1] = pack_bf16(y[2], y[3]);
                                }
                                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(
                                                 orow + hv * 64 + c * 32 + e * 16),
                                             "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                             : "memory");
                            }
                        }
                    }
                    tc_fence_before();
                    if (hv == 0) mbar_arrive(bar_p);   // the first half of X has been read
                }
                continue;
            }
            // ---- epilogue: O_t / l -> bf16 -> global                              (Eq. 6-7)
            if (!wait_bar(bars + 8 * (kBarOFinal0 + t), of_cnt & 1, ab, 40 + t)) return;
            ++of_cnt;
            tc_fence_after();
            __nv_bfloat16* orow = p.out + (((size_t)b * L + (valid_row ? row : 0)) * H + h) * kTile;
            if (kSplit && it.part >= 0) {
                // ---- one part of a split item: its rows of O_t, unnormalised (the readout in them
                // is scaled by this part's row sum, so that the merged sum carries gate * Q' S times
                // the total row sum), the reference maximum and the row sum go to the split buffers;
                // tc_split_merge_kernel combines the parts
                const size_t tp = ((size_t)it.slot * 2 + t) * p.k_split + it.part;
                float* mine = p.split_o + (tp * kTile + r) * kTile;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(o_addr + c * 32, o);
                    tmem_wait_ld();
                    if (valid_row) {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(
                                             mine + c * 32 + e * 8),
                                         "r"(o[e * 8]), "r"(o[e * 8 + 1]), "r"(o[e * 8 + 2]), "r"(o[e * 8 + 3]),
                                         "r"(o[e * 8 + 4]), "r"(o[e * 8 + 5]), "r"(o[e * 8 + 6]), "r"(o[e * 8 + 7])
                                         : "memory");
                    }
                }
                tc_fence_before();
                if (valid_row) *reinterpret_cast<float2*>(p.split_ml + (tp * kTile + r) * 2) = make_float2(m_ref, l_sum);
                continue;
            }
            const float inv_l = 1.0f / l_sum;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(o_addr + c * 32, o);
                tmem_wait_ld();
                if (valid_row) {
                    // 32-byte stores: each one fills a whole sector of the row
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            w[i] = pack_bf16(__uint_as_float(o[e * 16 + 2 * i]) * inv_l,
                                             __uint_as_float(o[e * 16 + 2 * i + 1]) * inv_l);
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(
                                         orow + c * 32 + e * 16),
                                     "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                     : "memory");
                    }
                }
            }
            tc_fence_before();
        }
    }
}

template <bool kElemGate, bool kSplit>
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
    volatile int* item_slots = reinterpret_cast<volatile int*>(smem + kOffBars + kNumBars * 8 + 8);
    const Abort ab{abort_flag, p.status, p.spin_limit};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_kv = p.n_kv;

    if (threadIdx.x == 0) {
        mbar_init(bars + 8 * kBarQFull, 1);
        mbar_init(bars + 8 * kBarQFree, 2);
        mbar_init(bars + 8 * kBarQRot0, 128);
        mbar_init(bars + 8 * kBarQRot1, 128);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bars + 8 * (kBarFull0 + s), 1);
            mbar_init(bars + 8 * (kBarEmpty0 + s), 2);   // both MMA issuers release every entry
        }
        mbar_init(bars + 8 * kBarSFull0, 1);
        mbar_init(bars + 8 * kBarSFull1, 1);
        mbar_init(bars + 8 * kBarPFull0, 128);
        mbar_init(bars + 8 * kBarPFull1, 128);
        mbar_init(bars + 8 * kBarOFinal0, 1);
        mbar_init(bars + 8 * kBarOFinal1, 1);
        mbar_init(bars + 8 * kBarTok0, 128);
        mbar_init(bars + 8 * kBarTok1, 128);
        mbar_init(bars + 8 * kBarDrain0, 1);
        mbar_init(bars + 8 * kBarDrain1, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        if (blockIdx.x == 0) *p.sched_next = 0;   // the next launch starts from a clean counter
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
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        softmax_role<kElemGate, kSplit>(p, smem, bars, tmem_base, ab, item_slots, warp >> 2, (warp & 3) * 32 + lane, warp & 3);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    }
    if (warp == 8) {
        // ---------------- TMA producer and scheduler ----------------
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_v);
            prefetch_tensormap(&tm_w);
            prefetch_tensormap(&tm_s);
            const uint32_t bar_q = bars + 8 * kBarQFull;
            uint32_t n = 0;       // ring entries produced so far (all items)
            bool ok = true;
            int q_item = -1;      // item whose Q tiles were requested last
            int id = (int)blockIdx.x;
            for (uint32_t item = 0; ok; ++item) {
                if (item > 0) ok = wait_bar(bars + 8 * kBarQFree, (item - 1) & 1, ab, 50);
                if (!ok) break;
                if (id >= p.n_sched) {
                    item_slots[item & 1] = -1;
                    mbar_arrive(bar_q);
                    break;
                }
                item_slots[item & 1] = id;
                const Item it = decode_item<kSplit>(id, p);
                const int j0 = kSplit ? it.j0 : 0, nj = kSplit ? it.nj : n_kv;
                const int ntile = it.ntile;
                mbar_expect_tx(bar_q, ntile * kTileBytes);
                q_item = (int)item;
                for (int t = 0; t < ntile; ++t) {
                    uint32_t dst = smem_base + kOffQ + t * kTileBytes;
                    tma_load_4d(dst, &tm_q, bar_q, 0, it.h[t], it.row0[t], it.b[t]);
                    tma_load_4d(dst + kHalfBytes, &tm_q, bar_q, 64, it.h[t], it.row0[t], it.b[t]);
                }
                const int entries = item_entries(it, nj);
                for (int e = 0; e < entries && ok; ++e, ++n) {
                    const uint32_t slot = n % kStages;
                    if (n >= (uint32_t)kStages)
                        ok = wait_bar(bars + 8 * (kBarEmpty0 + slot), ((n / kStages) - 1) & 1, ab, 51);
                    if (!ok) break;
                    const uint32_t bar = bars + 8 * (kBarFull0 + slot);
                    const uint32_t dst = smem_base + kOffRing + slot * kTileBytes;
                    mbar_expect_tx(bar, kTileBytes);
                    const Entry en = item_entry(it, nj, e);
                    const int tb = it.b[en.tile], th = it.h[en.tile];
                    if (en.kind == kEntK || en.kind == kEntV) {
                        const CUtensorMap* tm = en.kind == kEntV ? &tm_v : &tm_k;
                        tma_load_4d(dst, tm, bar, 0, th, (j0 + en.j) * kTile, tb);
                        tma_load_4d(dst + kHalfBytes, tm, bar, 64, th, (j0 + en.j) * kTile, tb);
                    } else if (en.kind == kEntW) {
                        tma_load_2d(dst, &tm_w, bar, 0, th * kTile);
                        tma_load_2d(dst + kHalfBytes, &tm_w, bar, 64, th * kTile);
                    } else if (en.kind == kEntQRaw) {
                        tma_load_4d(dst, &tm_q, bar, 0, th, it.row0[en.tile], tb);
                        tma_load_4d(dst + kHalfBytes, &tm_q, bar, 64, th, it.row0[en.tile], tb);
                    } else {
                        tma_load_2d(dst, &tm_s, bar, 0, (tb * p.s.H + th) * kTile);
                        tma_load_2d(dst + kHalfBytes, &tm_s, bar, 64, (tb * p.s.H + th) * kTile);
                    }
                }
                if (!ok) break;
                id = (int)gridDim.x + (int)atomicAdd(p.sched_counter, 1u);
            }
            if (!ok || *abort_flag) {
                // do not leave the CTA while bulk copies into its shared memory are in flight
                if (q_item >= 0) drain_bar(bar_q, (uint32_t)q_item & 1);
                for (uint32_t m = (n > (uint32_t)kStages ? n - kStages : 0); m < n; ++m)
                    drain_bar(bars + 8 * (kBarFull0 + m % kStages), (m / kStages) & 1);
            }
        }
    } else if (warp == 9 || warp == 10) {
        // ---------------- MMA issuers: warp 9 drives query tile 0, warp 10 tile 1 ----------------
        // Issuing a tcgen05.mma holds the thread until the tensor pipe accepts it, and every
        // wait / commit between two MMAs is time the pipe may idle; with one issuer per tile the
        // synchronisation of one tile overlaps the MMAs of the other.  Both issuers walk the
        // same sequence of ring entries and both release every entry (the empty barriers count
        // two arrivals), whether or not they read it.
        if (lane == 0) {
            const int t = warp - 9;
            constexpr uint32_t idesc_qk = idesc_bf16(kTile, kTile, 0, 0);  // A, B K-major
            constexpr uint32_t idesc_pv = idesc_bf16(kTile, kTile, 0, 1);  // A in TMEM, B N-contiguous
            const uint32_t q_tile = smem_base + kOffQ + t * kTileBytes;
            const uint32_t s_col = tmem_base + t * kTile;
            const uint32_t o_col = tmem_base + 2 * kTile + t * kTile;
            const uint32_t bar_s = bars + 8 * (kBarSFull0 + t);
            const uint32_t bar_p = bars + 8 * (kBarPFull0 + t);

            // Matrix descriptors are built once: the high word is constant (stride between 8-row
            // groups, version, swizzle) and a k-step only adds to the 16-byte-unit start address.
            const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
            constexpr uint32_t kLboK = 1u << 16;                                // K-major: unused field
            constexpr uint32_t kLboMN = (uint32_t)(kHalfBytes >> 4) << 16;      // 64-column groups of V
            auto desc64 = [&](uint32_t lo) {
                uint64_t d;
                asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
                return d;
            };
            // S_t (or U_t) = A_t * B^T with both operands K-major, 8 k-steps of 16
            auto issue_qk = [&](uint32_t a_tile, uint32_t b_tile) {
                const uint32_t a_lo = (a_tile >> 4) | kLboK, b_lo = (b_tile >> 4) | kLboK;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                    mma_ss(s_col, desc64(a_lo + koff), desc64(b_lo + koff), idesc_qk, ks > 0);
                }
            };
            // O_t (+)= P_t * V with P in TMEM and V rows = contraction index, 8 k-steps of 16
            auto issue_pv = [&](uint32_t v_tile, bool accumulate) {
                const uint32_t v_lo = (v_tile >> 4) | kLboMN;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(o_col, s_col + ks * 8, desc64(v_lo + (uint32_t)(ks * (2048 >> 4))), idesc_pv,
                           (accumulate || ks > 0) ? 1u : 0u);
            };
            auto slot_addr = [&](uint32_t entry) { return smem_base + kOffRing + (entry % kStages) * kTileBytes; };
            auto wait_full = [&](uint32_t entry, int site) {
                return wait_bar(bars + 8 * (kBarFull0 + entry % kStages), (entry / kStages) & 1, ab, site);
            };
            auto release = [&](uint32_t entry) { mma_commit(bars + 8 * (kBarEmpty0 + entry % kStages)); };

            uint32_t cons = 0;        // ring entries consumed so far (all items)
            uint32_t p_cnt = 0;       // phases of bar_p consumed
            uint32_t qrot_cnt = 0, of_cnt = 0;
            bool ok = true;
            for (uint32_t item = 0; ok; ++item) {
                ok = wait_bar(bars + 8 * kBarQFull, item & 1, ab, 60);
                if (!ok) break;
                const int id = item_slots[item & 1];
                if (id < 0) break;
                const Item it = decode_item<kSplit>(id, p);
                const int nj = kSplit ? it.nj : n_kv;   // key tiles of this item (a part walks its own range)
                const int ntile = it.ntile;
                const bool active = t < ntile;
                const bool shared = it.shared;
                // An entry both tiles read (K, V, W, S of a pair item) is released once by each
                // issuer; an entry only one tile reads is released twice by that tile's issuer
                // (the empty barriers always count two arrivals) and ignored by the other.
                auto release_mine = [&](uint32_t e, bool exclusive) {
                    release(e);
                    if (exclusive) release(e);
                };
                auto q_free = [&]() {
                    mma_commit(bars + 8 * kBarQFree);
                    if (ntile == 1) mma_commit(bars + 8 * kBarQFree);   // on behalf of the idle issuer
                };
                if (active) {
                    ok = wait_bar(bars + 8 * (kBarQRot0 + t), qrot_cnt & 1, ab, 61);
                    ++qrot_cnt;
                    if (!ok) break;
                    // S_t(0) = Q~_t K_0^T
                    const uint32_t e_k = cons + (shared ? 0 : t);
                    ok = wait_full(e_k, 62);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(q_tile, slot_addr(e_k));
                    mma_commit(bar_s);
                    release_mine(e_k, !shared);
                    if (nj == 1) q_free();
                }
                cons += shared ? 1 : ntile;

                for (int j = 0; j < nj && ok; ++j) {
                    const bool last = j + 1 == nj;       // then the next "S" is the inter branch's Q W
                    const int per_tile = last ? 3 : 2;   // ragged item: V, K or W, [Qraw] per tile
                    const int group = shared ? (last ? 2 + ntile : 2) : per_tile * ntile;
                    if (active) {
                        const uint32_t e_v = shared ? cons : cons + per_tile * t;   // V_j
                        const uint32_t e_b = e_v + 1;                               // K_{j+1} or W
                        const uint32_t e_q = shared ? cons + 2 + t : e_v + 2;       // raw Q tile (last only)
                        ok = wait_full(e_v, 63);
                        if (ok) ok = wait_full(e_b, 66);
                        if (ok && last) ok = wait_full(e_q, 68);
                        if (!ok) break;
                        ok = wait_bar(bar_p, p_cnt & 1, ab, 64 + t);
                        ++p_cnt;
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(slot_addr(e_v), j > 0);
                        issue_qk(last ? slot_addr(e_q) : q_tile, slot_addr(e_b));
                        mma_commit(bar_s);
                        release_mine(e_v, !shared);
                        release_mine(e_b, !shared);
                        if (last) release_mine(e_q, true);
                        if (j + 2 == nj) q_free();   // the last score MMA was the last use of Q~
                    }
                    cons += group;
                }
                if (!ok) break;
                // inter branch: O_t += Q''_t S
                if (active) {
                    const uint32_t e_s = cons + (shared ? 0 : t);
                    ok = wait_full(e_s, 69);
                    if (ok) ok = wait_bar(bar_p, p_cnt & 1, ab, 70 + t);
                    ++p_cnt;
                    if (!ok) break;
                    tc_fence_after();
                    if (kElemGate && p.gate_mode == 2 && p.gate != nullptr) {
                        // per-channel gates: X = Q' S kept apart from O_t, 64 channels at a time into
                        // columns 64-127 of S_t (Q' sits in columns 0-63)
                        constexpr uint32_t idesc_x = idesc_bf16(kTile, 64, 0, 1);
                        for (int hv = 0; hv < 2 && ok; ++hv) {
                            if (hv == 1) {
                                ok = wait_bar(bar_p, p_cnt & 1, ab, 72 + t);   // first half consumed
                                ++p_cnt;
                                if (!ok) break;
                                tc_fence_after();
                            }
                            const uint32_t x_lo = ((slot_addr(e_s) + hv * kHalfBytes) >> 4) | kLboMN;
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)
                                mma_ts(s_col + 64, s_col + ks * 8, desc64(x_lo + (uint32_t)(ks * (2048 >> 4))), idesc_x,
                                       ks > 0 ? 1u : 0u);
                            mma_commit(bar_s);
                        }
                        if (!ok) break;
                        release_mine(e_s, !shared);
                    } else {
                        issue_pv(slot_addr(e_s), true);
                        release_mine(e_s, !shared);
                        mma_commit(bars + 8 * (kBarOFinal0 + t));
                        ++of_cnt;
                    }
                }
                cons += shared ? 1 : ntile;
            }
            (void)of_cnt;
            if (!ok || *abort_flag) {
                // tensor memory is freed below: none of this thread's MMAs may still be running
                mma_commit(bars + 8 * (kBarDrain0 + t));
                drain_bar(bars + 8 * (kBarDrain0 + t), 0);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------------------------
// Token-sequential commit with per-token gates (Eq. 4 token by token), chunkwise, tensor cores.
// Notation as in the plain-FMA version: for a chunk of C = 64 tokens entering with state S_0,
//   U = U1 - W S_0,  S_C = g S_0 + Khat^T U,  U1 = T diag(beta) V',  W = T diag(beta g_{j-1}) K',
//   T = (I + A)^-1,  A_ji = beta_j (g_{j-1} / g_i) <K'_j, K'_i> (i < j),  Khat_i = (g / g_i) K'_i.
// tc_token_prepare_kernel: one CTA (128 threads, thread = token) per 128-token tile = two chunks.
//   U_k, U_v (MMA) -> K' -> Gram matrix K' K'^T (MMA) -> A (fp32, shared memory) -> T by forward
//   substitution (thread = column), stored as a bf16 block-diagonal 128 x 128 operand -> W and U1
//   (MMA, both chunks at once) -> global: W, Khat, U1 in bf16, chunk decays g in fp32.
// tc_token_scan_kernel: one CTA per (stream, head) walks the chunks in order (further down).
// ---------------------------------------------------------------------------------------------
constexpr int kTPOffWk = 0;                        // maps; later the fp32 matrix A (2 x 64 x 65)
constexpr int kTPOffWv = kTileBytes;
constexpr int kTPOffK = 2 * kTileBytes;            // raw K tile -> K' (bf16)
constexpr int kTPOffV = 3 * kTileBytes;            // raw V tile -> diag(beta) V'
constexpr int kTPOffKs = 4 * kTileBytes;           // diag(beta g_{j-1}) K'
constexpr int kTPOffT = 5 * kTileBytes;            // block-diagonal T
constexpr int kTPOffBars = 6 * kTileBytes;
constexpr int kTPSmemBytes = kTPOffBars + 1024 + 1024;   // barriers, gate scratch, alignment slack
constexpr int kTokC = 64;                          // tokens per chunk
constexpr int kLdA = kTokC + 4;   // 16-byte aligned rows, conflict-free 16-byte stores
static_assert(2 * kTokC * kLdA * 4 <= 2 * kTileBytes, "A fits over the two maps");

enum TPBar : int { kTPBarLoad = 0, kTPBarU, kTPBarG, kTPBarW, kTPBarDrain, kTPNumBars };

struct TcTokenParams {
    Shape s;
    const uint4* rope_h;
    const float* alpha;        // [B, L, H] logits or nullptr
    const float* beta;
    __nv_bfloat16* w;          // [B, H, rows_pad, 128]
    __nv_bfloat16* kh;         // [B, H, rows_pad, 128]
    __nv_bfloat16* u1;         // [B, H, rows_pad, 128]
    float* gc;                 // [B, H, 2 * ntile]
    float* state;              // scan kernel only
    __nv_bfloat16* state_bf16;
    uint32_t* status;
    uint32_t spin_limit;
    int ntile;                 // 128-token tiles; rows_pad = 128 * ntile
    int nchunk;                // ceil(L / 64): chunks the scan walks
    int decayed;               // prediction against alpha_j S_{j-1}
};

__global__ void __launch_bounds__(128, 1)
tc_token_prepare_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                        const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                        const TcTokenParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kTPOffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kTPOffBars + kTPNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kTPOffBars + kTPNumBars * 8 + 4);
    float* cl_s = reinterpret_cast<float*>(smem + kTPOffBars + 64);          // [128] log g_j (inclusive)
    float* wsum = reinterpret_cast<float*>(smem + kTPOffBars + 64 + 512);    // [4] warp totals
    const Abort ab{abort_flag, p.status, p.spin_limit};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int L = p.s.L, H = p.s.H;
    const int row = tile * kTile + tid;          // this thread's token
    const int chunk = tid >> 6, jj = tid & 63;   // chunk of the tile, index in the chunk

    if (tid == 0) {
        for (int i = 0; i < kTPNumBars; ++i) mbar_init(bars + 8 * i, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    // the off-diagonal blocks of T stay zero
    for (int i = tid; i < kTileBytes / 16; i += 128)
        reinterpret_cast<uint4*>(smem + kTPOffT)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);

    bool ok = true;
    if (tid == 0) {
        const uint32_t bar = bars + 8 * kTPBarLoad;
        mbar_expect_tx(bar, 4 * kTileBytes);
        tma_load_2d(smem_base + kTPOffWk, &tm_wk, bar, 0, h * kTile);
        tma_load_2d(smem_base + kTPOffWk + kHalfBytes, &tm_wk, bar, 64, h * kTile);
        tma_load_2d(smem_base + kTPOffWv, &tm_wv, bar, 0, h * kTile);
        tma_load_2d(smem_base + kTPOffWv + kHalfBytes, &tm_wv, bar, 64, h * kTile);
        tma_load_4d(smem_base + kTPOffK, &tm_k, bar, 0, h, tile * kTile, b);
        tma_load_4d(smem_base + kTPOffK + kHalfBytes, &tm_k, bar, 64, h, tile * kTile, b);
        tma_load_4d(smem_base + kTPOffV, &tm_v, bar, 0, h, tile * kTile, b);
        tma_load_4d(smem_base + kTPOffV + kHalfBytes, &tm_v, bar, 64, h, tile * kTile, b);
    }

    // ---- gates: log alpha_j, beta_j, cumulative decay within the chunk (tokens past L: 1 and 0)
    float la = 0.0f, be = 0.0f;
    if (row < L) {
        const size_t gi = ((size_t)b * L + row) * H + h;
        if (p.alpha != nullptr) {
            const float x = __ldg(p.alpha + gi);
            la = x >= 0.0f ? -log1pf(expf(-x)) : x - log1pf(expf(x));
        }
        be = p.beta != nullptr ? 1.0f / (1.0f + expf(-__ldg(p.beta + gi))) : 1.0f;
    }
    float cl = la;   // inclusive scan over the 64 tokens of the chunk (two warps)
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, cl, off);
        if (lane >= off) cl += up;
    }
    if (lane == 31) wsum[warp] = cl;
    __syncthreads();
    if (warp & 1) cl += wsum[warp - 1];
    cl_s[tid] = cl;
    __syncthreads();
    const float cl_total = cl_s[chunk * kTokC + kTokC - 1];
    const float cl_excl = cl - la;
    // log of the factor on K'_j S_0: g_{j-1} for Eq. 4 as printed, g_j when the token's prediction is made
    // against the state after its own forget gate
    const float cl_pred = p.decayed ? cl : cl_excl;

    constexpr uint32_t kLboK = 1u << 16;
    constexpr uint32_t kLboMN = (uint32_t)(kHalfBytes >> 4) << 16;
    const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
    auto desc64 = [&](uint32_t lo) {
        uint64_t d;
        asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
        return d;
    };
    constexpr uint32_t idesc_kk = idesc_bf16(kTile, kTile, 0, 0);   // both operands d-major
    constexpr uint32_t idesc_kn = idesc_bf16(kTile, kTile, 0, 1);   // A K-major, B rows = contraction index
    auto koff_k = [](int ks) { return (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4); };

    // ---- U_k = K W_phi_k, U_v = V W_phi_v
    if (tid == 0) {
        ok = wait_bar(bars + 8 * kTPBarLoad, 0, ab, 90);
        if (ok) {
            tc_fence_after();
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t a_lo = ((smem_base + (u ? kTPOffV : kTPOffK)) >> 4) | kLboK;
                const uint32_t b_lo = ((smem_base + (u ? kTPOffWv : kTPOffWk)) >> 4) | kLboK;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ss(tmem_base + u * kTile, desc64(a_lo + koff_k(ks)), desc64(b_lo + koff_k(ks)), idesc_kk, ks > 0);
            }
            mma_commit(bars + 8 * kTPBarU);
        }
    }
    uint32_t sreg[128];
    bool alive = wait_bar(bars + 8 * kTPBarU, 0, ab, 91);
    const size_t grow = (((size_t)b * H + h) * p.ntile + tile) * kTile + tid;   // row of the scratch tensors
    if (alive) {
        tc_fence_after();
        // ---- K' = L2Norm(RoPE(U_k)); three copies: K' (Gram), scaled for W, scaled for the scan
#pragma unroll
        for (int c = 0; c < 4; ++c)
            tmem_ld32(lane_base + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
        tmem_wait_ld();
        if (p.rope_h != nullptr) {
            const uint4* tab = p.rope_h + ((size_t)(row >> 5) * 16) * 32 + (row & 31);
            uint4 cs[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) cs[c] = __ldg(tab + c * 32);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint32_t h2[4] = {cs[c].x, cs[c].y, cs[c].z, cs[c].w};
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    float cc, s1;
                    unpack_cs(h2[m], cc, s1);
                    const float x0 = __uint_as_float(sreg[c * 8 + 2 * m]);
                    const float x1 = __uint_as_float(sreg[c * 8 + 2 * m + 1]);
                    sreg[c * 8 + 2 * m] = __float_as_uint(x0 * cc - x1 * s1);
                    sreg[c * 8 + 2 * m + 1] = __float_as_uint(x0 * s1 + x1 * cc);
                }
            }
        }
        float ss4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                ss4[k] = fmaf(__uint_as_float(sreg[c + k]), __uint_as_float(sreg[c + k]), ss4[k]);
        }
        const float f = rsqrtf((ss4[0] + ss4[1]) + (ss4[2] + ss4[3]) + p.s.eps);
        store_row_bf16_swizzled(smem + kTPOffK, tid, sreg, f);
        store_row_bf16_swizzled(smem + kTPOffKs, tid, sreg, f * be * expf(cl_pred));
        store_row_bf16_global(p.kh + grow * kTile, sreg, f * expf(cl_total - cl));
        // ---- diag(beta) V'
#pragma unroll
        for (int c = 0; c < 4; ++c)
            tmem_ld32(lane_base + kTile + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
        tmem_wait_ld();
        store_row_bf16_swizzled(smem + kTPOffV, tid, sreg, be);
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();

    // ---- Gram matrix K' K'^T -> TMEM columns 256-383 (row = token j, column = token i)
    if (tid == 0 && ok && !*abort_flag) {
        tc_fence_after();
        const uint32_t k_lo = ((smem_base + kTPOffK) >> 4) | kLboK;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            mma_ss(tmem_base + 2 * kTile, desc64(k_lo + koff_k(ks)), desc64(k_lo + koff_k(ks)), idesc_kk, ks > 0);
        mma_commit(bars + 8 * kTPBarG);
    }
    alive = alive && wait_bar(bars + 8 * kTPBarG, 0, ab, 92);
    float* As = reinterpret_cast<float*>(smem + kTPOffWk);   // the maps are dead: U_k, U_v are complete
    if (alive) {
        tc_fence_after();
        // this token's row of A: only the columns of its own chunk, strictly below the diagonal
        uint32_t g[64];
        tmem_ld32(lane_base + 2 * kTile + chunk * kTokC, *reinterpret_cast<uint32_t(*)[32]>(&g[0]));
        tmem_ld32(lane_base + 2 * kTile + chunk * kTokC + 32, *reinterpret_cast<uint32_t(*)[32]>(&g[32]));
        tmem_wait_ld();
        float* arow = As + (chunk * kTokC + jj) * kLdA;
#pragma unroll
        for (int i4 = 0; i4 < kTokC / 4; ++i4) {
            float v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = i4 * 4 + k;
                const float w = be * __expf(cl_pred - cl_s[chunk * kTokC + i]);
                v[k] = i < jj ? w * __uint_as_float(g[i]) : 0.0f;
            }
            *reinterpret_cast<float4*>(arow + i4 * 4) = make_float4(v[0], v[1], v[2], v[3]);
        }
    }
    __syncthreads();
    // ---- T = (I + A)^-1 by forward substitution; this thread owns column jj of its chunk's T
    if (alive) {
        const float* Ac = As + chunk * kTokC * kLdA;
        float t[kTokC];
#pragma unroll
        for (int j = 0; j < kTokC; ++j) {
            // row j of A in 16-byte pieces (the same address for the whole chunk: a broadcast),
            // four independent partial sums
            float acc[4] = {j == jj ? 1.0f : 0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int i4 = 0; i4 < (j + 3) / 4; ++i4) {
                const float4 a4 = *reinterpret_cast<const float4*>(Ac + j * kLdA + i4 * 4);
                const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (i4 * 4 + k < j) acc[k] -= av[k] * t[i4 * 4 + k];
            }
            t[j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
        }
        // element (row r = chunk*64 + j, column c = chunk*64 + jj) of the K-major swizzled bf16 tile
        const int cglob = chunk * kTokC + jj;
        uint8_t* tt = smem + kTPOffT + (cglob >> 6) * kHalfBytes + (cglob & 7) * 2;
        const int c16 = (cglob & 63) >> 3;
#pragma unroll
        for (int j = 0; j < kTokC; ++j) {
            const int r = chunk * kTokC + j;
            *reinterpret_cast<__nv_bfloat16*>(tt + r * 128 + ((c16 ^ (r & 7)) << 4)) = __float2bfloat16_rn(t[j]);
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();

    // ---- W = T diag(beta g_{j-1}) K' -> columns 0-127, U1 = T diag(beta) V' -> columns 128-255
    if (tid == 0 && ok && !*abort_flag) {
        tc_fence_after();
        const uint32_t t_lo = ((smem_base + kTPOffT) >> 4) | kLboK;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint32_t b_lo = ((smem_base + (u ? kTPOffV : kTPOffKs)) >> 4) | kLboMN;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(tmem_base + u * kTile, desc64(t_lo + koff_k(ks)), desc64(b_lo + (uint32_t)(ks * (2048 >> 4))),
                       idesc_kn, ks > 0);
        }
        mma_commit(bars + 8 * kTPBarW);
    }
    alive = alive && wait_bar(bars + 8 * kTPBarW, 0, ab, 93);
    if (alive) {
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c)
            tmem_ld32(lane_base + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
        tmem_wait_ld();
        store_row_bf16_global(p.w + grow * kTile, sreg, 1.0f);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            tmem_ld32(lane_base + kTile + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
        tmem_wait_ld();
        store_row_bf16_global(p.u1 + grow * kTile, sreg, 1.0f);
        if (jj == kTokC - 1)
            p.gc[(((size_t)b * H + h) * p.ntile + tile) * 2 + chunk] = expf(cl_total);
    }
    if (tid == 0 && (!ok || *abort_flag)) {
        drain_bar(bars + 8 * kTPBarLoad, 0);   // no bulk copy left in flight
        mma_commit(bars + 8 * kTPBarDrain);    // and no MMA still writing tensor memory
        drain_bar(bars + 8 * kTPBarDrain, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// tc_token_scan_kernel: one CTA (256 threads) per (stream, head); the fp32 state lives in TMEM
// (row = key dim d, 128 columns) for the whole walk.  Per chunk:
//   Y = W_c S            MMA, A = W tile (128 rows fetched, the first 64 are the chunk), B = bf16 copy of S
//   U = U1_c - Y         two threads per token (64 columns each), written as a bf16 operand tile
//   S += Khat_c^T U      MMA over the chunk's 64 tokens, accumulating on g_c S (scaled beforehand)
//   bf16 copy of the new S for the next chunk; S scaled by g_{c+1} in the same pass (two threads
//                        per state row, 64 columns each)
// The tiles of chunk c + 2 are fetched by TMA as soon as chunk c has released its buffers.
constexpr int kTSOffS = 0;                           // bf16 S, [d][e], 128 rows
constexpr int kTSOffW = kTileBytes;                  // 2 x 32 KB: W tiles (128 rows)
constexpr int kTSOffKh = 3 * kTileBytes;             // 2 x 16 KB: Khat chunks (64 rows)
constexpr int kTSOffU1 = 4 * kTileBytes;             // 2 x 16 KB: U1 chunks
constexpr int kTSOffU = 5 * kTileBytes;              // 16 KB: U operand
constexpr int kTSOffBars = 5 * kTileBytes + kHalfBytes;
constexpr int kTSSmemBytes = kTSOffBars + 128 + 1024;
constexpr int kChunkHalf = kTokC * 128;              // bytes of a 64-row, 64-column box
constexpr uint32_t kChunkTx = kTileBytes + 4 * kChunkHalf;   // W tile + Khat + U1 per chunk

enum TSBar : int { kTSBarS0 = 0, kTSBarFull0, kTSBarFull1, kTSBarY, kTSBarS2, kTSBarDrain, kTSNumBars };

constexpr int kTSThreads = 256;
__global__ void __launch_bounds__(kTSThreads, 1)
tc_token_scan_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_kh,
                     const __grid_constant__ CUtensorMap tm_u1, const __grid_constant__ CUtensorMap tm_s,
                     const TcTokenParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bars = smem_base + kTSOffBars;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kTSOffBars + kTSNumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kTSOffBars + kTSNumBars * 8 + 4);
    const Abort ab{abort_flag, p.status, p.spin_limit};

    const int tid = threadIdx.x, warp = tid >> 5;
    const int h = blockIdx.x, b = blockIdx.y;
    const size_t bh = (size_t)b * p.s.H + h;
    const int rows_pad = p.ntile * kTile;
    const int nchunk = p.nchunk;
    const float* gc = p.gc + bh * 2 * p.ntile;

    if (tid == 0) {
        for (int i = 0; i < kTSNumBars; ++i) mbar_init(bars + 8 * i, 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // warps w and w + 4 own the same 32 TMEM lanes (rows) and split the 128 columns in two
    const int rowid = (warp & 3) * 32 + (tid & 31);
    const int chalf = warp >> 2;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(chalf * 64);

    int loads_issued = 0;
    auto load_chunk = [&](int c) {
        const uint32_t bar = bars + 8 * (kTSBarFull0 + (c & 1));
        const int r0 = (int)(bh * rows_pad) + c * kTokC;
        mbar_expect_tx(bar, kChunkTx);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            tma_load_2d(smem_base + kTSOffW + (c & 1) * kTileBytes + half * kHalfBytes, &tm_w, bar, half * 64, r0);
            tma_load_2d(smem_base + kTSOffKh + (c & 1) * kHalfBytes + half * kChunkHalf, &tm_kh, bar, half * 64, r0);
            tma_load_2d(smem_base + kTSOffU1 + (c & 1) * kHalfBytes + half * kChunkHalf, &tm_u1, bar, half * 64, r0);
        }
        ++loads_issued;
    };
    if (tid == 0) {
        mbar_expect_tx(bars + 8 * kTSBarS0, kTileBytes);
        tma_load_2d(smem_base + kTSOffS, &tm_s, bars + 8 * kTSBarS0, 0, (int)bh * kTile);
        tma_load_2d(smem_base + kTSOffS + kHalfBytes, &tm_s, bars + 8 * kTSBarS0, 64, (int)bh * kTile);
        load_chunk(0);
        if (nchunk > 1) load_chunk(1);
    }

    // fp32 state row d = rowid (this thread's 64 columns) into TMEM columns 128-255, already scaled
    // by the first chunk's decay
    float* srow = p.state + (bh * kTile + rowid) * kTile + chalf * 64;
    {
        const float g0 = __ldg(gc);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t x[32];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float4 v = *reinterpret_cast<const float4*>(srow + c * 32 + e * 4);
                x[e * 4 + 0] = __float_as_uint(v.x * g0);
                x[e * 4 + 1] = __float_as_uint(v.y * g0);
                x[e * 4 + 2] = __float_as_uint(v.z * g0);
                x[e * 4 + 3] = __float_as_uint(v.w * g0);
            }
            tmem_st32(lane_base + kTile + c * 32, x);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();

    constexpr uint32_t kLboK = 1u << 16;
    constexpr uint32_t kLboMN = (uint32_t)(kHalfBytes >> 4) << 16;     // 128-row tiles
    constexpr uint32_t kLboMN64 = (uint32_t)(kChunkHalf >> 4) << 16;   // 64-row tiles
    const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0) >> 32);
    auto desc64 = [&](uint32_t lo) {
        uint64_t d;
        asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(desc_hi));
        return d;
    };
    constexpr uint32_t idesc_kn = idesc_bf16(kTile, kTile, 0, 1);
    constexpr uint32_t idesc_nn = idesc_bf16(kTile, kTile, 1, 1);

    bool ok = true, alive = true;
    for (int c = 0; c < nchunk; ++c) {
        const int s = c & 1;
        const uint32_t par = (uint32_t)((c >> 1) & 1);
        // ---- Y = W_c S
        if (tid == 0) {
            if (c == 0) ok = wait_bar(bars + 8 * kTSBarS0, 0, ab, 100);
            if (ok) ok = wait_bar(bars + 8 * (kTSBarFull0 + s), par, ab, 101);
            if (ok) {
                tc_fence_after();
                const uint32_t a_lo = ((smem_base + kTSOffW + s * kTileBytes) >> 4) | kLboK;
                const uint32_t b_lo = ((smem_base + kTSOffS) >> 4) | kLboMN;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
                    mma_ss(tmem_base, desc64(a_lo + koff), desc64(b_lo + (uint32_t)(ks * (2048 >> 4))), idesc_kn, ks > 0);
                }
                mma_commit(bars + 8 * kTSBarY);
            }
        }
        alive = wait_bar(bars + 8 * kTSBarY, (uint32_t)(c & 1), ab, 102);
        // the chunk's tiles landed before the MMA above was issued; waiting here as well makes
        // the bulk copy's writes visible to this thread
        if (alive) alive = wait_bar(bars + 8 * (kTSBarFull0 + s), par, ab, 103);
        tc_fence_after();
        // ---- U = U1_c - Y for the chunk's 64 tokens (threads 0-63), as a bf16 operand tile
        if (alive && rowid < kTokC) {
            const uint8_t* u1t = smem + kTSOffU1 + s * kHalfBytes + chalf * kChunkHalf;
            uint8_t* ut = smem + kTSOffU + chalf * kChunkHalf;
            uint32_t y[64];
            tmem_ld32(lane_base, *reinterpret_cast<uint32_t(*)[32]>(&y[0]));
            tmem_ld32(lane_base + 32, *reinterpret_cast<uint32_t(*)[32]>(&y[32]));
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < 8; ++q) {   // 16-byte chunk of this thread's 64-column half
                const int off = rowid * 128 + ((q ^ (rowid & 7)) << 4);
                const uint4 u1 = *reinterpret_cast<const uint4*>(u1t + off);
                const uint32_t uw[4] = {u1.x, u1.y, u1.z, u1.w};
                uint32_t o[4];
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const float lo = __uint_as_float(uw[m] << 16) - __uint_as_float(y[q * 8 + 2 * m]);
                    const float hi = __uint_as_float(uw[m] & 0xFFFF0000u) - __uint_as_float(y[q * 8 + 2 * m + 1]);
                    o[m] = pack_bf16(lo, hi);
                }
                *reinterpret_cast<uint4*>(ut + off) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        if (__syncthreads_or(!alive)) break;   // every thread leaves together
        // ---- S += Khat_c^T U
        if (tid == 0 && ok) {
            tc_fence_after();
            const uint32_t a_lo = ((smem_base + kTSOffKh + s * kHalfBytes) >> 4) | kLboMN64;
            const uint32_t b_lo = ((smem_base + kTSOffU) >> 4) | kLboMN64;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                mma_ss(tmem_base + kTile, desc64(a_lo + (uint32_t)(ks * (2048 >> 4))),
                       desc64(b_lo + (uint32_t)(ks * (2048 >> 4))), idesc_nn, 1u);
            mma_commit(bars + 8 * kTSBarS2);
        }
        alive = wait_bar(bars + 8 * kTSBarS2, (uint32_t)(c & 1), ab, 104);
        tc_fence_after();
        if (alive && tid == 0 && c + 2 < nchunk) load_chunk(c + 2);   // both MMAs that read slot s are done
        // ---- the new S: bf16 operand copy, and the fp32 rows scaled for the next chunk (or stored)
        const bool last = c + 1 == nchunk;
        const float gn = last ? 1.0f : __ldg(gc + c + 1);
        if (alive) {
            uint32_t x[64];
            tmem_ld32(lane_base + kTile, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
            tmem_ld32(lane_base + kTile + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
            tmem_wait_ld();
            if (!last) {
                uint8_t* sb = smem + kTSOffS + chalf * kHalfBytes + rowid * 128;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<uint4*>(sb + ((q ^ (rowid & 7)) << 4)) =
                        make_uint4(pack_bf16(__uint_as_float(x[q * 8 + 0]), __uint_as_float(x[q * 8 + 1])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 2]), __uint_as_float(x[q * 8 + 3])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 4]), __uint_as_float(x[q * 8 + 5])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 6]), __uint_as_float(x[q * 8 + 7])));
#pragma unroll
                for (int e = 0; e < 64; ++e) x[e] = __float_as_uint(__uint_as_float(x[e]) * gn);
                tmem_st32(lane_base + kTile, *reinterpret_cast<uint32_t(*)[32]>(&x[0]));
                tmem_st32(lane_base + kTile + 32, *reinterpret_cast<uint32_t(*)[32]>(&x[32]));
            } else {
                __nv_bfloat16* mrow = p.state_bf16 + (bh * kTile + rowid) * kTile + chalf * 64;
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    *reinterpret_cast<uint4*>(srow + e * 4) = make_uint4(x[e * 4], x[e * 4 + 1], x[e * 4 + 2], x[e * 4 + 3]);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<uint4*>(mrow + q * 8) =
                        make_uint4(pack_bf16(__uint_as_float(x[q * 8 + 0]), __uint_as_float(x[q * 8 + 1])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 2]), __uint_as_float(x[q * 8 + 3])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 4]), __uint_as_float(x[q * 8 + 5])),
                                   pack_bf16(__uint_as_float(x[q * 8 + 6]), __uint_as_float(x[q * 8 + 7])));
            }
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before();
        if (__syncthreads_or(!alive)) break;
    }
    if (tid == 0 && (!ok || *abort_flag)) {
        // leave no bulk copy in flight into this CTA's shared memory
        drain_bar(bars + 8 * kTSBarS0, 0);
        for (int m = (loads_issued > 2 ? loads_issued - 2 : 0); m < loads_issued; ++m)
            drain_bar(bars + 8 * (kTSBarFull0 + (m & 1)), (uint32_t)((m >> 1) & 1));
        mma_commit(bars + 8 * kTSBarDrain);    // no MMA still writing tensor memory when it is freed
        drain_bar(bars + 8 * kTSBarDrain, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 256);
    }
}

// The rotation table in the form the step kernel reads: half2 (cos, sin) per pair, 16 vectors of

// 4 pairs per token, stored so that the 32 tokens a warp owns are interleaved -- vector c of
// token l sits at uint4 index ((l / 32) * 16 + c) * 32 + l % 32 -- and each of a warp's 16 loads is
// one contiguous 512-byte segment.  Tokens past L (padding up to a whole tile) read as zero.
// fp16 keeps 11 bits of the unit-range values.
__global__ void pack_rope_kernel(const float* __restrict__ cos_t, const float* __restrict__ sin_t,
                                 __half2* __restrict__ out, int L, size_t total)
{
    size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int l = (int)(t / 64), m = (int)(t % 64);
    const int c = m >> 2, w = m & 3;
    const size_t dst = ((((size_t)(l >> 5) * 16 + c) * 32 + (l & 31)) << 2) + w;
    out[dst] = l < L ? __floats2half2_rn(cos_t[t], sin_t[t]) : __floats2half2_rn(0.0f, 0.0f);
}

// k_rot = RoPE(k) for bf16 [B, L, H, 128] from the packed half2 table: 8 elements (4 rotation pairs,
// one 16-byte table vector) per thread.  The same table rotates Q inside the step kernel.
__global__ void tc_rope_k_kernel(const uint4* __restrict__ k, const uint4* __restrict__ rope_h,
                                 uint4* __restrict__ out, int L, int H, size_t total8)
{
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total8) return;
    const int c = (int)(t & 15);                     // vector of the 128-element row
    const int l = (int)((t >> 4) / H % L);           // token
    const uint4 raw = __ldg(k + t);
    const uint4 cs = __ldg(rope_h + ((size_t)(l >> 5) * 16 + c) * 32 + (l & 31));
    uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    const uint32_t h2[4] = {cs.x, cs.y, cs.z, cs.w};
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        float cc, ss;
        unpack_cs(h2[m], cc, ss);
        const float x0 = __uint_as_float(w[m] << 16);
        const float x1 = __uint_as_float(w[m] & 0xFFFF0000u);
        w[m] = pack_bf16(x0 * cc - x1 * ss, x0 * ss + x1 * cc);
    }
    out[t] = make_uint4(w[0], w[1], w[2], w[3]);
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

// Combines the parts of the split items of a step launch: a warp takes kMergeRows consecutive query
// rows of one tile (the item is decoded once per warp), a lane four output channels of each.  With
// part q's reference maximum m_q, row sum l_q and unnormalised row O_q:
//   out = sum_q 2^(m_q - m) O_q / sum_q 2^(m_q - m) l_q,   m = max_q m_q,   summed in part order.
constexpr int kMergeRows = 4;
__global__ void __launch_bounds__(256)
tc_split_merge_kernel(const TcStepParams p)
{
    const int warp = (int)((blockIdx.x * 256u + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    constexpr int kWarpsPerTile = kTile / kMergeRows;
    const int r0 = (warp % kWarpsPerTile) * kMergeRows, t = (warp / kWarpsPerTile) & 1, slot = warp / (2 * kWarpsPerTile);
    const bool in_range = slot < p.n_items - p.n_whole;
    Item it;
    if (in_range) it = decode_item<false>(p.n_whole + slot, p);
    const int k = p.k_split;
    const size_t tp0 = ((size_t)slot * 2 + t) * k;
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the step kernel has finished, its writes are visible
    if (!in_range || t >= it.ntile || p.status[kStatusError] != 0u) return;
    const int row0 = it.row0[t] + r0;
    __nv_bfloat16* obase = p.out + (((size_t)it.b[t] * p.s.L + row0) * p.s.H + it.h[t]) * kTile + lane * 4;
    // all loads of the warp's rows go out before the first use
    float2 ml[kMergeRows][kMaxSplit];
    float4 x[kMergeRows][kMaxSplit];
#pragma unroll
    for (int i = 0; i < kMergeRows; ++i) {
#pragma unroll
        for (int q = 0; q < kMaxSplit; ++q) {
            if (q < k && row0 + i < p.s.L) {
                const size_t rr = (tp0 + q) * kTile + r0 + i;
                ml[i][q] = *reinterpret_cast<const float2*>(p.split_ml + rr * 2);
                x[i][q] = *reinterpret_cast<const float4*>(p.split_o + rr * kTile + lane * 4);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kMergeRows; ++i) {
        if (row0 + i >= p.s.L) break;
        float m_all = -INFINITY;
#pragma unroll
        for (int q = 0; q < kMaxSplit; ++q)
            if (q < k) m_all = fmaxf(m_all, ml[i][q].x);
        float l_all = 0.0f;
        float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
        for (int q = 0; q < kMaxSplit; ++q) {
            if (q < k) {
                const float wq = ex2_approx(ml[i][q].x - m_all);
                l_all = fmaf(wq, ml[i][q].y, l_all);
                acc.x = fmaf(wq, x[i][q].x, acc.x);
                acc.y = fmaf(wq, x[i][q].y, acc.y);
                acc.z = fmaf(wq, x[i][q].z, acc.z);
                acc.w = fmaf(wq, x[i][q].w, acc.w);
            }
        }
        const float inv = 1.0f / l_all;
        *reinterpret_cast<uint2*>(obase + (size_t)i * p.s.H * kTile) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    }
}

std::mutex g_setup_mutex;
DeviceSetup g_setup[kMaxDevices];

int device_setup(int* num_sms)
{
    return device_setup_once(g_setup_mutex, g_setup, [] {
        cudaError_t e = opt_in_smem(tc_step_kernel<false, false>, kSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_step_kernel<true, false>, kSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_step_kernel<false, true>, kSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_token_prepare_kernel, kTPSmemBytes);
        if (e == cudaSuccess) e = opt_in_smem(tc_token_scan_kernel, kTSSmemBytes);
        return e;
    }, num_sms);
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

int tc_rope_k(const Shape& s, const void* k, const void* rope_h, void* k_rot, cudaStream_t st)
{
    const size_t total8 = (size_t)s.B * s.L * s.H * kTile / 8;
    tc_rope_k_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, st>>>(
        static_cast<const uint4*>(k), static_cast<const uint4*>(rope_h), static_cast<uint4*>(k_rot), s.L, s.H, total8);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_rope_k_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

int tc_prepare_rope(const float* cos_t, const float* sin_t, void* out, int L, cudaStream_t st)
{
    size_t total = (size_t)((L + kTile - 1) / kTile) * kTile * (kTile / 2);   // padded to whole tiles
    pack_rope_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(cos_t, sin_t, static_cast<__half2*>(out), L,
                                                                         total);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of pack_rope_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 1;
}

int tc_step(const StepArgs& a, const __nv_bfloat16* wq_op, const __nv_bfloat16* state_bf16, cudaStream_t st)
{
    int num_sms = 0;
    if (int r = device_setup(&num_sms)) return r;
    CUtensorMap tm_q, tm_k, tm_v, tm_w, tm_s;
    if (int r = make_map_blhd(&tm_q, a.q, a.s)) return r;
    Shape ks = a.s;
    ks.L = a.Lk > 0 ? a.Lk : a.s.L;   // K and V may be a longer cache
    if (int r = make_map_blhd(&tm_k, a.k_rot, ks)) return r;
    if (int r = make_map_blhd(&tm_v, a.v, ks)) return r;
    if (int r = make_map_rows(&tm_w, wq_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_s, state_bf16, (size_t)a.s.B * a.s.H * kTile)) return r;
    TcStepParams p;
    p.s = a.s;
    p.gate = a.gate;
    p.gate_mode = a.gate_mode;
    p.rope_cos = a.rope_cos;
    p.rope_sin = a.rope_sin;
    p.rope_h = static_cast<const uint4*>(a.rope_h);
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.status = a.status;
    p.spin_limit = a.wait_limit ? a.wait_limit - 1 : kSpinLimit;
    p.Lk = ks.L;
    p.n_q = (a.s.L + kTile - 1) / kTile;
    p.n_kv = (ks.L + kTile - 1) / kTile;
    const int bh = a.s.B * a.s.H;
    p.n_pair_items = bh * (p.n_q / 2);
    p.n_items = p.n_pair_items + ((p.n_q & 1) ? (bh + 1) / 2 : 0);   // ragged tiles go two by two
    // two item counters alternate between launches: a launch consumes one and clears the other
    p.sched_counter = a.status + kStatusSched + (a.launch_parity & 1);
    p.sched_next = a.status + kStatusSched + ((a.launch_parity + 1) & 1);
    const bool elem_gate = p.gate_mode == 2 && p.gate != nullptr;
    // The last wave: `rem` items on num_sms SMs.  Cut into k key ranges, the wave takes
    // ceil(rem k / SMs) rounds of one part each; a part costs its share of the key iterations plus
    // what every item costs (the readout iteration, the hand-over between items) plus the exchange
    // of the partial rows -- measured: 3.7 k clk per iteration, 10.8 k per item, about 6 k for the
    // exchange.  Take the k that makes the wave shortest, if that is shorter than leaving it whole.
    p.n_whole = p.n_items;
    p.k_split = 1;
    if (!elem_gate && a.split_o != nullptr) {
        const int waves = (p.n_items + num_sms - 1) / num_sms;
        const int rem = p.n_items - (waves - 1) * num_sms;
        const float iter = 3.74f, fixed = 10.8f, exchange = 6.0f;
        float best = (p.n_kv + 1) * iter + fixed;
        for (int k = 2; k <= kMaxSplit; ++k) {
            if (p.n_kv < 4 * k || (long)rem * k * 2 > a.split_tile_parts) break;
            const float part = ((float)p.n_kv / k + 1.0f) * iter + fixed + exchange;
            const float cost = (float)((rem * k + num_sms - 1) / num_sms) * part;
            if (cost < 0.95f * best) { best = cost; p.k_split = k; }
        }
        if (p.k_split > 1) p.n_whole = p.n_items - rem;
    }
    p.n_sched = p.n_whole + (p.n_items - p.n_whole) * p.k_split;
    p.split_o = a.split_o;
    p.split_ml = a.split_ml;
    const int grid = p.n_sched < num_sms ? p.n_sched : num_sms;
    if (elem_gate)
        tc_step_kernel<true, false><<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_w, tm_s, p);
    else if (p.k_split > 1)
        tc_step_kernel<false, true><<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_w, tm_s, p);
    else
        tc_step_kernel<false, false><<<grid, kThreads, kSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_w, tm_s, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_step_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    if (p.k_split == 1) return 1;
    // the parts' rows are combined by a second, small kernel (one warp per row); it may start
    // before the step kernel ends and waits for it at its griddepcontrol.wait
    const long warps = (long)(p.n_items - p.n_whole) * 2 * (kTile / kMergeRows);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((warps + 7) / 8));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, tc_split_merge_kernel, p);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_split_merge_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 2;
}

// Eq. 4 token by token with per-token gates on the tensor-core path (bf16 I/O, D = 128).  The
// scratch tensors of `a` (sized for the fp32 plain-FMA version) are used as bf16 here.
int tc_commit_tokens(const TokenCommitArgs& a, const __nv_bfloat16* wk_op, const __nv_bfloat16* wv_op,
                     const void* rope_h, uint32_t* status, cudaStream_t st)
{
    int num_sms = 0;
    if (int r = device_setup(&num_sms)) return r;
    (void)num_sms;
    if (a.state_bf16 == nullptr) { set_error("tc_commit_tokens: needs the bf16 copy of the state"); return ARL2_ERR_INVALID_ARG; }
    TcTokenParams p;
    p.s = a.s;
    p.rope_h = static_cast<const uint4*>(rope_h);
    p.alpha = a.alpha;
    p.beta = a.beta;
    p.w = reinterpret_cast<__nv_bfloat16*>(a.w);
    p.kh = reinterpret_cast<__nv_bfloat16*>(a.kh);
    p.u1 = reinterpret_cast<__nv_bfloat16*>(a.u1);
    p.gc = a.gc;
    p.state = a.state;
    p.state_bf16 = a.state_bf16;
    p.status = status;
    p.spin_limit = a.wait_limit ? a.wait_limit - 1 : kSpinLimit;
    p.ntile = (a.s.L + kTile - 1) / kTile;
    p.nchunk = (a.s.L + kTokC - 1) / kTokC;
    p.decayed = a.decayed ? 1 : 0;
    const size_t rows = (size_t)a.s.B * a.s.H * p.ntile * kTile;
    if (rows >= ((size_t)1 << 31)) { set_error("tc_commit_tokens: too many rows"); return ARL2_ERR_UNSUPPORTED; }
    CUtensorMap tm_k, tm_v, tm_wk, tm_wv, tm_w, tm_kh, tm_u1, tm_s;
    if (int r = make_map_blhd(&tm_k, a.k, a.s)) return r;
    if (int r = make_map_blhd(&tm_v, a.v, a.s)) return r;
    if (int r = make_map_rows(&tm_wk, wk_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_wv, wv_op, (size_t)a.s.H * kTile)) return r;
    if (int r = make_map_rows(&tm_w, p.w, rows)) return r;
    if (int r = make_map_rows(&tm_kh, p.kh, rows, kTokC)) return r;
    if (int r = make_map_rows(&tm_u1, p.u1, rows, kTokC)) return r;
    if (int r = make_map_rows(&tm_s, a.state_bf16, (size_t)a.s.B * a.s.H * kTile)) return r;
    dim3 grid1(p.ntile, a.s.H, a.s.B);
    tc_token_prepare_kernel<<<grid1, 128, kTPSmemBytes, st>>>(tm_k, tm_v, tm_wk, tm_wv, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_token_prepare_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    dim3 grid2(a.s.H, a.s.B);
    tc_token_scan_kernel<<<grid2, kTSThreads, kTSSmemBytes, st>>>(tm_w, tm_kh, tm_u1, tm_s, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("launch of tc_token_scan_kernel failed: %s", cudaGetErrorString(e)); return ARL2_ERR_CUDA; }
    return 2;
}

}  // namespace arl2
