// HCA attention of the draft layer (Section 3.2; the appendix's attention listing) for sm_100a.
//
// One persistent, warp-specialised kernel, two CTAs per SM. A work item is one (sequence, query head,
// tile of 128 query positions); it sweeps its causal key tiles of 64 keys. Per key tile:
//   S = Q K_t^T            tcgen05.mma, 128 x 64 x 128, fp32 in TMEM (two S buffers)
//   softmax warps          read S (one query row per thread), hide the columns past t - m (the causal
//                          part and the m substituted entries), update the row's running reference
//                          and sum, write P = 2^(x - ref) as bf16 pairs back into tensor memory, over
//                          the scores they were made from
//   O += P V_t             tcgen05.mma with P read from tensor memory and V_t as an MN-major operand
//                          from shared memory, fp32 in TMEM
// The substituted entries (t, t - i), i < m, ride the same pipeline as extra half-height tiles:
//   before the key tiles   S_ih = Q K_d[i]^T for the two 64-key halves h of the K_d[i] tile fetched
//                          i rows early, so that the wanted scores <Q[t], K_d[i][t - i]> sit on the
//                          diagonal of half h for the rows of half h; each thread keeps its element
//   at the last key tile   the m scores join the row maximum and sum
//   after the key tiles    O += diag_h(p_i) V_d[i] (half h of V_d[i] fetched i rows early; the P
//                          buffer holds just the weights of the rows of half h on its diagonal)
// so no thread reads global memory. The running reference moves only when a tile's maximum exceeds it
// by more than 2^8 (the O accumulator in TMEM is then rescaled in place by the softmax warps), so P
// stays within bf16 range and most tiles skip the rescale.
//
// Two CTAs share an SM (96 KB of shared memory and 256 TMEM columns each): while one CTA's softmax
// warps wait for the tensor core, TMEM or a barrier, the other's keep the exp2 unit busy.
// Warps: 0 = TMA producer (Q once per item, K and V tiles through two-stage rings),
//        1 = MMA issuer and TMEM owner, 2-5 = softmax + epilogue (TMEM lane quadrant = warp % 4).
// Every wait is bounded (wait_barrier); a wait that gives up sets the status word and all roles leave.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace hass {
namespace hca {

constexpr int QT = 128;            // query rows per item
constexpr int KT = 64;             // keys per tile
constexpr int HD = 128;            // head dimension
constexpr int MAX_DRAFTS = 8;      // m <= 8
constexpr int NUM_THREADS = 192;
constexpr int Q_BYTES = QT * HD * 2;                 // two halves (64 columns of the head dimension) of 128 rows x 128 B
constexpr int Q_HALF = Q_BYTES / 2;
constexpr int KV_BYTES = KT * HD * 2;                // two halves of 64 rows x 128 B
constexpr int KV_HALF = KV_BYTES / 2;
constexpr int SMEM_Q = 0;
constexpr int SMEM_K = SMEM_Q + Q_BYTES;             // 2 stages
constexpr int SMEM_V = SMEM_K + 2 * KV_BYTES;        // 2 stages
constexpr int SMEM_BAR = SMEM_V + 2 * KV_BYTES;
constexpr int NUM_BARS = 19;
constexpr int SMEM_BYTES = SMEM_BAR + 256;           // 98560: two CTAs fit the SM's 228 KB
constexpr int TMEM_COLS = 256;     // S0 at 0, S1 at 64 (P as bf16 pairs overwrites the first 32 columns of its S), O at 128
constexpr float RESCALE_LOG2 = 8.f;

struct Params {
    CUtensorMap tmQ;               // [B, T, H * 128], box {64, 128, 1}, 128-byte swizzle
    CUtensorMap tmK, tmV;          // [B, T, Hkv * 128], box {64, 64, 1}
    CUtensorMap tmKd[MAX_DRAFTS];  // the draft passes' keys and values, same geometry; index = sub-diagonal
    CUtensorMap tmVd[MAX_DRAFTS];
    __nv_bfloat16* O;              // [B, T, H, 128]
    float* lse;                    // [B, H, T] or null
    int B, T, H, Hkv, m;
    int q_tiles;                   // ceil(T / 128)
    int k_tiles;                   // ceil(T / 64)
    int items;                     // B * H * q_tiles
    float c2;                      // scale * log2(e)
    unsigned int* status;
};

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap* tm, uint32_t bar, int x, int y,
                                            int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

__global__ void __launch_bounds__(NUM_THREADS, 2) hca_attention_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0u) {
        // the swizzled tiles need a 1024-byte aligned window; report instead of computing garbage
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (20u << 8) | 1u);
        return;
    }
    const uint32_t bar0 = base + SMEM_BAR;
    // barriers
    const uint32_t q_full = bar0, q_empty = bar0 + 8;
    auto k_full = [&](int b) { return bar0 + 8u * (2 + b); };
    auto k_empty = [&](int b) { return bar0 + 8u * (4 + b); };
    auto v_full = [&](int b) { return bar0 + 8u * (6 + b); };
    auto v_empty = [&](int b) { return bar0 + 8u * (8 + b); };
    auto s_full = [&](int b) { return bar0 + 8u * (10 + b); };
    auto s_empty = [&](int b) { return bar0 + 8u * (12 + b); };
    // one per S buffer: with a single barrier a warp one element ahead could arrive twice in one phase
    auto p_full = [&](int b) { return bar0 + 8u * (14 + b); };
    auto pv_done = [&](int b) { return bar0 + 8u * (16 + b); };     // PV product that read P from S buffer b
    const uint32_t o_free = bar0 + 8u * 18;
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_raw + SMEM_BAR + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(k_full(b), 1);
            mbar_init(k_empty(b), 1);
            mbar_init(v_full(b), 1);
            mbar_init(v_empty(b), 1);
            mbar_init(s_full(b), 1);
            mbar_init(s_empty(b), 4);
        }
        mbar_init(p_full(0), 4);
        mbar_init(p_full(1), 4);
        mbar_init(pv_done(0), 1);
        mbar_init(pv_done(1), 1);
        mbar_init(o_free, 4);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmQ);
        prefetch_tensormap(&p.tmK);
        prefetch_tensormap(&p.tmV);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_ptr_smem), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;

    const int BH = p.B * p.H;
    const int rep = p.H / p.Hkv;
    const int m = p.m;
    // item -> (query tile, sequence, head): the longest items (last query tiles) come first
    auto decode = [&](int item, int& qt, int& b, int& h) {
        qt = p.q_tiles - 1 - item / BH;
        const int bh = item - (item / BH) * BH;
        b = bh / p.H;
        h = bh - b * p.H;
    };
    // Items are sorted longest first; round k hands items k*G .. k*G + G-1 to the G CTAs, in alternating
    // direction, so that a CTA that got a long item in one round gets a short one in the next.
    auto first_item = [&](uint32_t k) {
        const int G = gridDim.x, c = blockIdx.x;
        return static_cast<int>(k) * G + ((k & 1u) ? G - 1 - c : c);
    };
    // key tiles of an item: 0 .. 2 qt + 1, cut at the end of the sequence
    auto key_tiles = [&](int qt) { return min(2 * qt + 2, p.k_tiles); };
    // Per item the tensor core runs two sequences, each with its own ring counter:
    //   score sequence (K ring, S buffers), length 2m + n: draft pass i, half h (element 2i + h), then key tiles 0 .. n-1
    //   value sequence (V ring, P buffer),  length n + 2m: key tiles 0 .. n-1, then draft pass i, half h

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            uint32_t gk = 0, gv = 0, it = 0;
            bool ok = true;
            auto load_k = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int s = gk & 1u;
                if (!wait_barrier(k_empty(s), ((gk >> 1) & 1u) ^ 1u, abort_flag, p.status, 2)) return false;
                mbar_arrive_expect_tx(k_full(s), KV_BYTES);
                tma_load_3d(base + SMEM_K + s * KV_BYTES, tm, k_full(s), col, row, b);
                tma_load_3d(base + SMEM_K + s * KV_BYTES + KV_HALF, tm, k_full(s), col + 64, row, b);
                ++gk;
                return true;
            };
            auto load_v = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int s = gv & 1u;
                if (!wait_barrier(v_empty(s), ((gv >> 1) & 1u) ^ 1u, abort_flag, p.status, 3)) return false;
                mbar_arrive_expect_tx(v_full(s), KV_BYTES);
                tma_load_3d(base + SMEM_V + s * KV_BYTES, tm, v_full(s), col, row, b);
                tma_load_3d(base + SMEM_V + s * KV_BYTES + KV_HALF, tm, v_full(s), col + 64, row, b);
                ++gv;
                return true;
            };
            for (int item = first_item(0); item < p.items && ok; item = first_item(++it)) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int col = (h / rep) * HD;
                const int n = key_tiles(qt);
                if (!wait_barrier(q_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(q_full, Q_BYTES);
                tma_load_3d(base + SMEM_Q, &p.tmQ, q_full, h * HD, qt * QT, b);
                tma_load_3d(base + SMEM_Q + Q_HALF, &p.tmQ, q_full, h * HD + 64, qt * QT, b);
                // draft keys start i rows early: row r of half hf is position qt*128 + 64 hf + r - i (zeros before the sequence)
                for (int e = 0; e < 2 * m && ok; ++e) ok = load_k(&p.tmKd[e >> 1], col, qt * QT + 64 * (e & 1) - (e >> 1), b);
                for (int j = 0; j < n && ok; ++j) {
                    ok = load_k(&p.tmK, col, j * KT, b);
                    if (ok) ok = load_v(&p.tmV, col, j * KT, b);
                }
                for (int e = 0; e < 2 * m && ok; ++e) ok = load_v(&p.tmVd[e >> 1], col, qt * QT + 64 * (e & 1) - (e >> 1), b);
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        // The whole warp runs this loop so that addresses and descriptors stay warp-uniform; one elected lane
        // issues the tensor-core instructions.
        {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(QT, HD, 0, 1);
            const uint32_t tmem_o = tmem_base + 2 * KT;
            uint32_t gk = 0, gv = 0, it = 0;
            bool ok = true;
            auto wait_all = [&](uint32_t bar, uint32_t parity, unsigned code) {
                return __all_sync(0xffffffffu, wait_barrier(bar, parity, abort_flag, p.status, code)) != 0;
            };
            // next element of the score sequence: S = Q K^T into S buffer gk & 1
            auto issue_s = [&]() -> bool {
                const int s = gk & 1u;
                const uint32_t ph = (gk >> 1) & 1u;
                if (!wait_all(k_full(s), ph, 4)) return false;
                if (!wait_all(s_empty(s), ph ^ 1u, 5)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint64_t a_desc = make_smem_desc_sw128(base + SMEM_Q + (k >> 2) * Q_HALF + (k & 3) * 32, 0, 1024);
                    const uint64_t b_desc =
                        make_smem_desc_sw128(base + SMEM_K + s * KV_BYTES + (k >> 2) * KV_HALF + (k & 3) * 32, 0, 1024);
                    if (leader) umma_bf16(tmem_base + s * KT, a_desc, b_desc, idesc_s, k != 0 ? 1u : 0u);
                }
                if (leader) {
                    umma_commit(k_empty(s));
                    umma_commit(s_full(s));
                }
                __syncwarp();
                ++gk;
                return true;
            };
            // next element of the value sequence: O (+)= P V
            auto issue_pv = [&](bool first) -> bool {
                const int s = gv & 1u;
                if (!wait_all(p_full(s), (gv >> 1) & 1u, 7)) return false;
                if (!wait_all(v_full(s), (gv >> 1) & 1u, 8)) return false;
                if (first && !wait_all(o_free, (it & 1u) ^ 1u, 9)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < KT / 16; ++k) {
                    // A = P from tensor memory (8 columns of bf16 pairs per 16 keys, in the S buffer the scores came
                    // from). B = V: 64-column groups KV_HALF apart, 16 keys further = 16 rows of 128 bytes.
                    const uint64_t b_desc =
                        make_smem_desc_sw128(base + SMEM_V + s * KV_BYTES + k * 16 * 128, KV_HALF, 1024);
                    if (leader) umma_bf16_ta(tmem_o, tmem_base + s * KT + 8 * k, b_desc, idesc_o, (!first || k != 0) ? 1u : 0u);
                }
                if (leader) {
                    umma_commit(v_empty(s));
                    umma_commit(pv_done(s));
                }
                __syncwarp();
                ++gv;
                return true;
            };
            for (int item = first_item(0); item < p.items && ok; item = first_item(++it)) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int n_s = 2 * m + key_tiles(qt);
                if (!wait_all(q_full, it & 1u, 6)) break;
                if (!issue_s()) break;
                if (n_s == 1 && elect_one()) umma_commit(q_empty);
                for (int a = 0; a < n_s && ok; ++a) {
                    if (a + 1 < n_s) {
                        ok = issue_s();
                        if (ok && a + 2 == n_s && elect_one()) umma_commit(q_empty);      // Q is free once the item's last S has read it
                    }
                    if (ok && a >= 2 * m) ok = issue_pv(a == 2 * m);
                }
                for (int e = 0; e < 2 * m && ok; ++e) ok = issue_pv(false);
            }
        }
    } else {
        // ===================== softmax + epilogue warps =====================
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                       // row of the tile = TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tmem_o = tmem_base + 2 * KT + lane_addr;
        uint32_t gk = 0, gv = 0;
        bool ok = true;
        // The weights of value-sequence element gv go, as bf16 pairs, into the first 32 columns of S buffer gv & 1:
        // for a key tile that is the buffer its scores came from (both sequences advance by the same even count
        // per item), already copied to registers; the tensor core takes products in issue order, so the next
        // score product into that buffer runs after the PV product that reads these weights.
        // PV(x) complete <=> pv_done(x & 1) has finished phase x >> 1.
        auto pv_wait = [&](uint32_t x, unsigned code) {
            return wait_barrier(pv_done(x & 1u), (x >> 1) & 1u, abort_flag, p.status, code);
        };
        for (int item = first_item(0), it = 0; item < p.items && ok; item = first_item(++it)) {
            int qt, b, h;
            decode(item, qt, b, h);
            const int n = key_tiles(qt);
            const int t = qt * QT + r;                        // position in the sequence
            const bool valid = t < p.T;
            // ---- draft passes of the score sequence: keep the diagonal element of each S_ih (raw, unscaled) ----
            float sd[MAX_DRAFTS];
#pragma unroll
            for (int i = 0; i < MAX_DRAFTS; ++i) sd[i] = 0.f;
#pragma unroll 1
            for (int e = 0; e < 2 * m; ++e, ++gk) {
                const int s = gk & 1u;
                if (!wait_barrier(s_full(s), (gk >> 1) & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                if ((quad >> 1) == (e & 1)) {                  // this warp's rows lie in half e & 1
                    uint32_t raw[32];
                    tmem_ld32(tmem_base + s * KT + lane_addr + 32 * (quad & 1), raw);     // this warp's diagonal block
                    tmem_ld_wait(raw);
                    float dv = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c == lane) dv = __uint_as_float(raw[c]);
#pragma unroll
                    for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                        if (ii == (e >> 1)) sd[ii] = dv;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(s));
            }
            if (!ok) break;
            float mref = -INFINITY, l = 0.f;
            for (int j = 0; j < n; ++j, ++gk, ++gv) {
                const int s = gk & 1u;
                if (!wait_barrier(s_full(s), (gk >> 1) & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * KT + lane_addr;
                const bool last = (j == n - 1);
                // Columns past t - m are hidden in the score tile: the causal part (s > t) and the m substituted
                // entries (t - m < s <= t), which enter the row's maximum and sum as scalars at the last tile.
                // Only tiles reaching past the first row's limit can hold such columns.
                const bool band = j * KT + KT - 1 > qt * QT - m;
                const int lim = t - m - j * KT;
                // the row's 64 scores into registers, then the S buffer goes back to the tensor core
                uint32_t raw[2][32];
                tmem_ld32(tmem_s, raw[0]);
                tmem_ld32(tmem_s + 32, raw[1]);
                tmem_ld_wait(raw[0]);
                tmem_ld_wait(raw[1]);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(s));
                float v[2][32];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) v[k][c] = __uint_as_float(raw[k][c]);
                    if (band) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (32 * k + c > lim) v[k][c] = -INFINITY;
                    }
                }
                float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = fmax3(mx0, v[k][c], v[k][c + 1]);
                        mx1 = fmax3(mx1, v[k][c + 2], v[k][c + 3]);
                    }
                }
                if (last) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) mx0 = fmaxf(mx0, sd[i]);
                }
                const float cand = fmaxf(mx0, mx1) * p.c2;
                if (j == 0) {
                    mref = cand;
                } else {
                    const bool grow = cand > mref + RESCALE_LOG2;      // also true when every earlier column of the row was hidden
                    if (__any_sync(0xffffffffu, grow)) {
                        // rescale the accumulator: O of this row *= 2^(old ref - new ref); needs the previous PV complete
                        const float f = grow ? ex2(mref - cand) : 1.f;
                        if (grow) {
                            mref = cand;
                            l *= f;
                        }
                        if (!pv_wait(gv - 1, 11)) { ok = false; break; }
                        tc_fence_after_sync();
#pragma unroll 1
                        for (int c0 = 0; c0 < HD; c0 += 32) {
                            uint32_t o[32];
                            tmem_ld32(tmem_o + c0, o);
                            tmem_ld_wait(o);
#pragma unroll
                            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
                            tmem_st32(tmem_o + c0, o);
                        }
                        tmem_st_wait();
                        tc_fence_before_sync();
                    }
                }
                // ---- P = 2^(x c2 - ref): row sum in fp32, bf16 into shared memory ----
                // (a row whose columns were all hidden so far has ref = -inf; it gets P = 0, not 2^(-inf + inf))
                const float nref = mref == -INFINITY ? 0.f : -mref;
                float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        ffma2(x0, x1, v[k][c], v[k][c + 1], p.c2, p.c2, nref, nref);
                        v[k][c] = ex2(x0);
                        v[k][c + 1] = ex2(x1);
                        fadd2(ls0, ls1, ls0, ls1, v[k][c], v[k][c + 1]);
                    }
                }
                l += ls0 + ls1;
                if (last) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) l += ex2(fmaf(sd[i], p.c2, nref));
                }
                if (gv >= 2 && !pv_wait(gv - 2, 12)) { ok = false; break; }     // the last weights in this buffer have been read
                {
                    uint32_t pk[32];
#pragma unroll
                    for (int k = 0; k < 2; ++k)
#pragma unroll
                        for (int c = 0; c < 32; c += 2) pk[16 * k + (c >> 1)] = pack_bf16(v[k][c], v[k][c + 1]);
                    tmem_st32(tmem_s, pk);
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(gv & 1u));
            }
            if (!ok) break;
            // ---- draft passes of the value sequence: P holds only the weights 2^(sd c2 - ref) of the rows of one
            //      half on its diagonal ----
            const float nref_f = mref == -INFINITY ? 0.f : -mref;
#pragma unroll 1
            for (int e = 0; e < 2 * m; ++e, ++gv) {
                const int i = e >> 1;
                float sdi = 0.f;
#pragma unroll
                for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                    if (ii == i) sdi = sd[ii];
                const bool mine = (r >> 6) == (e & 1) && t - i >= 0;
                const float pi = mine ? ex2(fmaf(sdi, p.c2, nref_f)) : 0.f;
                const uint32_t bits = pack_bf16(pi, 0.f) << ((r & 1) * 16);        // key r & 63 sits in word (r & 63) / 2
                if (gv >= 2 && !pv_wait(gv - 2, 14)) { ok = false; break; }
                {
                    uint32_t pk[32];
#pragma unroll
                    for (int w = 0; w < 32; ++w) pk[w] = (w == ((r & 63) >> 1)) ? bits : 0u;
                    tmem_st32(tmem_base + (gv & 1u) * KT + lane_addr, pk);
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(gv & 1u));
            }
            if (!ok) break;
            // ---- epilogue: O / l as bf16, each thread stores its own 256-byte row ----
            {
                if (!pv_wait(gv - 1, 13)) break;
                tc_fence_after_sync();
                const float inv = 1.f / l;
                if (valid && p.lse != nullptr)
                    p.lse[(static_cast<size_t>(b) * p.H + h) * p.T + t] = (mref + log2f(l)) * 0.6931471805599453f;
                __nv_bfloat16* orow = p.O + ((static_cast<size_t>(b) * p.T + (valid ? t : 0)) * p.H + h) * HD;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t raw[2][32];
                    tmem_ld32(tmem_o + 64 * hf, raw[0]);
                    tmem_ld32(tmem_o + 64 * hf + 32, raw[1]);
                    tmem_ld_wait(raw[0]);
                    tmem_ld_wait(raw[1]);
                    if (hf == 1) {
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(o_free);     // the accumulator may be overwritten by the next item
                    }
                    if (valid) {
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
#pragma unroll
                            for (int q8 = 0; q8 < 2; ++q8) {
                                const uint32_t* x = &raw[k][16 * q8];
                                st_global_v8(orow + 64 * hf + 32 * k + 16 * q8,
                                             pack_bf16(__uint_as_float(x[0]) * inv, __uint_as_float(x[1]) * inv),
                                             pack_bf16(__uint_as_float(x[2]) * inv, __uint_as_float(x[3]) * inv),
                                             pack_bf16(__uint_as_float(x[4]) * inv, __uint_as_float(x[5]) * inv),
                                             pack_bf16(__uint_as_float(x[6]) * inv, __uint_as_float(x[7]) * inv),
                                             pack_bf16(__uint_as_float(x[8]) * inv, __uint_as_float(x[9]) * inv),
                                             pack_bf16(__uint_as_float(x[10]) * inv, __uint_as_float(x[11]) * inv),
                                             pack_bf16(__uint_as_float(x[12]) * inv, __uint_as_float(x[13]) * inv),
                                             pack_bf16(__uint_as_float(x[14]) * inv, __uint_as_float(x[15]) * inv));
                            }
                        }
                    }
                }
            }
        }
    }

    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // a wait gave up: let copies that may still be in flight land before the CTA's memory is released
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace hca
}  // namespace hass
