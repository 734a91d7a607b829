// HCA attention of the draft layer (Section 3.2; the appendix's attention listing), forward, for sm_100a.
//
// One persistent, warp-specialised kernel, one CTA per SM. A CTA works on a PAIR of items at a time, an item
// being one (sequence, query head, tile of 128 query positions); the two items of a pair read the same
// key/value head, so every 128-key tile is fetched once and used by both:
//   - grouped heads with an even group size: two query heads of one group, same query tile;
//   - otherwise: two consecutive query tiles of one head (the lower one stops one key tile earlier).
// Each item owns a "slot": its Q tile in shared memory, a 128-column score buffer and a 128-column output
// accumulator in tensor memory, and four softmax warps. Per key tile and slot:
//   S = Q K_t^T            tcgen05.mma, 128 x 128 x 128, fp32 in TMEM
//   softmax warps          one query row per thread, its 128 scores in registers: hide the columns past t - m (the
//                          causal part and the m substituted entries), update the row's running reference and
//                          sum, write P = 2^(x - ref) as bf16 pairs back into tensor memory over the scores
//   O += P V_t             tcgen05.mma with P read from tensor memory, V_t an MN-major operand from shared memory
// The tensor core alternates between the slots, so one slot's products run while the other slot's rows are in
// their softmax. The products of a slot are issued in the order S(j), PV(j), S(j+1); the tensor core
// completes them in that order, so a finished S(j+1) means PV(j) has finished too and the softmax warps may
// touch the accumulator (rare rescale) without another barrier.
// The substituted entries (t, t - i), i < m, ride the same pipeline as extra products: before the key tiles
// S = Q K_d[i]^T with the K_d[i] tile fetched i rows early, so that the wanted scores sit on the diagonal and
// each row's thread keeps its own; the m scores join the row's maximum and sum at the last key tile; after
// the key tiles O += diag(p_i) V_d[i] with V_d[i] fetched i rows early. No thread reads global memory.
// The running reference moves only when a tile's maximum exceeds it by more than 2^8 (the accumulator is then
// rescaled in place by the row's thread), so P stays within bf16 range and almost every tile skips the rescale.
// Warps: 0 = TMA producer, 1 = MMA issuer and TMEM owner (2, 3 idle), 4-7 = softmax + epilogue of slot 0,
// 8-11 = of slot 1 (TMEM lane quadrant = warp % 4). The first warpgroup gives registers up (setmaxnreg) and the
// two softmax warpgroups take them: a row's 128 scores stay in registers. Every wait is bounded (wait_barrier); a wait that gives up sets the status
// word and all roles leave.
#pragma once
#include <cuda_bf16.h>

#include "hca_kernels.cuh"
#include "ptx.cuh"

namespace hass {
namespace hca2 {

using hca::ex2;
using hca::pack_bf16;
using hca::tma_load_3d;
using hca::tmem_st32;
using hca::tmem_st_wait;

constexpr int QT = 128;            // query rows per item
constexpr int KT = 128;            // keys per tile
constexpr int HD = 128;            // head dimension
constexpr int MAX_DRAFTS = 8;
constexpr int NUM_THREADS = 384;   // three warpgroups: {TMA, MMA, 2 idle warps}, softmax of slot 0, softmax of slot 1
constexpr int REGS_CONTROL = 56;   // registers per thread after the split (launch: 168 each; 56 + 2 * 224 = 3 * 168)
constexpr int REGS_SOFTMAX = 224;
constexpr int Q_BYTES = QT * HD * 2;                 // two halves (64 columns of the head dimension) of 128 rows x 128 B
constexpr int Q_HALF = Q_BYTES / 2;
constexpr int KV_BYTES = KT * HD * 2;
constexpr int KV_HALF = KV_BYTES / 2;
constexpr int KV_STAGES = 2;          // value tiles in flight
constexpr int K_STAGES = 3;           // key tiles in flight: one more, the draft passes' key tiles occupy the ring at an item's start
constexpr int SMEM_Q = 0;                            // 2 slots
constexpr int SMEM_K = SMEM_Q + 2 * Q_BYTES;
constexpr int SMEM_V = SMEM_K + K_STAGES * KV_BYTES;
constexpr int SMEM_BAR = SMEM_V + KV_STAGES * KV_BYTES;
constexpr int SCHED_DEPTH = 4;       // pair indices published ahead by the producer
constexpr int NUM_BARS = 4 + 2 * K_STAGES + 2 * KV_STAGES + 6 + 2 * SCHED_DEPTH;
constexpr int SMEM_BYTES = SMEM_BAR + 256;           // 229632
static_assert(8 * NUM_BARS + 4 * (2 + SCHED_DEPTH) <= 256 && SMEM_BYTES <= 232448, "shared-memory window");
constexpr int TMEM_COLS = 512;     // S of slot s at 128 s (P overwrites its first 64 columns), O of slot s at 256 + 128 s
constexpr float RESCALE_LOG2 = 8.f;

struct Params {
    CUtensorMap tmQ;               // [B, T, H * 128], box {64, 128, 1}, 128-byte swizzle
    CUtensorMap tmK, tmV;          // [B, T, Hkv * 128], box {64, 128, 1}
    CUtensorMap tmKd[MAX_DRAFTS];  // the draft passes' keys and values, same geometry; index = sub-diagonal
    CUtensorMap tmVd[MAX_DRAFTS];
    __nv_bfloat16* O;              // [B, T, H, 128]
    float* lse;                    // [B, H, T] or null
    int B, T, H, Hkv, m;
    int q_tiles;                   // ceil(T / 128)
    int pairs;                     // work units
    int head_pairing;              // 1: a pair = heads 2u, 2u + 1 at one query tile; 0: one head, query tiles qt - 1, qt
    float c2;                      // scale * log2(e)
    unsigned int* status;
};

struct Pair {
    int b, kv_col;                 // sequence; first column of the key/value head in [B, T, Hkv * 128]
    int h[2], qt[2];               // slot 0 / slot 1: query head and query tile
    bool act0;                     // slot 0 has an item (slot 1 always has one, and never the shorter one)
};

__device__ __forceinline__ Pair decode_pair(const Params& p, int idx) {
    Pair r;
    const int rep = p.H / p.Hkv;
    if (p.head_pairing) {
        const int per = p.B * (p.H >> 1);
        const int u = idx / per, rem = idx - u * per;
        r.b = rem / (p.H >> 1);
        const int hp = rem - r.b * (p.H >> 1);
        r.h[0] = 2 * hp;
        r.h[1] = 2 * hp + 1;
        r.qt[0] = r.qt[1] = p.q_tiles - 1 - u;          // longest first
        r.act0 = true;
    } else {
        const int per = p.B * p.H;
        const int u = idx / per, rem = idx - u * per;
        r.b = rem / p.H;
        r.h[0] = r.h[1] = rem - r.b * p.H;
        r.qt[1] = p.q_tiles - 1 - 2 * u;
        r.qt[0] = r.qt[1] - 1;
        r.act0 = r.qt[0] >= 0;
    }
    r.kv_col = (r.h[1] / rep) * HD;
    return r;
}

__global__ void __launch_bounds__(NUM_THREADS, 1) hca_attention_pair_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0u) {
        // the swizzled tiles need a 1024-byte aligned window; report instead of computing garbage
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (20u << 8) | 1u);
        return;
    }
    const uint32_t bar0 = base + SMEM_BAR;
    auto q_full = [&](int s) { return bar0 + 8u * s; };
    auto q_empty = [&](int s) { return bar0 + 8u * (2 + s); };
    auto k_full = [&](int st) { return bar0 + 8u * (4 + st); };
    constexpr int KVB = 2 * K_STAGES + 2 * KV_STAGES;      // barriers of the two rings
    auto k_empty = [&](int st) { return bar0 + 8u * (4 + K_STAGES + st); };
    auto v_full = [&](int st) { return bar0 + 8u * (4 + 2 * K_STAGES + st); };
    auto v_empty = [&](int st) { return bar0 + 8u * (4 + 2 * K_STAGES + KV_STAGES + st); };
    auto s_full = [&](int s) { return bar0 + 8u * (4 + KVB + s); };
    auto p_full = [&](int s) { return bar0 + 8u * (6 + KVB + s); };
    auto pv_done = [&](int s) { return bar0 + 8u * (8 + KVB + s); };
    auto sched_full = [&](int e) { return bar0 + 8u * (10 + KVB + e); };
    auto sched_empty = [&](int e) { return bar0 + 8u * (10 + KVB + SCHED_DEPTH + e); };
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_raw + SMEM_BAR + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);
    volatile int* sched_idx = reinterpret_cast<volatile int*>(tmem_ptr_smem + 2);      // [SCHED_DEPTH]

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(q_full(s), 1);
            mbar_init(q_empty(s), 1);
            mbar_init(s_full(s), 1);
            mbar_init(p_full(s), 4);
            mbar_init(pv_done(s), 1);
        }
        for (int st = 0; st < K_STAGES; ++st) {
            mbar_init(k_full(st), 1);
            mbar_init(k_empty(st), 1);
        }
        for (int st = 0; st < KV_STAGES; ++st) {
            mbar_init(v_full(st), 1);
            mbar_init(v_empty(st), 1);
        }
        for (int e = 0; e < SCHED_DEPTH; ++e) {
            mbar_init(sched_full(e), 1);
            mbar_init(sched_empty(e), 9);      // the MMA warp and the eight softmax warps
        }
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

    // Pairs are sorted longest first and handed out dynamically: the producer takes the next index from a counter in
    // the workspace (word 1, zeroed by the host before the launch) and publishes it to the other roles through a
    // small queue in shared memory, so a CTA that falls behind simply takes fewer pairs. An index >= pairs ends a role.
    // next_pair(k): the k-th index this CTA works on (every consumer warp calls it once per k).
    auto next_pair = [&](uint32_t k, unsigned code) -> int {
        const int e = k % SCHED_DEPTH;
        if (!wait_barrier(sched_full(e), (k / SCHED_DEPTH) & 1u, abort_flag, p.status, code)) return INT_MAX;
        const int idx = sched_idx[e];
        __syncwarp();
        if (lane == 0) mbar_arrive(sched_empty(e));
        return idx;
    };

    // Per item and slot the tensor core runs, in this order:
    //   m draft score products   S = Q K_d[i]^T with the K_d[i] tile fetched i rows early, so that the wanted
    //                            scores <Q[t], K_d[i][t - i]> sit on the tile's diagonal; the row's thread keeps its own
    //   n key tiles              S = Q K_t^T -> softmax -> O += P V_t
    //   m draft value products   O += diag(p_i) V_d[i] (V_d[i] fetched i rows early; P holds the row's weight on
    //                            the diagonal and zeros elsewhere), two passes per arrival of the softmax warps
    // Every product of a slot but the first S follows an arrival of the slot's softmax warps on p_full.
    // The K ring carries the draft key tiles, then the key tiles; the V ring the value tiles, then the draft
    // value tiles. A tile both slots use (always, when the pair is two heads of one group; the key/value
    // tiles otherwise) is one ring entry, released after the second slot's product.
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            uint32_t gq[2] = {0u, 0u}, gk = 0, gv = 0, it = 0;
            bool ok = true;
            auto load_k = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int st = gk % K_STAGES;
                if (!wait_barrier(k_empty(st), ((gk / K_STAGES) & 1u) ^ 1u, abort_flag, p.status, 2)) return false;
                mbar_arrive_expect_tx(k_full(st), KV_BYTES);
                tma_load_3d(base + SMEM_K + st * KV_BYTES, tm, k_full(st), col, row, b);
                tma_load_3d(base + SMEM_K + st * KV_BYTES + KV_HALF, tm, k_full(st), col + 64, row, b);
                ++gk;
                return true;
            };
            auto load_v = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int st = gv % KV_STAGES;
                if (!wait_barrier(v_empty(st), ((gv / KV_STAGES) & 1u) ^ 1u, abort_flag, p.status, 3)) return false;
                mbar_arrive_expect_tx(v_full(st), KV_BYTES);
                tma_load_3d(base + SMEM_V + st * KV_BYTES, tm, v_full(st), col, row, b);
                tma_load_3d(base + SMEM_V + st * KV_BYTES + KV_HALF, tm, v_full(st), col + 64, row, b);
                ++gv;
                return true;
            };
            for (;; ++it) {
                const int idx = static_cast<int>(atomicAdd(p.status + 1, 1u));
                {
                    const int e = it % SCHED_DEPTH;
                    if (!wait_barrier(sched_empty(e), ((it / SCHED_DEPTH) & 1u) ^ 1u, abort_flag, p.status, 15)) break;
                    sched_idx[e] = idx;
                    mbar_arrive(sched_full(e));
                }
                if (idx >= p.pairs || !ok) break;
                const Pair pr = decode_pair(p, idx);
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    if (s == 0 && !pr.act0) continue;
                    if (!wait_barrier(q_empty(s), (gq[s] & 1u) ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
                    mbar_arrive_expect_tx(q_full(s), Q_BYTES);
                    tma_load_3d(base + SMEM_Q + s * Q_BYTES, &p.tmQ, q_full(s), pr.h[s] * HD, pr.qt[s] * QT, pr.b);
                    tma_load_3d(base + SMEM_Q + s * Q_BYTES + Q_HALF, &p.tmQ, q_full(s), pr.h[s] * HD + 64, pr.qt[s] * QT, pr.b);
                    ++gq[s];
                }
                const int n = pr.qt[1] + 1;
                // draft keys start i rows early: row c of the tile is position qt * 128 + c - i (zeros before the sequence)
                for (int i = 0; i < p.m && ok; ++i) {
                    if (!p.head_pairing && pr.act0) ok = load_k(&p.tmKd[i], pr.kv_col, pr.qt[0] * QT - i, pr.b);
                    if (ok) ok = load_k(&p.tmKd[i], pr.kv_col, pr.qt[1] * QT - i, pr.b);
                }
                for (int j = 0; j < n && ok; ++j) {
                    ok = load_k(&p.tmK, pr.kv_col, j * KT, pr.b);
                    if (ok) ok = load_v(&p.tmV, pr.kv_col, j * KT, pr.b);
                }
                for (int i = 0; i < p.m && ok; ++i) {
                    if (!p.head_pairing && pr.act0) ok = load_v(&p.tmVd[i], pr.kv_col, pr.qt[0] * QT - i, pr.b);
                    if (ok) ok = load_v(&p.tmVd[i], pr.kv_col, pr.qt[1] * QT - i, pr.b);
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        // The whole warp runs this loop so that addresses and descriptors stay warp-uniform; one elected lane
        // issues the tensor-core instructions.
        constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
        constexpr uint32_t idesc_o = make_idesc_bf16(QT, HD, 0, 1);
        uint32_t gq[2] = {0u, 0u}, gp[2] = {0u, 0u}, gk = 0, gv = 0, it = 0;
        bool ok = true;
        // tcgen05.commit follows the products of the thread that issued them: one lane, elected once, issues all
        const bool leader = elect_one();
        auto wait_all = [&](uint32_t bar, uint32_t parity, unsigned code) {
            return __all_sync(0xffffffffu, wait_barrier(bar, parity, abort_flag, p.status, code)) != 0;
        };
        // S of slot s from K stage st; last: the item's last score product (its Q tile is free afterwards)
        auto issue_s = [&](int s, int st, bool last) {
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < HD / 16; ++k) {
                const uint64_t a_desc = make_smem_desc_sw128(base + SMEM_Q + s * Q_BYTES + (k >> 2) * Q_HALF + (k & 3) * 32, 0, 1024);
                const uint64_t b_desc = make_smem_desc_sw128(base + SMEM_K + st * KV_BYTES + (k >> 2) * KV_HALF + (k & 3) * 32, 0, 1024);
                if (leader) umma_bf16(tmem_base + s * KT, a_desc, b_desc, idesc_s, k != 0 ? 1u : 0u);
            }
            if (leader) {
                umma_commit(s_full(s));
                if (last) umma_commit(q_empty(s));
            }
            __syncwarp();
        };
        // O of slot s (+)= P V: keys [16 k0, 16 k1) of V stage st, P read from the slot's S buffer starting at column
        // a_col (8 columns of bf16 pairs per 16 keys). B = V: 64-column groups KV_HALF apart, 16 keys further = 16
        // rows of 128 bytes. first: the item's first product into O; commit: signal pv_done afterwards.
        auto issue_pv = [&](int s, int st, int a_col, int k0, int k1, bool first, bool commit) {
            tc_fence_after_sync();
#pragma unroll
            for (int k = k0; k < k1; ++k) {
                const uint64_t b_desc = make_smem_desc_sw128(base + SMEM_V + st * KV_BYTES + k * 16 * 128, KV_HALF, 1024);
                if (leader) umma_bf16_ta(tmem_base + 256 + s * HD, tmem_base + s * KT + a_col + 8 * (k - k0), b_desc, idesc_o, (!first || k != k0) ? 1u : 0u);
            }
            if (leader && commit) umma_commit(pv_done(s));
            __syncwarp();
        };
        auto k_acquire = [&](int& st) {
            st = gk % K_STAGES;
            return wait_all(k_full(st), (gk / K_STAGES) & 1u, 4);
        };
        auto k_release = [&](int st) {
            if (leader) umma_commit(k_empty(st));
            __syncwarp();
            ++gk;
        };
        auto v_acquire = [&](int& st) {
            st = gv % KV_STAGES;
            return wait_all(v_full(st), (gv / KV_STAGES) & 1u, 8);
        };
        auto v_release = [&](int st) {
            if (leader) umma_commit(v_empty(st));
            __syncwarp();
            ++gv;
        };
        auto p_wait = [&](int s) {
            const bool r = wait_all(p_full(s), gp[s] & 1u, 7);
            ++gp[s];
            return r;
        };

        for (int idx = next_pair(0, 16); idx < p.pairs && ok; idx = next_pair(++it, 16)) {
            const Pair pr = decode_pair(p, idx);
            const int m = p.m;
            const int n1 = pr.qt[1] + 1;
            const int n0 = pr.act0 ? pr.qt[0] + 1 : 0;
            const bool a_on = pr.act0;
            const bool shared = p.head_pairing != 0;         // the draft tiles serve both slots
            if (a_on) {
                if (!wait_all(q_full(0), gq[0] & 1u, 6)) break;
                ++gq[0];
            }
            if (!wait_all(q_full(1), gq[1] & 1u, 6)) break;
            ++gq[1];
            // S-type products: steps 0 .. m + n_s - 1 of slot s (m draft score products, then the key tiles). Step k + 1 of
            // a slot is issued after its softmax warps arrived for step k. Key tile j is ring entry shared by both slots.
            int st;
            // ---- step 0 of both slots ----
            if (m > 0 && !shared) {
                if (a_on) {
                    if (!k_acquire(st)) break;
                    issue_s(0, st, false);
                    k_release(st);
                }
                if (!k_acquire(st)) break;
                issue_s(1, st, false);
                k_release(st);
            } else {
                if (!k_acquire(st)) break;
                if (a_on && (m > 0 || n0 > 0)) issue_s(0, st, m == 0 && n0 == 1);
                issue_s(1, st, m == 0 && n1 == 1);
                k_release(st);
            }
            // ---- draft score steps: after the arrival for draft pass i, the slot's next S (pass i + 1, or key tile 0) ----
            for (int i = 0; i < m && ok; ++i) {
                const bool next_is_tile = (i + 1 == m);
                if (next_is_tile || shared) {
                    bool have = false;
                    if (a_on) {
                        if (!p_wait(0)) { ok = false; break; }
                        if (!k_acquire(st)) { ok = false; break; }
                        have = true;
                        issue_s(0, st, next_is_tile && n0 == 1);
                    }
                    if (!p_wait(1)) { ok = false; break; }
                    if (!have && !k_acquire(st)) { ok = false; break; }
                    issue_s(1, st, next_is_tile && n1 == 1);
                    k_release(st);
                } else {
                    if (a_on) {
                        if (!p_wait(0)) { ok = false; break; }
                        if (!k_acquire(st)) { ok = false; break; }
                        issue_s(0, st, false);
                        k_release(st);
                    }
                    if (!p_wait(1)) { ok = false; break; }
                    if (!k_acquire(st)) { ok = false; break; }
                    issue_s(1, st, false);
                    k_release(st);
                }
            }
            // ---- key tiles ----
            for (int j = 0; j < n1 && ok; ++j) {
                int vst;
                if (!v_acquire(vst)) { ok = false; break; }
                bool k_ready = false;
                if (j < n0) {
                    if (!p_wait(0)) { ok = false; break; }
                    issue_pv(0, vst, 0, 0, 8, j == 0, true);
                    if (j + 1 < n0) {
                        if (!k_acquire(st)) { ok = false; break; }
                        k_ready = true;
                        issue_s(0, st, j + 2 == n0);
                    }
                }
                if (!p_wait(1)) { ok = false; break; }
                issue_pv(1, vst, 0, 0, 8, j == 0, true);
                v_release(vst);
                if (j + 1 < n1) {
                    if (!k_ready && !k_acquire(st)) { ok = false; break; }
                    issue_s(1, st, j + 2 == n1);
                    k_release(st);
                }
            }
            // ---- draft value rounds: two passes per arrival (their weights sit in the two halves of the S buffer) ----
            for (int i0 = 0; i0 < m && ok; i0 += 2) {
                const bool two = i0 + 1 < m;
                bool waited0 = false, waited1 = false;
                for (int e = 0; e < (two ? 2 : 1) && ok; ++e) {
                    const bool fin = (e == 1) || !two;          // the slot's last product of the round
                    int vst;
                    if (shared) {
                        if (!v_acquire(vst)) { ok = false; break; }
                        if (a_on) {
                            if (!waited0 && !p_wait(0)) { ok = false; break; }
                            waited0 = true;
                            issue_pv(0, vst, 64 * e, 0, 8, false, fin);
                        }
                        if (!waited1 && !p_wait(1)) { ok = false; break; }
                        waited1 = true;
                        issue_pv(1, vst, 64 * e, 0, 8, false, fin);
                        v_release(vst);
                    } else {
                        if (a_on) {
                            if (!v_acquire(vst)) { ok = false; break; }
                            if (!waited0 && !p_wait(0)) { ok = false; break; }
                            waited0 = true;
                            issue_pv(0, vst, 64 * e, 0, 8, false, fin);
                            v_release(vst);
                        }
                        if (!v_acquire(vst)) { ok = false; break; }
                        if (!waited1 && !p_wait(1)) { ok = false; break; }
                        waited1 = true;
                        issue_pv(1, vst, 64 * e, 0, 8, false, fin);
                        v_release(vst);
                    }
                }
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
        // ===================== softmax + epilogue warps =====================
        const int slot = (warp - 4) >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                       // row of the tile = TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tmem_s = tmem_base + slot * KT + lane_addr;
        const uint32_t tmem_o = tmem_base + 256 + slot * HD + lane_addr;
        const int m = p.m;
        uint32_t gs = 0, gpv = 0, it = 0;                     // S-type products seen, PV-type products requested
        bool ok = true;
        for (int idx = next_pair(0, 17); idx < p.pairs && ok; idx = next_pair(++it, 17)) {
            const Pair pr = decode_pair(p, idx);
            if (slot == 0 && !pr.act0) continue;
            const int qt = pr.qt[slot], h = pr.h[slot], b = pr.b;
            const int n = qt + 1;
            const int t = qt * QT + r;                        // position in the sequence
            const bool valid = t < p.T;
            // ---- draft score steps: keep the diagonal element of each S (raw, unscaled) ----
            float sd[MAX_DRAFTS];
#pragma unroll
            for (int i = 0; i < MAX_DRAFTS; ++i) sd[i] = 0.f;
#pragma unroll 1
            for (int i = 0; i < m; ++i, ++gs) {
                if (!wait_barrier(s_full(slot), gs & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                uint32_t blk[32];
                tmem_ld32(tmem_s + 32 * quad, blk);           // this warp's diagonal block
                tmem_ld_wait(blk);
                float dv = 0.f;
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (c == lane) dv = __uint_as_float(blk[c]);
#pragma unroll
                for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                    if (ii == i) sd[ii] = dv;
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(slot));
            }
            if (!ok) break;
            float mref = -INFINITY, l = 0.f;
#pragma unroll 1
            for (int j = 0; j < n; ++j, ++gs) {
                if (!wait_barrier(s_full(slot), gs & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                const bool last = (j == n - 1);
                // the row's 128 scores into registers
                uint32_t raw[4][32];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld32(tmem_s + 32 * q, raw[q]);
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_wait(raw[q]);
                // Columns past t - m are hidden in the score tile: the causal part (s > t) and the m substituted
                // entries (t - m < s <= t), which enter the row's maximum and sum as scalars at the last tile.
                // Only tiles reaching past the first row's limit can hold such columns.
                if (j * KT + KT - 1 > qt * QT - m) {
                    const int lim = t - m - j * KT;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (32 * q + c > lim) raw[q][c] = 0xff800000u;      // -inf
                }
                float mx[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    mx[q] = fmaxf(__uint_as_float(raw[q][0]), __uint_as_float(raw[q][1]));
#pragma unroll
                    for (int c = 2; c < 32; c += 2) mx[q] = fmax3(mx[q], __uint_as_float(raw[q][c]), __uint_as_float(raw[q][c + 1]));
                }
                float mxa = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                if (last) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) mxa = fmaxf(mxa, sd[i]);
                }
                const float cand = mxa * p.c2;
                if (j == 0) {
                    mref = cand;
                } else {
                    const bool grow = cand > mref + RESCALE_LOG2;      // also true when every earlier column of the row was hidden
                    if (__any_sync(0xffffffffu, grow)) {
                        // Move the reference: this row's accumulator and sum are multiplied by 2^(old ref - new ref).
                        // The slot's products are complete up to this tile's S (the tensor core finishes them in
                        // issue order), so nothing else touches the accumulator now.
                        const float f = grow ? ex2(mref - cand) : 1.f;
                        if (grow) {
                            mref = cand;
                            l *= f;
                        }
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
                    }
                }
                // ---- P = 2^(x c2 - ref): row sum in fp32, bf16 pairs into tensor memory, 32 columns at a time ----
                // (a row whose columns were all hidden so far has ref = -inf; it gets P = 0, not 2^(-inf + inf))
                const float nref = mref == -INFINITY ? 0.f : -mref;
                float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t pk[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        ffma2(x0, x1, __uint_as_float(raw[q][c]), __uint_as_float(raw[q][c + 1]), p.c2, p.c2, nref, nref);
                        const float e0 = ex2(x0), e1 = ex2(x1);
                        fadd2(ls[(c >> 1) & 1], ls[2 + ((c >> 1) & 1)], ls[(c >> 1) & 1], ls[2 + ((c >> 1) & 1)], e0, e1);
                        pk[c >> 1] = pack_bf16(e0, e1);
                    }
                    hca::tmem_st16(tmem_s + 16 * q, pk);
                }
                l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
                if (last) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) l += ex2(fmaf(sd[i], p.c2, nref));
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(slot));
                ++gpv;
            }
            if (!ok) break;
            // ---- draft value rounds: two passes at a time; P holds only the weight 2^(sd c2 - ref) of each row, on the
            //      diagonal: pass i0 in the first 64 columns of the S buffer, pass i0 + 1 in the last 64 ----
            const float nref_f = mref == -INFINITY ? 0.f : -mref;
#pragma unroll 1
            for (int i0 = 0; i0 < m; i0 += 2) {
                // the products that last read these columns must be complete before they are overwritten
                if (!wait_barrier(pv_done(slot), (gpv - 1u) & 1u, abort_flag, p.status, 14)) { ok = false; break; }
                tc_fence_after_sync();
#pragma unroll 1
                for (int e = 0; e < 2 && i0 + e < m; ++e) {
                    const int i = i0 + e;
                    float sdi = 0.f;
#pragma unroll
                    for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                        if (ii == i) sdi = sd[ii];
                    const float pi = (t - i >= 0) ? ex2(fmaf(sdi, p.c2, nref_f)) : 0.f;
                    const uint32_t bits = pack_bf16(pi, 0.f) << ((r & 1) * 16);        // key r sits in word r / 2
#pragma unroll
                    for (int hw = 0; hw < 2; ++hw) {
                        uint32_t pk[32];
#pragma unroll
                        for (int w = 0; w < 32; ++w) pk[w] = (32 * hw + w == (r >> 1)) ? bits : 0u;
                        tmem_st32(tmem_s + 64 * e + 32 * hw, pk);
                    }
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(slot));
                ++gpv;
            }
            if (!ok) break;
            // ---- epilogue: O / l as bf16, each thread stores its own 256-byte row ----
            if (!wait_barrier(pv_done(slot), (gpv - 1u) & 1u, abort_flag, p.status, 13)) break;
            tc_fence_after_sync();
            const float inv = 1.f / l;
            if (valid && p.lse != nullptr)
                p.lse[(static_cast<size_t>(b) * p.H + h) * p.T + t] = (mref + log2f(l)) * 0.6931471805599453f;
            __nv_bfloat16* orow = p.O + ((static_cast<size_t>(b) * p.T + (valid ? t : 0)) * p.H + h) * HD;
            {
                uint32_t raw[4][32];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld32(tmem_o + 32 * q, raw[q]);
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_wait(raw[q]);
                if (valid) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
#pragma unroll
                        for (int q8 = 0; q8 < 2; ++q8) {
                            const uint32_t* x = &raw[q][16 * q8];
                            st_global_v8(orow + 32 * q + 16 * q8,
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
            // the accumulator and the score buffer go back to the tensor core with the next item's first step
            tc_fence_before_sync();
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

}  // namespace hca2
}  // namespace hass
