// Device code of the fused LM-head + Top-K distillation path (sm_100a).
//
// One warp-specialised, persistent GEMM kernel (TMA -> shared memory -> tcgen05.mma -> TMEM ->
// epilogue warps) is instantiated with three epilogues:
//   MODE_STATS  logits tile -> per-row softmax statistics, Top-K candidates (two variants: a sorted register
//               list for K <= 16, append buffers with warp-cooperative compaction otherwise) and, in the fused
//               forward+backward, a bf16 spill of 2^(z log2e - ref) that the second GEMM consumes
//   MODE_PROBS  draft logits tile -> dz_d tile = g (S_q p - q [v in Omega_hat]) in bf16 -> scratch
//               (the separate, recomputing backward)
//   MODE_OUT    dH_d tile: coef * acc - Omega_hat row (fused), coef * acc (q W of the combined objective)
//               or the accumulator as is (separate backward)
// plus small kernels: select (between the sweep of the target rows and the sweep of the draft rows: lse_t,
// Omega_hat, the set sorted by token id), loss_patch (after the draft sweep: lse_d, Eq. 1, row scale, the
// Omega_hat term into the spill), finalize (the single-sweep route: merge partial statistics, pick Omega_hat,
// Eq. 1 and its variants, the Omega_hat term of dH_d), ce_kernel (cross-entropy of the combined objective),
// bwd_prep (index-sorted Top-K lists for MODE_PROBS) and range_handled_kernel.
// Beside the four operand stages the kernel's shared memory holds 32 KB that the epilogue warps use: staging
// buffers for the TMA stores of the spill (draft sweep) or the logits waiting for admission to the register
// Top-K lists (target sweep).
#pragma once
#include <cuda_bf16.h>
#include <float.h>
#include <limits.h>

#include "ptx.cuh"

namespace hass {

constexpr int BM = 128;        // rows per tile (TMEM lanes)
constexpr int BN = 256;        // columns per tile (one UMMA N)
constexpr int BK = 64;         // contraction elements per pipeline stage (128 B of bf16: one swizzle row)
constexpr int UMMA_K = 16;     // contraction elements per tcgen05.mma (bf16)
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int B_STAGE_BYTES = BN * BK * 2;
constexpr int NUM_THREADS = 192;   // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int TMEM_COLS = 512;     // two accumulator buffers of BN fp32 columns
constexpr int MAX_PHASES = 48;
constexpr int K_CAP = 256;         // == HASS_K_MAX
constexpr int SPILL_STAGE_BYTES = 32 * 128;   // 32 rows x 64 bf16 of a spilled tile on their way to global memory
constexpr int SPILL_STAGES = 2;               // per epilogue warp
constexpr int SMEM_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 4 * SPILL_STAGES * SPILL_STAGE_BYTES +
                           1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr float LOG2E = 1.4426950408889634f;

enum { MODE_STATS = 0, MODE_PROBS = 1, MODE_OUT = 2 };

// A phase gives G consecutive row tiles S "lanes" each; lane l of a row tile sweeps the column
// tiles l, l + S, l + 2S, ... CTA b < G * S works on row tile row_tile_begin + b / S, lane b % S, and
// owns partial-result slot slot_base + b. All CTAs of a phase walk the column tiles in lockstep,
// so a column tile of B is fetched from HBM once and then served from L2 to the G row tiles.
struct Phase {
    int row_tile_begin, G, S, slot_base;
};
struct Schedule {
    int n_phases;
    int total_slots;
    int max_ctas;          // largest G * S over the phases = grid size
    int pad;
    Phase ph[MAX_PHASES];
};

struct GemmParams {
    CUtensorMap tmA0, tmA1, tmB;
    CUtensorMap tmSpill;   // MODE_STATS without Top-K lists (the draft sweep): the spill P as [chunk rows, p_pitch] bf16 with
                           // boxes of 64 columns x 32 rows, 128-byte swizzle, for TMA stores
    Schedule sched;
    int row_tiles0;        // row tiles [0, row_tiles0) read A0, the others A1 (tile index - row_tiles0)
    int topk_row_tiles;    // leading row tiles whose rows collect Top-K candidates (MODE_STATS)
    int a_row_offset;      // added to A0's row coordinate (chunked backward)
    int row_global_offset; // global row number of local row 0 (per-row inputs / outputs)
    int rows_valid;        // global rows >= rows_valid are padding
    int n_cols;            // extent of the tile-column dimension (V, or d for MODE_OUT)
    int col_tiles;
    int k_blocks;          // ceil(contraction extent / BK)
    int K;                 // Top-K
    int cap;               // capacity of a (row, slot) candidate buffer: cand_cap(K)
    int spill_begin;       // MODE_STATS: row tiles >= spill_begin also write the tile 2^(z log2e - ref2) in bf16 to
                           // P (row tile index - spill_begin); INT_MAX: none
    // MODE_STATS outputs (per slot)
    float* part_m;
    float* part_s;
    uint2* cand;           // [slot, row, cap] (logit bits, token id)
    int* cand_n;           // [slot, row] entries in use
    float* thr_share;      // [slot, row] each lane's current threshold, read by the other lanes of its row tile
                           // (initialised to NaN = "nothing published"; nullptr: no sharing)
    // MODE_PROBS
    const float* lse2;     // [N] lse_d * log2(e)
    const float* coef;     // [N] g * S_q
    const int* sidx;       // [N, K] Omega_hat sorted by token id
    const float* sgq;      // [N, K] g * q in the same order
    float* cap_z;          // MODE_STATS, TOPK_NONE: [N, K] out, z_d at the tokens of sidx (same order); slots of
                           // padding entries (token id INT_MAX) are left untouched
    __nv_bfloat16* P;      // [chunk rows, p_pitch]
    __nv_bfloat16* Pt;     // [chunk rows, p_pitch] spill of the target tiles, or nullptr
    long long p_pitch;
    // MODE_OUT. With sparse != nullptr the epilogue computes coef[row] * acc - sparse[local row, :] (row scale
    // and the Omega_hat term of dz_d W, precomputed by finalize); with coef alone coef[row] * acc; with neither
    // it stores the accumulator.
    const float* sparse;   // [chunk rows, out_pitch]
    void* out;
    int out_fp32;
    int out_align32;       // out base and row pitch are multiples of 32 bytes (256-bit stores allowed)
    long long out_pitch;   // elements
    unsigned int* status;
    const unsigned int* only_if_range;   // nullptr, or: run only if this status word reports a range overflow
    // The single-sweep route (spilling sweeps with Top-K lists): every spilling row leaves the ordered key of its
    // largest logit in row_zmax[row tile * 128 + row] (atomicMax over the lanes of the row tile; zeroed by the
    // host). A second sweep with use_row_zmax = 1 takes the row's fixed exponent from there instead of from
    // column tile 0, so that no logit of the row can exceed it.
    unsigned int* row_zmax;              // nullable
    int use_row_zmax;
};

// MODE_STATS: does this row tile also write its tiles 2^(z log2e - ref2) as bf16? Draft tiles from spill_begin
// on go to P; with Pt set, the target tiles (the leading topk_row_tiles) go to Pt (combined objective).
__device__ __forceinline__ bool spills(const GemmParams& p, int rt) {
    return rt >= p.spill_begin || (p.Pt != nullptr && rt < p.topk_row_tiles);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- streaming Top-K candidates ---------------------------------------------------------------------
// Each (row, slot) owns a buffer of `cap` (logit, token id) pairs in the workspace. The epilogue thread of
// the row appends every logit above its admission threshold; when a buffer is nearly full the whole warp
// compacts it to the row's K best and raises the threshold to the K-th largest logit. Entries stay in
// increasing token-id order, admission is strict (x > threshold), and among logits equal to the K-th the
// lowest token ids are kept, so equal logits resolve to the lower token id.
constexpr int CAND_CAP_MAX = 800;                 // largest buffer: K = 256
constexpr int CAND_REGS = CAND_CAP_MAX / 32;      // entries per lane during a compaction of the largest buffer
constexpr int CAND_REGS_SMALL = 13;               // ... of a buffer of up to 416 entries (K <= 128)
constexpr int CAND_SLACK = 32;                    // a compaction may leave up to K + CAND_SLACK entries

// K entries kept + room for max(2K, 96) new ones between compactions (each compaction then multiplies the
// number of columns a threshold has seen by about three) + the 32 entries before the end at which a
// compaction is triggered; a multiple of 32
__host__ __device__ constexpr int cand_cap(int K) { return (K + (2 * K > 96 ? 2 * K : 96) + 32 + 31) / 32 * 32; }

// order-preserving map from fp32 bit patterns to unsigned integers (and back); 0 is below every float
__device__ __forceinline__ uint32_t ordered_key(uint32_t bits) {
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
__device__ __forceinline__ uint32_t key_bits(uint32_t key) {
    return (key & 0x80000000u) ? (key ^ 0x80000000u) : ~key;
}

// Warp-collective: compacts the buffer `buf` holding n >= K entries, in place, keeping their order, and
// returns the bit pattern of the new admission threshold (only logits strictly above it can still belong to
// the row's K best); n_out = entries left. The K-th largest key is searched bit by bit from the top. After
// the upper 16 bits (bf16 resolution) the search stops if at most K + CAND_SLACK entries reach the prefix
// found so far: all of them are kept and the threshold is the value just below the prefix. Otherwise the
// search runs to the last bit, exactly K entries are kept (among logits equal to the K-th, the lowest token
// ids) and the threshold is the K-th largest logit itself.
template <int REGS>
__device__ __forceinline__ uint32_t compact_candidates(uint2* buf, int n, int K, int cap, int lane, int& n_out) {
    constexpr int CAND_REGS = REGS;
    uint32_t key[CAND_REGS];
    int id[CAND_REGS];
    const int groups = cap >> 5;
#pragma unroll
    for (int t = 0; t < CAND_REGS; ++t) {
        key[t] = 0u;
        id[t] = -1;
        const int e = lane + 32 * t;
        if (t < groups && e < n) {
            const uint2 v = __ldcg(buf + e);
            key[t] = ordered_key(v.x);
            id[t] = static_cast<int>(v.y);
        }
    }
    // largest T with at least K keys >= T, bit by bit; cT = number of keys >= T
    uint32_t T = 0u;
    int cT = n;
    bool exact = true;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
#pragma unroll
        for (int t = 0; t < CAND_REGS; ++t) c += (key[t] >= cand) ? 1 : 0;
        c = __reduce_add_sync(0xffffffffu, c);
        if (c >= K) {
            T = cand;
            cT = c;
        }
        if (bit == 16 && cT <= K + CAND_SLACK) {
            exact = false;
            break;
        }
    }
    const uint32_t lt_mask = (1u << lane) - 1u;
    int out = 0;
    if (!exact) {
        // keep every entry that reaches the 16-bit prefix
#pragma unroll
        for (int t = 0; t < CAND_REGS; ++t) {
            if (t < groups) {
                const bool keep = key[t] >= T;
                const uint32_t km = __ballot_sync(0xffffffffu, keep);
                if (keep) buf[out + __popc(km & lt_mask)] = make_uint2(key_bits(key[t]), static_cast<uint32_t>(id[t]));
                out += __popc(km);
            }
        }
        n_out = out;
        return key_bits(T - 1u);      // T >= 2^16 here: at least K keys reach it
    }
    int n_gt = 0;
#pragma unroll
    for (int t = 0; t < CAND_REGS; ++t) n_gt += (key[t] > T) ? 1 : 0;
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    const int need_eq = K - n_gt;             // >= 1: how many entries equal to the K-th are kept
    int run_eq = 0;
#pragma unroll
    for (int t = 0; t < CAND_REGS; ++t) {
        if (t < groups) {
            const bool eq = key[t] == T;
            const uint32_t em = __ballot_sync(0xffffffffu, eq);
            const bool keep = key[t] > T || (eq && run_eq + __popc(em & lt_mask) < need_eq);
            run_eq += __popc(em);
            const uint32_t km = __ballot_sync(0xffffffffu, keep);
            if (keep) buf[out + __popc(km & lt_mask)] = make_uint2(key_bits(key[t]), static_cast<uint32_t>(id[t]));
            out += __popc(km);
        }
    }
    n_out = out;
    return key_bits(T);
}

// TOPK selects how MODE_STATS keeps a row's Top-K candidates: TOPK_REG (K <= K_REG) a sorted list in
// registers, all lanes inserting in parallel - best while most rows still admit logits; TOPK_BUF (any K)
// append buffers with warp-cooperative compaction - cost nearly independent of K; TOPK_NONE: a sweep of draft
// rows whose Omega_hat is already known - no candidates are collected, instead each row's draft logits at its
// Omega_hat tokens are copied out of the accumulator as the sweep passes them (GemmParams::cap_z).
enum { TOPK_REG = 0, TOPK_BUF = 1, TOPK_NONE = 2 };
constexpr int K_REG = 16;

template <int MODE, int TOPK = TOPK_BUF>
__global__ void __launch_bounds__(NUM_THREADS, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    constexpr bool B_MN_MAJOR = (MODE == MODE_OUT);
    // conditional launch (the exact route that follows a fused call): nothing to do unless the fused sweep
    // reported a row beyond its exponent range
    if (p.only_if_range != nullptr && ((*p.only_if_range) & 0xffu) != 2u) return;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smemA = smem_base;
    const uint32_t smemB = smem_base + STAGES * A_STAGE_BYTES;
    const uint32_t spill_stage = smemB + STAGES * B_STAGE_BYTES;      // [epilogue warp][SPILL_STAGES] x SPILL_STAGE_BYTES
    const uint32_t bar_base = spill_stage + 4 * SPILL_STAGES * SPILL_STAGE_BYTES;
    // barriers: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]; then tmem pointer, abort flag
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint32_t* tmem_ptr_smem =
        reinterpret_cast<uint32_t*>(smem_gen + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 4 * SPILL_STAGES * SPILL_STAGE_BYTES +
                                    8 * (2 * STAGES + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmA0);
        prefetch_tensormap(&p.tmB);
        if (MODE == MODE_STATS) prefetch_tensormap(&p.tmA1);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_ptr_smem), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;

    // Calls f(row_tile, lane, S, slot) for every item of this CTA; f returns false to stop.
    auto for_each_item = [&](auto&& f) {
        for (int ph = 0; ph < p.sched.n_phases; ++ph) {
            const Phase P = p.sched.ph[ph];
            if (cta < P.G * P.S) {
                const int gi = cta / P.S;
                if (!f(P.row_tile_begin + gi, cta - gi * P.S, P.S, P.slot_base + cta)) return;
            }
        }
    };

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for_each_item([&](int rt, int ln, int S, int) {
                const bool second = (MODE == MODE_STATS) && rt >= p.row_tiles0;
                const CUtensorMap* tmA = second ? &p.tmA1 : &p.tmA0;
                const int row0 = p.a_row_offset + (second ? rt - p.row_tiles0 : rt) * BM;
                const int t0 = (MODE == MODE_STATS && spills(p, rt) && ln != 0) ? -1 : 0;
                const int nt = (p.col_tiles - ln + S - 1) / S;
                for (int t = t0; t < nt; ++t) {
                    const int ct = t < 0 ? 0 : ln + t * S;   // t = -1: column tile 0, for the row references only
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!wait_barrier(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) return false;
                        mbar_arrive_expect_tx(full_bar(stage), A_STAGE_BYTES + B_STAGE_BYTES);
                        tma_load_2d(smemA + stage * A_STAGE_BYTES, tmA, full_bar(stage), kb * BK, row0);
                        if (!B_MN_MAJOR) {
                            tma_load_2d(smemB + stage * B_STAGE_BYTES, &p.tmB, full_bar(stage), kb * BK, ct * BN);
                        } else {
                            // B tile = BK contraction rows x BN contiguous columns, fetched as BN/64 boxes
                            // of 64 columns (one 128-byte swizzle row) x BK rows
#pragma unroll
                            for (int j = 0; j < BN / 64; ++j)
                                tma_load_2d(smemB + stage * B_STAGE_BYTES + j * (BK * 128), &p.tmB, full_bar(stage),
                                            ct * BN + j * 64, kb * BK);
                        }
                        if (++stage == STAGES) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                }
                return true;
            });
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(BM, BN, 0, B_MN_MAJOR ? 1 : 0);
            int stage = 0;
            uint32_t phase = 0;
            int ab = 0;
            uint32_t aphase = 0;
            for_each_item([&](int rt, int ln, int S, int) {
                const int t0 = (MODE == MODE_STATS && spills(p, rt) && ln != 0) ? -1 : 0;
                const int nt = (p.col_tiles - ln + S - 1) / S;
                for (int t = t0; t < nt; ++t) {
                    if (!wait_barrier(tempty_bar(ab), aphase ^ 1u, abort_flag, p.status, 2)) return false;
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + ab * BN;
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!wait_barrier(full_bar(stage), phase, abort_flag, p.status, 3)) return false;
                        tc_fence_after_sync();
                        // A: K-major, 8-row groups 1024 B apart. B: K-major likewise, or MN-major with
                        // 64-column groups BK*128 B apart (LBO) and 8-row contraction groups 1024 B apart (SBO).
                        const uint64_t a_desc = make_smem_desc_sw128(smemA + stage * A_STAGE_BYTES, 0, 1024);
                        const uint64_t b_desc =
                            B_MN_MAJOR ? make_smem_desc_sw128(smemB + stage * B_STAGE_BYTES, BK * 128, 1024)
                                       : make_smem_desc_sw128(smemB + stage * B_STAGE_BYTES, 0, 1024);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            // advance the start address (>>4) along the contraction
                            const uint64_t a_adv = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                            const uint64_t b_adv = B_MN_MAJOR ? static_cast<uint64_t>((k * UMMA_K * 128) >> 4)
                                                              : static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                            umma_bf16(d_tmem, a_desc + a_adv, b_desc + b_adv, idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                        umma_commit(empty_bar(stage));   // frees the stage once these MMAs have read it
                        if (++stage == STAGES) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    umma_commit(tfull_bar(ab));          // accumulator complete
                    ab ^= 1;
                    if (ab == 0) aphase ^= 1u;
                }
                return true;
            });
        }
    } else {
        // ===================== epilogue warps =====================
        const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
        const int r_local = quad * 32 + lane;      // row inside the tile
        int ab = 0;
        uint32_t aphase = 0;
        // Top-K candidates of this thread's row (MODE_STATS): buffer in the workspace, entries in use
        uint2* cbuf = nullptr;
        int cnt = 0;
        uint32_t spill_boxes = 0;                  // chunks this warp has staged for TMA stores (two per box)
        // TOPK_REG: the K_REG largest logits so far sorted descending in tv[] (the admission threshold is the
        // K_REG-th largest: a list of exactly K entries with its K-th as threshold measured slower), and the
        // current chunk's admitted logits waiting in a small local-memory buffer
        constexpr bool USE_REG = MODE == MODE_STATS && TOPK == TOPK_REG;
        constexpr bool HAS_TOPK = MODE == MODE_STATS && TOPK != TOPK_NONE;
        constexpr bool CAPTURE = MODE == MODE_STATS && TOPK == TOPK_NONE;
        float tv[USE_REG ? K_REG : 1];
        int ti[USE_REG ? K_REG : 1];
        // ... waiting in shared memory: entry q of thread T at word q * 128 + T of the values' array and of the
        // tokens' array (16 KB each, the room the draft sweep uses for its spill boxes; this instantiation stores no
        // boxes). With 200 KB of shared memory carved out little L1 is left, and a per-thread array in local memory
        // cost about a thousand cycles per admitted logit here.
        static_assert(4 * SPILL_STAGES * SPILL_STAGE_BYTES >= 2 * 32 * 128 * 4, "room for the pending logits");
        const uint32_t pend_v = spill_stage + (threadIdx.x - 64) * 4;
        const uint32_t pend_i = pend_v + 32 * 128 * 4;
        constexpr int lo = 0;

        for_each_item([&](int rt, int ln, int S, int slot) {
            const int g_row = p.row_global_offset + rt * BM + r_local;
            const bool row_ok = g_row < p.rows_valid;
            // ---- per-item state ----
            float m = -INFINITY, s = 0.f, thr = -INFINITY;        // MODE_STATS; thr = admission threshold in force
            float thr_own = -INFINITY;                            // K-th (K_REG-th) largest logit of this lane's own list
            float thr_sh = -INFINITY;                             // just below the best threshold published by the other lanes
            bool want_topk = false;
            const bool spill = MODE == MODE_STATS && spills(p, rt);
            const bool track_zmax = MODE == MODE_STATS && TOPK != TOPK_NONE && spill && p.row_zmax != nullptr;
            float zmax = -INFINITY;                               // the row's largest logit in this lane's column tiles
            float ref2 = 0.f;                                     // spill rows: exponent offset (log2 units)
            float lse2 = 0.f, coef = 0.f;                         // MODE_PROBS / fused MODE_OUT
            const int* si = nullptr;
            const float* sg = nullptr;
            int cur = 0, nxt = INT_MAX;
            if (MODE == MODE_STATS) {
                want_topk = HAS_TOPK && rt < p.topk_row_tiles;
                if (HAS_TOPK) cbuf = p.cand + (static_cast<long long>(slot) * BM + r_local) * p.cap;
                cnt = 0;
                if (USE_REG) {
#pragma unroll
                    for (int i = 0; i < (USE_REG ? K_REG : 1); ++i) {
                        tv[i] = -INFINITY;
                        ti[i] = -1;
                    }
                }
            }
            if (MODE == MODE_PROBS && row_ok) {
                lse2 = p.lse2[g_row];
                coef = p.coef[g_row];
                si = p.sidx + static_cast<long long>(g_row) * p.K;
                sg = p.sgq + static_cast<long long>(g_row) * p.K;
                nxt = si[0];
            }
            if (MODE == MODE_OUT && p.coef != nullptr && row_ok) coef = p.coef[g_row];
            float* cz = nullptr;
            if (CAPTURE && row_ok && p.cap_z != nullptr) {
                // the row's Omega_hat in increasing token order; this lane meets its own column tiles in that order too
                si = p.sidx + static_cast<long long>(g_row) * p.K;
                cz = p.cap_z + static_cast<long long>(g_row) * p.K;
                nxt = si[0];
            }
            const int t0 = (spill && ln != 0) ? -1 : 0;
            const int nt = (p.col_tiles - ln + S - 1) / S;
            for (int t = t0; t < nt; ++t) {
                const int ct = t < 0 ? 0 : ln + t * S;
                // the whole warp must agree before the warp-collective TMEM loads below
                const bool ready = wait_barrier(tfull_bar(ab), aphase, abort_flag, p.status, 4);
                if (!__all_sync(0xffffffffu, ready)) return false;
                tc_fence_after_sync();
                const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + ab * BN;
                const int col_base = ct * BN;
                bool skip_tile = false;
                if (MODE == MODE_STATS && spill && t == t0) {
                    // Reference exponent of this row: its largest logit in column tile 0. Every lane of
                    // the row tile computes tile 0 first and so derives the same value.
                    float mx = -INFINITY;
                    if (TOPK != TOPK_NONE && p.use_row_zmax) {
                        // second sweep after a range report: the row's largest logit is known
                        mx = __uint_as_float(key_bits(p.row_zmax[rt * BM + r_local]));
                    } else {
#pragma unroll 1
                        for (int ch = 0; ch < BN / 32; ++ch) {
                            uint32_t r[32];
                            tmem_ld32(t_row + ch * 32, r);
                            tmem_ld_wait(r);
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (ch * 32 + j < p.n_cols) mx = fmaxf(mx, __uint_as_float(r[j]));
                        }
                    }
                    // spilled values are 2^(z log2e - ref2) <= about 2^-64 for typical rows, which leaves
                    // 2^191 of headroom above the reference before bf16 / fp32 overflow
                    ref2 = fmaf(mx, LOG2E, 64.f);
                    m = ref2 * (1.0f / LOG2E);
                    skip_tile = t < 0;
                }
                if (MODE == MODE_STATS && HAS_TOPK && !USE_REG && want_topk && t == 0 && p.n_cols - col_base >= BN) {
                    // First tile of the sweep, buffer empty, no threshold yet: admitting all 256 logits would fill
                    // the buffer and force a compaction of every row of the warp at once (32 warp-wide compactions
                    // in a row, during which the tensor core runs out of free accumulators). Instead each thread
                    // searches, bit by bit, the largest 12-bit prefix (sign, exponent, three mantissa bits) that at
                    // least K of its row's 256 logits reach - comparisons against the tile in tensor memory, the same
                    // instructions for every row - and starts from the threshold just below it: a valid lower bound
                    // of the row's K-th largest logit that admits little more than K of the tile's logits.
                    uint32_t T = 0u;
#pragma unroll 1
                    for (int bit = 31; bit >= 20; --bit) {
                        const uint32_t cand = T | (1u << bit);
                        const float fc = __uint_as_float(key_bits(cand));      // keys order like the floats they stand for
                        int c = 0;
#pragma unroll 1
                        for (int ch = 0; ch < BN / 32; ++ch) {
                            uint32_t r[32];
                            tmem_ld32(t_row + ch * 32, r);
                            tmem_ld_wait(r);
#pragma unroll
                            for (int j = 0; j < 32; ++j) c += (__uint_as_float(r[j]) >= fc) ? 1 : 0;
                        }
                        if (c >= p.K) T = cand;
                    }
                    if (T >= (1u << 20)) {
                        // the float just below the prefix; at the prefix of +0 that is -0, which compares equal to
                        // the zeros that were counted, so step down to a float that is really smaller
                        float below = __uint_as_float(key_bits(T - 1u));
                        if (below == 0.f) below = -1.17549435e-38f;
                        thr_own = below;
                        thr = fmaxf(thr_own, thr_sh);
                    }
                }
                if (CAPTURE && !skip_tile) {
                    while (nxt < col_base) {
                        ++cur;
                        nxt = cur < p.K ? si[cur] : INT_MAX;
                    }
                }
#pragma unroll 1
                for (int ch = 0; ch < BN / 32 && !skip_tile; ++ch) {
                    if (MODE == MODE_STATS && !USE_REG && want_topk) {
                        // make room for a whole chunk in every row's buffer (warp-uniform control flow), before the
                        // chunk's logits occupy registers
                        uint32_t full = __ballot_sync(0xffffffffu, cnt > p.cap - 32);
                        while (full) {
                            const int L = __ffs(full) - 1;
                            full &= full - 1u;
                            __syncwarp();
                            const unsigned long long bp = __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(cbuf), L);
                            const int n = __shfl_sync(0xffffffffu, cnt, L);
                            int left = 0;
                            const uint32_t tb = p.cap <= 32 * CAND_REGS_SMALL
                                                    ? compact_candidates<CAND_REGS_SMALL>(reinterpret_cast<uint2*>(bp), n, p.K, p.cap, lane, left)
                                                    : compact_candidates<CAND_REGS>(reinterpret_cast<uint2*>(bp), n, p.K, p.cap, lane, left);
                            __syncwarp();
                            if (lane == L) {
                                cnt = left;
                                thr_own = __uint_as_float(tb);
                                thr = fmaxf(thr_own, thr_sh);
                            }
                        }
                    }
                    uint32_t r[32];
                    tmem_ld32(t_row + ch * 32, r);
                    tmem_ld_wait(r);
                    const int col0 = col_base + ch * 32;
                    if (MODE == MODE_STATS) {
                        if (col0 + 32 > p.n_cols) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j >= p.n_cols) r[j] = __float_as_uint(-INFINITY);
                        }
                        if (CAPTURE) {
                            // draft logits at the row's Omega_hat, straight from the fp32 accumulator
                            while (nxt < col0 + 32) {
                                const int off = nxt - col0;
                                uint32_t zb = 0u;
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (j == off) zb = r[j];
                                cz[cur] = __uint_as_float(zb);
                                ++cur;
                                nxt = cur < p.K ? si[cur] : INT_MAX;
                            }
                        }
                        float cm = -INFINITY;     // the chunk's largest logit (not needed by a spill row without Top-K)
                        if (!spill || want_topk || track_zmax) {
                            cm = fmaxf(__uint_as_float(r[0]), __uint_as_float(r[1]));
#pragma unroll
                            for (int j = 2; j < 32; j += 2) cm = fmax3(cm, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
                            zmax = fmaxf(zmax, cm);
                        }
                        if (!spill) {
                            if (cm > m) {
                                s *= ex2((m - cm) * LOG2E);
                                m = cm;
                            }
                            const float mneg = -m * LOG2E;
                            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                float t0, t1;
                                ffma2(t0, t1, __uint_as_float(r[j]), __uint_as_float(r[j + 1]), LOG2E, LOG2E, mneg, mneg);
                                fadd2(acc0, acc1, acc0, acc1, ex2(t0), ex2(t1));
                            }
                            s += acc0 + acc1;
                        } else {
                            // one exponential per logit serves both the row's sum and the spilled tile; a
                            // logit beyond the exponent range gives inf here and is reported at the item's end
                            float e[32];
                            float acc0 = 0.f, acc1 = 0.f;
                            const float nref2 = -ref2;
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                float t0, t1;
                                ffma2(t0, t1, __uint_as_float(r[j]), __uint_as_float(r[j + 1]), LOG2E, LOG2E, nref2, nref2);
                                e[j] = ex2(t0);
                                e[j + 1] = ex2(t1);
                                fadd2(acc0, acc1, acc0, acc1, e[j], e[j + 1]);
                            }
                            s += acc0 + acc1;
                            if (TOPK == TOPK_NONE) {
                                // The draft sweep hands its spill to the TMA unit: the row's 32 values go into the warp's
                                // staging buffer (128-byte rows, swizzled), and after every second chunk one lane
                                // requests the store of the 32 x 64 box. That is one request per 4 KB from this warp
                                // instead of 64 store instructions that each touch 32 rows.
                                const uint32_t buf = spill_stage + (quad * SPILL_STAGES + ((spill_boxes >> 1) & 1)) * SPILL_STAGE_BYTES;
                                if ((ch & 1) == 0) {
                                    // the store that read this buffer two boxes ago must have finished reading it
                                    if (lane == 0) bulk_wait_group_read<SPILL_STAGES - 1>();
                                    __syncwarp();
                                }
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    st_shared_v4(buf + lane * 128 + ((((ch & 1) * 4 + j) ^ (lane & 7)) << 4),
                                                 pack_bf16x2(e[8 * j + 0], e[8 * j + 1]), pack_bf16x2(e[8 * j + 2], e[8 * j + 3]),
                                                 pack_bf16x2(e[8 * j + 4], e[8 * j + 5]), pack_bf16x2(e[8 * j + 6], e[8 * j + 7]));
                                if (ch & 1) {
                                    fence_proxy_async_smem();
                                    __syncwarp();
                                    if (lane == 0) {
                                        tma_store_2d(&p.tmSpill, buf, col0 - 32, (rt - p.spill_begin) * BM + quad * 32);
                                        bulk_commit_group();
                                    }
                                }
                                ++spill_boxes;
                            } else {
                                __nv_bfloat16* dst = (rt >= p.spill_begin
                                                          ? p.P + static_cast<long long>((rt - p.spill_begin) * BM + r_local) * p.p_pitch
                                                          : p.Pt + static_cast<long long>(rt * BM + r_local) * p.p_pitch) + col0;
#pragma unroll
                                for (int g16 = 0; g16 < 2; ++g16)
                                    st_global_v8(dst + 16 * g16, pack_bf16x2(e[16 * g16 + 0], e[16 * g16 + 1]),
                                                 pack_bf16x2(e[16 * g16 + 2], e[16 * g16 + 3]),
                                                 pack_bf16x2(e[16 * g16 + 4], e[16 * g16 + 5]),
                                                 pack_bf16x2(e[16 * g16 + 6], e[16 * g16 + 7]),
                                                 pack_bf16x2(e[16 * g16 + 8], e[16 * g16 + 9]),
                                                 pack_bf16x2(e[16 * g16 + 10], e[16 * g16 + 11]),
                                                 pack_bf16x2(e[16 * g16 + 12], e[16 * g16 + 13]),
                                                 pack_bf16x2(e[16 * g16 + 14], e[16 * g16 + 15]));
                            }
                        }
                        if (!USE_REG && want_topk && cm > thr) {
                            // predicated stores, no branches: as 32 conditional blocks this section took about 5000
                            // cycles whenever any row of the warp admitted a logit
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const bool in = __uint_as_float(r[j]) > thr;
                                st_global_v2_if(cbuf + cnt, r[j], static_cast<uint32_t>(col0 + j), in);
                                cnt += in ? 1 : 0;
                            }
                        }
                        if (USE_REG && want_topk && cm > thr) {
                            // collect the chunk's candidates, then admit them one by one (the
                            // threshold only rises, so each is re-checked against the current one)
                            int np = 0;
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float x = __uint_as_float(r[j]);
                                const bool in = x > thr;       // predicated stores, no branches
                                st_shared_b32_if(pend_v + np * 512, __float_as_uint(x), in);
                                st_shared_b32_if(pend_i + np * 512, static_cast<uint32_t>(col0 + j), in);
                                np += in ? 1 : 0;
                            }
                            for (int q = 0; q < np; ++q) {
                                const float x = __uint_as_float(ld_shared_b32(pend_v + q * 512));
                                const int id = static_cast<int>(ld_shared_b32(pend_i + q * 512));
                                if (!(x > thr)) continue;
                                // sorted insertion; equal logits stay behind earlier (lower) token ids
#pragma unroll
                                for (int i = (USE_REG ? K_REG : 1) - 1; i >= 0; --i) {
                                    if (i > 0 && i > lo) {
                                        const bool shift = x > tv[i > 0 ? i - 1 : 0];
                                        const bool here = !shift && x > tv[i];
                                        tv[i] = shift ? tv[i > 0 ? i - 1 : 0] : (here ? x : tv[i]);
                                        ti[i] = shift ? ti[i > 0 ? i - 1 : 0] : (here ? id : ti[i]);
                                    } else if (i == lo) {
                                        if (x > tv[i]) {
                                            tv[i] = x;
                                            ti[i] = id;
                                        }
                                    }
                                }
                                thr_own = tv[(USE_REG ? K_REG : 1) - 1];
                                thr = fmaxf(thr_own, thr_sh);
                            }
                        }
                    } else if (MODE == MODE_PROBS) {
                        while (nxt < col0) {
                            ++cur;
                            nxt = cur < p.K ? si[cur] : INT_MAX;
                        }
                        float e[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) e[j] = coef * ex2(fmaf(__uint_as_float(r[j]), LOG2E, -lse2));
                        while (nxt < col0 + 32) {
                            const int off = nxt - col0;
                            const float gq = sg[cur];
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j == off) e[j] -= gq;
                            ++cur;
                            nxt = cur < p.K ? si[cur] : INT_MAX;
                        }
                        if (col0 + 32 > p.n_cols) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j >= p.n_cols) e[j] = 0.f;
                        }
                        uint4* dst = reinterpret_cast<uint4*>(p.P + static_cast<long long>(rt * BM + r_local) * p.p_pitch + col0);
#pragma unroll
                        for (int g8 = 0; g8 < 4; ++g8) {
                            uint4 w;
                            w.x = pack_bf16x2(e[8 * g8 + 0], e[8 * g8 + 1]);
                            w.y = pack_bf16x2(e[8 * g8 + 2], e[8 * g8 + 3]);
                            w.z = pack_bf16x2(e[8 * g8 + 4], e[8 * g8 + 5]);
                            w.w = pack_bf16x2(e[8 * g8 + 6], e[8 * g8 + 7]);
                            dst[g8] = w;
                        }
                    } else if (row_ok) {
                        float o[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(r[j]);
                        const bool full = col0 + 32 <= p.n_cols;
                        if (p.sparse != nullptr) {
                            // dH_d = coef * (spilled tile x W) - sum_{x in Omega_hat} g q(x) W[x, :]
                            const float* sp = p.sparse + static_cast<long long>(rt * BM + r_local) * p.out_pitch + col0;
                            if (full) {
#pragma unroll
                                for (int g8 = 0; g8 < 4; ++g8) {
                                    float v[8];
                                    ld_global_v8(sp + 8 * g8, v);
#pragma unroll
                                    for (int u = 0; u < 8; ++u) o[8 * g8 + u] = fmaf(coef, o[8 * g8 + u], -v[u]);
                                }
                            } else {
#pragma unroll
                                for (int g4 = 0; g4 < 8; ++g4) {
                                    if (col0 + 4 * g4 < p.n_cols) {
                                        const float4 v = *reinterpret_cast<const float4*>(sp + 4 * g4);
                                        o[4 * g4 + 0] = fmaf(coef, o[4 * g4 + 0], -v.x);
                                        o[4 * g4 + 1] = fmaf(coef, o[4 * g4 + 1], -v.y);
                                        o[4 * g4 + 2] = fmaf(coef, o[4 * g4 + 2], -v.z);
                                        o[4 * g4 + 3] = fmaf(coef, o[4 * g4 + 3], -v.w);
                                    }
                                }
                            }
                        }
                        if (p.sparse == nullptr && p.coef != nullptr) {
                            // row scale only (the target side's q W of the combined objective)
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] *= coef;
                        }
                        if (p.out_fp32) {
                            float* dst = reinterpret_cast<float*>(p.out) + static_cast<long long>(g_row) * p.out_pitch + col0;
                            if (full && p.out_align32) {
#pragma unroll
                                for (int g8 = 0; g8 < 4; ++g8)
                                    st_global_v8(dst + 8 * g8, __float_as_uint(o[8 * g8]), __float_as_uint(o[8 * g8 + 1]),
                                                 __float_as_uint(o[8 * g8 + 2]), __float_as_uint(o[8 * g8 + 3]),
                                                 __float_as_uint(o[8 * g8 + 4]), __float_as_uint(o[8 * g8 + 5]),
                                                 __float_as_uint(o[8 * g8 + 6]), __float_as_uint(o[8 * g8 + 7]));
                            } else {
#pragma unroll
                                for (int g4 = 0; g4 < 8; ++g4)
                                    if (col0 + 4 * g4 < p.n_cols)
                                        *reinterpret_cast<float4*>(dst + 4 * g4) =
                                            make_float4(o[4 * g4], o[4 * g4 + 1], o[4 * g4 + 2], o[4 * g4 + 3]);
                            }
                        } else {
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + static_cast<long long>(g_row) * p.out_pitch + col0;
                            if (full && p.out_align32) {
#pragma unroll
                                for (int g16 = 0; g16 < 2; ++g16)
                                    st_global_v8(dst + 16 * g16, pack_bf16x2(o[16 * g16 + 0], o[16 * g16 + 1]),
                                                 pack_bf16x2(o[16 * g16 + 2], o[16 * g16 + 3]),
                                                 pack_bf16x2(o[16 * g16 + 4], o[16 * g16 + 5]),
                                                 pack_bf16x2(o[16 * g16 + 6], o[16 * g16 + 7]),
                                                 pack_bf16x2(o[16 * g16 + 8], o[16 * g16 + 9]),
                                                 pack_bf16x2(o[16 * g16 + 10], o[16 * g16 + 11]),
                                                 pack_bf16x2(o[16 * g16 + 12], o[16 * g16 + 13]),
                                                 pack_bf16x2(o[16 * g16 + 14], o[16 * g16 + 15]));
                            } else {
#pragma unroll
                                for (int g8 = 0; g8 < 4; ++g8) {
                                    if (col0 + 8 * g8 < p.n_cols) {
                                        uint4 w;
                                        w.x = pack_bf16x2(o[8 * g8 + 0], o[8 * g8 + 1]);
                                        w.y = pack_bf16x2(o[8 * g8 + 2], o[8 * g8 + 3]);
                                        w.z = pack_bf16x2(o[8 * g8 + 4], o[8 * g8 + 5]);
                                        w.w = pack_bf16x2(o[8 * g8 + 6], o[8 * g8 + 7]);
                                        *reinterpret_cast<uint4*>(dst + 8 * g8) = w;
                                    }
                                }
                            }
                        }
                    }
                }
                // accumulator drained: hand the buffer back to the MMA warp
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(ab));
                ab ^= 1;
                if (ab == 0) aphase ^= 1u;
                if (MODE == MODE_STATS && want_topk && p.thr_share != nullptr && S > 1) {
                    // The K-th largest logit of ANY lane's part of the row is a lower bound of the row's K-th
                    // largest, so a lane may adopt the other lanes' thresholds: publish ours, read up to three
                    // neighbours. A logit equal to a foreign threshold must still be admitted (ties are settled
                    // by token id when the lists are merged), hence the step just below it. Stale or missing
                    // (NaN) values only leave the threshold lower than it could be.
                    volatile float* sh = p.thr_share + static_cast<long long>(slot - ln) * BM + r_local;
                    sh[static_cast<long long>(ln) * BM] = thr_own;
                    const int nn = S - 1 < 3 ? S - 1 : 3;
                    for (int q = 1; q <= nn; ++q) {
                        const float v = sh[static_cast<long long>((ln + q) % S) * BM];
                        thr_sh = fmaxf(thr_sh, nextafterf(v, -INFINITY));
                    }
                    thr = fmaxf(thr, thr_sh);
                }
            }
            if (MODE == MODE_STATS) {
                const long long so = static_cast<long long>(slot) * BM + r_local;
                p.part_m[so] = m;
                p.part_s[so] = s;
                // a spilled value reached the top of the fp32 range: the row's logits spread too far
                // above its reference for the fixed-exponent spill
                if (spill && !(s < 1e38f)) atomicCAS(p.status, 0u, (5u << 8) | 2u);
                if (track_zmax && !p.use_row_zmax) atomicMax(p.row_zmax + rt * BM + r_local, ordered_key(__float_as_uint(zmax)));
                if (USE_REG && want_topk) {
                    // the register list goes out as a full buffer of K_REG entries (unused ones carry id -1)
#pragma unroll
                    for (int k = 0; k < (USE_REG ? K_REG : 1); ++k)
                        cbuf[k] = make_uint2(__float_as_uint(tv[k]), static_cast<uint32_t>(ti[k]));
                    cnt = K_REG;
                }
                if (want_topk) p.cand_n[static_cast<long long>(slot) * BM + r_local] = cnt;
            }
            return true;
        });
        // shared memory must outlive the TMA stores that read it
        if (MODE == MODE_STATS && TOPK == TOPK_NONE && lane == 0) bulk_wait_group0();
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

// ---------------------------------------------------------------------------------------------
// finalize: one warp per row. Merges the per-slot (max, sum-exp) pairs into lse_t / lse_d, selects
// Omega_hat from the slots' candidates (or takes it as an input), gathers the draft logits at
// Omega_hat with K dot products, and evaluates Eq. 1.
struct FinalizeParams {
    Schedule sched;
    int d, K;
    int cap;               // capacity of a (row, slot) candidate buffer
    int row_begin, rows;   // global rows [row_begin, row_begin + rows) = local row tiles 0.. of the schedule
    int row_tiles_t;       // row tiles of the target matrix in the schedule (0: Omega_hat is an input)
    const float* part_m;
    const float* part_s;
    const uint2* cand;
    const int* cand_n;
    const __nv_bfloat16* H_d;
    const __nv_bfloat16* W;
    const int* idx_in;     // [N,K] when row_tiles_t == 0
    const float* q_in;
    float* loss;
    int* idx_out;
    float* q_out;
    float* lse_t;
    float* lse_d;
    // fused backward (all nullable): per-row scale of the spilled tiles and g * q of Omega_hat
    const float* grad_loss;
    float* coef_out;       // [N]   g * S_q * exp(m_spill - lse_d), m_spill = the row's spill reference
    float* gq_out;         // [N,K] g * q, in the order of topk_idx
    float* sparse_out;     // [rows, d] sum_{x in Omega_hat} g q(x) W[x, :], indexed by local row
    // combined objective CE(q, p) + w * Top-K (coef_t_out != nullptr): the target tiles were spilled as well
    float w_topk;          // weight w of the Top-K term
    float* coef_t_out;     // [N] e^(m_spill_t - lse_t): scale that turns (target spill x W) into q W
    const __nv_bfloat16* Pt;   // target spill of the chunk [rows, p_pitch]
    long long p_pitch;
    float* ce_corr_out;    // [N] sum_{x in Omega_hat} (q(x) - bf16 q(x)) z_d(x): the cross-entropy is formed from
                           // the bf16 spill; its largest terms are put back in fp32
    // loss variants of Section 4.3
    float top_p;           // > 0: Omega_hat is cut to the shortest sorted prefix with cumulative q > top_p (Top-P)
    int* n_out;            // [N] |Omega_hat| (nullable)
    int normed;            // 1: Normed Top-K - q, p renormalised over Omega_hat; no draft sweep exists, and the
                           // gradient row sum_x g (pn(x) - qn(x)) W[x,:] goes straight to dH_out
    void* dH_out;          // [N, d] (normed only)
    int dH_fp32;
    int bidir;             // 1: Bi-directional Top-K - Omega_hat also takes the draft's K most probable tokens (the draft
                           // rows collected candidates too); idx_out / q_out then have 2K entries per row
    const __nv_bfloat16* H_t;   // target features (bidir: target logits of the draft's tokens)
    const unsigned int* only_if_range;   // as in GemmParams
};

__device__ __forceinline__ void find_slots(const Schedule& sc, int row_tile, int& slot0, int& S) {
    slot0 = 0;
    S = 0;
    for (int ph = 0; ph < sc.n_phases; ++ph) {
        const Phase P = sc.ph[ph];
        if (row_tile >= P.row_tile_begin && row_tile < P.row_tile_begin + P.G) {
            slot0 = P.slot_base + (row_tile - P.row_tile_begin) * P.S;
            S = P.S;
            return;
        }
    }
}

__device__ __forceinline__ float warp_lse(const float* pm, const float* ps, int slot0, int S, int r, int lane) {
    float m = -INFINITY;
    for (int j = lane; j < S; j += 32) m = fmaxf(m, pm[static_cast<long long>(slot0 + j) * BM + r]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float s = 0.f;
    for (int j = lane; j < S; j += 32) {
        const long long so = static_cast<long long>(slot0 + j) * BM + r;
        s += ps[so] * exp2f((pm[so] - m) * LOG2E);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return m + logf(s);
}

constexpr int FIN_GRP = 16;   // tokens of Omega_hat whose W rows finalize reads together

__global__ void __launch_bounds__(256) finalize_kernel(const __grid_constant__ FinalizeParams p) {
    if (p.only_if_range != nullptr && ((*p.only_if_range) & 0xffu) != 2u) return;
    const int lane = threadIdx.x & 31;
    const int local = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (local >= p.rows) return;
    const int row = p.row_begin + local;
    const int rt = local / BM, r = local % BM;
    const int K = p.K;
    int slot0, S;

    // draft statistics (the Normed Top-K variant has none: it needs the draft logits on Omega_hat only)
    float lse_d = 0.f, m_spill = 0.f;
    int slot0_d = 0, S_d = 0;
    if (!p.normed) {
        find_slots(p.sched, p.row_tiles_t + rt, slot0, S);
        slot0_d = slot0;
        S_d = S;
        lse_d = warp_lse(p.part_m, p.part_s, slot0, S, r, lane);
        if (lane == 0) p.lse_d[row] = lse_d;
        m_spill = p.part_m[static_cast<long long>(slot0) * BM + r];
    }
    const float g = p.grad_loss ? p.grad_loss[row] : 1.f;
    float S_q = 0.f;

    float lse_t = 0.f;
    if (p.row_tiles_t > 0) {
        find_slots(p.sched, rt, slot0, S);
        lse_t = warp_lse(p.part_m, p.part_s, slot0, S, r, lane);
        if (lane == 0) {
            p.lse_t[row] = lse_t;
            if (p.coef_t_out) p.coef_t_out[row] = expf(p.part_m[static_cast<long long>(slot0) * BM + r] - lse_t);
        }
    }
    const bool combined = p.coef_t_out != nullptr;
    const float coef_t = combined ? expf(p.part_m[static_cast<long long>(slot0) * BM + r] - lse_t) : 0.f;
    float ce_corr = 0.f;
    const float gw = combined ? g * p.w_topk : g;     // weight of the Omega_hat term q 1[Omega_hat] in dz_d

    const __nv_bfloat16* hrow = p.H_d + static_cast<long long>(row) * p.d;
    float loss = 0.f;
    float prev_v = INFINITY;
    int prev_i = -1;
    const int cap = p.cap;
    __shared__ int sh_tok[8][K_CAP];      // Omega_hat of the warp's row (the bi-directional set needs 2K <= K_CAP)
    __shared__ float sh_q[8][K_CAP];
    __shared__ float sh_dot[8][K_CAP];
    float cum_q = 0.f;
    int n_sel = 0;
    const int wib = threadIdx.x >> 5;
    // next candidate of the slots [sl0, sl0 + nS) after (pv, pi) in the order: logit descending, then token id
    // ascending (warp-collective; every lane gets the result)
    auto select_next = [&](int sl0, int nS, float pv, int pi, float& bv, int& bi) {
        bv = -INFINITY;
        bi = INT_MAX;
        for (int sl = 0; sl < nS; ++sl) {
            const long long so = static_cast<long long>(sl0 + sl) * BM + r;
            const int n = p.cand_n[so];
            for (int e = lane; e < n; e += 32) {
                const uint2 ce = p.cand[so * cap + e];
                const float v = __uint_as_float(ce.x);
                const int i = static_cast<int>(ce.y);
                if (i < 0) continue;
                const bool after_prev = (v < pv) || (v == pv && i > pi);
                const bool better = (v > bv) || (v == bv && i < bi);
                if (after_prev && better) {
                    bv = v;
                    bi = i;
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
            }
        }
    };
    const int ostride = p.bidir ? 2 * K : K;     // entries per row of idx_out / q_out
    for (int j = 0; j < K; ++j) {
        int tok;
        float qv;
        if (p.row_tiles_t > 0) {
            float bv;
            int bi;
            select_next(slot0, S, prev_v, prev_i, bv, bi);
            prev_v = bv;
            prev_i = bi;
            tok = bi == INT_MAX ? 0 : bi;     // cannot happen for K <= V; keeps the gather in range
            qv = expf(bv - lse_t);
            int tok_out = tok;
            if (p.top_p > 0.f) {
                // Top-P: a token belongs to Omega_hat while the probability of those before it is <= P
                if (cum_q > p.top_p) {
                    tok_out = -1;
                    tok = 0;
                    qv = 0.f;
                } else {
                    ++n_sel;
                }
                cum_q += qv;
            } else {
                ++n_sel;
            }
            if (lane == 0) {
                p.idx_out[static_cast<long long>(row) * ostride + j] = tok_out;
                p.q_out[static_cast<long long>(row) * ostride + j] = qv;
            }
        } else {
            tok = p.idx_in[static_cast<long long>(row) * K + j];
            qv = p.q_in[static_cast<long long>(row) * K + j];
        }
        S_q += qv;
        if (lane == 0) {
            if (p.gq_out) p.gq_out[static_cast<long long>(row) * K + j] = g * qv;
            sh_tok[wib][j] = tok;
            sh_q[wib][j] = qv;
        }
    }
    __syncwarp();
    int Ku = K;                                   // |Omega_hat| slots in use (2K at most for the bi-directional set)
    if (p.bidir) {
        // the draft's own K most probable tokens, in descending p; those not in the target's set join Omega_hat
        float pv = INFINITY;
        int pi = -1;
        for (int j = 0; j < K; ++j) {
            float bv;
            int bi;
            select_next(slot0_d, S_d, pv, pi, bv, bi);
            pv = bv;
            pi = bi;
            if (bi == INT_MAX) break;
            bool dup = false;
            for (int t = lane; t < K; t += 32) dup |= (sh_tok[wib][t] == bi);
            if (__any_sync(0xffffffffu, dup)) continue;
            // target probability of this token: q = exp(<H_t[row], W[tok]> - lse_t)
            const __nv_bfloat16* trow = p.H_t + static_cast<long long>(row) * p.d;
            const __nv_bfloat16* wrow = p.W + static_cast<long long>(bi) * p.d;
            float acc = 0.f;
            for (int k0 = lane * 8; k0 < p.d; k0 += 256) {
                const uint4 hv = *reinterpret_cast<const uint4*>(trow + k0);
                const uint4 wv = *reinterpret_cast<const uint4*>(wrow + k0);
                const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
                const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float2 a2 = __bfloat1622float2(hp[t]);
                    const float2 b2 = __bfloat1622float2(wp[t]);
                    acc = fmaf(a2.x, b2.x, acc);
                    acc = fmaf(a2.y, b2.y, acc);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            const float qv = expf(acc - lse_t);
            S_q += qv;
            if (lane == 0) {
                sh_tok[wib][Ku] = bi;
                sh_q[wib][Ku] = qv;
                p.idx_out[static_cast<long long>(row) * ostride + Ku] = bi;
                p.q_out[static_cast<long long>(row) * ostride + Ku] = qv;
            }
            ++Ku;
        }
        for (int u = Ku + lane; u < 2 * K; u += 32) {
            p.idx_out[static_cast<long long>(row) * ostride + u] = -1;
            p.q_out[static_cast<long long>(row) * ostride + u] = 0.f;
        }
        n_sel = Ku;
        __syncwarp();
    }
    // Draft logits at Omega_hat (K dot products with rows of W) and, for the fused backward, the row
    // sum_{x in Omega_hat} g q(x) W[x, :]. The W rows are read once: FIN_GRP tokens at a time, 256 columns
    // (8 per lane) per step; the fp32 row is accumulated across token groups.
    float* so = (p.sparse_out && !p.normed) ? p.sparse_out + static_cast<long long>(local) * p.d : nullptr;
    for (int g0 = 0; g0 < Ku; g0 += FIN_GRP) {
        const int ng = Ku - g0 < FIN_GRP ? Ku - g0 : FIN_GRP;
        float dot[FIN_GRP];
#pragma unroll
        for (int jj = 0; jj < FIN_GRP; ++jj) dot[jj] = 0.f;
        for (int k0 = lane * 8; k0 < p.d; k0 += 256) {
            const uint4 hv = *reinterpret_cast<const uint4*>(hrow + k0);
            const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
            float h[8];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float2 f2 = __bfloat1622float2(hp[t]);
                h[2 * t] = f2.x;
                h[2 * t + 1] = f2.y;
            }
            float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (so && g0 > 0) {
                const float4 a0 = *reinterpret_cast<const float4*>(so + k0);
                const float4 a1 = *reinterpret_cast<const float4*>(so + k0 + 4);
                a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w;
                a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            }
#pragma unroll
            for (int jj = 0; jj < FIN_GRP; ++jj) {
                if (jj < ng) {
                    const float gq = gw * sh_q[wib][g0 + jj];
                    const uint4 wv = *reinterpret_cast<const uint4*>(p.W + static_cast<long long>(sh_tok[wib][g0 + jj]) * p.d + k0);
                    const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float2 b = __bfloat1622float2(wp[t]);
                        dot[jj] = fmaf(h[2 * t], b.x, dot[jj]);
                        dot[jj] = fmaf(h[2 * t + 1], b.y, dot[jj]);
                        a[2 * t] = fmaf(gq, b.x, a[2 * t]);
                        a[2 * t + 1] = fmaf(gq, b.y, a[2 * t + 1]);
                    }
                }
            }
            if (so) {
                *reinterpret_cast<float4*>(so + k0) = make_float4(a[0], a[1], a[2], a[3]);
                *reinterpret_cast<float4*>(so + k0 + 4) = make_float4(a[4], a[5], a[6], a[7]);
            }
        }
#pragma unroll
        for (int jj = 0; jj < FIN_GRP; ++jj) {
            float acc = dot[jj];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (jj < ng) {
                const float qv = sh_q[wib][g0 + jj];
                if (lane == 0) sh_dot[wib][g0 + jj] = acc;
                loss += qv * (lse_d - acc);     // -q log p,  log p = z_d - lse_d
                if (combined) {
                    const float q_spill = __bfloat162float(p.Pt[static_cast<long long>(local) * p.p_pitch + sh_tok[wib][g0 + jj]]) * coef_t;
                    ce_corr += (qv - q_spill) * acc;
                }
            }
        }
    }
    if (lane == 0 && p.n_out) p.n_out[row] = (p.top_p > 0.f && !(cum_q > p.top_p)) ? -n_sel : n_sel;
    if (p.normed) {
        // Normed Top-K: qn = q / S_q, pn = softmax of the draft logits restricted to Omega_hat
        __syncwarp();
        float mx = -INFINITY;
        for (int j = lane; j < K; j += 32) mx = fmaxf(mx, sh_dot[wib][j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int j = lane; j < K; j += 32) se += expf(sh_dot[wib][j] - mx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float lse_k = mx + logf(se);
        float ln = 0.f;
        for (int j = lane; j < K; j += 32) {
            const float qn = sh_q[wib][j] / S_q;
            const float zj = sh_dot[wib][j];
            ln += qn * (lse_k - zj);
            sh_dot[wib][j] = g * (expf(zj - lse_k) - qn);      // dL/dz_d on Omega_hat
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ln += __shfl_xor_sync(0xffffffffu, ln, o);
        loss = ln;
        __syncwarp();
        for (int k0 = lane * 8; k0 < p.d; k0 += 256) {
            float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int j = 0; j < K; ++j) {
                const float c = sh_dot[wib][j];
                const uint4 wv = *reinterpret_cast<const uint4*>(p.W + static_cast<long long>(sh_tok[wib][j]) * p.d + k0);
                const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float2 b = __bfloat1622float2(wp[t]);
                    a[2 * t] = fmaf(c, b.x, a[2 * t]);
                    a[2 * t + 1] = fmaf(c, b.y, a[2 * t + 1]);
                }
            }
            if (p.dH_fp32) {
                float* o = reinterpret_cast<float*>(p.dH_out) + static_cast<long long>(row) * p.d + k0;
                *reinterpret_cast<float4*>(o) = make_float4(a[0], a[1], a[2], a[3]);
                *reinterpret_cast<float4*>(o + 4) = make_float4(a[4], a[5], a[6], a[7]);
            } else {
                uint4 w;
                w.x = pack_bf16x2(a[0], a[1]);
                w.y = pack_bf16x2(a[2], a[3]);
                w.z = pack_bf16x2(a[4], a[5]);
                w.w = pack_bf16x2(a[6], a[7]);
                *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.dH_out) + static_cast<long long>(row) * p.d + k0) = w;
            }
        }
    }
    if (lane == 0) {
        if (combined) p.ce_corr_out[row] = ce_corr;
        p.loss[row] = loss;
        // dense part of dz_d: g S_q p (Top-K loss) or g (1 + w S_q) p (combined objective)
        if (p.coef_out) p.coef_out[row] = (combined ? g * (1.f + p.w_topk * S_q) : g * S_q) * expf(m_spill - lse_d);
    }
}

// ---------------------------------------------------------------------------------------------
// select_kernel: one warp per row, between the sweep of the target rows and the sweep of the draft rows of
// the fused call. Merges the target's partial statistics into lse_t, picks Omega_hat from the sweep's
// candidates (or takes it as an input), writes topk_idx / topk_q in descending q, and leaves the same set
// sorted by token id (sidx, sq) for the draft sweep, which copies z_d at those tokens out of its accumulators.
constexpr int SEL_WARPS = 4;          // warps (rows) per block
constexpr int SEL_MAX = 768;          // candidates of one row that fit its shared-memory window (> K_CAP + 32)

struct SelectParams {
    Schedule sched;        // schedule of the target sweep; its row tile t = rows [128 t, 128 t + 128) of the chunk
    int K, cap;
    int row_begin, rows;   // global rows [row_begin, row_begin + rows)
    int from_sweep;        // 1: Omega_hat from the sweep's candidates; 0: idx_in / q_in are given
    const float* part_m;
    const float* part_s;
    const uint2* cand;
    const int* cand_n;
    const int* idx_in;     // [N, K]
    const float* q_in;
    int* idx_out;          // [N, K] (from_sweep)
    float* q_out;
    float* lse_t;
    int* n_out;            // [N] |Omega_hat| (nullable)
    float top_p;           // > 0: Omega_hat is cut to the shortest sorted prefix with cumulative q > top_p
    int* sidx;             // [N, K] Omega_hat in increasing token id; unused entries INT_MAX
    float* sq;             // [N, K] q in the same order; unused entries 0
    const unsigned int* only_if_range;
};

// Warp-collective: the largest t such that at least `want` of the n keys satisfy key >= t (keys pass the
// filter `use`); bit by bit from the top.
template <typename KeyFn>
__device__ __forceinline__ uint32_t kth_largest_key(int n, int want, int lane, KeyFn key_of) {
    uint32_t T = 0u;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t c2 = T | (1u << bit);
        int c = 0;
        for (int e = lane; e < n; e += 32) {
            uint32_t k;
            if (key_of(e, k)) c += (k >= c2) ? 1 : 0;
        }
        c = __reduce_add_sync(0xffffffffu, c);
        if (c >= want) T = c2;
    }
    return T;
}

__global__ void __launch_bounds__(SEL_WARPS * 32) select_kernel(const __grid_constant__ SelectParams p) {
    if (p.only_if_range != nullptr && ((*p.only_if_range) & 0xffu) != 2u) return;
    __shared__ uint32_t sh_key[SEL_WARPS][SEL_MAX];   // ordered keys of the row's candidates
    __shared__ int sh_id[SEL_WARPS][SEL_MAX];
    __shared__ int sel_tok[SEL_WARPS][K_CAP];         // Omega_hat in descending q
    __shared__ float sel_q[SEL_WARPS][K_CAP];
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int local = blockIdx.x * SEL_WARPS + wib;
    if (local >= p.rows) return;
    const int row = p.row_begin + local;
    const int rt = local / BM, r = local % BM;
    const int K = p.K;
    const long long ro = static_cast<long long>(row) * K;

    if (p.from_sweep) {
        int slot0, S;
        find_slots(p.sched, rt, slot0, S);
        const float lse_t = warp_lse(p.part_m, p.part_s, slot0, S, r, lane);
        if (lane == 0) p.lse_t[row] = lse_t;
        // Pool of candidates in shared memory. The slots' lists are appended 32 entries at a time; whenever the
        // next 32 might not fit, the pool is cut to its K best (logit descending, lower token id first among
        // equal logits) and the K-th logit becomes a floor below which later candidates are not even copied.
        uint32_t* kk = sh_key[wib];
        int* ii = sh_id[wib];
        int n = 0;
        uint32_t floor_key = 0u;
        const uint32_t lt_mask = (1u << lane) - 1u;
        auto cut_to_k = [&]() {
            // K-th largest logit, then (only if several candidates share it) the id bound among those
            const uint32_t T = kth_largest_key(n, K, lane, [&](int e, uint32_t& k) { k = kk[e]; return true; });
            int n_gt = 0, n_eq = 0;
            for (int e = lane; e < n; e += 32) {
                n_gt += kk[e] > T ? 1 : 0;
                n_eq += kk[e] == T ? 1 : 0;
            }
            n_gt = __reduce_add_sync(0xffffffffu, n_gt);
            n_eq = __reduce_add_sync(0xffffffffu, n_eq);
            const int need_eq = K - n_gt;
            uint32_t T2 = 0u;      // among the candidates equal to T: those with ~id >= T2 (the lowest ids) are kept
            if (n_eq > need_eq)
                T2 = kth_largest_key(n, need_eq, lane, [&](int e, uint32_t& k) { k = ~static_cast<uint32_t>(ii[e]); return kk[e] == T; });
            int np = 0;
            for (int e0 = 0; e0 < n; e0 += 32) {
                const int e = e0 + lane;
                uint32_t ke = 0u;
                int ie = 0;
                if (e < n) {
                    ke = kk[e];
                    ie = ii[e];
                }
                const bool take = e < n && (ke > T || (ke == T && ~static_cast<uint32_t>(ie) >= T2));
                const uint32_t bm = __ballot_sync(0xffffffffu, take);
                __syncwarp();
                if (take) {
                    const int at = np + __popc(bm & lt_mask);      // at <= e: in place
                    kk[at] = ke;
                    ii[at] = ie;
                }
                np += __popc(bm);
                __syncwarp();
            }
            n = np;
            floor_key = T;
        };
        for (int sl = 0; sl < S; ++sl) {
            const long long so = static_cast<long long>(slot0 + sl) * BM + r;
            const int cn = p.cand_n[so];
            for (int e0 = 0; e0 < cn; e0 += 32) {
                if (n + 32 > SEL_MAX) cut_to_k();      // n > K here: the window holds more than K_CAP + 32 entries
                const int e = e0 + lane;
                bool ok = false;
                uint2 ce = make_uint2(0u, 0u);
                uint32_t key = 0u;
                if (e < cn) {
                    ce = p.cand[so * p.cap + e];
                    key = ordered_key(ce.x);
                    // unused register-list entries carry id -1; anything below the floor cannot be among the K best
                    ok = static_cast<int>(ce.y) >= 0 && key >= floor_key;
                }
                const uint32_t bm = __ballot_sync(0xffffffffu, ok);
                if (ok) {
                    const int at = n + __popc(bm & lt_mask);
                    kk[at] = key;
                    ii[at] = static_cast<int>(ce.y);
                }
                n += __popc(bm);
            }
            __syncwarp();
        }
        if (n > K) cut_to_k();
        __syncwarp();
        // order the K picks: logit descending, token id ascending
        for (int j = lane; j < K; j += 32) {
            const uint32_t kj = j < n ? kk[j] : 0u;
            const int ij = j < n ? ii[j] : 0;
            int rank = 0;
            for (int i = 0; i < K; ++i) {
                const uint32_t ki = i < n ? kk[i] : 0u;
                const int i2 = i < n ? ii[i] : 0;
                rank += (ki > kj || (ki == kj && (i2 < ij || (i2 == ij && i < j)))) ? 1 : 0;
            }
            sel_tok[wib][rank] = ij;
            sel_q[wib][rank] = j < n ? expf(__uint_as_float(key_bits(kj)) - lse_t) : 0.f;
        }
        __syncwarp();
        int n_sel = K;
        if (p.top_p > 0.f) {
            // Top-P: a token belongs to Omega_hat while the probability of those before it is <= P
            int n = 0;
            if (lane == 0) {
                float cum = 0.f;
                for (int j = 0; j < K; ++j) {
                    if (cum > p.top_p) {
                        sel_tok[wib][j] = -1;
                        sel_q[wib][j] = 0.f;
                    } else {
                        ++n;
                    }
                    cum += sel_q[wib][j];
                }
                if (!(cum > p.top_p)) n = -n;      // all K tokens taken and P still not exceeded: the cap cut the prefix
            }
            __syncwarp();
            n_sel = __shfl_sync(0xffffffffu, n, 0);
        }
        for (int j = lane; j < K; j += 32) {
            p.idx_out[ro + j] = sel_tok[wib][j];
            p.q_out[ro + j] = sel_q[wib][j];
        }
        if (lane == 0 && p.n_out) p.n_out[row] = n_sel;
    } else {
        for (int j = lane; j < K; j += 32) {
            sel_tok[wib][j] = p.idx_in[ro + j];
            sel_q[wib][j] = p.q_in[ro + j];
        }
        if (lane == 0 && p.n_out) p.n_out[row] = K;
    }
    __syncwarp();
    // the same set in increasing token id (entries cut by Top-P go to the end as INT_MAX / 0)
    for (int j = lane; j < K; j += 32) {
        const int tj = sel_tok[wib][j] < 0 ? INT_MAX : sel_tok[wib][j];
        int rank = 0;
        for (int i = 0; i < K; ++i) {
            const int ti = sel_tok[wib][i] < 0 ? INT_MAX : sel_tok[wib][i];
            rank += (ti < tj || (ti == tj && i < j)) ? 1 : 0;
        }
        p.sidx[ro + rank] = tj;
        p.sq[ro + rank] = tj == INT_MAX ? 0.f : sel_q[wib][j];
    }
}

// ---------------------------------------------------------------------------------------------
// loss_patch_kernel: one warp per row, after the sweep of the draft rows of the fused call. Merges the draft's
// partial statistics into lse_d, evaluates Eq. 1 from the captured draft logits, writes the per-row scale of the
// spilled tiles, and puts the Omega_hat term of dz_d into the spill itself: with the spilled value
// P~(v) = 2^(z_d(v) log2e - ref2), dz_d(v) = coef (P~(v) - [v in Omega_hat] q(v) / (S_q e^(m_spill - lse_d))),
// so the K entries of the row at its Omega_hat tokens are lowered in place (bf16) and the second GEMM needs
// nothing but the row scale in its epilogue.
struct LossPatchParams {
    Schedule sched;        // schedule of the draft sweep
    int K;
    int row_begin, rows;
    const float* part_m;
    const float* part_s;
    const int* sidx;       // [N, K]
    const float* sq;
    const float* cap_z;    // [N, K] z_d at sidx
    const float* grad_loss;
    float* loss;
    float* lse_d;
    float* coef_out;       // [N] g S_q e^(m_spill - lse_d)
    __nv_bfloat16* P;      // spill of the chunk [rows, p_pitch]
    long long p_pitch;
};

__global__ void __launch_bounds__(256) loss_patch_kernel(const __grid_constant__ LossPatchParams p) {
    const int lane = threadIdx.x & 31;
    const int local = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (local >= p.rows) return;
    const int row = p.row_begin + local;
    const int rt = local / BM, r = local % BM;
    const int K = p.K;
    int slot0, S;
    find_slots(p.sched, rt, slot0, S);
    const float lse_d = warp_lse(p.part_m, p.part_s, slot0, S, r, lane);
    const float m_spill = p.part_m[static_cast<long long>(slot0) * BM + r];
    const float g = p.grad_loss ? p.grad_loss[row] : 1.f;
    const long long ro = static_cast<long long>(row) * K;
    float S_q = 0.f, loss = 0.f;
    for (int j = lane; j < K; j += 32) {
        if (p.sidx[ro + j] != INT_MAX) {
            const float qv = p.sq[ro + j];
            S_q += qv;
            loss += qv * (lse_d - p.cap_z[ro + j]);     // -q log p,  log p = z_d - lse_d
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        S_q += __shfl_xor_sync(0xffffffffu, S_q, o);
        loss += __shfl_xor_sync(0xffffffffu, loss, o);
    }
    const float scale = S_q * expf(m_spill - lse_d);     // coef / g
    if (lane == 0) {
        p.loss[row] = loss;
        p.lse_d[row] = lse_d;
        if (p.coef_out) p.coef_out[row] = g * scale;
    }
    if (p.P != nullptr && g != 0.f && scale > 0.f && scale < INFINITY) {      // P == nullptr: forward only, nothing to patch
        const float inv = 1.f / scale;
        __nv_bfloat16* prow = p.P + static_cast<long long>(local) * p.p_pitch;
        for (int j = lane; j < K; j += 32) {
            const int tok = p.sidx[ro + j];
            if (tok != INT_MAX) prow[tok] = __float2bfloat16_rn(__bfloat162float(prow[tok]) - p.sq[ro + j] * inv);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// ce_kernel (combined objective): one warp per row of a chunk. T[local, :] = q W of the row (from the second
// GEMM over the target spill). Full-vocabulary cross-entropy -sum_v q log p = lse_d - <H_d[row], q W>, and the
// (with the fp32 correction of the Omega_hat terms from finalize) the q W row joins the row's Omega_hat term so that dH_d = coef (draft spill x W) - sparse.
__global__ void __launch_bounds__(256) ce_kernel(int rows, int row_begin, int d, const __nv_bfloat16* __restrict__ H_d,
                                                 const float* __restrict__ T, const float* __restrict__ lse_d,
                                                 const float* __restrict__ grad_loss, const float* __restrict__ ce_corr,
                                                 float* __restrict__ loss_ce, float* __restrict__ sparse,
                                                 const unsigned int* __restrict__ only_if_range) {
    if (only_if_range != nullptr && ((*only_if_range) & 0xffu) != 2u) return;
    const int lane = threadIdx.x & 31;
    const int local = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (local >= rows) return;
    const int row = row_begin + local;
    const float g = grad_loss ? grad_loss[row] : 1.f;
    const __nv_bfloat16* hrow = H_d + static_cast<long long>(row) * d;
    const float* trow = T + static_cast<long long>(local) * d;
    float* srow = sparse + static_cast<long long>(local) * d;
    float dot = 0.f;
    for (int k0 = lane * 8; k0 < d; k0 += 256) {
        const uint4 hv = *reinterpret_cast<const uint4*>(hrow + k0);
        const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
        const float4 t0 = *reinterpret_cast<const float4*>(trow + k0);
        const float4 t1 = *reinterpret_cast<const float4*>(trow + k0 + 4);
        float4 s0 = *reinterpret_cast<const float4*>(srow + k0);
        float4 s1 = *reinterpret_cast<const float4*>(srow + k0 + 4);
        const float2 h0 = __bfloat1622float2(hp[0]), h1 = __bfloat1622float2(hp[1]);
        const float2 h2 = __bfloat1622float2(hp[2]), h3 = __bfloat1622float2(hp[3]);
        dot += h0.x * t0.x + h0.y * t0.y + h1.x * t0.z + h1.y * t0.w + h2.x * t1.x + h2.y * t1.y + h3.x * t1.z + h3.y * t1.w;
        s0.x = fmaf(g, t0.x, s0.x); s0.y = fmaf(g, t0.y, s0.y); s0.z = fmaf(g, t0.z, s0.z); s0.w = fmaf(g, t0.w, s0.w);
        s1.x = fmaf(g, t1.x, s1.x); s1.y = fmaf(g, t1.y, s1.y); s1.z = fmaf(g, t1.z, s1.z); s1.w = fmaf(g, t1.w, s1.w);
        *reinterpret_cast<float4*>(srow + k0) = s0;
        *reinterpret_cast<float4*>(srow + k0 + 4) = s1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (lane == 0) loss_ce[row] = lse_d[row] - dot - ce_corr[row];
}

// Self-test of the bounded waits (hass_selftest_wait_expiry): one CTA, no TMA, no tensor memory. Every thread
// waits for a phase of an mbarrier that nothing ever completes; thread 0 with the caller's short limit, the
// others with the library's normal limit. Thread 0 runs out of time, records its code in the status word and
// raises the CTA's abort flag, which ends the other threads' waits; the kernel then returns by itself.
// report[0] = threads whose wait gave up, report[1] = nanoseconds the CTA spent waiting.
__global__ void wait_expiry_selftest_kernel(unsigned int* status, unsigned long long limit_ns, unsigned int* report) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    __shared__ int gave_up;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        gave_up = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const unsigned long long t0 = globaltimer_ns();
    const bool done = wait_barrier(smem_u32(&bar), 0u, &abort_flag, status, 15u, threadIdx.x == 0 ? limit_ns : kWaitLimitNs);
    if (!done) atomicAdd(&gave_up, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        report[0] = static_cast<unsigned int>(gave_up);
        report[1] = static_cast<unsigned int>(globaltimer_ns() - t0);
    }
}

// Ends the exact route after a fused call: the range report has been dealt with. Word 2 of the status block
// records that the route ran (the host-buffer entry then copies dH_d to the host once more).
__global__ void range_handled_kernel(unsigned int* status) {
    if (((*status) & 0xffu) == 2u) {
        *status = 0u;
        status[2] = 1u;
    }
}

// ---------------------------------------------------------------------------------------------
// bwd_prep: one warp per row. Sorts Omega_hat by token id (the MODE_PROBS epilogue walks the vocabulary in
// increasing order; entries cut by Top-P carry id -1 and come first) by ranking every entry against the
// others, and precomputes g * q, g * S_q and lse_d * log2(e).
constexpr int PREP_WARPS = 4;
__global__ void __launch_bounds__(PREP_WARPS * 32) bwd_prep_kernel(int N, int K, const int* __restrict__ idx,
                                                                    const float* __restrict__ q,
                                                                    const float* __restrict__ lse_d,
                                                                    const float* __restrict__ grad_loss,
                                                                    int* __restrict__ sidx, float* __restrict__ sgq,
                                                                    float* __restrict__ coef, float* __restrict__ lse2,
                                                                    const unsigned int* __restrict__ only_if_range) {
    if (only_if_range != nullptr && ((*only_if_range) & 0xffu) != 2u) return;
    __shared__ int s_tok[PREP_WARPS][K_CAP];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int row = blockIdx.x * PREP_WARPS + wib;
    if (row >= N) return;
    const long long ro = static_cast<long long>(row) * K;
    const float g = grad_loss ? grad_loss[row] : 1.f;
    float S_q = 0.f;
    for (int j = lane; j < K; j += 32) {
        s_tok[wib][j] = idx[ro + j];
        S_q += q[ro + j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S_q += __shfl_xor_sync(0xffffffffu, S_q, o);
    __syncwarp();
    for (int j = lane; j < K; j += 32) {
        const int tj = s_tok[wib][j];
        int rank = 0;
        for (int i = 0; i < K; ++i) {
            const int ti = s_tok[wib][i];
            rank += (ti < tj || (ti == tj && i < j)) ? 1 : 0;
        }
        sidx[ro + rank] = tj;
        sgq[ro + rank] = g * q[ro + j];
    }
    if (lane == 0) {
        coef[row] = g * S_q;
        lse2[row] = lse_d[row] * LOG2E;
    }
}

}  // namespace hass
