// HCA attention of the draft layer (Section 3.2; the appendix's attention listing) for sm_100a.
//
// One persistent, warp-specialised kernel. A work item is one (sequence, query head, tile of 128
// query positions); it sweeps the key tiles 0 .. its own (causal). The key tiles of an item are dealt
// alternately to two softmax groups (even tiles: group 0, odd tiles: group 1), each with its own S
// buffer, P buffer, O accumulator and running (reference, sum); the two partial results are merged in
// the epilogue. The groups never synchronise inside the sweep, so while one waits for the tensor core
// or for TMEM the other keeps the exp unit busy. Per key tile:
//   S = Q K_t^T            tcgen05.mma, 128 x 128 x 128, fp32 in TMEM
//   softmax warps          read S (one query row per thread), hide the columns past t - m (the causal
//                          part and the m substituted entries), update the row's running reference
//                          and sum, write P = 2^(x - ref) as bf16 into shared memory in the swizzled
//                          layout the tensor core reads
//   O += P V_t             tcgen05.mma with V_t as an MN-major operand, fp32 in TMEM
// The substituted entries (t, t - i), i < m, ride the same pipeline as extra tiles of the item:
//   before the key tiles   S_i = Q K_d[i]^T with the K_d[i] tile fetched i rows early, so that the
//                          wanted scores <Q[t], K_d[i][t - i]> sit on the tile's main diagonal; each
//                          softmax thread keeps its diagonal element
//   at the diagonal tile   the m scores join the row maximum and sum
//   after the key tiles    O += diag(p_i) V_d[i], V_d[i] again fetched i rows early and the P buffer
//                          holding just the weights on its diagonal
// so no thread reads global memory; the epilogue divides by the row sum, stages bf16 rows in shared
// memory and stores them with TMA.
// The running reference moves only when a tile's maximum exceeds it by more than 2^8 (the O
// accumulator in TMEM is then rescaled in place by the softmax warps), so P stays within bf16
// range and most tiles skip the rescale.
//
// Warps: 0 = TMA producer (Q once per item, K and V tiles through two-stage rings),
//        1 = MMA issuer and TMEM owner, 2-5 = softmax group 0 + epilogue, 6-9 = softmax group 1
//        (TMEM lane quadrant = warp % 4). The diagonal tile's group also takes the draft passes.
//        320 threads leave 168 registers per thread, so a softmax thread reads its row of S from TMEM
//        twice, 64 columns at a time (maximum first, exponentials second), instead of holding all 128.
// Every wait is bounded (wait_barrier); a wait that gives up sets the status word and all roles leave.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace hass {
namespace hca {

constexpr int QT = 128;            // query rows per item
constexpr int KT = 128;            // keys per tile
constexpr int HD = 128;            // head dimension
constexpr int MAX_DRAFTS = 8;      // m <= 8
constexpr int NUM_THREADS = 320;
constexpr int TILE_BYTES = 128 * 128 * 2;           // any 128 x 128 bf16 tile: two 16 KB halves of 64 columns
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int SMEM_Q = 0;
constexpr int SMEM_K = SMEM_Q + TILE_BYTES;          // 2 stages
constexpr int SMEM_V = SMEM_K + 2 * TILE_BYTES;      // 2 stages
constexpr int SMEM_P = SMEM_V + 2 * TILE_BYTES;      // one buffer per softmax group
constexpr int SMEM_BAR = SMEM_P + 2 * TILE_BYTES;
constexpr int NUM_BARS = 21;
constexpr int SMEM_XCH = SMEM_BAR + 256;             // group 1's (reference, sum) per row for the merge: 128 x float2
constexpr int SMEM_BYTES = SMEM_XCH + 1024 + 1024 /*alignment slack*/;
constexpr int TMEM_COLS = 512;     // S of group 0 / 1 at columns 0 / 128, O of group 0 / 1 at 256 / 384
constexpr float RESCALE_LOG2 = 8.f;

struct Params {
    CUtensorMap tmQ, tmK, tmV;     // 3-D maps {heads * 128, T, B}, box {64, 128, 1}, 128-byte swizzle
    CUtensorMap tmKd[MAX_DRAFTS];  // the draft passes' keys and values, same geometry; index = sub-diagonal
    CUtensorMap tmVd[MAX_DRAFTS];
    CUtensorMap tmO;               // O [B, T, H * 128], box {64, 32, 1}: one warp's rows of half a tile
    float* lse;                    // [B, H, T] or null
    int B, T, H, Hkv, m;
    int q_tiles;                   // ceil(T / 128)
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
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Tiled store shared -> global (rows past the tensor's extent are clipped), tracked by bulk groups.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t smem_src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(tm)),
                 "r"(smem_src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__global__ void __launch_bounds__(NUM_THREADS, 1) hca_attention_kernel(const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + SMEM_BAR;
    // barriers (g = softmax group)
    const uint32_t q_full = bar0, q_empty = bar0 + 8;
    auto k_full = [&](int b) { return bar0 + 8u * (2 + b); };
    auto k_empty = [&](int b) { return bar0 + 8u * (4 + b); };
    auto v_full = [&](int b) { return bar0 + 8u * (6 + b); };
    auto v_empty = [&](int b) { return bar0 + 8u * (8 + b); };
    auto s_full = [&](int g) { return bar0 + 8u * (10 + g); };    // S of group g written by the tensor core
    auto s_empty = [&](int g) { return bar0 + 8u * (12 + g); };   // ... and read into registers by the group
    auto p_full = [&](int g) { return bar0 + 8u * (14 + g); };    // P of group g written
    auto pv_done = [&](int g) { return bar0 + 8u * (16 + g); };   // ... and consumed by its PV product
    const uint32_t o_free = bar0 + 8u * 18;                       // both accumulators read by the epilogue
    const uint32_t b_done = bar0 + 8u * 19;                       // group 1 posted its (reference, sum)
    const uint32_t x_free = bar0 + 8u * 20;                       // ... and group 0 has read them
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + SMEM_BAR + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);
    float2* xch = reinterpret_cast<float2*>(smem_gen + SMEM_XCH);

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
            mbar_init(p_full(b), 4);
            mbar_init(pv_done(b), 1);
        }
        mbar_init(o_free, 4);
        mbar_init(b_done, 4);
        mbar_init(x_free, 4);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmQ);
        prefetch_tensormap(&p.tmK);
        prefetch_tensormap(&p.tmV);
        prefetch_tensormap(&p.tmO);
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
    // The tensor core's program for one item, in issue order (e = 0 .. qt + m):
    //   e < qt          key tile e                 group e & 1        S and PV
    //   qt <= e < qt+m  draft pass e - qt (keys)   group qt & 1       S only
    //   e == qt + m     key tile qt (diagonal)     group qt & 1       S and PV
    // followed by the m draft passes' values (PV only, group qt & 1). S(e + 1) is issued before PV(e).

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            uint32_t gk = 0, gv = 0, it = 0;
            bool ok = true;
            auto load_k = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int s = gk & 1u;
                if (!wait_barrier(k_empty(s), ((gk >> 1) & 1u) ^ 1u, abort_flag, p.status, 2)) return false;
                mbar_arrive_expect_tx(k_full(s), TILE_BYTES);
                tma_load_3d(base + SMEM_K + s * TILE_BYTES, tm, k_full(s), col, row, b);
                tma_load_3d(base + SMEM_K + s * TILE_BYTES + HALF_BYTES, tm, k_full(s), col + 64, row, b);
                ++gk;
                return true;
            };
            auto load_v = [&](const CUtensorMap* tm, int col, int row, int b) -> bool {
                const int s = gv & 1u;
                if (!wait_barrier(v_empty(s), ((gv >> 1) & 1u) ^ 1u, abort_flag, p.status, 3)) return false;
                mbar_arrive_expect_tx(v_full(s), TILE_BYTES);
                tma_load_3d(base + SMEM_V + s * TILE_BYTES, tm, v_full(s), col, row, b);
                tma_load_3d(base + SMEM_V + s * TILE_BYTES + HALF_BYTES, tm, v_full(s), col + 64, row, b);
                ++gv;
                return true;
            };
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++it) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int col = (h / rep) * HD;
                const int n_e = qt + m + 1;
                if (!wait_barrier(q_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(q_full, TILE_BYTES);
                tma_load_3d(base + SMEM_Q, &p.tmQ, q_full, h * HD, qt * QT, b);
                tma_load_3d(base + SMEM_Q + HALF_BYTES, &p.tmQ, q_full, h * HD + 64, qt * QT, b);
                // keys of element e; a draft pass's tile starts i rows early (zeros before the sequence), so that
                // row r of the tile is position qt*128 + r - i
                auto keys = [&](int e) -> bool {
                    if (e < qt) return load_k(&p.tmK, col, e * KT, b);
                    if (e < qt + m) return load_k(&p.tmKd[e - qt], col, qt * QT - (e - qt), b);
                    return load_k(&p.tmK, col, qt * KT, b);
                };
                ok = keys(0);
                for (int e = 0; e < n_e && ok; ++e) {
                    if (e + 1 < n_e) ok = keys(e + 1);
                    if (ok && e < qt) ok = load_v(&p.tmV, col, e * KT, b);
                    if (ok && e == qt + m) ok = load_v(&p.tmV, col, qt * KT, b);
                }
                for (int i = 0; i < m && ok; ++i) ok = load_v(&p.tmVd[i], col, qt * QT - i, b);
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(QT, HD, 0, 1);
            uint32_t gk = 0, gv = 0, it = 0;
            uint32_t cs[2] = {0, 0}, cp[2] = {0, 0};      // S / PV elements issued per group so far
            bool ok = true;
            // S = Q K^T of the next key ring stage into group g's S buffer
            auto issue_s = [&](int g) -> bool {
                const int s = gk & 1u;
                if (!wait_barrier(k_full(s), (gk >> 1) & 1u, abort_flag, p.status, 4)) return false;
                if (!wait_barrier(s_empty(g), (cs[g] & 1u) ^ 1u, abort_flag, p.status, 5)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t off = (k >> 2) * HALF_BYTES + (k & 3) * 32;
                    const uint64_t a_desc = make_smem_desc_sw128(base + SMEM_Q + off, 0, 1024);
                    const uint64_t b_desc = make_smem_desc_sw128(base + SMEM_K + s * TILE_BYTES + off, 0, 1024);
                    umma_bf16(tmem_base + g * KT, a_desc, b_desc, idesc_s, k != 0 ? 1u : 0u);
                }
                umma_commit(k_empty(s));
                umma_commit(s_full(g));
                ++gk;
                ++cs[g];
                return true;
            };
            // O_g (+)= P_g V of the next value ring stage
            auto issue_pv = [&](int g, bool first) -> bool {
                const int s = gv & 1u;
                if (!wait_barrier(p_full(g), cp[g] & 1u, abort_flag, p.status, 7)) return false;
                if (!wait_barrier(v_full(s), (gv >> 1) & 1u, abort_flag, p.status, 8)) return false;
                if (first && !wait_barrier(o_free, (it & 1u) ^ 1u, abort_flag, p.status, 9)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < KT / 16; ++k) {
                    // A = P: K-major halves of 64 keys. B = V: 16 keys further = 16 rows of 128 bytes.
                    const uint64_t a_desc = make_smem_desc_sw128(
                        base + SMEM_P + g * TILE_BYTES + (k >> 2) * HALF_BYTES + (k & 3) * 32, 0, 1024);
                    const uint64_t b_desc =
                        make_smem_desc_sw128(base + SMEM_V + s * TILE_BYTES + k * 16 * 128, HALF_BYTES, 1024);
                    umma_bf16(tmem_base + (2 + g) * KT, a_desc, b_desc, idesc_o, (!first || k != 0) ? 1u : 0u);
                }
                umma_commit(v_empty(s));
                umma_commit(pv_done(g));
                ++gv;
                ++cp[g];
                return true;
            };
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++it) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int n_e = qt + m + 1;
                const int gd = qt & 1;
                auto group_of = [&](int e) { return e < qt ? (e & 1) : gd; };
                bool first[2] = {true, true};
                if (!wait_barrier(q_full, it & 1u, abort_flag, p.status, 6)) break;
                if (!issue_s(group_of(0))) break;
                if (n_e == 1) umma_commit(q_empty);
                for (int e = 0; e < n_e && ok; ++e) {
                    if (e + 1 < n_e) {
                        ok = issue_s(group_of(e + 1));
                        if (ok && e + 2 == n_e) umma_commit(q_empty);      // Q is free once the item's last S has read it
                    }
                    if (ok && (e < qt || e == qt + m)) {
                        const int g = group_of(e);
                        ok = issue_pv(g, first[g]);
                        first[g] = false;
                    }
                }
                for (int i = 0; i < m && ok; ++i) ok = issue_pv(gd, false);
            }
        }
    } else {
        // ===================== softmax groups (+ epilogue in group 0) =====================
        const int grp = (warp - 2) >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                       // row of the tile = TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tmem_s = tmem_base + grp * KT + lane_addr;
        const uint32_t tmem_o = tmem_base + (2 + grp) * KT + lane_addr;
        uint32_t cs = 0, cp = 0;         // S / PV elements of this group so far
        uint32_t cp_other = 0;           // group 0 only: PV elements of group 1 so far
        uint32_t nx = 0;                 // items in which group 1 took part (exchange barrier phases)
        bool ok = true;
        bool store_pending = false;      // lane 0 of group 0: a TMA store of this warp may still be reading its staging rows
        // 16-byte unit `chunk` (0..15) of this thread's 256-byte row of this group's P buffer, as the tensor core
        // and TMA see it
        auto p_addr = [&](int chunk) {
            return base + SMEM_P + grp * TILE_BYTES + (chunk >> 3) * HALF_BYTES + r * 128 + ((((chunk & 7) ^ (r & 7))) << 4);
        };
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x) {
            int qt, b, h;
            decode(item, qt, b, h);
            const int gd = qt & 1;
            const int t = qt * QT + r;                        // position in the sequence
            const bool valid = t < p.T;
            float sd[MAX_DRAFTS];
#pragma unroll
            for (int i = 0; i < MAX_DRAFTS; ++i) sd[i] = 0.f;
            float mref = -INFINITY, l = 0.f;
            bool fresh = true;          // no tile of this item seen yet by this group
            // this group's key tiles: grp, grp + 2, ... and, for the diagonal's group, the draft passes and tile qt
            for (int j = grp;; j += 2) {
                const bool diag = j >= qt;
                if (diag) {
                    if (grp != gd) break;
                    // ---- draft passes of the score sequence: keep the diagonal element of each S_i (raw, unscaled) ----
#pragma unroll 1
                    for (int i = 0; i < m; ++i, ++cs) {
                        if (!wait_barrier(s_full(grp), cs & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                        tc_fence_after_sync();
                        uint32_t raw[32];
                        tmem_ld32(tmem_s + 32 * quad, raw);     // columns of this warp's diagonal block
                        tmem_ld_wait(raw);
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(s_empty(grp));
                        float dv = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == lane) dv = __uint_as_float(raw[c]);
#pragma unroll
                        for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                            if (ii == i) sd[ii] = dv;
                    }
                    if (!ok) break;
                }
                if (!wait_barrier(s_full(grp), cs & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                // Columns past t - m are hidden in the score tile: the causal part (s > t) and the m substituted
                // entries (t - m < s <= t), which enter the row's maximum and sum as scalars at the diagonal tile.
                // Only the last two tiles can hold such columns.
                const bool band = diag || (m > 0 && j + 1 == qt);
                const int lim = t - m - j * KT;
                // ---- pass 1: row maximum, 64 columns at a time ----
                float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t ra[32], rb[32];
                    tmem_ld32(tmem_s + 64 * hf, ra);
                    tmem_ld32(tmem_s + 64 * hf + 32, rb);
                    tmem_ld_wait(ra);
                    tmem_ld_wait(rb);
                    if (band) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            if (64 * hf + c > lim) ra[c] = 0xff800000u;          // -inf
                            if (64 * hf + 32 + c > lim) rb[c] = 0xff800000u;
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        mx0 = fmax3(mx0, __uint_as_float(ra[c]), __uint_as_float(ra[c + 1]));
                        mx1 = fmax3(mx1, __uint_as_float(rb[c]), __uint_as_float(rb[c + 1]));
                    }
                }
                if (diag) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) mx0 = fmaxf(mx0, sd[i]);
                }
                const float cand = fmaxf(mx0, mx1) * p.c2;
                if (fresh) {
                    mref = cand;
                    fresh = false;
                } else {
                    const bool grow = cand > mref + RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rescale the accumulator: O of this row *= 2^(old ref - new ref); needs this group's previous PV complete
                        const float f = grow ? ex2(mref - cand) : 1.f;
                        if (grow) {
                            mref = cand;
                            l *= f;
                        }
                        if (!wait_barrier(pv_done(grp), (cp & 1u) ^ 1u, abort_flag, p.status, 11)) { ok = false; break; }
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
                // ---- pass 2: P = 2^(x c2 - ref), row sum in fp32, bf16 into shared memory ----
                if (!wait_barrier(pv_done(grp), (cp & 1u) ^ 1u, abort_flag, p.status, 12)) { ok = false; break; }   // P has been read
                if (store_pending) {
                    bulk_wait_read();          // (lane 0) the previous item's O store has read this warp's staging rows
                    store_pending = false;
                }
                __syncwarp();
                const float nref = -mref;
                float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t ra[32], rb[32];
                    tmem_ld32(tmem_s + 64 * hf, ra);
                    tmem_ld32(tmem_s + 64 * hf + 32, rb);
                    tmem_ld_wait(ra);
                    tmem_ld_wait(rb);
                    if (hf == 1) {
                        // the row is in registers for the last time: the S buffer goes back to the tensor core
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(s_empty(grp));
                    }
                    if (band) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            if (64 * hf + c > lim) ra[c] = 0xff800000u;
                            if (64 * hf + 32 + c > lim) rb[c] = 0xff800000u;
                        }
                    }
                    float va[32], vb[32];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1;
                        ffma2(x0, x1, __uint_as_float(ra[c]), __uint_as_float(ra[c + 1]), p.c2, p.c2, nref, nref);
                        va[c] = ex2(x0);
                        va[c + 1] = ex2(x1);
                        fadd2(ls0, ls1, ls0, ls1, va[c], va[c + 1]);
                        ffma2(x0, x1, __uint_as_float(rb[c]), __uint_as_float(rb[c + 1]), p.c2, p.c2, nref, nref);
                        vb[c] = ex2(x0);
                        vb[c + 1] = ex2(x1);
                        fadd2(ls0, ls1, ls0, ls1, vb[c], vb[c + 1]);
                    }
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        st_shared_v4(p_addr(8 * hf + q4), pack_bf16(va[8 * q4], va[8 * q4 + 1]),
                                     pack_bf16(va[8 * q4 + 2], va[8 * q4 + 3]), pack_bf16(va[8 * q4 + 4], va[8 * q4 + 5]),
                                     pack_bf16(va[8 * q4 + 6], va[8 * q4 + 7]));
                        st_shared_v4(p_addr(8 * hf + 4 + q4), pack_bf16(vb[8 * q4], vb[8 * q4 + 1]),
                                     pack_bf16(vb[8 * q4 + 2], vb[8 * q4 + 3]), pack_bf16(vb[8 * q4 + 4], vb[8 * q4 + 5]),
                                     pack_bf16(vb[8 * q4 + 6], vb[8 * q4 + 7]));
                    }
                }
                l += ls0 + ls1;
                ++cs;
                fence_proxy_async_smem();      // P visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(grp));
                ++cp;
                if (diag) {
                    // ---- draft passes of the value sequence: P holds only the weight 2^(sd c2 - ref) on its diagonal ----
#pragma unroll 1
                    for (int i = 0; i < m; ++i, ++cp) {
                        float sdi = 0.f;
#pragma unroll
                        for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                            if (ii == i) sdi = sd[ii];
                        const float pi = (t - i >= 0) ? ex2(fmaf(sdi, p.c2, -mref)) : 0.f;
                        l += pi;
                        const uint32_t bits = pack_bf16(pi, 0.f) << ((r & 1) * 16);        // column r sits in word (r & 7) / 2
                        if (!wait_barrier(pv_done(grp), (cp & 1u) ^ 1u, abort_flag, p.status, 14)) { ok = false; break; }
#pragma unroll
                        for (int chunk = 0; chunk < 16; ++chunk) {
                            const bool here = chunk == (r >> 3);
                            const int w = (r & 7) >> 1;
                            st_shared_v4(p_addr(chunk), here && w == 0 ? bits : 0u, here && w == 1 ? bits : 0u,
                                         here && w == 2 ? bits : 0u, here && w == 3 ? bits : 0u);
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(p_full(grp));
                    }
                    break;
                }
            }
            if (!ok) break;
            if (qt == 0 && grp == 1) continue;       // a one-tile item has nothing for group 1
            if (grp == 1) {
                // ---- post this group's (reference, sum); group 0 merges and stores ----
                if (!wait_barrier(x_free, (nx & 1u) ^ 1u, abort_flag, p.status, 15)) break;
                xch[r] = make_float2(mref, l);
                __syncwarp();
                if (lane == 0) mbar_arrive(b_done);
                ++nx;
                continue;
            }
            // ---- epilogue (group 0): merge the two partial results, O / l as bf16 staged in this warp's rows of
            //      its P buffer, stored with TMA ----
            {
                const bool two = qt >= 1;
                // group 1's PV elements in this item: its key tiles, and the diagonal's extras if it owns the diagonal
                cp_other += (qt / 2) + (gd == 1 ? 1 + m : 0);
                if (!wait_barrier(pv_done(0), (cp & 1u) ^ 1u, abort_flag, p.status, 13)) break;
                float fa = 1.f, fb = 0.f, lb = 0.f, mm = mref;
                if (two) {
                    if (!wait_barrier(b_done, nx & 1u, abort_flag, p.status, 16)) break;
                    if (!wait_barrier(pv_done(1), (cp_other & 1u) ^ 1u, abort_flag, p.status, 17)) break;
                    const float2 o = xch[r];
                    ++nx;
                    mm = fmaxf(mref, o.x);
                    fa = ex2(mref - mm);
                    fb = ex2(o.x - mm);
                    lb = o.y;
                }
                tc_fence_after_sync();
                const float lsum = l * fa + lb * fb;
                const float inv = 1.f / lsum;
                fa *= inv;
                fb *= inv;
                if (valid && p.lse != nullptr)
                    p.lse[(static_cast<size_t>(b) * p.H + h) * p.T + t] = (mm + log2f(lsum)) * 0.6931471805599453f;
                if (store_pending) {
                    bulk_wait_read();
                    store_pending = false;
                }
                __syncwarp();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint32_t ra[32], rb[32];
                    tmem_ld32(tmem_o + 32 * k, ra);
                    if (two) tmem_ld32(tmem_o + KT + 32 * k, rb);
                    tmem_ld_wait(ra);
                    if (two) tmem_ld_wait(rb);
                    float o[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        o[c] = __uint_as_float(ra[c]) * fa;
                        if (two) o[c] = fmaf(__uint_as_float(rb[c]), fb, o[c]);
                    }
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        st_shared_v4(p_addr(4 * k + q4), pack_bf16(o[8 * q4], o[8 * q4 + 1]),
                                     pack_bf16(o[8 * q4 + 2], o[8 * q4 + 3]), pack_bf16(o[8 * q4 + 4], o[8 * q4 + 5]),
                                     pack_bf16(o[8 * q4 + 6], o[8 * q4 + 7]));
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(o_free);         // both accumulators may be overwritten by the next item
                    if (two) mbar_arrive(x_free);
                    if (qt * QT + quad * 32 < p.T) {
                        const uint32_t src = base + SMEM_P + quad * 32 * 128;
                        tma_store_3d(&p.tmO, src, h * HD, qt * QT + quad * 32, b);
                        tma_store_3d(&p.tmO, src + HALF_BYTES, h * HD + 64, qt * QT + quad * 32, b);
                        bulk_commit();
                        store_pending = true;
                    }
                }
            }
        }
        if (lane == 0) bulk_wait_all();      // O stores complete before the CTA's shared memory goes away
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
