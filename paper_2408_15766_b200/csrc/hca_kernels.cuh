// HCA attention of the draft layer (Section 3.2; the appendix's attention listing) for sm_100a.
//
// One persistent, warp-specialised kernel. A work item is one (sequence, query head, tile of 128
// query positions); it sweeps the key tiles 0 .. its own (causal). Per key tile:
//   S = Q K_t^T            tcgen05.mma, 128 x 128 x 128, fp32 in TMEM (two S buffers)
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
//        1 = MMA issuer and TMEM owner, 2-5 = softmax + epilogue (TMEM lane quadrant = warp % 4).
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
constexpr int NUM_THREADS = 192;
constexpr int TILE_BYTES = 128 * 128 * 2;           // any 128 x 128 bf16 tile: two 16 KB halves of 64 columns
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int SMEM_Q = 0;
constexpr int SMEM_K = SMEM_Q + TILE_BYTES;          // 2 stages
constexpr int SMEM_V = SMEM_K + 2 * TILE_BYTES;      // 2 stages
constexpr int SMEM_P = SMEM_V + 2 * TILE_BYTES;      // 2 buffers
constexpr int SMEM_BAR = SMEM_P + 2 * TILE_BYTES;
constexpr int NUM_BARS = 19;
constexpr int SMEM_BYTES = SMEM_BAR + 256 + 1024 /*alignment slack*/;
constexpr int TMEM_COLS = 512;     // S0 at 0, S1 at 128, O at 256
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
    // barriers
    const uint32_t q_full = bar0, q_empty = bar0 + 8;
    auto k_full = [&](int b) { return bar0 + 8u * (2 + b); };
    auto k_empty = [&](int b) { return bar0 + 8u * (4 + b); };
    auto v_full = [&](int b) { return bar0 + 8u * (6 + b); };
    auto v_empty = [&](int b) { return bar0 + 8u * (8 + b); };
    auto s_full = [&](int b) { return bar0 + 8u * (10 + b); };
    auto s_empty = [&](int b) { return bar0 + 8u * (12 + b); };
    auto p_full = [&](int b) { return bar0 + 8u * (14 + b); };
    auto pv_done = [&](int b) { return bar0 + 8u * (16 + b); };
    const uint32_t o_free = bar0 + 8u * 18;
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + SMEM_BAR + 8 * NUM_BARS);
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
            mbar_init(p_full(b), 4);
            mbar_init(pv_done(b), 1);
        }
        mbar_init(o_free, 4);
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
    // Per item the tensor core runs two sequences, each with its own ring counter:
    //   score sequence (K ring, S buffers), length m + qt + 1: draft pass 0 .. m-1, then key tiles 0 .. qt
    //   value sequence (V ring, P buffers), length qt + 1 + m: key tiles 0 .. qt, then draft pass 0 .. m-1

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
                if (!wait_barrier(q_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(q_full, TILE_BYTES);
                tma_load_3d(base + SMEM_Q, &p.tmQ, q_full, h * HD, qt * QT, b);
                tma_load_3d(base + SMEM_Q + HALF_BYTES, &p.tmQ, q_full, h * HD + 64, qt * QT, b);
                // draft keys start i rows early: row r of the tile is position qt*128 + r - i (zeros before the sequence)
                for (int i = 0; i < m && ok; ++i) ok = load_k(&p.tmKd[i], col, qt * QT - i, b);
                for (int j = 0; j <= qt && ok; ++j) {
                    ok = load_k(&p.tmK, col, j * KT, b);
                    if (ok) ok = load_v(&p.tmV, col, j * KT, b);
                }
                for (int i = 0; i < m && ok; ++i) ok = load_v(&p.tmVd[i], col, qt * QT - i, b);
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(QT, HD, 0, 1);
            const uint32_t tmem_o = tmem_base + 2 * KT;
            uint32_t gk = 0, gv = 0, it = 0;
            bool ok = true;
            // next element of the score sequence: S = Q K^T into S buffer gk & 1
            auto issue_s = [&]() -> bool {
                const int s = gk & 1u;
                const uint32_t ph = (gk >> 1) & 1u;
                if (!wait_barrier(k_full(s), ph, abort_flag, p.status, 4)) return false;
                if (!wait_barrier(s_empty(s), ph ^ 1u, abort_flag, p.status, 5)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t off = (k >> 2) * HALF_BYTES + (k & 3) * 32;
                    const uint64_t a_desc = make_smem_desc_sw128(base + SMEM_Q + off, 0, 1024);
                    const uint64_t b_desc = make_smem_desc_sw128(base + SMEM_K + s * TILE_BYTES + off, 0, 1024);
                    umma_bf16(tmem_base + s * KT, a_desc, b_desc, idesc_s, k != 0 ? 1u : 0u);
                }
                umma_commit(k_empty(s));
                umma_commit(s_full(s));
                ++gk;
                return true;
            };
            // next element of the value sequence: O (+)= P V
            auto issue_pv = [&](bool first) -> bool {
                const int s = gv & 1u;
                const uint32_t ph = (gv >> 1) & 1u;
                if (!wait_barrier(p_full(s), ph, abort_flag, p.status, 7)) return false;
                if (!wait_barrier(v_full(s), ph, abort_flag, p.status, 8)) return false;
                if (first && !wait_barrier(o_free, (it & 1u) ^ 1u, abort_flag, p.status, 9)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < KT / 16; ++k) {
                    // A = P: K-major halves of 64 keys. B = V: 16 keys further = 16 rows of 128 bytes.
                    const uint64_t a_desc = make_smem_desc_sw128(
                        base + SMEM_P + s * TILE_BYTES + (k >> 2) * HALF_BYTES + (k & 3) * 32, 0, 1024);
                    const uint64_t b_desc =
                        make_smem_desc_sw128(base + SMEM_V + s * TILE_BYTES + k * 16 * 128, HALF_BYTES, 1024);
                    umma_bf16(tmem_o, a_desc, b_desc, idesc_o, (!first || k != 0) ? 1u : 0u);
                }
                umma_commit(v_empty(s));
                umma_commit(pv_done(s));
                ++gv;
                return true;
            };
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++it) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int n_s = m + qt + 1;
                if (!wait_barrier(q_full, it & 1u, abort_flag, p.status, 6)) break;
                if (!issue_s()) break;
                if (n_s == 1) umma_commit(q_empty);
                for (int a = 0; a < n_s && ok; ++a) {
                    if (a + 1 < n_s) {
                        ok = issue_s();
                        if (ok && a + 2 == n_s) umma_commit(q_empty);      // Q is free once the item's last S has read it
                    }
                    if (ok && a >= m) ok = issue_pv(a == m);
                }
                for (int i = 0; i < m && ok; ++i) ok = issue_pv(false);
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
        bool store_pending = false;      // lane 0: a TMA store of this warp may still be reading its staging rows
        // 16-byte unit `chunk` (0..15) of this thread's 256-byte row of P buffer s, as the tensor core and TMA see it
        auto p_addr = [&](int s, int chunk) {
            return base + SMEM_P + s * TILE_BYTES + (chunk >> 3) * HALF_BYTES + r * 128 + ((((chunk & 7) ^ (r & 7))) << 4);
        };
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x) {
            int qt, b, h;
            decode(item, qt, b, h);
            const int t = qt * QT + r;                        // position in the sequence
            const bool valid = t < p.T;
            // ---- draft passes of the score sequence: keep the diagonal element of each S_i (raw, unscaled) ----
            float sd[MAX_DRAFTS];
#pragma unroll
            for (int i = 0; i < MAX_DRAFTS; ++i) sd[i] = 0.f;
#pragma unroll 1
            for (int i = 0; i < m; ++i, ++gk) {
                const int s = gk & 1u;
                if (!wait_barrier(s_full(s), (gk >> 1) & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                uint32_t raw[32];
                tmem_ld32(tmem_base + s * KT + lane_addr + 32 * quad, raw);     // columns of this warp's diagonal block
                tmem_ld_wait(raw);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(s));
                float dv = 0.f;
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (c == lane) dv = __uint_as_float(raw[c]);
#pragma unroll
                for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                    if (ii == i) sd[ii] = dv;
            }
            if (!ok) break;
            float mref = -INFINITY, l = 0.f;
            for (int j = 0; j <= qt; ++j, ++gk, ++gv) {
                const int s = gk & 1u;
                if (!wait_barrier(s_full(s), (gk >> 1) & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * KT + lane_addr;
                const bool diag = (j == qt);
                // Columns past t - m are hidden in the score tile: the causal part (s > t) and the m substituted
                // entries (t - m < s <= t), which enter the row's maximum and sum as scalars at the diagonal tile.
                // Only the last two tiles can hold such columns.
                const bool band = diag || (m > 0 && j + 1 == qt);
                const int lim = t - m - j * KT;
                // the whole row of S into registers, then the S buffer goes back to the tensor core
                uint32_t raw[4][32];
#pragma unroll
                for (int k = 0; k < 4; ++k) tmem_ld32(tmem_s + 32 * k, raw[k]);
#pragma unroll
                for (int k = 0; k < 4; ++k) tmem_ld_wait(raw[k]);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(s));
                float v[4][32];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
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
                for (int k = 0; k < 4; ++k) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = fmax3(mx0, v[k][c], v[k][c + 1]);
                        mx1 = fmax3(mx1, v[k][c + 2], v[k][c + 3]);
                    }
                }
                if (diag) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < m && t - i >= 0) mx0 = fmaxf(mx0, sd[i]);
                }
                const float cand = fmaxf(mx0, mx1) * p.c2;
                if (j == 0) {
                    mref = cand;
                } else {
                    const bool grow = cand > mref + RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rescale the accumulator: O of this row *= 2^(old ref - new ref); needs the previous PV complete
                        const float f = grow ? ex2(mref - cand) : 1.f;
                        if (grow) {
                            mref = cand;
                            l *= f;
                        }
                        const uint32_t gp = gv - 1;
                        if (!wait_barrier(pv_done(gp & 1u), (gp >> 1) & 1u, abort_flag, p.status, 11)) { ok = false; break; }
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
                const float nref = -mref;
                float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
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
                const int ps = gv & 1u;
                if (!wait_barrier(pv_done(ps), ((gv >> 1) & 1u) ^ 1u, abort_flag, p.status, 12)) { ok = false; break; }   // P[ps] has been read
                if (store_pending) {
                    bulk_wait_read();          // (lane 0) the previous item's O store has read this warp's staging rows
                    store_pending = false;
                }
                __syncwarp();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        st_shared_v4(p_addr(ps, 4 * k + q4), pack_bf16(v[k][8 * q4], v[k][8 * q4 + 1]),
                                     pack_bf16(v[k][8 * q4 + 2], v[k][8 * q4 + 3]), pack_bf16(v[k][8 * q4 + 4], v[k][8 * q4 + 5]),
                                     pack_bf16(v[k][8 * q4 + 6], v[k][8 * q4 + 7]));
                }
                fence_proxy_async_smem();      // P visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(ps));
            }
            if (!ok) break;
            // ---- draft passes of the value sequence: P holds only the weight 2^(sd c2 - ref) on its diagonal ----
#pragma unroll 1
            for (int i = 0; i < m; ++i, ++gv) {
                float sdi = 0.f;
#pragma unroll
                for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                    if (ii == i) sdi = sd[ii];
                const float pi = (t - i >= 0) ? ex2(fmaf(sdi, p.c2, -mref)) : 0.f;
                l += pi;
                const uint32_t bits = pack_bf16(pi, 0.f) << ((r & 1) * 16);        // column r sits in word (r & 7) / 2
                const int ps = gv & 1u;
                if (!wait_barrier(pv_done(ps), ((gv >> 1) & 1u) ^ 1u, abort_flag, p.status, 14)) { ok = false; break; }
#pragma unroll
                for (int chunk = 0; chunk < 16; ++chunk) {
                    const bool here = chunk == (r >> 3);
                    const int w = (r & 7) >> 1;
                    st_shared_v4(p_addr(ps, chunk), here && w == 0 ? bits : 0u, here && w == 1 ? bits : 0u,
                                 here && w == 2 ? bits : 0u, here && w == 3 ? bits : 0u);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(ps));
            }
            if (!ok) break;
            // ---- epilogue: O / l as bf16, staged in this warp's rows of P buffer 0 and stored with TMA ----
            {
                const uint32_t gp = gv - 1;
                if (!wait_barrier(pv_done(gp & 1u), (gp >> 1) & 1u, abort_flag, p.status, 13)) break;
                tc_fence_after_sync();
                const float inv = 1.f / l;
                if (valid && p.lse != nullptr)
                    p.lse[(static_cast<size_t>(b) * p.H + h) * p.T + t] = (mref + log2f(l)) * 0.6931471805599453f;
                uint32_t raw[4][32];
#pragma unroll
                for (int k = 0; k < 4; ++k) tmem_ld32(tmem_o + 32 * k, raw[k]);
#pragma unroll
                for (int k = 0; k < 4; ++k) tmem_ld_wait(raw[k]);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(o_free);         // the accumulator may be overwritten by the next item
                // every PV product of the item is complete, so both P buffers are idle; the bytes used are this
                // warp's own rows, which no other warp writes
#pragma unroll
                for (int k = 0; k < 4; ++k) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const uint32_t* x = &raw[k][8 * q4];
                        st_shared_v4(p_addr(0, 4 * k + q4),
                                     pack_bf16(__uint_as_float(x[0]) * inv, __uint_as_float(x[1]) * inv),
                                     pack_bf16(__uint_as_float(x[2]) * inv, __uint_as_float(x[3]) * inv),
                                     pack_bf16(__uint_as_float(x[4]) * inv, __uint_as_float(x[5]) * inv),
                                     pack_bf16(__uint_as_float(x[6]) * inv, __uint_as_float(x[7]) * inv));
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && qt * QT + quad * 32 < p.T) {
                    const uint32_t src = base + SMEM_P + quad * 32 * 128;
                    tma_store_3d(&p.tmO, src, h * HD, qt * QT + quad * 32, b);
                    tma_store_3d(&p.tmO, src + HALF_BYTES, h * HD + 64, qt * QT + quad * 32, b);
                    bulk_commit();
                    store_pending = true;
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
