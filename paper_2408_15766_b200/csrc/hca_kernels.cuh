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
// The substituted entries (t, t - i), i < m, never pass through the tensor core: their scores against
// the i-th draft pass's keys are 128-long dot products the softmax warps compute up front (coalesced,
// one warp per 32 rows); they join the row maximum and sum at the diagonal tile, and their weight times
// the draft pass's value row is added in the epilogue, which also divides by the row sum.
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
    const __nv_bfloat16* Q;        // [B, T, H, 128]
    const __nv_bfloat16* K_d[MAX_DRAFTS];   // [B, T, Hkv, 128] each; index = sub-diagonal
    const __nv_bfloat16* V_d[MAX_DRAFTS];
    __nv_bfloat16* O;              // [B, T, H, 128]
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
__device__ __forceinline__ void prefetch_l2(const void* ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Dot product of two 128-element bf16 rows (16-byte aligned), fp32 accumulation.
__device__ __forceinline__ float dot128(const __nv_bfloat16* a, const __nv_bfloat16* b) {
    const uint4* pa = reinterpret_cast<const uint4*>(a);
    const uint4* pb = reinterpret_cast<const uint4*>(b);
    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
        const uint4 x = __ldg(pa + i), y = __ldg(pb + i);
        acc0 = fmaf(bf16_lo(x.x), bf16_lo(y.x), acc0);
        acc1 = fmaf(bf16_hi(x.x), bf16_hi(y.x), acc1);
        acc0 = fmaf(bf16_lo(x.y), bf16_lo(y.y), acc0);
        acc1 = fmaf(bf16_hi(x.y), bf16_hi(y.y), acc1);
        acc0 = fmaf(bf16_lo(x.z), bf16_lo(y.z), acc0);
        acc1 = fmaf(bf16_hi(x.z), bf16_hi(y.z), acc1);
        acc0 = fmaf(bf16_lo(x.w), bf16_lo(y.w), acc0);
        acc1 = fmaf(bf16_hi(x.w), bf16_hi(y.w), acc1);
    }
    return acc0 + acc1;
}

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
    // item -> (query tile, sequence, head): the longest items (last query tiles) come first
    auto decode = [&](int item, int& qt, int& b, int& h) {
        qt = p.q_tiles - 1 - item / BH;
        const int bh = item - (item / BH) * BH;
        b = bh / p.H;
        h = bh - b * p.H;
    };

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            uint32_t g = 0, it = 0;    // key tiles and items done by this CTA
            for (int item = blockIdx.x; item < p.items; item += gridDim.x, ++it) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int gkv = h / rep;
                if (!wait_barrier(q_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(q_full, TILE_BYTES);
                tma_load_3d(base + SMEM_Q, &p.tmQ, q_full, h * HD, qt * QT, b);
                tma_load_3d(base + SMEM_Q + HALF_BYTES, &p.tmQ, q_full, h * HD + 64, qt * QT, b);
                bool ok = true;
                for (int j = 0; j <= qt; ++j, ++g) {
                    const int s = g & 1u;
                    const uint32_t ph = (g >> 1) & 1u;
                    if (!wait_barrier(k_empty(s), ph ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
                    mbar_arrive_expect_tx(k_full(s), TILE_BYTES);
                    tma_load_3d(base + SMEM_K + s * TILE_BYTES, &p.tmK, k_full(s), gkv * HD, j * KT, b);
                    tma_load_3d(base + SMEM_K + s * TILE_BYTES + HALF_BYTES, &p.tmK, k_full(s), gkv * HD + 64, j * KT, b);
                    if (!wait_barrier(v_empty(s), ph ^ 1u, abort_flag, p.status, 3)) { ok = false; break; }
                    mbar_arrive_expect_tx(v_full(s), TILE_BYTES);
                    tma_load_3d(base + SMEM_V + s * TILE_BYTES, &p.tmV, v_full(s), gkv * HD, j * KT, b);
                    tma_load_3d(base + SMEM_V + s * TILE_BYTES + HALF_BYTES, &p.tmV, v_full(s), gkv * HD + 64, j * KT, b);
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_o = make_idesc_bf16(QT, HD, 0, 1);
            const uint32_t tmem_o = tmem_base + 2 * KT;
            uint32_t g = 0, it = 0;
            bool ok = true;
            // S(g) = Q K^T into S buffer g & 1
            auto issue_s = [&](uint32_t gg) -> bool {
                const int s = gg & 1u;
                const uint32_t ph = (gg >> 1) & 1u;
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
                return true;
            };
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++it) {
                int qt, b, h;
                decode(item, qt, b, h);
                if (!wait_barrier(q_full, it & 1u, abort_flag, p.status, 6)) break;
                if (!issue_s(g)) break;
                if (qt == 0) umma_commit(q_empty);
                for (int j = 0; j <= qt; ++j, ++g) {
                    if (j + 1 <= qt) {
                        if (!issue_s(g + 1)) { ok = false; break; }
                        if (j + 1 == qt) umma_commit(q_empty);      // Q is free once the item's last S has read it
                    }
                    const int s = g & 1u;
                    const uint32_t ph = (g >> 1) & 1u;
                    if (!wait_barrier(p_full(s), ph, abort_flag, p.status, 7)) { ok = false; break; }
                    if (!wait_barrier(v_full(s), ph, abort_flag, p.status, 8)) { ok = false; break; }
                    if (j == 0 && !wait_barrier(o_free, (it & 1u) ^ 1u, abort_flag, p.status, 9)) { ok = false; break; }
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < KT / 16; ++k) {
                        // A = P: K-major halves of 64 keys. B = V: 16 keys further = 16 rows of 128 bytes.
                        const uint64_t a_desc = make_smem_desc_sw128(
                            base + SMEM_P + s * TILE_BYTES + (k >> 2) * HALF_BYTES + (k & 3) * 32, 0, 1024);
                        const uint64_t b_desc =
                            make_smem_desc_sw128(base + SMEM_V + s * TILE_BYTES + k * 16 * 128, HALF_BYTES, 1024);
                        umma_bf16(tmem_o, a_desc, b_desc, idesc_o, (j | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(v_empty(s));
                    umma_commit(pv_done(s));
                }
            }
        }
    } else {
        // ===================== softmax + epilogue warps =====================
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                       // row of the tile = TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tmem_o = tmem_base + 2 * KT + lane_addr;
        uint32_t g = 0, it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++it) {
            int qt, b, h;
            decode(item, qt, b, h);
            const int gkv = h / rep;
            const int t = qt * QT + r;                        // position in the sequence
            const bool valid = t < p.T;
            const int t_warp = qt * QT + quad * 32;           // first row of this warp
            // ---- scores against the draft passes' keys on this row's substituted entries (raw, unscaled).
            // The warp takes its 32 rows one by one with coalesced 256-byte reads (lane = 4 columns), then a
            // transposing butterfly leaves row rr's dot product on lane rr.
            float sd[MAX_DRAFTS];
#pragma unroll
            for (int i = 0; i < MAX_DRAFTS; ++i) sd[i] = 0.f;
            if (p.m > 0 && item + static_cast<int>(gridDim.x) < p.items) {
                // pull the draft rows of this CTA's next item towards L2 while this item is processed
                int qt2, b2, h2;
                decode(item + gridDim.x, qt2, b2, h2);
                const int g2 = h2 / rep;
#pragma unroll 1
                for (int i = 0; i < p.m; ++i) {
                    int ts = qt2 * QT + r - i;
                    ts = ts < 0 ? 0 : (ts >= p.T ? p.T - 1 : ts);
                    const size_t off = ((static_cast<size_t>(b2) * p.T + ts) * p.Hkv + g2) * HD;
                    prefetch_l2(p.K_d[i] + off);
                    prefetch_l2(p.K_d[i] + off + 64);
                    prefetch_l2(p.V_d[i] + off);
                    prefetch_l2(p.V_d[i] + off + 64);
                }
            }
            if (p.m > 0) {
                uint2 qv[32];
#pragma unroll
                for (int rr = 0; rr < 32; ++rr) {
                    int tr = t_warp + rr;
                    tr = tr >= p.T ? p.T - 1 : tr;
                    qv[rr] = __ldg(reinterpret_cast<const uint2*>(
                                       p.Q + ((static_cast<size_t>(b) * p.T + tr) * p.H + h) * HD) + lane);
                }
#pragma unroll 1
                for (int i = 0; i < p.m; ++i) {
                    {
                        float acc[32];
                        const __nv_bfloat16* kd = p.K_d[i];
#pragma unroll
                        for (int rr = 0; rr < 32; ++rr) {
                            // rows outside the sequence read a clamped row (no branch around the load); their
                            // result is never used
                            int ts = t_warp + rr - i;
                            ts = ts < 0 ? 0 : (ts >= p.T ? p.T - 1 : ts);
                            const uint2 kv = __ldg(reinterpret_cast<const uint2*>(
                                                       kd + ((static_cast<size_t>(b) * p.T + ts) * p.Hkv + gkv) * HD) + lane);
                            acc[rr] = fmaf(bf16_lo(qv[rr].x), bf16_lo(kv.x),
                                           fmaf(bf16_hi(qv[rr].x), bf16_hi(kv.x),
                                                fmaf(bf16_lo(qv[rr].y), bf16_lo(kv.y), bf16_hi(qv[rr].y) * bf16_hi(kv.y))));
                        }
#pragma unroll
                        for (int sft = 16; sft >= 1; sft >>= 1) {
                            const bool up = (lane & sft) != 0;
#pragma unroll
                            for (int k = 0; k < sft; ++k) {
                                const float keep = up ? acc[k + sft] : acc[k];
                                const float send = up ? acc[k] : acc[k + sft];
                                acc[k] = keep + __shfl_xor_sync(0xffffffffu, send, sft);
                            }
                        }
#pragma unroll
                        for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                            if (ii == i) sd[ii] = acc[0];
                    }
                }
            }
            float mref = -INFINITY, l = 0.f;
            for (int j = 0; j <= qt; ++j, ++g) {
                const int s = g & 1u;
                const uint32_t ph = (g >> 1) & 1u;
                if (!wait_barrier(s_full(s), ph, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * KT + lane_addr;
                const bool diag = (j == qt);
                // Columns past t - m are hidden in the score tile: the causal part (s > t) and the m substituted
                // entries (t - m < s <= t), which enter the row's maximum and sum as scalars at the diagonal tile
                // and meet their value rows in the epilogue. Only the last two tiles can hold such columns.
                const bool band = diag || (p.m > 0 && j + 1 == qt);
                const int lim = t - p.m - j * KT;
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
                        if (i < p.m && t - i >= 0) mx0 = fmaxf(mx0, sd[i]);
                }
                const float cand = fmaxf(mx0, mx1) * p.c2;
                if (j == 0) {
                    mref = cand;
                } else {
                    const bool grow = cand > mref + RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rescale the accumulator: O of this row *= 2^(old ref - new ref); needs PV(g-1) complete
                        const float f = grow ? ex2(mref - cand) : 1.f;
                        if (grow) {
                            mref = cand;
                            l *= f;
                        }
                        const uint32_t gp = g - 1;
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
                if (diag) {
#pragma unroll
                    for (int i = 0; i < MAX_DRAFTS; ++i)
                        if (i < p.m && t - i >= 0) l += ex2(fmaf(sd[i], p.c2, nref));
                }
                if (!wait_barrier(pv_done(s), ph ^ 1u, abort_flag, p.status, 12)) { ok = false; break; }   // PV(g-2) has read P[s]
                const uint32_t p_row = base + SMEM_P + s * TILE_BYTES + r * 128;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t half = p_row + (k >> 1) * HALF_BYTES;
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int chunk = (k & 1) * 4 + q4;                // 16-byte unit inside the 128-byte row
                        st_shared_v4(half + (((chunk ^ (r & 7)) & 7) << 4), pack_bf16(v[k][8 * q4], v[k][8 * q4 + 1]),
                                     pack_bf16(v[k][8 * q4 + 2], v[k][8 * q4 + 3]), pack_bf16(v[k][8 * q4 + 4], v[k][8 * q4 + 5]),
                                     pack_bf16(v[k][8 * q4 + 6], v[k][8 * q4 + 7]));
                    }
                }
                fence_proxy_async_smem();      // P visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(s));
            }
            if (!ok) break;
            // ---- epilogue: O / l, plus the substituted entries' weight times the draft value rows ----
            {
                const uint32_t gp = g - 1;
                if (!wait_barrier(pv_done(gp & 1u), (gp >> 1) & 1u, abort_flag, p.status, 13)) break;
                tc_fence_after_sync();
                const float inv = 1.f / l;
                float pd[MAX_DRAFTS];
#pragma unroll
                for (int i = 0; i < MAX_DRAFTS; ++i)
                    pd[i] = (i < p.m && valid && t - i >= 0) ? ex2(fmaf(sd[i], p.c2, -mref)) * inv : 0.f;
                if (valid && p.lse != nullptr)
                    p.lse[(static_cast<size_t>(b) * p.H + h) * p.T + t] = (mref + log2f(l)) * 0.6931471805599453f;
                // Stage this warp's 32 rows of O (fp32, normalised) in shared memory. Both PV products that read
                // the P buffers are complete, and the bytes used are exactly this warp's own rows of the two
                // P buffers (4 pieces of 128 bytes per row), which no other warp writes.
                auto piece = [&](int rr, int k) {   // 128-byte piece k (columns 32k .. 32k+31) of row rr of this warp
                    return base + SMEM_P + (k >> 1) * TILE_BYTES + (k & 1) * HALF_BYTES + (quad * 32 + rr) * 128;
                };
                {
                    uint32_t raw[4][32];
#pragma unroll
                    for (int k = 0; k < 4; ++k) tmem_ld32(tmem_o + 32 * k, raw[k]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) tmem_ld_wait(raw[k]);
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(o_free);     // the accumulator may be overwritten by the next item
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
#pragma unroll
                        for (int c8 = 0; c8 < 8; ++c8)
                            st_shared_v4(piece(lane, k) + (((c8 ^ lane) & 7) << 4),
                                         __float_as_uint(__uint_as_float(raw[k][4 * c8]) * inv),
                                         __float_as_uint(__uint_as_float(raw[k][4 * c8 + 1]) * inv),
                                         __float_as_uint(__uint_as_float(raw[k][4 * c8 + 2]) * inv),
                                         __float_as_uint(__uint_as_float(raw[k][4 * c8 + 3]) * inv));
                    }
                }
                __syncwarp();
                // row by row with the warp across the 128 columns (lane = 4 columns): coalesced reads of the draft
                // value rows and coalesced stores of O
                const int kq = lane >> 3, cq = lane & 7;
#pragma unroll 1
                for (int rr0 = 0; rr0 < 32; rr0 += 16) {
                    float4 o[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u)
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(o[u].x), "=f"(o[u].y), "=f"(o[u].z), "=f"(o[u].w)
                                     : "r"(piece(rr0 + u, kq) + (((cq ^ (rr0 + u)) & 7) << 4)));
#pragma unroll 1
                    for (int i = 0; i < p.m; ++i) {
                        float pdi = 0.f;
#pragma unroll
                        for (int ii = 0; ii < MAX_DRAFTS; ++ii)
                            if (ii == i) pdi = pd[ii];
                        const __nv_bfloat16* vd = p.V_d[i];
                        uint2 vv[16];
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            int ts = t_warp + rr0 + u - i;
                            ts = ts < 0 ? 0 : (ts >= p.T ? p.T - 1 : ts);
                            vv[u] = __ldg(reinterpret_cast<const uint2*>(
                                              vd + ((static_cast<size_t>(b) * p.T + ts) * p.Hkv + gkv) * HD) + lane);
                        }
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            const float w = __shfl_sync(0xffffffffu, pdi, rr0 + u);    // 0 where the entry does not exist
                            o[u].x = fmaf(w, bf16_lo(vv[u].x), o[u].x);
                            o[u].y = fmaf(w, bf16_hi(vv[u].x), o[u].y);
                            o[u].z = fmaf(w, bf16_lo(vv[u].y), o[u].z);
                            o[u].w = fmaf(w, bf16_hi(vv[u].y), o[u].w);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        const int tr = t_warp + rr0 + u;
                        if (tr < p.T)
                            *(reinterpret_cast<uint2*>(p.O + ((static_cast<size_t>(b) * p.T + tr) * p.H + h) * HD) + lane) =
                                make_uint2(pack_bf16(o[u].x, o[u].y), pack_bf16(o[u].z, o[u].w));
                    }
                }
                __syncwarp();      // the staging bytes are this warp's P rows of the next tiles
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
