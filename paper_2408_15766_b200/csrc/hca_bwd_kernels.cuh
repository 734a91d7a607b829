// Backward of the HCA attention (Section 3.2) for sm_100a. With P = softmax weights (recomputed from the
// forward's row normaliser), D[t] = <dO[t], O[t]> and dS = P * (dP - D) * scale, dP[t,s] = <dO[t], v(t,s)>:
//   dQ[t]    = sum_s dS[t,s] k(t,s)                                  hca_dq_kernel (query tiles stationary)
//   dK_t[s]  = sum_{t: t-s >= m} dS[t,s] Q[t],  dV_t[s] = sum_{t: t-s >= m} P[t,s] dO[t]
//                                                                    hca_dkv_kernel (key tiles stationary)
//   dK_d[i][s] = dS[s+i,s] Q[s+i],  dV_d[i][s] = P[s+i,s] dO[s+i]    hca_draft_grad_kernel (one term per
//                                                                    query head of the group: row scalings)
// hca_dq_kernel also leaves P and dS of the substituted entries (t, t-i) in the workspace for the last one.
//
// Both tensor-core kernels follow the forward kernel's organisation (warp 0 TMA producer, warp 1 MMA issuer
// and TMEM owner, then row-owning warps - here two groups of four, taking alternate elements (dQ) or half of
// a tile's columns (dK/dV), which needs no exchange because the backward has no running row statistics) and
// its bounded waits. The A operands of the products come from tensor memory wherever they fit.
#pragma once
#include "hca_kernels.cuh"

namespace hass {
namespace hca_bwd {

using hca::ex2;
using hca::pack_bf16;
using hca::st_shared_v4;
using hca::tma_load_3d;

constexpr int QT = 128;
constexpr int KT = 64;
constexpr int HD = 128;
constexpr int MAX_DRAFTS = hca::MAX_DRAFTS;
constexpr int NUM_THREADS = 320;        // producer, MMA issuer, two groups of four row-owning warps
constexpr int Q_BYTES = QT * HD * 2;
constexpr int Q_HALF = Q_BYTES / 2;
constexpr int KV_BYTES = KT * HD * 2;
constexpr int KV_HALF = KV_BYTES / 2;
constexpr int DS_BYTES = QT * KT * 2;

// D[b, h, t] = <dO[b, t, h, :], O[b, t, h, :]>, half a warp per row of 128 (16 bytes per lane and tensor).
__global__ void hca_bwd_prep_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO,
                                    float* __restrict__ D, int B, int T, int H) {
    const long long row = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 4;   // (b, t, h)
    const int sub = threadIdx.x & 15;
    const bool live = row < static_cast<long long>(B) * T * H;
    auto lo = [](uint32_t w) { return __uint_as_float(w << 16); };
    auto hi = [](uint32_t w) { return __uint_as_float(w & 0xffff0000u); };
    float acc = 0.f;
    if (live) {
        const uint4 a = __ldg(reinterpret_cast<const uint4*>(O + row * HD) + sub);
        const uint4 c = __ldg(reinterpret_cast<const uint4*>(dO + row * HD) + sub);
        acc = lo(a.x) * lo(c.x) + hi(a.x) * hi(c.x) + lo(a.y) * lo(c.y) + hi(a.y) * hi(c.y) + lo(a.z) * lo(c.z) +
              hi(a.z) * hi(c.z) + lo(a.w) * lo(c.w) + hi(a.w) * hi(c.w);
    }
#pragma unroll
    for (int sft = 8; sft >= 1; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    if (live && sub == 0) {
        const int h = static_cast<int>(row % H);
        const long long bt = row / H;
        const int t = static_cast<int>(bt % T);
        const int b = static_cast<int>(bt / T);
        D[(static_cast<long long>(b) * H + h) * T + t] = acc;
    }
}

// ------------------------------------------------------------------------------------------------------
// dQ: a work item is (sequence, query head, tile of 128 query positions). Every element of its sweep - a key
// tile of 64 keys, or half h of draft pass i fetched i rows early (the substituted entries sit on its
// diagonal) - takes the same route: K and V stage by TMA; S = Q K^T and dP = dO V^T into TMEM; the row's
// thread forms dS (full row, or its diagonal element only) as bf16 pairs in tensor memory, over the scores it
// came from; dQ += dS K with dS read from tensor memory and the same K stage read MN-major. Q and dO are copied
// into tensor memory once per item, so the S / dP products read only their B operands from shared memory.
constexpr int DQ_SMEM_Q = 0;
constexpr int DQ_SMEM_DO = DQ_SMEM_Q + Q_BYTES;
constexpr int DQ_STAGES = 4;        // a K/V stage is held until its dQ product is done, long after the next S/dP products need theirs
constexpr int DQ_SMEM_K = DQ_SMEM_DO + Q_BYTES;
constexpr int DQ_SMEM_V = DQ_SMEM_K + DQ_STAGES * KV_BYTES;
constexpr int DQ_SMEM_BAR = DQ_SMEM_V + DQ_STAGES * KV_BYTES;
constexpr int DQ_NUM_BARS = 2 * DQ_STAGES + 14;
constexpr int DQ_SMEM_BYTES = DQ_SMEM_BAR + 256 + 1024 /*alignment slack*/;
constexpr int DQ_TMEM_COLS = 512;   // buffer sb: S at 128 sb (dS as bf16 pairs later overwrites its first 32 columns), dP at
                                    // 128 sb + 64; dQ at 256; Q at 384 and dO at 448 as bf16 pairs
constexpr int DQ_TMEM_Q = 384, DQ_TMEM_DO = 448;

struct DqParams {
    CUtensorMap tmQ, tmdO;         // [B, T, H * 128], box {64, 128, 1}
    CUtensorMap tmK, tmV;          // [B, T, Hkv * 128], box {64, 64, 1}
    CUtensorMap tmKd[MAX_DRAFTS];
    CUtensorMap tmVd[MAX_DRAFTS];
    __nv_bfloat16* dQ;             // [B, T, H, 128]
    const float* lse;              // [B, H, T] natural-log normaliser from the forward
    const float* D;                // [B, H, T]
    float* Pd;                     // [B, H, T, m] weight of the substituted entry (t, t - i)
    float* dSd;                    // [B, H, T, m] its dS
    int B, T, H, Hkv, m;
    int q_tiles, k_tiles, items;
    float c2;                      // scale * log2(e)
    float scale;
    unsigned int* status;
};

__global__ void __launch_bounds__(NUM_THREADS, 1) hca_dq_kernel(const __grid_constant__ DqParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + DQ_SMEM_BAR;
    const uint32_t qdo_full = bar0, qdo_empty = bar0 + 8;
    auto kv_full = [&](int s) { return bar0 + 8u * (2 + s); };
    auto kv_empty = [&](int s) { return bar0 + 8u * (2 + DQ_STAGES + s); };
    auto sdp_full = [&](int s) { return bar0 + 8u * (2 + 2 * DQ_STAGES + s); };
    auto sdp_empty = [&](int s) { return bar0 + 8u * (4 + 2 * DQ_STAGES + s); };
    auto ds_full = [&](int s) { return bar0 + 8u * (6 + 2 * DQ_STAGES + s); };
    auto ds_empty = [&](int s) { return bar0 + 8u * (8 + 2 * DQ_STAGES + s); };
    const uint32_t dq_done = bar0 + 8u * (10 + 2 * DQ_STAGES), dq_free = bar0 + 8u * (11 + 2 * DQ_STAGES);
    const uint32_t qt_ready = bar0 + 8u * (12 + 2 * DQ_STAGES);    // Q and dO of the item copied into tensor memory
    const uint32_t qt_free = bar0 + 8u * (13 + 2 * DQ_STAGES);     // ... and read by the item's last S / dP product
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + DQ_SMEM_BAR + 8 * DQ_NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(qdo_full, 1);
        mbar_init(qdo_empty, 8);
        mbar_init(qt_ready, 8);
        mbar_init(qt_free, 1);
        for (int s = 0; s < DQ_STAGES; ++s) {
            mbar_init(kv_full(s), 1);
            mbar_init(kv_empty(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(sdp_full(s), 1);
            mbar_init(sdp_empty(s), 4);
            mbar_init(ds_full(s), 4);
            mbar_init(ds_empty(s), 1);
        }
        mbar_init(dq_done, 1);
        mbar_init(dq_free, 8);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmQ);
        prefetch_tensormap(&p.tmdO);
        prefetch_tensormap(&p.tmK);
        prefetch_tensormap(&p.tmV);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_ptr_smem), DQ_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;
    // items are sorted longest first; round k deals items k*G .. k*G + G-1 to the G CTAs in alternating direction
    auto round_item = [&](uint32_t k) {
        const int G = gridDim.x, c = blockIdx.x;
        return static_cast<int>(k) * G + ((k & 1u) ? G - 1 - c : c);
    };

    const int BH = p.B * p.H;
    const int rep = p.H / p.Hkv;
    const int m = p.m;
    auto decode = [&](int item, int& qt, int& b, int& h) {
        qt = p.q_tiles - 1 - item / BH;
        const int bh = item - (item / BH) * BH;
        b = bh / p.H;
        h = bh - b * p.H;
    };
    auto key_tiles = [&](int qt) { return min(2 * qt + 2, p.k_tiles); };
    // elements of an item: key tiles 0 .. n-1, then draft pass i, half h (element n + 2i + h)

    if (warp == 0) {
        if (lane == 0) {
            uint32_t g = 0, it = 0;
            bool ok = true;
            for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int col = (h / rep) * HD;
                const int n = key_tiles(qt);
                if (!wait_barrier(qdo_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(qdo_full, 2 * Q_BYTES);
                tma_load_3d(base + DQ_SMEM_Q, &p.tmQ, qdo_full, h * HD, qt * QT, b);
                tma_load_3d(base + DQ_SMEM_Q + Q_HALF, &p.tmQ, qdo_full, h * HD + 64, qt * QT, b);
                tma_load_3d(base + DQ_SMEM_DO, &p.tmdO, qdo_full, h * HD, qt * QT, b);
                tma_load_3d(base + DQ_SMEM_DO + Q_HALF, &p.tmdO, qdo_full, h * HD + 64, qt * QT, b);
                for (int e = 0; e < n + 2 * m && ok; ++e, ++g) {
                    const int s = g % DQ_STAGES;
                    if (!wait_barrier(kv_empty(s), ((g / DQ_STAGES) & 1u) ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
                    const int d = e - n;
                    const CUtensorMap* tk = e < n ? &p.tmK : &p.tmKd[d >> 1];
                    const CUtensorMap* tv = e < n ? &p.tmV : &p.tmVd[d >> 1];
                    const int row = e < n ? e * KT : qt * QT + 64 * (d & 1) - (d >> 1);
                    mbar_arrive_expect_tx(kv_full(s), 2 * KV_BYTES);
                    tma_load_3d(base + DQ_SMEM_K + s * KV_BYTES, tk, kv_full(s), col, row, b);
                    tma_load_3d(base + DQ_SMEM_K + s * KV_BYTES + KV_HALF, tk, kv_full(s), col + 64, row, b);
                    tma_load_3d(base + DQ_SMEM_V + s * KV_BYTES, tv, kv_full(s), col, row, b);
                    tma_load_3d(base + DQ_SMEM_V + s * KV_BYTES + KV_HALF, tv, kv_full(s), col + 64, row, b);
                }
            }
        }
    } else if (warp == 1) {
        // The whole warp runs this loop so that addresses and descriptors stay warp-uniform; one elected lane
        // issues the tensor-core instructions.
        {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_q = make_idesc_bf16(QT, HD, 0, 1);
            uint32_t gs = 0, gq = 0, it = 0;      // elements whose S/dP, resp. dQ product has been issued
            bool ok = true;
            auto wait_all = [&](uint32_t bar, uint32_t parity, unsigned code) {
                return __all_sync(0xffffffffu, wait_barrier(bar, parity, abort_flag, p.status, code)) != 0;
            };
            auto issue_sdp = [&]() -> bool {
                const int s = gs & 1u;                  // S / dP buffer
                const int ks = gs % DQ_STAGES;          // K / V stage
                const uint32_t ph = (gs >> 1) & 1u;
                if (!wait_all(kv_full(ks), (gs / DQ_STAGES) & 1u, 4)) return false;
                if (!wait_all(sdp_empty(s), ph ^ 1u, 5)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t ko = (k >> 2) * KV_HALF + (k & 3) * 32;
                    // A (Q, dO) comes from tensor memory, 8 columns per K step: only B is read from shared memory
                    const uint64_t dk_ = make_smem_desc_sw128(base + DQ_SMEM_K + ks * KV_BYTES + ko, 0, 1024);
                    const uint64_t dv_ = make_smem_desc_sw128(base + DQ_SMEM_V + ks * KV_BYTES + ko, 0, 1024);
                    if (leader) {
                        umma_bf16_ta(tmem_base + s * 128, tmem_base + DQ_TMEM_Q + 8 * k, dk_, idesc_s, k != 0 ? 1u : 0u);
                        umma_bf16_ta(tmem_base + s * 128 + 64, tmem_base + DQ_TMEM_DO + 8 * k, dv_, idesc_s, k != 0 ? 1u : 0u);
                    }
                }
                if (leader) umma_commit(sdp_full(s));
                __syncwarp();
                ++gs;
                return true;
            };
            auto issue_dq = [&](bool first, bool last) -> bool {
                const int s = gq & 1u;                  // dS buffer
                const int ks = gq % DQ_STAGES;          // K stage
                if (!wait_all(ds_full(s), (gq >> 1) & 1u, 7)) return false;
                if (first && !wait_all(dq_free, (it & 1u) ^ 1u, 9)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < KT / 16; ++k) {
                    // A = dS from tensor memory, in the buffer its S came from (the next S / dP product into that
                    // buffer is issued after this one and the tensor core keeps issue order)
                    const uint64_t db_ = make_smem_desc_sw128(base + DQ_SMEM_K + ks * KV_BYTES + k * 16 * 128, KV_HALF, 1024);
                    if (leader) umma_bf16_ta(tmem_base + 256, tmem_base + s * 128 + 8 * k, db_, idesc_q, (!first || k != 0) ? 1u : 0u);
                }
                if (leader) {
                    umma_commit(kv_empty(ks));
                    umma_commit(ds_empty(s));
                    if (last) umma_commit(dq_done);
                }
                __syncwarp();
                ++gq;
                return true;
            };
            for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
                int qt, b, h;
                decode(item, qt, b, h);
                const int n_e = key_tiles(qt) + 2 * m;
                if (!wait_all(qt_ready, it & 1u, 6)) break;
                if (!issue_sdp()) break;
                if (n_e == 1 && elect_one()) umma_commit(qt_free);
                for (int a = 0; a < n_e && ok; ++a) {
                    if (a + 1 < n_e) {
                        ok = issue_sdp();
                        if (ok && a + 2 == n_e && elect_one()) umma_commit(qt_free);
                    }
                    if (ok) ok = issue_dq(a == 0, a + 1 == n_e);
                }
            }
        }
    } else {
        // two groups of four warps: group grp takes the elements with (running index & 1) == grp, i.e. always the
        // S / dP buffer and the dS buffer of its own index, so each group has two element slots of time for its
        // chain TMEM load -> row math -> dS store (nothing is carried from one element to the next); in the
        // epilogue each group stores half of the dQ row
        const int grp = (warp - 2) >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        uint32_t g = 0, it = 0;
        bool ok = true;
        // This row of Q (group 0) or dO (group 1) of this CTA's item number `n_it`, from shared memory into tensor
        // memory, where the S and dP products read it as their A operand. Done for the first item up front and
        // for every later item as soon as the group has finished the previous item's elements, before its
        // epilogue, so that the tensor core can start on the next item meanwhile.
        auto copy_item = [&](uint32_t n_it) -> bool {
            if (!wait_barrier(qdo_full, n_it & 1u, abort_flag, p.status, 16)) return false;
            if (!wait_barrier(qt_free, (n_it & 1u) ^ 1u, abort_flag, p.status, 17)) return false;
            tc_fence_after_sync();
            const uint32_t src = base + (grp == 0 ? DQ_SMEM_Q : DQ_SMEM_DO) + r * 128;
            const uint32_t dst = tmem_base + lane_addr + (grp == 0 ? DQ_TMEM_Q : DQ_TMEM_DO);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t w[32];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(w[4 * j]), "=r"(w[4 * j + 1]), "=r"(w[4 * j + 2]), "=r"(w[4 * j + 3])
                                 : "r"(src + hf * Q_HALF + (((j ^ (r & 7)) & 7) << 4)));
                hca::tmem_st32(dst + 32 * hf, w);
            }
            hca::tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(qt_ready);
                mbar_arrive(qdo_empty);     // the shared-memory copies may be refilled for the item after
            }
            return true;
        };
        if (round_item(0) < p.items) ok = copy_item(0);
        for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
            int qt, b, h;
            decode(item, qt, b, h);
            const int n = key_tiles(qt);
            const int t = qt * QT + r;
            const bool valid = t < p.T;
            const size_t row_idx = (static_cast<size_t>(b) * p.H + h) * p.T + (valid ? t : 0);
            // P = 2^(S c2 - lse2); a row outside the sequence gets P = 0 through lse2 = +inf
            const float nlse2 = valid ? -p.lse[row_idx] * 1.4426950408889634f : -INFINITY;
            const float Dt = valid ? p.D[row_idx] : 0.f;
            const float nDs = -Dt * p.scale;
            for (int e = 0; e < n + 2 * m; ++e, ++g) {
                if ((g & 1u) != static_cast<uint32_t>(grp)) continue;
                const int s = grp;
                const uint32_t ph = (g >> 1) & 1u;
                if (!wait_barrier(sdp_full(s), ph, abort_flag, p.status, 10)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * 128 + lane_addr;
                if (e < n) {
                    // ---- key tile: dS for the row, 32 columns at a time ----
                    const bool band = e * KT + KT - 1 > qt * QT - m;
                    bool stop = false;
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        const int lim = t - m - e * KT - 32 * hc;
                        uint32_t sr[32], dr[32];
                        tmem_ld32(tmem_s + 32 * hc, sr);
                        tmem_ld32(tmem_s + 64 + 32 * hc, dr);
                        tmem_ld_wait(sr);
                        tmem_ld_wait(dr);
                        if (hc == 1) {
                            tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(sdp_empty(s));
                        }
                        if (band) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c > lim) sr[c] = 0xff800000u;       // -inf: weight 0
                        }
                        // dS = P (dP - D) scale = 2^(S c2 - lse2) (dP scale - D scale), two columns per instruction
                        float ds[32];
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            float x0, x1, y0, y1;
                            ffma2(x0, x1, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]), p.c2, p.c2, nlse2, nlse2);
                            ffma2(y0, y1, __uint_as_float(dr[c]), __uint_as_float(dr[c + 1]), p.scale, p.scale, nDs, nDs);
                            fmul2(ds[c], ds[c + 1], ex2(x0), ex2(x1), y0, y1);
                        }
                        if (hc == 0 && !wait_barrier(ds_empty(s), ph ^ 1u, abort_flag, p.status, 12)) { stop = true; break; }
                        // as bf16 pairs over the S columns already in registers (columns 16 hc .. 16 hc + 15)
                        uint32_t pk[16];
#pragma unroll
                        for (int c = 0; c < 32; c += 2) pk[c >> 1] = pack_bf16(ds[c], ds[c + 1]);
                        hca::tmem_st16(tmem_s + 16 * hc, pk);
                    }
                    if (stop) { ok = false; break; }
                } else {
                    // ---- draft pass i, half hf: only the diagonal element of the rows of that half ----
                    const int i = (e - n) >> 1, hf = (e - n) & 1;
                    const bool holder = (r >> 6) == hf;        // warp-uniform
                    float sv = 0.f, dv = 0.f;
                    if (holder) {
                        uint32_t sr[32], dr[32];
                        tmem_ld32(tmem_s + 32 * (quad & 1), sr);
                        tmem_ld32(tmem_s + 64 + 32 * (quad & 1), dr);
                        tmem_ld_wait(sr);
                        tmem_ld_wait(dr);
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            if (c == lane) {
                                sv = __uint_as_float(sr[c]);
                                dv = __uint_as_float(dr[c]);
                            }
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(sdp_empty(s));
                    const bool mine = holder && t - i >= 0 && valid;
                    const float pw = mine ? ex2(fmaf(sv, p.c2, nlse2)) : 0.f;
                    const float dsv = mine ? pw * fmaf(dv, p.scale, nDs) : 0.f;
                    if (holder && valid) {
                        p.Pd[row_idx * m + i] = pw;
                        p.dSd[row_idx * m + i] = dsv;
                    }
                    const uint32_t bits = pack_bf16(dsv, 0.f) << ((r & 1) * 16);
                    if (!wait_barrier(ds_empty(s), ph ^ 1u, abort_flag, p.status, 14)) { ok = false; break; }
                    uint32_t pk[32];
#pragma unroll
                    for (int w = 0; w < 32; ++w) pk[w] = (holder && w == ((r & 63) >> 1)) ? bits : 0u;
                    hca::tmem_st32(tmem_s, pk);
                }
                hca::tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(ds_full(s));
            }
            if (!ok) break;
            if (round_item(it + 1) < p.items && !copy_item(it + 1)) { ok = false; break; }
            // ---- epilogue: this group's half of the dQ row as bf16 ----
            if (!wait_barrier(dq_done, it & 1u, abort_flag, p.status, 13)) break;
            tc_fence_after_sync();
            __nv_bfloat16* orow = p.dQ + ((static_cast<size_t>(b) * p.T + (valid ? t : 0)) * p.H + h) * HD + 64 * grp;
            {
                uint32_t raw[2][32];
                tmem_ld32(tmem_base + 256 + lane_addr + 64 * grp, raw[0]);
                tmem_ld32(tmem_base + 256 + lane_addr + 64 * grp + 32, raw[1]);
                tmem_ld_wait(raw[0]);
                tmem_ld_wait(raw[1]);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(dq_free);
                if (valid) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
#pragma unroll
                        for (int q8 = 0; q8 < 2; ++q8) {
                            const uint32_t* x = &raw[k][16 * q8];
                            st_global_v8(orow + 32 * k + 16 * q8,
                                         pack_bf16(__uint_as_float(x[0]), __uint_as_float(x[1])),
                                         pack_bf16(__uint_as_float(x[2]), __uint_as_float(x[3])),
                                         pack_bf16(__uint_as_float(x[4]), __uint_as_float(x[5])),
                                         pack_bf16(__uint_as_float(x[6]), __uint_as_float(x[7])),
                                         pack_bf16(__uint_as_float(x[8]), __uint_as_float(x[9])),
                                         pack_bf16(__uint_as_float(x[10]), __uint_as_float(x[11])),
                                         pack_bf16(__uint_as_float(x[12]), __uint_as_float(x[13])),
                                         pack_bf16(__uint_as_float(x[14]), __uint_as_float(x[15])));
                        }
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, DQ_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------------
// dK_t, dV_t: a work item is (sequence, key/value head, tile of 128 key positions), kept in shared memory; it
// sweeps the query heads of its group and, per head, the tiles of 64 queries at or after it. Per element:
//   S^T = K Q^T and dP^T = V dO^T      tcgen05.mma, 128 x 64 x 128, into TMEM (rows = keys, one per thread)
//   threads                             P^T = 2^(S^T c2 - lse2[t]) on the entries the target's keys really met
//                                       (t - s >= m), dS^T = P^T (dP^T - D[t]) scale; both as bf16 pairs back into
//                                       tensor memory, over the columns they were made from
//   dV += P^T dO, dK += dS^T Q          A from tensor memory, the Q / dO stage read MN-major from shared memory
// The per-query vectors -lse2[t] and -D[t] scale of an element travel with its Q / dO stage: the producer warp's
// lanes copy them into shared memory next to the TMA loads.
constexpr int KV_SMEM_K = 0;                               // 128 keys x 128: two halves of 16 KB
constexpr int KV_SMEM_V = KV_SMEM_K + Q_BYTES;
constexpr int KV_STAGES = 4;        // a Q/dO stage is held until its dV/dK products are done
constexpr int KV_SMEM_Q = KV_SMEM_V + Q_BYTES;             // stages of 64 queries
constexpr int KV_SMEM_DO = KV_SMEM_Q + KV_STAGES * KV_BYTES;
constexpr int KV_SMEM_VEC = KV_SMEM_DO + KV_STAGES * KV_BYTES;     // per stage: 64 x -lse2, 64 x -D scale (floats)
constexpr int KV_SMEM_BAR = KV_SMEM_VEC + KV_STAGES * 512;
constexpr int KV_NUM_BARS = 2 * KV_STAGES + 10;
constexpr int KV_SMEM_BYTES = KV_SMEM_BAR + 256 + 1024 /*alignment slack*/;
constexpr int KV_TMEM_COLS = 512;   // buffer sb: S^T at 128 sb, dP^T at 128 sb + 64 (P^T and dS^T as bf16 pairs later overwrite
                                    // columns 0..15 and 32..47 of each); dV at 256, dK at 384

struct DkvParams {
    CUtensorMap tmK, tmV;          // [B, T, Hkv * 128], box {64, 128, 1}
    CUtensorMap tmQ, tmdO;         // [B, T, H * 128], box {64, 64, 1}
    __nv_bfloat16* dK;             // [B, T, Hkv, 128]
    __nv_bfloat16* dV;
    const float* lse;              // [B, H, T]
    const float* D;                // [B, H, T]
    int B, T, H, Hkv, m;
    int kt_tiles;                  // ceil(T / 128) key tiles
    int q_tiles64;                 // ceil(T / 64) query tiles
    int items;                     // B * Hkv * kt_tiles
    float c2, scale;
    unsigned int* status;
};

__global__ void __launch_bounds__(NUM_THREADS, 1) hca_dkv_kernel(const __grid_constant__ DkvParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + KV_SMEM_BAR;
    const uint32_t kv_full = bar0, kv_empty = bar0 + 8;
    auto qd_full = [&](int s) { return bar0 + 8u * (2 + s); };
    auto qd_empty = [&](int s) { return bar0 + 8u * (2 + KV_STAGES + s); };
    auto st_full = [&](int s) { return bar0 + 8u * (2 + 2 * KV_STAGES + s); };
    auto st_empty = [&](int s) { return bar0 + 8u * (4 + 2 * KV_STAGES + s); };
    const uint32_t pds_full = bar0 + 8u * (6 + 2 * KV_STAGES), pds_empty = bar0 + 8u * (7 + 2 * KV_STAGES);
    const uint32_t acc_done = bar0 + 8u * (8 + 2 * KV_STAGES), acc_free = bar0 + 8u * (9 + 2 * KV_STAGES);
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_gen + KV_SMEM_BAR + 8 * KV_NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);
    float* vec = reinterpret_cast<float*>(smem_gen + KV_SMEM_VEC);     // [stage][0..63 -lse2 | 64..127 D]

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        mbar_init(kv_empty, 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(qd_full(s), 2);      // the TMA transaction's arrival and the producer warp's vectors
            mbar_init(qd_empty(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(st_full(s), 1);
            mbar_init(st_empty(s), 8);
        }
        mbar_init(pds_full, 8);
        mbar_init(pds_empty, 1);
        mbar_init(acc_done, 1);
        mbar_init(acc_free, 8);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmK);
        prefetch_tensormap(&p.tmV);
        prefetch_tensormap(&p.tmQ);
        prefetch_tensormap(&p.tmdO);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_ptr_smem), KV_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;
    // items are sorted longest first; round k deals items k*G .. k*G + G-1 to the G CTAs in alternating direction
    auto round_item = [&](uint32_t k) {
        const int G = gridDim.x, c = blockIdx.x;
        return static_cast<int>(k) * G + ((k & 1u) ? G - 1 - c : c);
    };

    const int BG = p.B * p.Hkv;
    const int rep = p.H / p.Hkv;
    const int m = p.m;
    // item -> (key tile, sequence, key/value head): the first key tiles meet the most queries and come first
    auto decode = [&](int item, int& kt, int& b, int& g) {
        kt = item / BG;
        const int bg = item - kt * BG;
        b = bg / p.Hkv;
        g = bg - b * p.Hkv;
    };
    // elements of an item: for each head of the group, the 64-query tiles 2 kt .. q_tiles64 - 1
    auto q_count = [&](int kt) { return p.q_tiles64 - 2 * kt; };

    if (warp == 0) {
        // ===================== producer: TMA by lane 0, the per-query vectors by all lanes =====================
        uint32_t gq = 0, it = 0;
        bool ok = true;
        for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
            int kt, b, g;
            decode(item, kt, b, g);
            const int nq = q_count(kt);
            if (lane == 0) {
                ok = wait_barrier(kv_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1);
                if (ok) {
                    mbar_arrive_expect_tx(kv_full, 2 * Q_BYTES);
                    tma_load_3d(base + KV_SMEM_K, &p.tmK, kv_full, g * HD, kt * QT, b);
                    tma_load_3d(base + KV_SMEM_K + Q_HALF, &p.tmK, kv_full, g * HD + 64, kt * QT, b);
                    tma_load_3d(base + KV_SMEM_V, &p.tmV, kv_full, g * HD, kt * QT, b);
                    tma_load_3d(base + KV_SMEM_V + Q_HALF, &p.tmV, kv_full, g * HD + 64, kt * QT, b);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            for (int e = 0; e < rep * nq && ok; ++e, ++gq) {
                const int h = g * rep + e / nq;
                const int jq = 2 * kt + e % nq;
                const int s = gq % KV_STAGES;
                if (lane == 0) ok = wait_barrier(qd_empty(s), ((gq / KV_STAGES) & 1u) ^ 1u, abort_flag, p.status, 2);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(qd_full(s), 2 * KV_BYTES);
                    tma_load_3d(base + KV_SMEM_Q + s * KV_BYTES, &p.tmQ, qd_full(s), h * HD, jq * KT, b);
                    tma_load_3d(base + KV_SMEM_Q + s * KV_BYTES + KV_HALF, &p.tmQ, qd_full(s), h * HD + 64, jq * KT, b);
                    tma_load_3d(base + KV_SMEM_DO + s * KV_BYTES, &p.tmdO, qd_full(s), h * HD, jq * KT, b);
                    tma_load_3d(base + KV_SMEM_DO + s * KV_BYTES + KV_HALF, &p.tmdO, qd_full(s), h * HD + 64, jq * KT, b);
                }
                // -lse2[t] (or -inf past the sequence, which zeroes the weight) and -D[t] scale for the 64 queries
                const size_t rowbase = (static_cast<size_t>(b) * p.H + h) * p.T;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int c = lane + 32 * u;
                    const int t = jq * KT + c;
                    vec[s * 128 + c] = t < p.T ? -p.lse[rowbase + t] * 1.4426950408889634f : -INFINITY;
                    vec[s * 128 + 64 + c] = t < p.T ? -p.D[rowbase + t] * p.scale : 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(qd_full(s));
            }
        }
    } else if (warp == 1) {
        // whole warp in the loop, one elected lane issues (see hca_dq_kernel)
        {
            constexpr uint32_t idesc_s = make_idesc_bf16(QT, KT, 0, 0);
            constexpr uint32_t idesc_a = make_idesc_bf16(QT, HD, 0, 1);
            uint32_t gs = 0, ga = 0, it = 0;
            bool ok = true;
            auto wait_all = [&](uint32_t bar, uint32_t parity, unsigned code) {
                return __all_sync(0xffffffffu, wait_barrier(bar, parity, abort_flag, p.status, code)) != 0;
            };
            auto issue_st = [&]() -> bool {
                const int s = gs & 1u;                  // S^T / dP^T buffer
                const int qs = gs % KV_STAGES;          // Q / dO stage
                const uint32_t ph = (gs >> 1) & 1u;
                if (!wait_all(qd_full(qs), (gs / KV_STAGES) & 1u, 4)) return false;
                if (!wait_all(st_empty(s), ph ^ 1u, 5)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t ao = (k >> 2) * Q_HALF + (k & 3) * 32, bo = (k >> 2) * KV_HALF + (k & 3) * 32;
                    const uint64_t ak_ = make_smem_desc_sw128(base + KV_SMEM_K + ao, 0, 1024);
                    const uint64_t bq_ = make_smem_desc_sw128(base + KV_SMEM_Q + qs * KV_BYTES + bo, 0, 1024);
                    const uint64_t av_ = make_smem_desc_sw128(base + KV_SMEM_V + ao, 0, 1024);
                    const uint64_t bd_ = make_smem_desc_sw128(base + KV_SMEM_DO + qs * KV_BYTES + bo, 0, 1024);
                    if (leader) {
                        umma_bf16(tmem_base + s * 128, ak_, bq_, idesc_s, k != 0 ? 1u : 0u);
                        umma_bf16(tmem_base + s * 128 + 64, av_, bd_, idesc_s, k != 0 ? 1u : 0u);
                    }
                }
                if (leader) umma_commit(st_full(s));
                __syncwarp();
                ++gs;
                return true;
            };
            auto issue_acc = [&](bool first, bool last) -> bool {
                const int s = ga % KV_STAGES;           // Q / dO stage
                if (!wait_all(pds_full, ga & 1u, 7)) return false;
                if (first && !wait_all(acc_free, (it & 1u) ^ 1u, 9)) return false;
                tc_fence_after_sync();
                const bool leader = elect_one();
#pragma unroll
                for (int k = 0; k < KT / 16; ++k) {
                    // A from tensor memory: queries 16 k .. 16 k + 15 of P^T (dS^T) sit as 8 columns of bf16 pairs in
                    // the part of the S^T (dP^T) buffer their own column group read: 0..15 for k < 2, 32..47 for k >= 2
                    const uint32_t a_col = (ga & 1u) * 128 + (k < 2 ? 8 * k : 32 + 8 * (k - 2));
                    const uint64_t bd_ = make_smem_desc_sw128(base + KV_SMEM_DO + s * KV_BYTES + k * 16 * 128, KV_HALF, 1024);
                    const uint64_t bq_ = make_smem_desc_sw128(base + KV_SMEM_Q + s * KV_BYTES + k * 16 * 128, KV_HALF, 1024);
                    if (leader) {
                        umma_bf16_ta(tmem_base + 256, tmem_base + a_col, bd_, idesc_a, (!first || k != 0) ? 1u : 0u);
                        umma_bf16_ta(tmem_base + 384, tmem_base + a_col + 64, bq_, idesc_a, (!first || k != 0) ? 1u : 0u);
                    }
                }
                if (leader) {
                    umma_commit(qd_empty(s));
                    umma_commit(pds_empty);
                    if (last) umma_commit(acc_done);
                }
                __syncwarp();
                ++ga;
                return true;
            };
            for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
                int kt, b, g;
                decode(item, kt, b, g);
                const int n_e = rep * q_count(kt);
                if (!wait_all(kv_full, it & 1u, 6)) break;
                if (!issue_st()) break;
                if (n_e == 1 && elect_one()) umma_commit(kv_empty);
                for (int a = 0; a < n_e && ok; ++a) {
                    if (a + 1 < n_e) {
                        ok = issue_st();
                        if (ok && a + 2 == n_e && elect_one()) umma_commit(kv_empty);     // K and V are free once the last S^T / dP^T has read them
                    }
                    if (ok) ok = issue_acc(a == 0, a + 1 == n_e);
                }
            }
        }
    } else {
        // two groups of four warps share every key row: group grp takes the query columns 32 grp .. 32 grp + 31
        // of each element, and in the epilogue dV (group 0) or dK (group 1)
        const int grp = (warp - 2) >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                 // key row of the tile
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        uint32_t gq = 0, it = 0;
        bool ok = true;
        for (int item = round_item(0); item < p.items && ok; item = round_item(++it)) {
            int kt, b, g;
            decode(item, kt, b, g);
            const int nq = q_count(kt);
            const int spos = kt * QT + r;               // key position
            for (int e = 0; e < rep * nq; ++e, ++gq) {
                const int jq = 2 * kt + e % nq;
                const int s = gq & 1u;                  // S^T / dP^T buffer
                const int qs = gq % KV_STAGES;          // the element's Q / dO stage, for its vectors
                const uint32_t ph = (gq >> 1) & 1u;
                if (!wait_barrier(st_full(s), ph, abort_flag, p.status, 10)) { ok = false; break; }
                if (!wait_barrier(qd_full(qs), (gq / KV_STAGES) & 1u, abort_flag, p.status, 15)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * 128 + lane_addr + 32 * grp;
                // the target's key at spos met query t only if t - spos >= m: columns below lo are empty
                const int lo = spos + m - jq * KT - 32 * grp;
                const bool band = spos + m - jq * KT > 0;
                uint32_t sr[32], dr[32];
                tmem_ld32(tmem_s, sr);
                tmem_ld32(tmem_s + 64, dr);
                tmem_ld_wait(sr);
                tmem_ld_wait(dr);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(st_empty(s));
                if (band) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c < lo) sr[c] = 0xff800000u;       // -inf: weight 0
                }
                // P^T = 2^(S^T c2 - lse2[t]), dS^T = P^T (dP^T scale - D[t] scale), two columns per instruction
                const float4* nl = reinterpret_cast<const float4*>(vec + qs * 128 + 32 * grp);
                const float4* dd = reinterpret_cast<const float4*>(vec + qs * 128 + 64 + 32 * grp);
                float pw[32], ds[32];
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4) {
                    const float4 a = nl[c4], d = dd[c4];
                    const int c = 4 * c4;
                    float x0, x1, y0, y1;
                    ffma2(x0, x1, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]), p.c2, p.c2, a.x, a.y);
                    ffma2(y0, y1, __uint_as_float(dr[c]), __uint_as_float(dr[c + 1]), p.scale, p.scale, d.x, d.y);
                    pw[c] = ex2(x0);
                    pw[c + 1] = ex2(x1);
                    fmul2(ds[c], ds[c + 1], pw[c], pw[c + 1], y0, y1);
                    ffma2(x0, x1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]), p.c2, p.c2, a.z, a.w);
                    ffma2(y0, y1, __uint_as_float(dr[c + 2]), __uint_as_float(dr[c + 3]), p.scale, p.scale, d.z, d.w);
                    pw[c + 2] = ex2(x0);
                    pw[c + 3] = ex2(x1);
                    fmul2(ds[c + 2], ds[c + 3], pw[c + 2], pw[c + 3], y0, y1);
                }
                if (!wait_barrier(pds_empty, (gq & 1u) ^ 1u, abort_flag, p.status, 12)) { ok = false; break; }
                {
                    // bf16 pairs over the first 16 of the 32 columns this group read (S^T, resp. dP^T)
                    uint32_t pk[16], dk[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        pk[c >> 1] = pack_bf16(pw[c], pw[c + 1]);
                        dk[c >> 1] = pack_bf16(ds[c], ds[c + 1]);
                    }
                    hca::tmem_st16(tmem_s, pk);
                    hca::tmem_st16(tmem_s + 64, dk);
                    hca::tmem_st_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(pds_full);
            }
            if (!ok) break;
            // ---- epilogue: this key row of dV (group 0) or dK (group 1) as bf16 ----
            if (!wait_barrier(acc_done, it & 1u, abort_flag, p.status, 13)) break;
            tc_fence_after_sync();
            const bool valid = spos < p.T;
            const size_t orow = ((static_cast<size_t>(b) * p.T + (valid ? spos : 0)) * p.Hkv + g) * HD;
#pragma unroll
            for (int part = 0; part < 2; ++part) {      // columns 0..63, 64..127
                __nv_bfloat16* dst = (grp == 0 ? p.dV : p.dK) + orow + 64 * part;
                uint32_t raw[2][32];
                tmem_ld32(tmem_base + 256 + 128 * grp + lane_addr + 64 * part, raw[0]);
                tmem_ld32(tmem_base + 256 + 128 * grp + lane_addr + 64 * part + 32, raw[1]);
                tmem_ld_wait(raw[0]);
                tmem_ld_wait(raw[1]);
                if (part == 1) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_free);
                }
                if (valid) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
#pragma unroll
                        for (int q8 = 0; q8 < 2; ++q8) {
                            const uint32_t* x = &raw[k][16 * q8];
                            st_global_v8(dst + 32 * k + 16 * q8, pack_bf16(__uint_as_float(x[0]), __uint_as_float(x[1])),
                                         pack_bf16(__uint_as_float(x[2]), __uint_as_float(x[3])),
                                         pack_bf16(__uint_as_float(x[4]), __uint_as_float(x[5])),
                                         pack_bf16(__uint_as_float(x[6]), __uint_as_float(x[7])),
                                         pack_bf16(__uint_as_float(x[8]), __uint_as_float(x[9])),
                                         pack_bf16(__uint_as_float(x[10]), __uint_as_float(x[11])),
                                         pack_bf16(__uint_as_float(x[12]), __uint_as_float(x[13])),
                                         pack_bf16(__uint_as_float(x[14]), __uint_as_float(x[15])));
                        }
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, KV_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------------
// Gradients of the draft passes' keys and values: position s of pass i meets exactly one query per head,
// t = s + i, so dK_d[i][s] = sum over the group's query heads of dS[t, s] Q[t] and likewise for the values.
// Half a warp per (sequence, query position t, key/value head): it reads the group's Q[t] and dO[t] rows once
// and writes row t - i of every pass i; the last i rows of pass i have no query and are zeroed by the half-warp
// of the same index. A thread covers 8 of the 128 columns (16-byte accesses).
struct DraftGradParams {
    __nv_bfloat16* dKd[MAX_DRAFTS];
    __nv_bfloat16* dVd[MAX_DRAFTS];
};

__global__ void hca_draft_grad_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ dO,
                                      const float* __restrict__ Pd, const float* __restrict__ dSd,
                                      const __grid_constant__ DraftGradParams out, int m, int B, int T, int H, int Hkv) {
    const long long w = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 4;   // (b, t, g)
    const int sub = threadIdx.x & 15;       // 8 of the 128 columns (16 bytes) per thread
    if (w >= static_cast<long long>(B) * T * Hkv) return;
    const int g = static_cast<int>(w % Hkv);
    const long long bt = w / Hkv;
    const int t = static_cast<int>(bt % T);
    const int b = static_cast<int>(bt / T);
    const int rep = H / Hkv;
    auto lo = [](uint32_t x) { return __uint_as_float(x << 16); };
    auto hi = [](uint32_t x) { return __uint_as_float(x & 0xffff0000u); };
    auto widen = [&](const uint4& v, float (&f)[8]) {
        f[0] = lo(v.x); f[1] = hi(v.x); f[2] = lo(v.y); f[3] = hi(v.y);
        f[4] = lo(v.z); f[5] = hi(v.z); f[6] = lo(v.w); f[7] = hi(v.w);
    };
    auto narrow = [&](const float (&f)[8]) {
        return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
    };
    // two passes at a time (the group's rows are re-read from cache for further pairs): few registers, many rows in flight
    for (int i0 = 0; i0 < m; i0 += 2) {
        float kacc[2][8], vacc[2][8];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int c = 0; c < 8; ++c) kacc[j][c] = vacc[j][c] = 0.f;
        // two heads of the group at a time, all their loads issued before any is used
        for (int h0 = 0; h0 < rep; h0 += 2) {
            uint4 q[2], d[2];
            float pw[2][2], ds[2][2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const bool on = h0 + u < rep;
                const int h = g * rep + (on ? h0 + u : 0);
                const size_t row = ((static_cast<size_t>(b) * T + t) * H + h) * HD;
                q[u] = __ldg(reinterpret_cast<const uint4*>(Q + row) + sub);
                d[u] = __ldg(reinterpret_cast<const uint4*>(dO + row) + sub);
                const size_t ri = ((static_cast<size_t>(b) * H + h) * T + t) * m;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const bool use = on && i0 + j < m;
                    pw[u][j] = use ? __ldg(Pd + ri + i0 + j) : 0.f;      // zero where t - i < 0
                    ds[u][j] = use ? __ldg(dSd + ri + i0 + j) : 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                float qf[8], df[8];
                widen(q[u], qf);
                widen(d[u], df);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        kacc[j][c] = fmaf(ds[u][j], qf[c], kacc[j][c]);
                        vacc[j][c] = fmaf(pw[u][j], df[c], vacc[j][c]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = i0 + j;
            if (i < m) {
                if (t - i >= 0) {
                    const size_t orow = ((static_cast<size_t>(b) * T + (t - i)) * Hkv + g) * HD;
                    *(reinterpret_cast<uint4*>(out.dKd[i] + orow) + sub) = narrow(kacc[j]);
                    *(reinterpret_cast<uint4*>(out.dVd[i] + orow) + sub) = narrow(vacc[j]);
                }
                if (t + i >= T) {       // position t of pass i would meet query t + i, past the sequence
                    const size_t orow = ((static_cast<size_t>(b) * T + t) * Hkv + g) * HD;
                    *(reinterpret_cast<uint4*>(out.dKd[i] + orow) + sub) = make_uint4(0u, 0u, 0u, 0u);
                    *(reinterpret_cast<uint4*>(out.dVd[i] + orow) + sub) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
    }
}

}  // namespace hca_bwd
}  // namespace hass
