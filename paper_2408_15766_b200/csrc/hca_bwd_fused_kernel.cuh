// Backward of the HCA attention (Section 3.2) for sm_100a, one tensor-core kernel for all three target-side
// gradients. With P = softmax weights (recomputed from the forward's row normaliser), D[t] = <dO[t], O[t]>,
// dP[t,s] = <dO[t], v(t,s)> and dS = P * (dP - D) * scale:
//   dQ[t]    = sum_s dS[t,s] k(t,s)
//   dK_t[s]  = sum_{t: t-s >= m} dS[t,s] Q[t],   dV_t[s] = sum_{t: t-s >= m} P[t,s] dO[t]
//   dK_d[i][s] = dS[s+i,s] Q[s+i],               dV_d[i][s] = P[s+i,s] dO[s+i]
// Three launches:
//   hca_bwd_rows_kernel    everything that is one row of 128 per (query, head): D, the m substituted entries
//                          (t, t-i) - their scores, weights and dS as plain dot products -, the gradients of the
//                          draft passes' keys and values, and the substituted entries' share of dQ, which
//                          initialises the fp32 dQ accumulator
//   hca_bwd_fused_kernel   key tiles stationary: S^T and dP^T are formed once per (key tile, query tile, head)
//                          and feed dV += P^T dO, dK += dS^T Q and dQ^T = K^T dS^T; the last one is a
//                          per-element partial result that goes through shared memory into the fp32 accumulator
//                          in global memory by TMA reduction (cp.reduce.async.bulk.tensor, add.f32)
//   hca_dq_convert_kernel  the accumulator as bf16
// Five tensor products per (key tile, query tile) pair, the number the chain rule needs.
#pragma once
#include "hca_kernels.cuh"

namespace hass {
namespace hca_bwd {

using hca::ex2;
using hca::pack_bf16;
using hca::tma_load_3d;

constexpr int KEYS = 128;               // keys per item (stationary tile)
constexpr int QE = 64;                  // queries per element of an item's sweep
constexpr int HD = 128;
constexpr int MAX_DRAFTS = hca::MAX_DRAFTS;
constexpr int NUM_THREADS = 352;        // producer, MMA issuer, two groups of four row-owning warps, the vector warp
constexpr int VEC_WARP = 10;
constexpr int K_BYTES = KEYS * HD * 2;  // two halves (64 columns of the head dimension) of 128 rows x 128 B
constexpr int K_HALF = K_BYTES / 2;
constexpr int QE_BYTES = QE * HD * 2;
constexpr int QE_HALF = QE_BYTES / 2;
constexpr int DS_BYTES = KEYS * QE * 2; // dS^T of an element: 128 key rows x 64 queries, 128-byte rows

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void widen8(const uint4& v, float (&f)[8]) {
    f[0] = bf_lo(v.x); f[1] = bf_hi(v.x); f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
    f[4] = bf_lo(v.z); f[5] = bf_hi(v.z); f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}
__device__ __forceinline__ uint4 narrow8(const float (&f)[8]) {
    return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}
__device__ __forceinline__ float dot8(const float (&a)[8], const float (&b)[8]) {
    float s = a[0] * b[0];
#pragma unroll
    for (int c = 1; c < 8; ++c) s = fmaf(a[c], b[c], s);
    return s;
}
// Adds a [1, rows, cols] fp32 box from shared memory into global memory through the tensor map (element type and
// box come from the map; parts outside the tensor are dropped). Completion is tracked by the thread's bulk groups.
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* tm, uint32_t smem_src, int x, int y, int z) {
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(tm)),
                 "r"(smem_src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
// sum over the 16 lanes of a half-warp
__device__ __forceinline__ float sum16(float v) {
#pragma unroll
    for (int sft = 8; sft >= 1; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
    return v;
}

// ------------------------------------------------------------------------------------------------------
// Row work. Half a warp per (sequence, query position t, key/value head g); a lane covers 8 of the 128
// columns (16-byte accesses). For every query head h of the group Q[t], dO[t], O[t] are read once and give
//   D[t] = <dO, O>;  for i < m:  s_i = <Q[t], K_d[i][t-i]>,  dp_i = <dO[t], V_d[i][t-i]>,
//   P_i = 2^(s_i c2 - lse2[t]),  dS_i = P_i (dp_i - D) scale          (zero where t - i < 0)
//   dQacc[t] = sum_i dS_i K_d[i][t-i]                                  (fp32; zero for m = 0)
//   dK_d[i][t-i] = sum_h dS_i Q[t],  dV_d[i][t-i] = sum_h P_i dO[t]
// Position s of pass i meets exactly one query per head (t = s + i), so each output row has one writer; the
// last i rows of pass i meet none and are zeroed by the half-warp of the same index. Passes are taken two at
// a time; the rows of the next head are requested before the current head is worked on.
struct RowsParams {
    const __nv_bfloat16* Q;        // [B, T, H, 128]
    const __nv_bfloat16* O;
    const __nv_bfloat16* dO;
    const __nv_bfloat16* Kd[MAX_DRAFTS];   // [B, T, Hkv, 128]
    const __nv_bfloat16* Vd[MAX_DRAFTS];
    __nv_bfloat16* dKd[MAX_DRAFTS];
    __nv_bfloat16* dVd[MAX_DRAFTS];
    const float* lse;              // [B, H, T]
    float* D;                      // [B, H, T]
    float* dQacc;                  // [B, T, H, 128] fp32
    int m, B, T, H, Hkv;
    float c2, scale;
};

__global__ void __launch_bounds__(256, 2) hca_bwd_rows_kernel(const __grid_constant__ RowsParams p) {
    const long long w = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 4;   // (b, t, g)
    const int sub = threadIdx.x & 15;
    // no thread leaves early: the shuffles below name all 32 lanes, so a half-warp past the end runs on clamped
    // indices with its stores switched off
    const long long total = static_cast<long long>(p.B) * p.T * p.Hkv;
    const bool live = w < total;
    const long long wc = live ? w : total - 1;
    const int g = static_cast<int>(wc % p.Hkv);
    const long long bt = wc / p.Hkv;
    const int t = static_cast<int>(bt % p.T);
    const int b = static_cast<int>(bt / p.T);
    const int rep = p.H / p.Hkv;
    const int m = p.m;
    const int passes = m > 0 ? m : 1;
    const size_t row0 = ((static_cast<size_t>(b) * p.T + t) * p.H + g * rep) * HD;      // head g * rep; the group's heads follow
    const size_t ri0 = (static_cast<size_t>(b) * p.H + g * rep) * p.T + t;              // ... at distance T here
    for (int i0 = 0; i0 < passes; i0 += 2) {
        uint4 kraw[2], vraw[2];         // kept packed; widened where they are used
        float kacc[2][8], vacc[2][8];
        bool use[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = i0 + j;
            use[j] = i < m && t - i >= 0;
            kraw[j] = vraw[j] = make_uint4(0u, 0u, 0u, 0u);
            if (use[j]) {
                const size_t row = ((static_cast<size_t>(b) * p.T + (t - i)) * p.Hkv + g) * HD;
                kraw[j] = __ldg(reinterpret_cast<const uint4*>(p.Kd[i] + row) + sub);
                vraw[j] = __ldg(reinterpret_cast<const uint4*>(p.Vd[i] + row) + sub);
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) kacc[j][c] = vacc[j][c] = 0.f;
        }
        uint4 qn = __ldg(reinterpret_cast<const uint4*>(p.Q + row0) + sub);
        uint4 dn = __ldg(reinterpret_cast<const uint4*>(p.dO + row0) + sub);
        uint4 on = i0 == 0 ? __ldg(reinterpret_cast<const uint4*>(p.O + row0) + sub) : make_uint4(0u, 0u, 0u, 0u);
        float ln = __ldg(p.lse + ri0);
        for (int hh = 0; hh < rep; ++hh) {
            const size_t row = row0 + static_cast<size_t>(hh) * HD;
            const size_t ri = ri0 + static_cast<size_t>(hh) * p.T;
            float qf[8], df[8];
            widen8(qn, qf);
            widen8(dn, df);
            const uint4 oc = on;
            const float nlse2 = -ln * 1.4426950408889634f;
            if (hh + 1 < rep) {
                qn = __ldg(reinterpret_cast<const uint4*>(p.Q + row + HD) + sub);
                dn = __ldg(reinterpret_cast<const uint4*>(p.dO + row + HD) + sub);
                if (i0 == 0) on = __ldg(reinterpret_cast<const uint4*>(p.O + row + HD) + sub);
                ln = __ldg(p.lse + ri + p.T);
            }
            float Dt;
            if (i0 == 0) {
                float of[8];
                widen8(oc, of);
                Dt = sum16(dot8(df, of));
                if (live && sub == 0) p.D[ri] = Dt;
            } else {
                Dt = p.D[ri];           // written by this half-warp's first lane in the first round
                Dt = __shfl_sync(0xffffffffu, Dt, threadIdx.x & 16);
            }
            float dq[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) dq[c] = 0.f;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float kdf[8], vdf[8];
                widen8(kraw[j], kdf);
                widen8(vraw[j], vdf);
                const float sv = sum16(dot8(qf, kdf));
                const float dv = sum16(dot8(df, vdf));
                const float pw = use[j] ? ex2(fmaf(sv, p.c2, nlse2)) : 0.f;
                const float ds = pw * (dv - Dt) * p.scale;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    dq[c] = fmaf(ds, kdf[c], dq[c]);
                    kacc[j][c] = fmaf(ds, qf[c], kacc[j][c]);
                    vacc[j][c] = fmaf(pw, df[c], vacc[j][c]);
                }
            }
            if (live) {
                float* dst = p.dQacc + row + 8 * sub;
                if (i0 != 0) {
                    float a[8];
                    ld_global_v8(dst, a);
#pragma unroll
                    for (int c = 0; c < 8; ++c) dq[c] += a[c];
                }
                st_global_v8(dst, __float_as_uint(dq[0]), __float_as_uint(dq[1]), __float_as_uint(dq[2]),
                             __float_as_uint(dq[3]), __float_as_uint(dq[4]), __float_as_uint(dq[5]),
                             __float_as_uint(dq[6]), __float_as_uint(dq[7]));
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = i0 + j;
            if (live && i < m) {
                if (t - i >= 0) {
                    const size_t orow = ((static_cast<size_t>(b) * p.T + (t - i)) * p.Hkv + g) * HD;
                    *(reinterpret_cast<uint4*>(p.dKd[i] + orow) + sub) = narrow8(kacc[j]);
                    *(reinterpret_cast<uint4*>(p.dVd[i] + orow) + sub) = narrow8(vacc[j]);
                }
                if (t + i >= p.T) {     // position t of pass i would meet query t + i, past the sequence
                    const size_t orow = ((static_cast<size_t>(b) * p.T + t) * p.Hkv + g) * HD;
                    *(reinterpret_cast<uint4*>(p.dKd[i] + orow) + sub) = make_uint4(0u, 0u, 0u, 0u);
                    *(reinterpret_cast<uint4*>(p.dVd[i] + orow) + sub) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
    }
}

// dQ = the fp32 accumulator as bf16; 8 values per thread.
__global__ void __launch_bounds__(256) hca_dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dQ,
                                                             long long n8) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    float v[8];
    ld_global_v8(acc + 8 * i, v);
    *(reinterpret_cast<uint4*>(dQ) + i) = narrow8(v);
}

// ------------------------------------------------------------------------------------------------------
// The tensor-core kernel. A work item is (sequence, key/value head, tile of 128 key positions); its K and V
// tiles stay in shared memory while it sweeps the query heads of its group and, per head, the tiles of 64
// queries at or after it. Per element (one head, 64 queries), in tensor-memory set sb = element & 1:
//   S^T = K Q^T, dP^T = V dO^T        tcgen05.mma, 128 x 64 x 128 each (rows = keys, one per thread)
//   threads                            P^T = 2^(S^T c2 - lse2[t]) on the entries the target's keys really met
//                                      (t - s >= m), dS^T = P^T (dP^T - D[t]) scale; both as bf16 pairs back into
//                                      the S^T columns they were read from (A operands), dS^T also into shared
//                                      memory as 128-byte rows (the B operand of the dQ^T product)
//   dV += P^T dO, dK += dS^T Q         A from tensor memory, the Q / dO stage read MN-major
//   dQ^T = K^T dS^T                    128 (head dimension) x 64 (queries) x 128 (keys), K read MN-major as A,
//                                      into the columns dP^T came from; not accumulated on chip
//   threads                            dQ^T out of tensor memory into a staging buffer in shared memory (transposed
//                                      back: 32 queries x 128 floats per group), from where one TMA reduction per
//                                      group adds it into the accumulator; rows past the sequence are clipped by
//                                      the tensor map. (Plain red.global.add.f32 from the threads - 32 per thread
//                                      and element - is limited to about 16 bytes per clock and SM and made the
//                                      threads the slowest stage.)
// The tensor core completes products in issue order, so the issue order S^T(e+2) after the three products of
// element e needs no barrier for the S^T columns; dP^T(e+2) waits until the threads have taken dQ^T(e) out.
// The per-query vectors -lse2[t] and -D[t] scale of an element travel with its Q / dO stage (written by a warp
// that does nothing else).
constexpr int F_STAGES = 3;             // a Q / dO stage is held until the element's last product is done
constexpr int F_SMEM_K = 0;
constexpr int F_SMEM_V = F_SMEM_K + K_BYTES;
constexpr int F_SMEM_Q = F_SMEM_V + K_BYTES;
constexpr int F_SMEM_DO = F_SMEM_Q + F_STAGES * QE_BYTES;
constexpr int F_SMEM_DS = F_SMEM_DO + F_STAGES * QE_BYTES;          // two buffers
constexpr int DQ_STAGE_BYTES = 32 * HD * 4;                         // one group's share of dQ: 32 queries x 128 floats
constexpr int F_SMEM_DQ = F_SMEM_DS + 2 * DS_BYTES;                 // one staging buffer per group
constexpr int F_SMEM_VEC = F_SMEM_DQ + 2 * DQ_STAGE_BYTES;          // per stage: 64 x -lse2, 64 x -D scale (floats)
constexpr int F_SMEM_BAR = F_SMEM_VEC + F_STAGES * 512;
constexpr int F_NUM_BARS = 2 + 2 * F_STAGES + 8 + 2 + 4;
constexpr int F_SMEM_TAIL = 256;
constexpr int F_SMEM_BYTES = F_SMEM_BAR + F_SMEM_TAIL;
static_assert(8 * F_NUM_BARS + 8 <= F_SMEM_TAIL, "barriers, tensor-memory pointer and abort flag must fit the tail");
static_assert(F_SMEM_BYTES <= 232448, "shared memory of one CTA");
constexpr int F_TMEM_COLS = 512;        // set sb at 128 sb: S^T in columns 0..63, dP^T (later dQ^T) in 64..127; dV at 256, dK at 384

struct FusedParams {
    CUtensorMap tmK, tmV;          // [B, T, Hkv * 128], box {64, 128, 1}, 128-byte swizzle
    CUtensorMap tmQ, tmdO;         // [B, T, H * 128], box {64, 64, 1}
    CUtensorMap tmdQ;              // the fp32 accumulator [B, T, H * 128], box {128, 32, 1}, no swizzle; initialised by
                                   // hca_bwd_rows_kernel
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

__global__ void __launch_bounds__(NUM_THREADS, 1) hca_bwd_fused_kernel(const __grid_constant__ FusedParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0u) {
        // the swizzled tiles need a 1024-byte aligned window; report instead of computing garbage
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (20u << 8) | 1u);
        return;
    }
    const uint32_t bar0 = base + F_SMEM_BAR;
    const uint32_t kv_full = bar0, kv_empty = bar0 + 8;
    auto qd_full = [&](int s) { return bar0 + 8u * (2 + s); };
    auto qd_empty = [&](int s) { return bar0 + 8u * (2 + F_STAGES + s); };
    auto st_full = [&](int s) { return bar0 + 8u * (2 + 2 * F_STAGES + s); };      // S^T and dP^T of the set are complete
    auto dp_free = [&](int s) { return bar0 + 8u * (4 + 2 * F_STAGES + s); };      // dQ^T taken out: the dP^T columns may be rewritten
    auto pds_full = [&](int s) { return bar0 + 8u * (6 + 2 * F_STAGES + s); };     // P^T, dS^T written
    auto dq_full = [&](int s) { return bar0 + 8u * (8 + 2 * F_STAGES + s); };      // the element's three products are complete
    const uint32_t acc_done = bar0 + 8u * (10 + 2 * F_STAGES), acc_free = bar0 + 8u * (11 + 2 * F_STAGES);
    auto stage_free = [&](int g) { return bar0 + 8u * (12 + 2 * F_STAGES + g); };  // group g's staging buffer has been read by its last reduction
    auto stage_full = [&](int g) { return bar0 + 8u * (14 + 2 * F_STAGES + g); };  // ... has been written by the group's four warps
    uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(smem_raw + F_SMEM_BAR + 8 * F_NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_ptr_smem + 1);
    float* vec = reinterpret_cast<float*>(smem_raw + F_SMEM_VEC);      // [stage][0..63 -lse2 | 64..127 -D scale]

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        mbar_init(kv_empty, 1);
        for (int s = 0; s < F_STAGES; ++s) {
            mbar_init(qd_full(s), 2);      // the TMA transaction's arrival and the vector warp's
            mbar_init(qd_empty(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(st_full(s), 1);
            mbar_init(dp_free(s), 8);
            mbar_init(pds_full(s), 8);
            mbar_init(dq_full(s), 1);
            mbar_init(stage_free(s), 1);
            mbar_init(stage_full(s), 4);
        }
        mbar_init(acc_done, 1);
        mbar_init(acc_free, 8);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&p.tmK);
        prefetch_tensormap(&p.tmV);
        prefetch_tensormap(&p.tmQ);
        prefetch_tensormap(&p.tmdO);
        prefetch_tensormap(&p.tmdQ);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_ptr_smem), F_TMEM_COLS);
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
    // Every CTA walks the rounds in rotated order, starting at round (its index mod rounds): its share of the work
    // is the same, but at any moment different CTAs are in rounds of different item lengths, so that their item
    // boundaries (pipeline drained, a burst of loads) do not coincide. next_item steps the round counter k to this
    // CTA's next existing item and returns it, or -1.
    const int n_rounds = (p.items + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    auto next_item = [&](int& k) {
        while (k < n_rounds) {
            const int item = round_item(static_cast<uint32_t>((k + static_cast<int>(blockIdx.x)) % n_rounds));
            ++k;
            if (item < p.items) return item;
        }
        return -1;
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
        // ===================== producer: TMA =====================
        if (lane == 0) {
            uint32_t gq = 0, it = 0;
            bool ok = true;
            for (int rk = 0, item = next_item(rk); item >= 0 && ok; item = next_item(rk), ++it) {
                int kt, b, g;
                decode(item, kt, b, g);
                const int nq = q_count(kt);
                if (!wait_barrier(kv_empty, (it & 1u) ^ 1u, abort_flag, p.status, 1)) break;
                mbar_arrive_expect_tx(kv_full, 2 * K_BYTES);
                tma_load_3d(base + F_SMEM_K, &p.tmK, kv_full, g * HD, kt * KEYS, b);
                tma_load_3d(base + F_SMEM_K + K_HALF, &p.tmK, kv_full, g * HD + 64, kt * KEYS, b);
                tma_load_3d(base + F_SMEM_V, &p.tmV, kv_full, g * HD, kt * KEYS, b);
                tma_load_3d(base + F_SMEM_V + K_HALF, &p.tmV, kv_full, g * HD + 64, kt * KEYS, b);
                for (int e = 0; e < rep * nq; ++e, ++gq) {
                    const int h = g * rep + e / nq;
                    const int jq = 2 * kt + e % nq;
                    const int s = gq % F_STAGES;
                    if (!wait_barrier(qd_empty(s), ((gq / F_STAGES) & 1u) ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
                    mbar_arrive_expect_tx(qd_full(s), 2 * QE_BYTES);
                    tma_load_3d(base + F_SMEM_Q + s * QE_BYTES, &p.tmQ, qd_full(s), h * HD, jq * QE, b);
                    tma_load_3d(base + F_SMEM_Q + s * QE_BYTES + QE_HALF, &p.tmQ, qd_full(s), h * HD + 64, jq * QE, b);
                    tma_load_3d(base + F_SMEM_DO + s * QE_BYTES, &p.tmdO, qd_full(s), h * HD, jq * QE, b);
                    tma_load_3d(base + F_SMEM_DO + s * QE_BYTES + QE_HALF, &p.tmdO, qd_full(s), h * HD + 64, jq * QE, b);
                }
            }
        }
    } else if (warp == VEC_WARP) {
        // ===================== the per-query vectors of every element, next to its Q / dO stage =====================
        // -lse2[t] (or -inf past the sequence, which zeroes the weight) and -D[t] scale for the 64 queries, two per
        // lane. A warp of its own: the loads' latency then delays neither the TMA requests nor anything else.
        uint32_t gq = 0, it = 0;
        bool ok = true;
        for (int rk = 0, item = next_item(rk); item >= 0 && ok; item = next_item(rk), ++it) {
            int kt, b, g;
            decode(item, kt, b, g);
            const int nq = q_count(kt);
            for (int e = 0; e < rep * nq && ok; ++e, ++gq) {
                const int h = g * rep + e / nq;
                const int jq = 2 * kt + e % nq;
                const int s = gq % F_STAGES;
                const size_t rowbase = (static_cast<size_t>(b) * p.H + h) * p.T;
                float nl[2], nd[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int t = jq * QE + lane + 32 * u;
                    nl[u] = t < p.T ? -__ldg(p.lse + rowbase + t) * 1.4426950408889634f : -INFINITY;
                    nd[u] = t < p.T ? -__ldg(p.D + rowbase + t) * p.scale : 0.f;
                }
                if (lane == 0) ok = wait_barrier(qd_empty(s), ((gq / F_STAGES) & 1u) ^ 1u, abort_flag, p.status, 3);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    vec[s * 128 + lane + 32 * u] = nl[u];
                    vec[s * 128 + 64 + lane + 32 * u] = nd[u];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(qd_full(s));
            }
        }
    } else if (warp == 1) {
        // The whole warp runs this loop so that addresses and descriptors stay warp-uniform; one elected lane
        // issues the tensor-core instructions.
        constexpr uint32_t idesc_s = make_idesc_bf16(KEYS, QE, 0, 0);     // S^T, dP^T: both operands K-major
        constexpr uint32_t idesc_a = make_idesc_bf16(KEYS, HD, 0, 1);     // dV, dK: A from tensor memory, B MN-major
        constexpr uint32_t idesc_q = make_idesc_bf16(HD, QE, 1, 1);       // dQ^T: K^T and dS^T, both MN-major
        uint32_t gs = 0, ga = 0, it = 0;      // elements whose S^T/dP^T, resp. whose three accumulating products have been issued
        bool ok = true;
        auto wait_all = [&](uint32_t bar, uint32_t parity, unsigned code) {
            return __all_sync(0xffffffffu, wait_barrier(bar, parity, abort_flag, p.status, code)) != 0;
        };
        auto issue_st = [&]() -> bool {
            const int s = gs & 1u;                  // tensor-memory set
            const int qs = gs % F_STAGES;           // Q / dO stage
            if (!wait_all(qd_full(qs), (gs / F_STAGES) & 1u, 4)) return false;
            tc_fence_after_sync();
            bool leader = elect_one();
#pragma unroll
            for (int k = 0; k < HD / 16; ++k) {
                const uint32_t ao = (k >> 2) * K_HALF + (k & 3) * 32, bo = (k >> 2) * QE_HALF + (k & 3) * 32;
                const uint64_t ak_ = make_smem_desc_sw128(base + F_SMEM_K + ao, 0, 1024);
                const uint64_t bq_ = make_smem_desc_sw128(base + F_SMEM_Q + qs * QE_BYTES + bo, 0, 1024);
                if (leader) umma_bf16(tmem_base + s * 128, ak_, bq_, idesc_s, k != 0 ? 1u : 0u);
            }
            __syncwarp();
            // the dP^T columns held dQ^T of the element two before: its threads must have taken it out
            if (!wait_all(dp_free(s), ((gs >> 1) & 1u) ^ 1u, 5)) return false;
            tc_fence_after_sync();
            leader = elect_one();
#pragma unroll
            for (int k = 0; k < HD / 16; ++k) {
                const uint32_t ao = (k >> 2) * K_HALF + (k & 3) * 32, bo = (k >> 2) * QE_HALF + (k & 3) * 32;
                const uint64_t av_ = make_smem_desc_sw128(base + F_SMEM_V + ao, 0, 1024);
                const uint64_t bd_ = make_smem_desc_sw128(base + F_SMEM_DO + qs * QE_BYTES + bo, 0, 1024);
                if (leader) umma_bf16(tmem_base + s * 128 + 64, av_, bd_, idesc_s, k != 0 ? 1u : 0u);
            }
            if (leader) umma_commit(st_full(s));
            __syncwarp();
            ++gs;
            return true;
        };
        auto issue_acc = [&](bool first, bool last) -> bool {
            const int s = ga & 1u;
            const int qs = ga % F_STAGES;
            if (!wait_all(pds_full(s), (ga >> 1) & 1u, 7)) return false;
            if (first && !wait_all(acc_free, (it & 1u) ^ 1u, 9)) return false;
            tc_fence_after_sync();
            const bool leader = elect_one();
#pragma unroll
            for (int k = 0; k < QE / 16; ++k) {
                // A from tensor memory: queries 16 k .. 16 k + 15 of P^T sit as 8 columns of bf16 pairs at the start of
                // the 32 columns their group read (0..15 for k < 2, 32..47 for k >= 2), dS^T 16 columns further
                const uint32_t a_col = s * 128 + (k < 2 ? 8 * k : 32 + 8 * (k - 2));
                const uint64_t bd_ = make_smem_desc_sw128(base + F_SMEM_DO + qs * QE_BYTES + k * 16 * 128, QE_HALF, 1024);
                const uint64_t bq_ = make_smem_desc_sw128(base + F_SMEM_Q + qs * QE_BYTES + k * 16 * 128, QE_HALF, 1024);
                if (leader) {
                    umma_bf16_ta(tmem_base + 256, tmem_base + a_col, bd_, idesc_a, (!first || k != 0) ? 1u : 0u);
                    umma_bf16_ta(tmem_base + 384, tmem_base + a_col + 16, bq_, idesc_a, (!first || k != 0) ? 1u : 0u);
                }
            }
#pragma unroll
            for (int k = 0; k < KEYS / 16; ++k) {
                // keys 16 k .. 16 k + 15: rows of the K tile (A, the head dimension contiguous: two halves of 64) and of
                // the dS^T buffer (B, the 64 queries contiguous)
                const uint64_t ak_ = make_smem_desc_sw128(base + F_SMEM_K + k * 16 * 128, K_HALF, 1024);
                const uint64_t bs_ = make_smem_desc_sw128(base + F_SMEM_DS + s * DS_BYTES + k * 16 * 128, 0, 1024);
                if (leader) umma_bf16(tmem_base + s * 128 + 64, ak_, bs_, idesc_q, k != 0 ? 1u : 0u);
            }
            if (leader) {
                umma_commit(qd_empty(qs));
                umma_commit(dq_full(s));
                if (last) {
                    umma_commit(acc_done);
                    umma_commit(kv_empty);
                }
            }
            __syncwarp();
            ++ga;
            return true;
        };
        for (int rk = 0, item = next_item(rk); item >= 0 && ok; item = next_item(rk), ++it) {
            int kt, b, g;
            decode(item, kt, b, g);
            const int n_e = rep * q_count(kt);
            if (!wait_all(kv_full, it & 1u, 6)) break;
            ok = issue_st();
            if (ok && n_e > 1) ok = issue_st();
            for (int a = 0; a < n_e && ok; ++a) {
                ok = issue_acc(a == 0, a + 1 == n_e);
                if (ok && a + 2 < n_e) ok = issue_st();
            }
        }
    } else if (warp < VEC_WARP) {
        // two groups of four warps share every key row: group grp takes the query columns 32 grp .. 32 grp + 31
        // of each element, and in the epilogue dV (group 0) or dK (group 1)
        const int grp = (warp - 2) >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                 // key row of the tile; row of dQ^T (head dimension) when reading that
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        uint32_t gq = 0, it = 0;
        bool ok = true;
        // dQ^T of the element with running index ge (head h, 64-query tile jq): this thread's row (one of the 128
        // head dimensions) for the group's 32 queries goes into the group's staging buffer as column r of a
        // [32 queries][128] fp32 tile, which one thread of the group hands to the TMA unit for reduction into the
        // accumulator.
        const bool issuer = quad == 0 && lane == 0;
        const uint32_t stage = base + F_SMEM_DQ + grp * DQ_STAGE_BYTES;
        uint32_t nd = 0;                            // reductions of this group so far
        auto take_dq = [&](uint32_t ge, int b, int h, int jq) -> bool {
            const int s = ge & 1u;
            if (!wait_barrier(dq_full(s), (ge >> 1) & 1u, abort_flag, p.status, 11)) return false;
            tc_fence_after_sync();
            uint32_t v[32];
            tmem_ld32(tmem_base + s * 128 + 64 + 32 * grp + lane_addr, v);
            tmem_ld_wait(v);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(dp_free(s));
            if (issuer) {
                bulk_wait_group_read<0>();            // the previous reduction has read the staging buffer
                mbar_arrive(stage_free(grp));
            }
            if (!wait_barrier(stage_free(grp), nd & 1u, abort_flag, p.status, 16)) return false;
#pragma unroll
            for (int c = 0; c < 32; ++c) st_shared_b32(stage + c * (HD * 4) + r * 4, v[c]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(stage_full(grp));
            if (issuer) {
                if (!wait_barrier(stage_full(grp), nd & 1u, abort_flag, p.status, 17)) return false;
                if (jq * QE + 32 * grp < p.T) {     // a ragged last tile may leave the second group nothing
                    tma_reduce_add_3d(&p.tmdQ, stage, h * HD, jq * QE + 32 * grp, b);
                    bulk_commit_group();
                }
            }
            __syncwarp();
            ++nd;
            return true;
        };
        for (int rk = 0, item = next_item(rk); item >= 0 && ok; item = next_item(rk), ++it) {
            int kt, b, g;
            decode(item, kt, b, g);
            const int nq = q_count(kt);
            const int spos = kt * KEYS + r;             // key position
            const int n_e = rep * nq;
            for (int e = 0; e < n_e; ++e, ++gq) {
                const int jq = 2 * kt + e % nq;
                const int s = gq & 1u;                  // tensor-memory set
                const int qs = gq % F_STAGES;           // the element's Q / dO stage, for its vectors
                if (!wait_barrier(st_full(s), (gq >> 1) & 1u, abort_flag, p.status, 10)) { ok = false; break; }
                if (!wait_barrier(qd_full(qs), (gq / F_STAGES) & 1u, abort_flag, p.status, 15)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_s = tmem_base + s * 128 + lane_addr + 32 * grp;
                // the target's key at spos met query t only if t - spos >= m: columns below lo are empty
                const int lo = spos + m - jq * QE - 32 * grp;
                const bool band = spos + m - jq * QE > 0;
                uint32_t sr[32], dr[32];
                tmem_ld32(tmem_s, sr);
                tmem_ld32(tmem_s + 64, dr);
                tmem_ld_wait(sr);
                tmem_ld_wait(dr);
                if (band) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c < lo) sr[c] = 0xff800000u;       // -inf: weight 0
                }
                // P^T = 2^(S^T c2 - lse2[t]), dS^T = P^T (dP^T scale - D[t] scale), two columns per instruction
                const float4* nl = reinterpret_cast<const float4*>(vec + qs * 128 + 32 * grp);
                const float4* dd = reinterpret_cast<const float4*>(vec + qs * 128 + 64 + 32 * grp);
                uint32_t pk[16], dk[16];
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4) {
                    const float4 a = nl[c4], d = dd[c4];
                    const int c = 4 * c4;
                    float x0, x1, y0, y1, p0, p1, p2, p3, d0, d1, d2, d3;
                    ffma2(x0, x1, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]), p.c2, p.c2, a.x, a.y);
                    ffma2(y0, y1, __uint_as_float(dr[c]), __uint_as_float(dr[c + 1]), p.scale, p.scale, d.x, d.y);
                    p0 = ex2(x0);
                    p1 = ex2(x1);
                    fmul2(d0, d1, p0, p1, y0, y1);
                    ffma2(x0, x1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]), p.c2, p.c2, a.z, a.w);
                    ffma2(y0, y1, __uint_as_float(dr[c + 2]), __uint_as_float(dr[c + 3]), p.scale, p.scale, d.z, d.w);
                    p2 = ex2(x0);
                    p3 = ex2(x1);
                    fmul2(d2, d3, p2, p3, y0, y1);
                    pk[2 * c4] = pack_bf16(p0, p1);
                    pk[2 * c4 + 1] = pack_bf16(p2, p3);
                    dk[2 * c4] = pack_bf16(d0, d1);
                    dk[2 * c4 + 1] = pack_bf16(d2, d3);
                }
                // bf16 pairs over the 32 columns this group read: P^T in the first 16, dS^T in the last 16. The set's
                // previous user of these columns as operands (the products of the element two before) finished before
                // this element's S^T was written, and so did its read of the dS^T buffer in shared memory.
                hca::tmem_st16(tmem_s, pk);
                hca::tmem_st16(tmem_s + 16, dk);
                {
                    // dS^T row r, queries 32 grp .. 32 grp + 31: four 16-byte chunks of the 128-byte row, swizzled
                    const uint32_t rowaddr = base + F_SMEM_DS + s * DS_BYTES + r * 128;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        st_shared_v4(rowaddr + ((((4 * grp + j) ^ (r & 7)) & 7) << 4), dk[4 * j], dk[4 * j + 1], dk[4 * j + 2],
                                     dk[4 * j + 3]);
                }
                hca::tmem_st_wait();
                fence_proxy_async_smem();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(pds_full(s));
                // the element before this one: its products were issued when its P^T / dS^T arrived and run while this
                // element's were being formed
                if (e > 0) {
                    const int ep = e - 1;
                    if (!take_dq(gq - 1, b, g * rep + ep / nq, 2 * kt + ep % nq)) { ok = false; break; }
                }
            }
            if (!ok) break;
            if (!take_dq(gq - 1, b, g * rep + (n_e - 1) / nq, 2 * kt + (n_e - 1) % nq)) break;
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
        if (issuer) bulk_wait_group0();     // shared memory must outlive the reductions that read it
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, F_TMEM_COLS);
    }
}

}  // namespace hca_bwd
}  // namespace hass
