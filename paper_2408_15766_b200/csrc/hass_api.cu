// Host side of the C ABI declared in include/hass.h: argument checks, tile schedules, TMA
// descriptors, workspace layout and kernel launches. No allocation, no synchronisation except in
// hass_check and the *_host entry.
#include <atomic>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "../../include/hass.h"
#include "kernels.cuh"
#include "hca_kernels.cuh"
#include "hca_pair_kernel.cuh"
#include "hca_bwd_fused_kernel.cuh"

namespace hass {

static std::atomic<long long> g_launches{0};

// ---- optional per-kernel timing (hass_profile_*) ------------------------------------------------
// When enabled, every kernel launch is bracketed by a pair of CUDA events on its own stream; the
// summary adds up the elapsed time per kernel kind. Off by default; not thread-safe.
enum { KIND_STATS = 0, KIND_PROBS = 1, KIND_OUT = 2, KIND_FINALIZE = 3, KIND_PREP = 4, KIND_CONDITIONAL = 5, KIND_HCA = 6, KIND_HCA_DQ_CONVERT = 7, KIND_HCA_BWD_FUSED = 8, KIND_HCA_BWD_ROWS = 9, KIND_STATS_DRAFT = 10, NUM_KINDS = 11 };
constexpr int kMaxRecords = 8192;
struct Profiler {
    bool on = false;
    int n = 0;
    std::vector<cudaEvent_t> ev;     // 2 per record
    std::vector<int> kind;
};
static Profiler g_prof;

struct KernelTimer {
    int rec = -1;
    cudaStream_t st;
    KernelTimer(int kind, cudaStream_t s) : st(s) {
        if (g_prof.on && g_prof.n < kMaxRecords) {
            rec = g_prof.n++;
            g_prof.kind[rec] = kind;
            cudaEventRecord(g_prof.ev[2 * rec], st);
        }
    }
    ~KernelTimer() {
        if (rec >= 0) cudaEventRecord(g_prof.ev[2 * rec + 1], st);
    }
};

// ---- device info ------------------------------------------------------------------------------
struct DeviceInfo {
    int ok = 0;   // 0 unknown, 1 usable, <0 hass_status
    int sms = 148;
};
static DeviceInfo g_dev[64];

static int device_info(DeviceInfo* out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    DeviceInfo& di = g_dev[dev];
    if (di.ok == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        if (major != 10) {
            di.ok = HASS_ERR_ARCH;
        } else {
            di.sms = sms;
            cudaError_t e0 = cudaFuncSetAttribute(gemm_kernel<MODE_STATS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            cudaError_t e1 = cudaFuncSetAttribute(gemm_kernel<MODE_PROBS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            cudaError_t e2 = cudaFuncSetAttribute(gemm_kernel<MODE_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            cudaError_t e3 = cudaFuncSetAttribute(gemm_kernel<MODE_STATS, TOPK_REG>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            if (e3 == cudaSuccess) e3 = cudaFuncSetAttribute(gemm_kernel<MODE_STATS, TOPK_NONE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            cudaError_t e4 = cudaFuncSetAttribute(hca2::hca_attention_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, hca2::SMEM_BYTES);
            if (e4 == cudaSuccess) e4 = cudaFuncSetAttribute(hca_bwd::hca_bwd_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, hca_bwd::F_SMEM_BYTES);
            if (e0 != cudaSuccess || e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess || e4 != cudaSuccess) {
                cudaGetLastError();
                return HASS_ERR_CUDA;
            }
            di.ok = 1;
        }
    }
    if (di.ok < 0) return di.ok;
    *out = di;
    return HASS_OK;
}

static int sm_count_or_default() {
    DeviceInfo di;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return 148;
    }
    return device_info(&di) == HASS_OK ? di.sms : 148;
}

// ---- tile schedule ----------------------------------------------------------------------------
// Splits RT row tiles into phases (G row tiles x S lanes, G * S <= sms) minimising the summed phase
// durations ceil(CT / S), by dynamic programming over the number of row tiles already covered.
static int plan_schedule(int RT, int CT, int sms, Schedule* out) {
    if (RT < 1 || CT < 1 || sms < 1) return HASS_ERR_INVALID_ARG;
    const int INF = 1 << 30;
    std::vector<int> best(RT + 1, INF), nph(RT + 1, INF), choice(RT + 1, 0);
    best[0] = 0;
    nph[0] = 0;
    for (int n = 1; n <= RT; ++n) {
        for (int G = 1; G <= n && G <= sms; ++G) {
            int S = sms / G;
            if (S > CT) S = CT;
            const int cost = best[n - G] + (CT + S - 1) / S;
            const int ph = nph[n - G] + 1;
            if (cost < best[n] || (cost == best[n] && ph < nph[n])) {
                best[n] = cost;
                nph[n] = ph;
                choice[n] = G;
            }
        }
    }
    if (nph[RT] > MAX_PHASES) return HASS_ERR_UNSUPPORTED;
    std::vector<int> groups;
    for (int n = RT; n > 0; n -= choice[n]) groups.push_back(choice[n]);
    std::memset(out, 0, sizeof(*out));
    int rt = 0, slot = 0, maxc = 0;
    // largest groups first: the widest phases start together
    for (size_t i = 0; i < groups.size(); ++i)
        for (size_t j = i + 1; j < groups.size(); ++j)
            if (groups[j] > groups[i]) std::swap(groups[i], groups[j]);
    for (size_t i = 0; i < groups.size(); ++i) {
        const int G = groups[i];
        int S = sms / G;
        if (S > CT) S = CT;
        out->ph[i] = Phase{rt, G, S, slot};
        rt += G;
        slot += G * S;
        if (G * S > maxc) maxc = G * S;
    }
    out->n_phases = static_cast<int>(groups.size());
    out->total_slots = slot;
    out->max_ctas = maxc;
    return HASS_OK;
}

// ---- TMA descriptors --------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

static int get_encode() {
    if (g_encode) return HASS_OK;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return HASS_OK;
}

// bf16 row-major matrix [rows, cols] with `pitch` elements between rows; box = box_cols x box_rows,
// 128-byte swizzle (box_cols must be 64), out-of-range elements read as zero.
static int make_tmap(CUtensorMap* tm, const void* base, long long rows, long long cols, long long pitch,
                     int box_cols, int box_rows) {
    cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    cuuint64_t gstride[1] = {static_cast<cuuint64_t>(pitch) * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HASS_OK : HASS_ERR_CUDA;
}

// bf16 tensor [B, T, heads * 128] (dense): box = 64 columns x box_rows positions of one sequence, 128-byte
// swizzle. Positions past T read as zeros, so a ragged last tile never sees the next sequence.
static int make_tmap_seq(CUtensorMap* tm, const void* base, long long B, long long T, long long cols,
                         int box_rows = 128) {
    cuuint64_t gdim[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(B)};
    cuuint64_t gstride[2] = {static_cast<cuuint64_t>(cols) * 2, static_cast<cuuint64_t>(cols) * 2 * static_cast<cuuint64_t>(T)};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HASS_OK : HASS_ERR_CUDA;
}

// capacity of a (row, slot) candidate buffer for this K
static int topk_cap(int K) { return K <= K_REG ? K_REG : cand_cap(K); }

// ---- workspace layout -------------------------------------------------------------------------
static inline size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

struct Layout {
    size_t status, part_m, part_s, cand_v, cand_i, thr_share, fwd_end, sidx, sgq, coef, lse2, capz, zmax, sparse, scratch, fixed_end;
    size_t scratch_row_tile_bytes;   // bytes of dz_d scratch per 128-row tile
    long long p_pitch;
    int pref_chunk_tiles;
    int slot_cap;
    size_t total_pref;
};

static int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

// The forward schedule covers 2 * RT row tiles (target then draft).
static int make_layout(long long N, long long d, long long V, int K, int sms, Layout* L, Schedule* fwd_sched) {
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN);
    Schedule s;
    int rc = plan_schedule(2 * RT, CT, sms, &s);
    if (rc != HASS_OK) return rc;
    if (fwd_sched) *fwd_sched = s;
    int pref = sms / 4;
    if (pref < 1) pref = 1;
    if (pref > RT) pref = RT;
    // partial-statistics slots: enough for the whole-batch forward and for the per-chunk forward
    // sweeps of the fused path (target + draft tiles, or draft tiles only, of a full or last chunk)
    int slot_cap = s.total_slots;
    {
        const int rem = RT % pref;
        const int cands[5] = {RT, 2 * pref, pref, 2 * rem, rem};
        for (int i = 0; i < 5; ++i) {
            if (cands[i] < 1) continue;
            Schedule t;
            rc = plan_schedule(cands[i], CT, sms, &t);
            if (rc != HASS_OK) return rc;
            if (t.total_slots > slot_cap) slot_cap = t.total_slots;
        }
    }
    if (slot_cap < sms) slot_cap = sms;     // any single-phase schedule (a caller-limited, smaller chunk) fits
    L->slot_cap = slot_cap;
    size_t off = 0;
    L->status = off;
    off += 256;
    const size_t slots = static_cast<size_t>(slot_cap);
    L->part_m = off;
    off = align256(off + slots * BM * 4);
    L->part_s = off;
    off = align256(off + slots * BM * 4);
    L->cand_v = off;                        // candidate buffers: (logit, token id) pairs, cand_cap(K) per (row, slot)
    off = align256(off + slots * BM * 8 * topk_cap(K));
    L->cand_i = off;                        // entries in use per (row, slot)
    off = align256(off + slots * BM * 4);
    L->thr_share = off;                     // admission thresholds the lanes of a row tile publish to each other
    off = align256(off + slots * BM * 4);
    L->fwd_end = off;                       // what the forward-only entry points use
    L->sidx = off;
    off = align256(off + static_cast<size_t>(N) * K * 4);
    L->sgq = off;
    off = align256(off + static_cast<size_t>(N) * K * 4);
    L->coef = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    L->lse2 = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    L->capz = off;                          // fused path: draft logits at Omega_hat, captured by the draft sweep, [N, K]
    off = align256(off + static_cast<size_t>(N) * K * 4);
    L->zmax = off;                          // single-sweep route: every spilling row's largest logit (target and draft rows)
    off = align256(off + static_cast<size_t>(2 * RT) * BM * 4);
    L->sparse = off;                        // fused path: Omega_hat term of one chunk of rows, fp32 [chunk rows, d]
    off = align256(off + static_cast<size_t>(pref) * BM * d * 4);
    L->scratch = off;
    L->fixed_end = off;
    L->p_pitch = static_cast<long long>(CT) * BN;
    L->scratch_row_tile_bytes = static_cast<size_t>(BM) * L->p_pitch * 2;
    L->pref_chunk_tiles = pref;
    L->total_pref = off + L->scratch_row_tile_bytes * pref;
    return HASS_OK;
}

// ---- argument checks --------------------------------------------------------------------------
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_sizes(long long N, long long d, long long V, int K) {
    if (N < 1 || d < 8 || V < 1 || K < 1) return HASS_ERR_INVALID_ARG;
    if (d % 8 != 0) return HASS_ERR_INVALID_ARG;
    if (K > V || K > HASS_K_MAX) return HASS_ERR_INVALID_ARG;
    if (N > (1ll << 30) || V > (1ll << 30) || d > (1ll << 20)) return HASS_ERR_UNSUPPORTED;
    return HASS_OK;
}

static const bool kLog = [] {
    const char* e = std::getenv("HASS_LOG");
    return e && e[0] == '1';
}();

static void log_schedule(const char* what, const Schedule& s) {
    if (!kLog) return;
    std::fprintf(stderr, "[hass] %s: %d phases, %d slots, grid %d:", what, s.n_phases, s.total_slots, s.max_ctas);
    for (int i = 0; i < s.n_phases; ++i)
        std::fprintf(stderr, " (rt0=%d G=%d S=%d)", s.ph[i].row_tile_begin, s.ph[i].G, s.ph[i].S);
    std::fprintf(stderr, "\n");
}

template <int MODE>
static int launch_gemm(const GemmParams& p, cudaStream_t st, int kind = -1) {
    KernelTimer timer(p.only_if_range ? KIND_CONDITIONAL : (kind >= 0 ? kind : MODE), st);
    if (MODE == MODE_STATS && p.topk_row_tiles == 0 && p.cap_z != nullptr)
        gemm_kernel<MODE_STATS, TOPK_NONE><<<p.sched.max_ctas, NUM_THREADS, SMEM_BYTES, st>>>(p);
    else if (MODE == MODE_STATS && p.K <= K_REG)
        gemm_kernel<MODE_STATS, TOPK_REG><<<p.sched.max_ctas, NUM_THREADS, SMEM_BYTES, st>>>(p);
    else
        gemm_kernel<MODE><<<p.sched.max_ctas, NUM_THREADS, SMEM_BYTES, st>>>(p);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? HASS_OK : HASS_ERR_CUDA;
}

// ---- forward ----------------------------------------------------------------------------------
// with_target: both projections + Omega_hat selection; otherwise draft only with Omega_hat given.
static int forward_impl(bool with_target, const void* H_t, const void* H_d, const void* W, long long N, long long d,
                        long long V, int K, const int* idx_in, const float* q_in, float* loss, int* idx_out,
                        float* q_out, float* lse_t, float* lse_d, void* workspace, size_t workspace_bytes,
                        cudaStream_t st, const unsigned int* only_if_range = nullptr, float top_p = 0.f,
                        int* topk_n = nullptr) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_d || !W || !loss || !lse_d || !aligned16(H_d) || !aligned16(W)) return HASS_ERR_INVALID_ARG;
    if (with_target && (!H_t || !idx_out || !q_out || !lse_t || !aligned16(H_t))) return HASS_ERR_INVALID_ARG;
    if (!with_target && (!idx_in || !q_in)) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;

    Layout L;
    Schedule full;
    rc = make_layout(N, d, V, K, di.sms, &L, &full);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.fwd_end) return HASS_ERR_WORKSPACE;
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    // every public call starts with a clean status word (a conditional follow-up keeps the one it reads)
    if (!only_if_range && cudaMemsetAsync(ws + L.status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }

    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    if (with_target) {
        p.sched = full;
        p.row_tiles0 = RT;
        p.topk_row_tiles = RT;
        rc = make_tmap(&p.tmA0, H_t, N, d, d, BK, BM);
        if (rc == HASS_OK) rc = make_tmap(&p.tmA1, H_d, N, d, d, BK, BM);
    } else {
        rc = plan_schedule(RT, CT, di.sms, &p.sched);   // never needs more slots than the full schedule
        if (rc != HASS_OK) return rc;
        if (p.sched.total_slots > L.slot_cap) return HASS_ERR_WORKSPACE;
        p.row_tiles0 = RT;
        p.topk_row_tiles = 0;
        rc = make_tmap(&p.tmA0, H_d, N, d, d, BK, BM);
        if (rc == HASS_OK) rc = make_tmap(&p.tmA1, H_d, N, d, d, BK, BM);
    }
    if (rc == HASS_OK) rc = make_tmap(&p.tmB, W, V, d, d, BK, BN);
    if (rc != HASS_OK) return rc;
    log_schedule(with_target ? "fwd stats" : "fwd stats (draft)", p.sched);
    p.spill_begin = INT_MAX;
    p.a_row_offset = 0;
    p.row_global_offset = 0;
    p.rows_valid = static_cast<int>(N);
    p.n_cols = static_cast<int>(V);
    p.col_tiles = CT;
    p.k_blocks = ceil_div(d, BK);
    p.K = K;
    p.cap = topk_cap(K);
    p.part_m = reinterpret_cast<float*>(ws + L.part_m);
    p.part_s = reinterpret_cast<float*>(ws + L.part_s);
    p.cand = reinterpret_cast<uint2*>(ws + L.cand_v);
    p.cand_n = reinterpret_cast<int*>(ws + L.cand_i);
    p.status = reinterpret_cast<unsigned int*>(ws + L.status);
    p.only_if_range = only_if_range;
    p.thr_share = reinterpret_cast<float*>(ws + L.thr_share);
    if (cudaMemsetAsync(p.thr_share, 0xff, static_cast<size_t>(p.sched.total_slots) * BM * 4, st) != cudaSuccess) {   // NaN
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    rc = launch_gemm<MODE_STATS>(p, st);
    if (rc != HASS_OK) return rc;

    FinalizeParams f;
    std::memset(&f, 0, sizeof(f));
    f.sched = p.sched;
    f.row_begin = 0;
    f.rows = static_cast<int>(N);
    f.d = static_cast<int>(d);
    f.K = K;
    f.cap = topk_cap(K);
    f.row_tiles_t = with_target ? RT : 0;
    f.part_m = p.part_m;
    f.part_s = p.part_s;
    f.cand = p.cand;
    f.cand_n = p.cand_n;
    f.H_d = static_cast<const __nv_bfloat16*>(H_d);
    f.W = static_cast<const __nv_bfloat16*>(W);
    f.idx_in = idx_in;
    f.q_in = q_in;
    f.loss = loss;
    f.idx_out = idx_out;
    f.q_out = q_out;
    f.lse_t = lse_t;
    f.lse_d = lse_d;
    f.only_if_range = only_if_range;
    f.top_p = top_p;
    f.n_out = topk_n;
    const int warps_per_block = 8;
    {
        KernelTimer timer(only_if_range ? KIND_CONDITIONAL : KIND_FINALIZE, st);
        finalize_kernel<<<ceil_div(N, warps_per_block), warps_per_block * 32, 0, st>>>(f);
    }
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? HASS_OK : HASS_ERR_CUDA;
}

// ---- backward ---------------------------------------------------------------------------------
static int backward_impl(const void* H_d, const void* W, long long N, long long d, long long V, int K,
                         const int* topk_idx, const float* topk_q, const float* lse_d, const float* grad_loss,
                         void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes, cudaStream_t st,
                         bool clear_status, const unsigned int* only_if_range = nullptr) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_d || !W || !topk_idx || !topk_q || !lse_d || !dH_d) return HASS_ERR_INVALID_ARG;
    if (!aligned16(H_d) || !aligned16(W) || !aligned16(dH_d)) return HASS_ERR_INVALID_ARG;
    if (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;

    Layout L;
    rc = make_layout(N, d, V, K, di.sms, &L, nullptr);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.fixed_end + L.scratch_row_tile_bytes) return HASS_ERR_WORKSPACE;
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN), DT = ceil_div(d, BN);
    long long fit = static_cast<long long>((workspace_bytes - L.fixed_end) / L.scratch_row_tile_bytes);
    int chunk_tiles = L.pref_chunk_tiles;
    if (fit < chunk_tiles) chunk_tiles = static_cast<int>(fit);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* sidx = reinterpret_cast<int*>(ws + L.sidx);
    float* sgq = reinterpret_cast<float*>(ws + L.sgq);
    float* coef = reinterpret_cast<float*>(ws + L.coef);
    float* lse2 = reinterpret_cast<float*>(ws + L.lse2);
    __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(ws + L.scratch);
    if (clear_status && cudaMemsetAsync(ws + L.status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }

    {
        KernelTimer timer(only_if_range ? KIND_CONDITIONAL : KIND_PREP, st);
        bwd_prep_kernel<<<ceil_div(N, PREP_WARPS), PREP_WARPS * 32, 0, st>>>(static_cast<int>(N), K, topk_idx, topk_q, lse_d, grad_loss,
                                                           sidx, sgq, coef, lse2, only_if_range);
    }
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;

    CUtensorMap tmHd, tmWk, tmWn, tmP;
    rc = make_tmap(&tmHd, H_d, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = make_tmap(&tmWk, W, V, d, d, BK, BN);      // B of z_d = H_d W^T: K-major
    if (rc == HASS_OK) rc = make_tmap(&tmWn, W, V, d, d, 64, BK);      // B of dH_d = dz_d W: MN-major boxes
    if (rc == HASS_OK) rc = make_tmap(&tmP, P, static_cast<long long>(chunk_tiles) * BM, V, L.p_pitch, BK, BM);
    if (rc != HASS_OK) return rc;

    for (int t0 = 0; t0 < RT; t0 += chunk_tiles) {
        const int tiles = (RT - t0 < chunk_tiles) ? RT - t0 : chunk_tiles;
        // (1) dz_d tiles of this chunk of rows -> scratch
        GemmParams p;
        std::memset(&p, 0, sizeof(p));
        rc = plan_schedule(tiles, CT, di.sms, &p.sched);
        if (rc != HASS_OK) return rc;
        log_schedule("bwd dz_d", p.sched);
        p.tmA0 = tmHd;
        p.tmA1 = tmHd;
        p.tmB = tmWk;
        p.row_tiles0 = tiles;
        p.a_row_offset = t0 * BM;
        p.row_global_offset = t0 * BM;
        p.rows_valid = static_cast<int>(N);
        p.n_cols = static_cast<int>(V);
        p.col_tiles = CT;
        p.k_blocks = ceil_div(d, BK);
        p.K = K;
        p.lse2 = lse2;
        p.coef = coef;
        p.sidx = sidx;
        p.sgq = sgq;
        p.P = P;
        p.p_pitch = L.p_pitch;
        p.status = reinterpret_cast<unsigned int*>(ws + L.status);
        p.only_if_range = only_if_range;
        rc = launch_gemm<MODE_PROBS>(p, st);
        if (rc != HASS_OK) return rc;
        // (2) dH_d rows of this chunk = dz_d chunk x W
        GemmParams o;
        std::memset(&o, 0, sizeof(o));
        rc = plan_schedule(tiles, DT, di.sms, &o.sched);
        if (rc != HASS_OK) return rc;
        log_schedule("bwd dH_d", o.sched);
        o.tmA0 = tmP;
        o.tmA1 = tmP;
        o.tmB = tmWn;
        o.row_tiles0 = tiles;
        o.a_row_offset = 0;
        o.row_global_offset = t0 * BM;
        o.rows_valid = static_cast<int>(N);
        o.n_cols = static_cast<int>(d);
        o.col_tiles = DT;
        o.k_blocks = ceil_div(V, BK);
        o.K = K;
        o.out = dH_d;
        o.out_fp32 = dH_dtype == HASS_FP32 ? 1 : 0;
        o.out_align32 = ((reinterpret_cast<uintptr_t>(dH_d) | static_cast<uintptr_t>(d * (dH_dtype == HASS_FP32 ? 4 : 2))) & 31u) == 0 ? 1 : 0;
        o.out_pitch = d;
        o.status = p.status;
        o.only_if_range = only_if_range;
        rc = launch_gemm<MODE_OUT>(o, st);
        if (rc != HASS_OK) return rc;
    }
    return HASS_OK;
}

// ---- fused forward + backward with one sweep over target and draft rows ----------------------------
// The route of the combined objective and of the Bi-directional variant (the plain Top-K call, its _draft form
// and Top-P use fused2_impl below). Per chunk of row tiles: (1) one sweep computes the logits of the chunk's target and draft rows,
// their statistics and Top-K candidates, and spills the draft tiles as 2^(z log2e - ref2) in bf16;
// (2) finalize gives loss, Omega_hat, lse and the per-row scale of the spilled tiles; (3) the second
// GEMM contracts the spilled tiles with W and applies scale and sparse term in its epilogue. No
// logit is computed twice. with_target = false: Omega_hat is an input (aligning steps >= 2).
// Extra buffers and outputs of the combined objective CE(q, p) + w * Top-K (nullptr: Top-K loss alone).
struct Combined {
    float w;               // weight of the Top-K term
    float* loss_ce;        // [N] out: full-vocabulary cross-entropy per row
    float* coef_t;         // [N] scratch: scale of the target spill
    float* T;              // [chunk rows, d] scratch: q W of the chunk's rows
    __nv_bfloat16* Pt;     // [chunk rows, p_pitch] scratch: spill of the target tiles
};

static int fused_impl(bool with_target, const void* H_t, const void* H_d, const void* W, long long N, long long d,
                      long long V, int K, const float* grad_loss, const int* idx_in, const float* q_in, float* loss,
                      int* idx_out, float* q_out, float* lse_t, float* lse_d, void* dH_d, int dH_dtype,
                      void* workspace, size_t workspace_bytes, cudaStream_t st, const Combined* cmb = nullptr,
                      int* topk_n = nullptr, bool bidir = false) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_d || !W || !loss || !lse_d || !dH_d || !aligned16(H_d) || !aligned16(W) || !aligned16(dH_d))
        return HASS_ERR_INVALID_ARG;
    if (with_target && (!H_t || !idx_out || !q_out || !lse_t || !aligned16(H_t))) return HASS_ERR_INVALID_ARG;
    if (!with_target && (!idx_in || !q_in)) return HASS_ERR_INVALID_ARG;
    if (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32) return HASS_ERR_INVALID_ARG;
    if (bidir && (!with_target || 2 * K > K_CAP)) return HASS_ERR_UNSUPPORTED;   // the union holds up to 2K tokens
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    Layout L;
    rc = make_layout(N, d, V, K, di.sms, &L, nullptr);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.fixed_end + L.scratch_row_tile_bytes) return HASS_ERR_WORKSPACE;
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN), DT = ceil_div(d, BN);
    long long fit = static_cast<long long>((workspace_bytes - L.fixed_end) / L.scratch_row_tile_bytes);
    int chunk_tiles = L.pref_chunk_tiles;
    if (fit < chunk_tiles) chunk_tiles = static_cast<int>(fit);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* gq = bidir ? nullptr : reinterpret_cast<float*>(ws + L.sgq);    // [N, K]: too small for the 2K-token union
    float* coef = reinterpret_cast<float*>(ws + L.coef);
    float* sparse = reinterpret_cast<float*>(ws + L.sparse);
    __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(ws + L.scratch);
    unsigned int* status = reinterpret_cast<unsigned int*>(ws + L.status);
    if (cudaMemsetAsync(status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    CUtensorMap tmHt, tmHd, tmWk, tmWn, tmP;
    rc = make_tmap(&tmHd, H_d, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = with_target ? make_tmap(&tmHt, H_t, N, d, d, BK, BM) : make_tmap(&tmHt, H_d, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = make_tmap(&tmWk, W, V, d, d, BK, BN);
    if (rc == HASS_OK) rc = make_tmap(&tmWn, W, V, d, d, 64, BK);
    if (rc == HASS_OK) rc = make_tmap(&tmP, P, static_cast<long long>(chunk_tiles) * BM, V, L.p_pitch, BK, BM);
    CUtensorMap tmPt;
    if (rc == HASS_OK && cmb) rc = make_tmap(&tmPt, cmb->Pt, static_cast<long long>(chunk_tiles) * BM, V, L.p_pitch, BK, BM);
    if (rc != HASS_OK) return rc;

    // Every spilling row records its largest logit. If the sweep reports a row beyond the exponent range of its spill
    // (reference from column tile 0), the same sequence runs a second time as conditional launches with each row's
    // reference taken from that record, which no logit of the row can exceed.
    unsigned int* zmax = reinterpret_cast<unsigned int*>(ws + L.zmax);
    if (cudaMemsetAsync(zmax, 0, static_cast<size_t>(2 * RT) * BM * 4, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    auto run = [&](bool retry) -> int {
    const unsigned int* gate = retry ? status : nullptr;
    for (int t0 = 0; t0 < RT; t0 += chunk_tiles) {
        const int tiles = (RT - t0 < chunk_tiles) ? RT - t0 : chunk_tiles;
        const int rows = static_cast<int>((N - static_cast<long long>(t0) * BM < static_cast<long long>(tiles) * BM)
                                              ? N - static_cast<long long>(t0) * BM
                                              : static_cast<long long>(tiles) * BM);
        // (1) logits sweep with statistics, candidates and spill
        GemmParams p;
        std::memset(&p, 0, sizeof(p));
        rc = plan_schedule(with_target ? 2 * tiles : tiles, CT, di.sms, &p.sched);
        if (rc != HASS_OK) return rc;
        if (p.sched.total_slots > L.slot_cap) return HASS_ERR_WORKSPACE;
        log_schedule("fused stats", p.sched);
        p.tmA0 = tmHt;
        p.tmA1 = tmHd;
        p.tmB = tmWk;
        p.row_tiles0 = tiles;
        p.topk_row_tiles = with_target ? (bidir ? 2 * tiles : tiles) : 0;
        p.spill_begin = with_target ? tiles : 0;
        p.a_row_offset = t0 * BM;
        p.row_global_offset = t0 * BM;
        p.rows_valid = static_cast<int>(N);
        p.n_cols = static_cast<int>(V);
        p.col_tiles = CT;
        p.k_blocks = ceil_div(d, BK);
        p.K = K;
        p.cap = topk_cap(K);
        p.part_m = reinterpret_cast<float*>(ws + L.part_m);
        p.part_s = reinterpret_cast<float*>(ws + L.part_s);
        p.cand = reinterpret_cast<uint2*>(ws + L.cand_v);
        p.cand_n = reinterpret_cast<int*>(ws + L.cand_i);
        p.P = P;
        p.Pt = cmb ? cmb->Pt : nullptr;
        p.p_pitch = L.p_pitch;
        p.status = status;
        p.thr_share = reinterpret_cast<float*>(ws + L.thr_share);
        p.row_zmax = zmax + static_cast<size_t>(with_target ? 2 : 1) * t0 * BM;
        p.use_row_zmax = retry ? 1 : 0;
        p.only_if_range = gate;
    if (cudaMemsetAsync(p.thr_share, 0xff, static_cast<size_t>(p.sched.total_slots) * BM * 4, st) != cudaSuccess) {   // NaN
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    rc = launch_gemm<MODE_STATS>(p, st);
        if (rc != HASS_OK) return rc;
        // (2) statistics -> loss, Omega_hat, per-row scale
        FinalizeParams f;
        std::memset(&f, 0, sizeof(f));
        f.sched = p.sched;
        f.d = static_cast<int>(d);
        f.K = K;
        f.cap = topk_cap(K);
        f.row_begin = t0 * BM;
        f.rows = rows;
        f.row_tiles_t = with_target ? tiles : 0;
        f.part_m = p.part_m;
        f.part_s = p.part_s;
        f.cand = p.cand;
        f.cand_n = p.cand_n;
        f.H_d = static_cast<const __nv_bfloat16*>(H_d);
        f.W = static_cast<const __nv_bfloat16*>(W);
        f.idx_in = idx_in;
        f.q_in = q_in;
        f.loss = loss;
        f.idx_out = idx_out;
        f.q_out = q_out;
        f.lse_t = lse_t;
        f.lse_d = lse_d;
        f.grad_loss = grad_loss;
        f.coef_out = coef;
        f.gq_out = gq;
        f.sparse_out = sparse;
        f.n_out = topk_n;
        f.bidir = bidir ? 1 : 0;
        f.H_t = static_cast<const __nv_bfloat16*>(H_t);
        f.w_topk = cmb ? cmb->w : 1.f;
        f.coef_t_out = cmb ? cmb->coef_t : nullptr;
        f.Pt = cmb ? cmb->Pt : nullptr;
        f.p_pitch = L.p_pitch;
        f.ce_corr_out = reinterpret_cast<float*>(ws + L.lse2);    // [N] floats, otherwise used by the split backward
        f.only_if_range = gate;
        {
            KernelTimer timer(retry ? KIND_CONDITIONAL : KIND_FINALIZE, st);
            finalize_kernel<<<ceil_div(rows, 8), 256, 0, st>>>(f);
        }
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
        // (3) dH_d rows of the chunk
        GemmParams o;
        std::memset(&o, 0, sizeof(o));
        rc = plan_schedule(tiles, DT, di.sms, &o.sched);
        if (rc != HASS_OK) return rc;
        log_schedule("fused dH_d", o.sched);
        if (cmb) {
            // (2b) q W of the chunk's rows from the target spill, then the cross-entropy and its gradient term
            GemmParams t = o;
            t.tmA0 = tmPt;
            t.tmA1 = tmPt;
            t.tmB = tmWn;
            t.row_tiles0 = tiles;
            t.spill_begin = INT_MAX;
            t.row_global_offset = 0;
            t.rows_valid = rows;
            t.n_cols = static_cast<int>(d);
            t.col_tiles = DT;
            t.k_blocks = ceil_div(V, BK);
            t.K = K;
            t.coef = cmb->coef_t + static_cast<long long>(t0) * BM;
            t.out = cmb->T;
            t.out_fp32 = 1;
            t.out_align32 = 1;
            t.out_pitch = d;
            t.status = status;
            t.only_if_range = gate;
            rc = launch_gemm<MODE_OUT>(t, st);
            if (rc != HASS_OK) return rc;
            {
                KernelTimer timer(retry ? KIND_CONDITIONAL : KIND_FINALIZE, st);
                ce_kernel<<<ceil_div(rows, 8), 256, 0, st>>>(rows, t0 * BM, static_cast<int>(d),
                                                             static_cast<const __nv_bfloat16*>(H_d), cmb->T, lse_d, grad_loss,
                                                             reinterpret_cast<const float*>(ws + L.lse2), cmb->loss_ce, sparse, gate);
            }
            g_launches.fetch_add(1);
            if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
        }
        o.tmA0 = tmP;
        o.tmA1 = tmP;
        o.tmB = tmWn;
        o.row_tiles0 = tiles;
        o.spill_begin = INT_MAX;
        o.a_row_offset = 0;
        o.row_global_offset = t0 * BM;
        o.rows_valid = static_cast<int>(N);
        o.n_cols = static_cast<int>(d);
        o.col_tiles = DT;
        o.k_blocks = ceil_div(V, BK);
        o.K = K;
        o.coef = coef;
        o.sparse = sparse;
        o.out = dH_d;
        o.out_fp32 = dH_dtype == HASS_FP32 ? 1 : 0;
        o.out_align32 = ((reinterpret_cast<uintptr_t>(dH_d) | static_cast<uintptr_t>(d * (dH_dtype == HASS_FP32 ? 4 : 2))) & 31u) == 0 ? 1 : 0;
        o.out_pitch = d;
        o.status = status;
        o.only_if_range = gate;
        rc = launch_gemm<MODE_OUT>(o, st);
        if (rc != HASS_OK) return rc;
    }
    return HASS_OK;
    };
    rc = run(false);
    if (rc != HASS_OK) return rc;
    rc = run(true);
    if (rc != HASS_OK) return rc;
    {
        KernelTimer timer(KIND_CONDITIONAL, st);
        range_handled_kernel<<<1, 1, 0, st>>>(status);
    }
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
    return HASS_OK;
}

// ---- fused forward + backward, Omega_hat known before the draft rows are swept -------------------------
// The route of hass_topk_distill_fwd_bwd, its _draft form and the Top-P variant. Per chunk of row tiles:
// (1) sweep of the chunk's TARGET rows: statistics and Top-K candidates; (2) select_kernel: lse_t, Omega_hat,
// and the same set sorted by token id; (3) sweep of the chunk's DRAFT rows: statistics, the bf16 spill of
// 2^(z_d log2e - ref2), and z_d at the row's Omega_hat copied out of the accumulator as the sweep passes those
// columns; (4) loss_patch_kernel: lse_d, Eq. 1, the per-row scale, and the Omega_hat term of dz_d subtracted
// from the K spilled entries it concerns; (5) the second GEMM with the row scale in its epilogue. No logit
// is computed twice and no row of W is gathered, so the cost does not depend on K beyond the candidate
// handling of (1). with_target = false: (1) is skipped and (2) only sorts the given Omega_hat.
// Hand-over between two copy streams and the compute stream, used by the host-buffer entry: the rows of a chunk
// are copied to the device while the previous chunk computes, and a chunk's dH_d rows go back to the host while
// the next chunk computes. H_t / H_d / dH_d of fused2_impl are then the device staging buffers.
struct ChunkPipe {
    cudaStream_t h2d, d2h;
    const uint8_t* Ht_host;
    const uint8_t* Hd_host;
    uint8_t* dH_host;
    size_t in_row_bytes, out_row_bytes;
    cudaEvent_t* events;       // pool
    int n_events, used;
    cudaEvent_t next() { return used < n_events ? events[used++] : nullptr; }
};

static int fused2_impl(bool with_target, const void* H_t, const void* H_d, const void* W, long long N, long long d,
                       long long V, int K, const float* grad_loss, const int* idx_in, const float* q_in, float* loss,
                       int* idx_out, float* q_out, float* lse_t, float* lse_d, void* dH_d, int dH_dtype,
                       void* workspace, size_t workspace_bytes, cudaStream_t st, float top_p = 0.f,
                       int* topk_n = nullptr, ChunkPipe* pipe = nullptr) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_d || !W || !loss || !lse_d || !dH_d || !aligned16(H_d) || !aligned16(W) || !aligned16(dH_d))
        return HASS_ERR_INVALID_ARG;
    if (with_target && (!H_t || !idx_out || !q_out || !lse_t || !aligned16(H_t))) return HASS_ERR_INVALID_ARG;
    if (!with_target && (!idx_in || !q_in)) return HASS_ERR_INVALID_ARG;
    if (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    Layout L;
    rc = make_layout(N, d, V, K, di.sms, &L, nullptr);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.fixed_end + L.scratch_row_tile_bytes) return HASS_ERR_WORKSPACE;
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN), DT = ceil_div(d, BN);
    long long fit = static_cast<long long>((workspace_bytes - L.fixed_end) / L.scratch_row_tile_bytes);
    int chunk_tiles = L.pref_chunk_tiles;
    if (fit < chunk_tiles) chunk_tiles = static_cast<int>(fit);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* sidx = reinterpret_cast<int*>(ws + L.sidx);
    float* sq = reinterpret_cast<float*>(ws + L.sgq);
    float* coef = reinterpret_cast<float*>(ws + L.coef);
    float* capz = reinterpret_cast<float*>(ws + L.capz);
    __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(ws + L.scratch);
    unsigned int* status = reinterpret_cast<unsigned int*>(ws + L.status);
    if (cudaMemsetAsync(status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    CUtensorMap tmHt, tmHd, tmWk, tmWn, tmP;
    rc = make_tmap(&tmHd, H_d, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = with_target ? make_tmap(&tmHt, H_t, N, d, d, BK, BM) : make_tmap(&tmHt, H_d, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = make_tmap(&tmWk, W, V, d, d, BK, BN);
    if (rc == HASS_OK) rc = make_tmap(&tmWn, W, V, d, d, 64, BK);
    if (rc == HASS_OK) rc = make_tmap(&tmP, P, static_cast<long long>(chunk_tiles) * BM, V, L.p_pitch, BK, BM);
    // the same buffer as the draft sweep's TMA stores see it: boxes of 64 columns x 32 rows, every column up to the pitch
    CUtensorMap tmPst;
    if (rc == HASS_OK) rc = make_tmap(&tmPst, P, static_cast<long long>(chunk_tiles) * BM, L.p_pitch, L.p_pitch, 64, 32);
    if (rc != HASS_OK) return rc;

    for (int t0 = 0; t0 < RT; t0 += chunk_tiles) {
        const int tiles = (RT - t0 < chunk_tiles) ? RT - t0 : chunk_tiles;
        const int rows = static_cast<int>((N - static_cast<long long>(t0) * BM < static_cast<long long>(tiles) * BM)
                                              ? N - static_cast<long long>(t0) * BM
                                              : static_cast<long long>(tiles) * BM);
        // both sweeps cover `tiles` row tiles and share one schedule
        GemmParams p;
        std::memset(&p, 0, sizeof(p));
        rc = plan_schedule(tiles, CT, di.sms, &p.sched);
        if (rc != HASS_OK) return rc;
        if (p.sched.total_slots > L.slot_cap) return HASS_ERR_WORKSPACE;
        log_schedule("fused sweep (target / draft)", p.sched);
        p.tmB = tmWk;
        p.row_tiles0 = tiles;
        p.a_row_offset = t0 * BM;
        p.row_global_offset = t0 * BM;
        p.rows_valid = static_cast<int>(N);
        p.n_cols = static_cast<int>(V);
        p.col_tiles = CT;
        p.k_blocks = ceil_div(d, BK);
        p.K = K;
        p.cap = topk_cap(K);
        p.part_m = reinterpret_cast<float*>(ws + L.part_m);
        p.part_s = reinterpret_cast<float*>(ws + L.part_s);
        p.cand = reinterpret_cast<uint2*>(ws + L.cand_v);
        p.cand_n = reinterpret_cast<int*>(ws + L.cand_i);
        p.p_pitch = L.p_pitch;
        p.status = status;
        cudaEvent_t ev_d = nullptr;
        if (pipe) {
            // this chunk's rows of H_t, then of H_d, on the inbound copy stream; the sweeps wait for them
            const size_t off = static_cast<size_t>(t0) * BM * pipe->in_row_bytes, bytes = static_cast<size_t>(rows) * pipe->in_row_bytes;
            cudaEvent_t ev_t = pipe->next();
            ev_d = pipe->next();
            if (!ev_t || !ev_d) return HASS_ERR_UNSUPPORTED;
            bool ok = cudaMemcpyAsync(const_cast<uint8_t*>(static_cast<const uint8_t*>(H_t)) + off, pipe->Ht_host + off, bytes,
                                      cudaMemcpyHostToDevice, pipe->h2d) == cudaSuccess;
            ok = ok && cudaEventRecord(ev_t, pipe->h2d) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(const_cast<uint8_t*>(static_cast<const uint8_t*>(H_d)) + off, pipe->Hd_host + off, bytes,
                                       cudaMemcpyHostToDevice, pipe->h2d) == cudaSuccess;
            ok = ok && cudaEventRecord(ev_d, pipe->h2d) == cudaSuccess;
            ok = ok && cudaStreamWaitEvent(st, ev_t, 0) == cudaSuccess;
            if (!ok) {
                cudaGetLastError();
                return HASS_ERR_CUDA;
            }
        }
        if (with_target) {
            // (1) target rows: statistics + candidates
            GemmParams t = p;
            t.tmA0 = tmHt;
            t.tmA1 = tmHt;
            t.topk_row_tiles = tiles;
            t.spill_begin = INT_MAX;
            t.thr_share = reinterpret_cast<float*>(ws + L.thr_share);
            if (cudaMemsetAsync(t.thr_share, 0xff, static_cast<size_t>(t.sched.total_slots) * BM * 4, st) != cudaSuccess) {   // NaN
                cudaGetLastError();
                return HASS_ERR_CUDA;
            }
            rc = launch_gemm<MODE_STATS>(t, st);
            if (rc != HASS_OK) return rc;
        }
        // (2) Omega_hat of the chunk's rows
        SelectParams sp;
        std::memset(&sp, 0, sizeof(sp));
        sp.sched = p.sched;
        sp.K = K;
        sp.cap = p.cap;
        sp.row_begin = t0 * BM;
        sp.rows = rows;
        sp.from_sweep = with_target ? 1 : 0;
        sp.part_m = p.part_m;
        sp.part_s = p.part_s;
        sp.cand = p.cand;
        sp.cand_n = p.cand_n;
        sp.idx_in = idx_in;
        sp.q_in = q_in;
        sp.idx_out = idx_out;
        sp.q_out = q_out;
        sp.lse_t = lse_t;
        sp.n_out = topk_n;
        sp.top_p = top_p;
        sp.sidx = sidx;
        sp.sq = sq;
        {
            KernelTimer timer(KIND_FINALIZE, st);
            select_kernel<<<ceil_div(rows, SEL_WARPS), SEL_WARPS * 32, 0, st>>>(sp);
        }
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
        // (3) draft rows: statistics, spill, z_d at Omega_hat
        if (pipe && cudaStreamWaitEvent(st, ev_d, 0) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        {
            GemmParams q = p;
            q.tmA0 = tmHd;
            q.tmA1 = tmHd;
            q.topk_row_tiles = 0;
            q.spill_begin = 0;
            q.sidx = sidx;
            q.cap_z = capz;
            q.P = P;
            q.tmSpill = tmPst;
            rc = launch_gemm<MODE_STATS>(q, st, KIND_STATS_DRAFT);
            if (rc != HASS_OK) return rc;
        }
        // (4) lse_d, loss, row scale, Omega_hat term into the spill
        LossPatchParams lp;
        std::memset(&lp, 0, sizeof(lp));
        lp.sched = p.sched;
        lp.K = K;
        lp.row_begin = t0 * BM;
        lp.rows = rows;
        lp.part_m = p.part_m;
        lp.part_s = p.part_s;
        lp.sidx = sidx;
        lp.sq = sq;
        lp.cap_z = capz;
        lp.grad_loss = grad_loss;
        lp.loss = loss;
        lp.lse_d = lse_d;
        lp.coef_out = coef;
        lp.P = P;
        lp.p_pitch = L.p_pitch;
        {
            KernelTimer timer(KIND_FINALIZE, st);
            loss_patch_kernel<<<ceil_div(rows, 8), 256, 0, st>>>(lp);
        }
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
        // (5) dH_d rows of the chunk = row scale x (patched spill x W)
        GemmParams o;
        std::memset(&o, 0, sizeof(o));
        rc = plan_schedule(tiles, DT, di.sms, &o.sched);
        if (rc != HASS_OK) return rc;
        log_schedule("fused dH_d", o.sched);
        o.tmA0 = tmP;
        o.tmA1 = tmP;
        o.tmB = tmWn;
        o.row_tiles0 = tiles;
        o.spill_begin = INT_MAX;
        o.a_row_offset = 0;
        o.row_global_offset = t0 * BM;
        o.rows_valid = static_cast<int>(N);
        o.n_cols = static_cast<int>(d);
        o.col_tiles = DT;
        o.k_blocks = ceil_div(V, BK);
        o.K = K;
        o.coef = coef;
        o.out = dH_d;
        o.out_fp32 = dH_dtype == HASS_FP32 ? 1 : 0;
        o.out_align32 = ((reinterpret_cast<uintptr_t>(dH_d) | static_cast<uintptr_t>(d * (dH_dtype == HASS_FP32 ? 4 : 2))) & 31u) == 0 ? 1 : 0;
        o.out_pitch = d;
        o.status = status;
        rc = launch_gemm<MODE_OUT>(o, st);
        if (rc != HASS_OK) return rc;
        if (pipe) {
            // the chunk's dH_d rows on the outbound copy stream
            const size_t off = static_cast<size_t>(t0) * BM * pipe->out_row_bytes, bytes = static_cast<size_t>(rows) * pipe->out_row_bytes;
            cudaEvent_t ev_o = pipe->next();
            if (!ev_o) return HASS_ERR_UNSUPPORTED;
            bool ok = cudaEventRecord(ev_o, st) == cudaSuccess;
            ok = ok && cudaStreamWaitEvent(pipe->d2h, ev_o, 0) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(pipe->dH_host + off, static_cast<const uint8_t*>(dH_d) + off, bytes, cudaMemcpyDeviceToHost,
                                       pipe->d2h) == cudaSuccess;
            if (!ok) {
                cudaGetLastError();
                return HASS_ERR_CUDA;
            }
        }
    }
    {
        // Exact route, enqueued behind every call of this route: if a sweep reported a row beyond its exponent
        // range, the separate forward and the recomputing backward (which have no such limit) redo the call
        // and the report is withdrawn; otherwise each of these launches returns at once.
        rc = forward_impl(with_target, H_t, H_d, W, N, d, V, K, idx_in, q_in, loss, idx_out, q_out, lse_t, lse_d,
                          workspace, workspace_bytes, st, status, top_p, topk_n);
        if (rc != HASS_OK) return rc;
        rc = backward_impl(H_d, W, N, d, V, K, with_target ? idx_out : idx_in, with_target ? q_out : q_in, lse_d,
                           grad_loss, dH_d, dH_dtype, workspace, workspace_bytes, st, false, status);
        if (rc != HASS_OK) return rc;
        {
            KernelTimer timer(KIND_CONDITIONAL, st);
            range_handled_kernel<<<1, 1, 0, st>>>(status);
        }
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
    }
    return HASS_OK;
}

// ---- forward alone, Omega_hat known before the draft rows are swept -----------------------------------
// hass_topk_distill_fwd and hass_topk_distill_fwd_draft: the sweep of the target rows (statistics, candidates),
// select_kernel, the sweep of the draft rows (statistics and z_d at the row's Omega_hat, copied out of the
// accumulator) and loss_patch_kernel (lse_d, Eq. 1). Nothing is spilled and no row of W is gathered. Needs the
// [N, K] lists of the workspace beyond the statistics; with a workspace that ends before them the older
// single-sweep forward (forward_impl) runs instead.
static int forward2_impl(bool with_target, const void* H_t, const void* H_d, const void* W, long long N, long long d,
                         long long V, int K, const int* idx_in, const float* q_in, float* loss, int* idx_out,
                         float* q_out, float* lse_t, float* lse_d, void* workspace, size_t workspace_bytes,
                         cudaStream_t st) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_d || !W || !loss || !lse_d || !aligned16(H_d) || !aligned16(W)) return HASS_ERR_INVALID_ARG;
    if (with_target && (!H_t || !idx_out || !q_out || !lse_t || !aligned16(H_t))) return HASS_ERR_INVALID_ARG;
    if (!with_target && (!idx_in || !q_in)) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    Layout L;
    rc = make_layout(N, d, V, K, di.sms, &L, nullptr);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.sparse)
        return forward_impl(with_target, H_t, H_d, W, N, d, V, K, idx_in, q_in, loss, idx_out, q_out, lse_t, lse_d,
                            workspace, workspace_bytes, st);
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws + L.status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    rc = plan_schedule(RT, CT, di.sms, &p.sched);
    if (rc != HASS_OK) return rc;
    if (p.sched.total_slots > L.slot_cap) return HASS_ERR_WORKSPACE;
    log_schedule("fwd sweep (target / draft)", p.sched);
    rc = make_tmap(&p.tmB, W, V, d, d, BK, BN);
    if (rc != HASS_OK) return rc;
    p.row_tiles0 = RT;
    p.spill_begin = INT_MAX;
    p.rows_valid = static_cast<int>(N);
    p.n_cols = static_cast<int>(V);
    p.col_tiles = CT;
    p.k_blocks = ceil_div(d, BK);
    p.K = K;
    p.cap = topk_cap(K);
    p.part_m = reinterpret_cast<float*>(ws + L.part_m);
    p.part_s = reinterpret_cast<float*>(ws + L.part_s);
    p.cand = reinterpret_cast<uint2*>(ws + L.cand_v);
    p.cand_n = reinterpret_cast<int*>(ws + L.cand_i);
    p.status = reinterpret_cast<unsigned int*>(ws + L.status);
    int* sidx = reinterpret_cast<int*>(ws + L.sidx);
    float* sq = reinterpret_cast<float*>(ws + L.sgq);
    float* capz = reinterpret_cast<float*>(ws + L.capz);
    if (with_target) {
        GemmParams t = p;
        rc = make_tmap(&t.tmA0, H_t, N, d, d, BK, BM);
        if (rc != HASS_OK) return rc;
        t.tmA1 = t.tmA0;
        t.topk_row_tiles = RT;
        t.thr_share = reinterpret_cast<float*>(ws + L.thr_share);
        if (cudaMemsetAsync(t.thr_share, 0xff, static_cast<size_t>(t.sched.total_slots) * BM * 4, st) != cudaSuccess) {   // NaN
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        rc = launch_gemm<MODE_STATS>(t, st);
        if (rc != HASS_OK) return rc;
    }
    SelectParams sp;
    std::memset(&sp, 0, sizeof(sp));
    sp.sched = p.sched;
    sp.K = K;
    sp.cap = p.cap;
    sp.row_begin = 0;
    sp.rows = static_cast<int>(N);
    sp.from_sweep = with_target ? 1 : 0;
    sp.part_m = p.part_m;
    sp.part_s = p.part_s;
    sp.cand = p.cand;
    sp.cand_n = p.cand_n;
    sp.idx_in = idx_in;
    sp.q_in = q_in;
    sp.idx_out = idx_out;
    sp.q_out = q_out;
    sp.lse_t = lse_t;
    sp.sidx = sidx;
    sp.sq = sq;
    {
        KernelTimer timer(KIND_FINALIZE, st);
        select_kernel<<<ceil_div(N, SEL_WARPS), SEL_WARPS * 32, 0, st>>>(sp);
    }
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
    {
        GemmParams q = p;
        rc = make_tmap(&q.tmA0, H_d, N, d, d, BK, BM);
        if (rc != HASS_OK) return rc;
        q.tmA1 = q.tmA0;
        q.topk_row_tiles = 0;
        q.sidx = sidx;
        q.cap_z = capz;
        rc = launch_gemm<MODE_STATS>(q, st, KIND_STATS_DRAFT);
        if (rc != HASS_OK) return rc;
    }
    LossPatchParams lp;
    std::memset(&lp, 0, sizeof(lp));
    lp.sched = p.sched;
    lp.K = K;
    lp.row_begin = 0;
    lp.rows = static_cast<int>(N);
    lp.part_m = p.part_m;
    lp.part_s = p.part_s;
    lp.sidx = sidx;
    lp.sq = sq;
    lp.cap_z = capz;
    lp.loss = loss;
    lp.lse_d = lse_d;
    {
        KernelTimer timer(KIND_FINALIZE, st);
        loss_patch_kernel<<<ceil_div(N, 8), 256, 0, st>>>(lp);
    }
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? HASS_OK : HASS_ERR_CUDA;
}

// ---- Normed Top-K variant -----------------------------------------------------------------------------
// Both distributions are renormalised over Omega_hat, so the loss and its gradient involve the draft
// logits on Omega_hat only: one sweep over the TARGET rows (statistics + Top-K), then finalize computes the
// K draft logits per row, the loss and the gradient row directly. No draft sweep, no second GEMM.
static int normed_impl(const void* H_t, const void* H_d, const void* W, long long N, long long d, long long V, int K,
                       const float* grad_loss, float* loss, int* idx_out, float* q_out, int* topk_n, float* lse_t,
                       void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_t || !H_d || !W || !loss || !idx_out || !q_out || !lse_t || !dH_d) return HASS_ERR_INVALID_ARG;
    if (!aligned16(H_t) || !aligned16(H_d) || !aligned16(W) || !aligned16(dH_d)) return HASS_ERR_INVALID_ARG;
    if (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    Layout L;
    rc = make_layout(N, d, V, K, di.sms, &L, nullptr);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < L.fwd_end) return HASS_ERR_WORKSPACE;
    const int RT = ceil_div(N, BM), CT = ceil_div(V, BN);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws + L.status, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    rc = plan_schedule(RT, CT, di.sms, &p.sched);
    if (rc != HASS_OK) return rc;
    if (p.sched.total_slots > L.slot_cap) return HASS_ERR_WORKSPACE;
    log_schedule("normed stats (target)", p.sched);
    rc = make_tmap(&p.tmA0, H_t, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = make_tmap(&p.tmA1, H_t, N, d, d, BK, BM);
    if (rc == HASS_OK) rc = make_tmap(&p.tmB, W, V, d, d, BK, BN);
    if (rc != HASS_OK) return rc;
    p.row_tiles0 = RT;
    p.topk_row_tiles = RT;
    p.spill_begin = INT_MAX;
    p.rows_valid = static_cast<int>(N);
    p.n_cols = static_cast<int>(V);
    p.col_tiles = CT;
    p.k_blocks = ceil_div(d, BK);
    p.K = K;
    p.cap = topk_cap(K);
    p.part_m = reinterpret_cast<float*>(ws + L.part_m);
    p.part_s = reinterpret_cast<float*>(ws + L.part_s);
    p.cand = reinterpret_cast<uint2*>(ws + L.cand_v);
    p.cand_n = reinterpret_cast<int*>(ws + L.cand_i);
    p.status = reinterpret_cast<unsigned int*>(ws + L.status);
    p.thr_share = reinterpret_cast<float*>(ws + L.thr_share);
    if (cudaMemsetAsync(p.thr_share, 0xff, static_cast<size_t>(p.sched.total_slots) * BM * 4, st) != cudaSuccess) {   // NaN
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    rc = launch_gemm<MODE_STATS>(p, st);
    if (rc != HASS_OK) return rc;
    FinalizeParams f;
    std::memset(&f, 0, sizeof(f));
    f.sched = p.sched;
    f.d = static_cast<int>(d);
    f.K = K;
    f.cap = p.cap;
    f.row_begin = 0;
    f.rows = static_cast<int>(N);
    f.row_tiles_t = RT;
    f.part_m = p.part_m;
    f.part_s = p.part_s;
    f.cand = p.cand;
    f.cand_n = p.cand_n;
    f.H_d = static_cast<const __nv_bfloat16*>(H_d);
    f.W = static_cast<const __nv_bfloat16*>(W);
    f.loss = loss;
    f.idx_out = idx_out;
    f.q_out = q_out;
    f.lse_t = lse_t;
    f.grad_loss = grad_loss;
    f.n_out = topk_n;
    f.normed = 1;
    f.dH_out = dH_d;
    f.dH_fp32 = dH_dtype == HASS_FP32 ? 1 : 0;
    {
        KernelTimer timer(KIND_FINALIZE, st);
        finalize_kernel<<<ceil_div(N, 8), 256, 0, st>>>(f);
    }
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? HASS_OK : HASS_ERR_CUDA;
}

}  // namespace hass

using namespace hass;

extern "C" {

const char* hass_status_string(int status) {
    switch (status) {
        case HASS_OK: return "HASS_OK";
        case HASS_ERR_INVALID_ARG: return "HASS_ERR_INVALID_ARG";
        case HASS_ERR_UNSUPPORTED: return "HASS_ERR_UNSUPPORTED";
        case HASS_ERR_WORKSPACE: return "HASS_ERR_WORKSPACE";
        case HASS_ERR_CUDA: return "HASS_ERR_CUDA";
        case HASS_ERR_TIMEOUT: return "HASS_ERR_TIMEOUT";
        case HASS_ERR_ARCH: return "HASS_ERR_ARCH";
        case HASS_ERR_RANGE: return "HASS_ERR_RANGE";
        default: return "HASS_ERR_UNKNOWN";
    }
}

int hass_version(void) { return 10410; }

int64_t hass_kernel_launch_count(void) { return g_launches.load(); }

int hass_profile_enable(int on) {
    if (on && g_prof.ev.empty()) {
        g_prof.ev.resize(2 * kMaxRecords);
        g_prof.kind.resize(kMaxRecords);
        for (auto& e : g_prof.ev)
            if (cudaEventCreate(&e) != cudaSuccess) {
                cudaGetLastError();
                g_prof.ev.clear();
                return HASS_ERR_CUDA;
            }
    }
    g_prof.on = on != 0;
    g_prof.n = 0;
    return HASS_OK;
}

int hass_profile_summary(double* ms_by_kind, int64_t* launches_by_kind, int n_kinds) {
    if (!ms_by_kind || !launches_by_kind || n_kinds < NUM_KINDS) return HASS_ERR_INVALID_ARG;
    for (int k = 0; k < n_kinds; ++k) {
        ms_by_kind[k] = 0.0;
        launches_by_kind[k] = 0;
    }
    for (int r = 0; r < g_prof.n; ++r) {
        if (cudaEventSynchronize(g_prof.ev[2 * r + 1]) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_prof.ev[2 * r], g_prof.ev[2 * r + 1]) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        ms_by_kind[g_prof.kind[r]] += ms;
        launches_by_kind[g_prof.kind[r]] += 1;
    }
    g_prof.n = 0;
    return HASS_OK;
}

int hass_topk_distill_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes) {
    if (!bytes) return HASS_ERR_INVALID_ARG;
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    Layout L;
    rc = make_layout(N, d, V, K, sm_count_or_default(), &L, nullptr);
    if (rc != HASS_OK) return rc;
    *bytes = L.total_pref;
    return HASS_OK;
}

int hass_topk_distill_fwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d, int64_t V, int32_t K,
                          float* loss, int32_t* topk_idx, float* topk_q, float* lse_t, float* lse_d, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
    return forward2_impl(true, H_t, H_d, W, N, d, V, K, nullptr, nullptr, loss, topk_idx, topk_q, lse_t, lse_d,
                         workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int hass_topk_distill_fwd_draft(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V, int32_t K,
                                const int32_t* topk_idx, const float* topk_q, float* loss, float* lse_d,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return forward2_impl(false, nullptr, H_d, W, N, d, V, K, topk_idx, topk_q, loss, nullptr, nullptr, nullptr, lse_d,
                         workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int hass_topk_distill_bwd(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V, int32_t K,
                          const int32_t* topk_idx, const float* topk_q, const float* lse_d, const float* grad_loss,
                          void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_impl(H_d, W, N, d, V, K, topk_idx, topk_q, lse_d, grad_loss, dH_d, dH_dtype, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(cuda_stream), true);
}

int hass_topk_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                              int32_t K, const float* grad_loss, float* loss, int32_t* topk_idx, float* topk_q,
                              float* lse_t, float* lse_d, void* dH_d, int dH_dtype, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
    return fused2_impl(true, H_t, H_d, W, N, d, V, K, grad_loss, nullptr, nullptr, loss, topk_idx, topk_q, lse_t, lse_d,
                       dH_d, dH_dtype, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int hass_topk_distill_fwd_bwd_draft(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V, int32_t K,
                                    const int32_t* topk_idx, const float* topk_q, const float* grad_loss, float* loss,
                                    float* lse_d, void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
    return fused2_impl(false, nullptr, H_d, W, N, d, V, K, grad_loss, topk_idx, topk_q, loss, nullptr, nullptr, nullptr,
                       lse_d, dH_d, dH_dtype, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int hass_variant_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                                 int32_t K, int variant, float param, const float* grad_loss, float* loss,
                                 int32_t* topk_idx, float* topk_q, int32_t* topk_n, float* lse_t, float* lse_d,
                                 void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    switch (variant) {
        case HASS_LOSS_TOPK:
            return fused2_impl(true, H_t, H_d, W, N, d, V, K, grad_loss, nullptr, nullptr, loss, topk_idx, topk_q, lse_t,
                               lse_d, dH_d, dH_dtype, workspace, workspace_bytes, st, 0.f, topk_n);
        case HASS_LOSS_TOP_P:
            if (!(param > 0.f)) return HASS_ERR_INVALID_ARG;
            return fused2_impl(true, H_t, H_d, W, N, d, V, K, grad_loss, nullptr, nullptr, loss, topk_idx, topk_q, lse_t,
                               lse_d, dH_d, dH_dtype, workspace, workspace_bytes, st, param, topk_n);
        case HASS_LOSS_BIDIR_TOPK:
            return fused_impl(true, H_t, H_d, W, N, d, V, K, grad_loss, nullptr, nullptr, loss, topk_idx, topk_q, lse_t,
                              lse_d, dH_d, dH_dtype, workspace, workspace_bytes, st, nullptr, topk_n, true);
        case HASS_LOSS_NORMED_TOPK:
            return normed_impl(H_t, H_d, W, N, d, V, K, grad_loss, loss, topk_idx, topk_q, topk_n, lse_t, dH_d, dH_dtype,
                               workspace, workspace_bytes, st);
        default:
            return HASS_ERR_INVALID_ARG;
    }
}

// Buffers appended to the normal workspace by the combined-objective entry.
struct CombinedStage {
    size_t coef_t, T, Pt, total;
};
static int combined_stage(int64_t N, int64_t d, int64_t V, int32_t K, size_t base, CombinedStage* c) {
    Layout L;
    int rc = make_layout(N, d, V, K, sm_count_or_default(), &L, nullptr);
    if (rc != HASS_OK) return rc;
    size_t off = align256(base);
    c->coef_t = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    c->T = off;
    off = align256(off + static_cast<size_t>(L.pref_chunk_tiles) * BM * d * 4);
    c->Pt = off;
    off = align256(off + L.scratch_row_tile_bytes * L.pref_chunk_tiles);
    c->total = off;
    return HASS_OK;
}

int hass_combined_distill_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes) {
    if (!bytes) return HASS_ERR_INVALID_ARG;
    size_t base = 0;
    int rc = hass_topk_distill_workspace_bytes(N, d, V, K, &base);
    if (rc != HASS_OK) return rc;
    CombinedStage c;
    rc = combined_stage(N, d, V, K, base, &c);
    if (rc != HASS_OK) return rc;
    *bytes = c.total;
    return HASS_OK;
}

int hass_combined_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                                  int32_t K, float w_topk, const float* grad_loss, float* loss_ce, float* loss_topk,
                                  int32_t* topk_idx, float* topk_q, float* lse_t, float* lse_d, void* dH_d,
                                  int dH_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!loss_ce || !(w_topk == w_topk)) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    size_t base = 0;
    rc = hass_topk_distill_workspace_bytes(N, d, V, K, &base);
    if (rc != HASS_OK) return rc;
    CombinedStage c;
    rc = combined_stage(N, d, V, K, base, &c);
    if (rc != HASS_OK) return rc;
    if (workspace_bytes < c.total) return HASS_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    Combined cmb;
    cmb.w = w_topk;
    cmb.loss_ce = loss_ce;
    cmb.coef_t = reinterpret_cast<float*>(ws + c.coef_t);
    cmb.T = reinterpret_cast<float*>(ws + c.T);
    cmb.Pt = reinterpret_cast<__nv_bfloat16*>(ws + c.Pt);
    return fused_impl(true, H_t, H_d, W, N, d, V, K, grad_loss, nullptr, nullptr, loss_topk, topk_idx, topk_q, lse_t,
                      lse_d, dH_d, dH_dtype, workspace, base, static_cast<cudaStream_t>(cuda_stream), &cmb);
}

// Device staging appended to the normal workspace by the *_host entry.
struct HostStage {
    size_t H_t, H_d, grad, loss, idx, q, lse_t, lse_d, dH, total;
};
static int host_stage(int64_t N, int64_t d, int64_t V, int32_t K, int dH_dtype, size_t base, HostStage* s) {
    size_t off = align256(base);
    s->H_t = off;
    off = align256(off + static_cast<size_t>(N) * d * 2);
    s->H_d = off;
    off = align256(off + static_cast<size_t>(N) * d * 2);
    s->grad = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    s->loss = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    s->idx = off;
    off = align256(off + static_cast<size_t>(N) * K * 4);
    s->q = off;
    off = align256(off + static_cast<size_t>(N) * K * 4);
    s->lse_t = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    s->lse_d = off;
    off = align256(off + static_cast<size_t>(N) * 4);
    s->dH = off;
    off = align256(off + static_cast<size_t>(N) * d * (dH_dtype == HASS_FP32 ? 4 : 2));
    s->total = off;
    (void)V;
    return HASS_OK;
}

int hass_topk_distill_host_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, int dH_dtype, size_t* bytes) {
    if (!bytes || (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32)) return HASS_ERR_INVALID_ARG;
    size_t base = 0;
    int rc = hass_topk_distill_workspace_bytes(N, d, V, K, &base);
    if (rc != HASS_OK) return rc;
    HostStage s;
    host_stage(N, d, V, K, dH_dtype, base, &s);
    *bytes = s.total;
    return HASS_OK;
}

// Copy streams and events of the host-buffer entry, created on a device's first call (no device memory).
struct HostPipeResources {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t events[256];
};
static HostPipeResources g_host_pipe[64];

static int host_pipe_resources(HostPipeResources** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    HostPipeResources& r = g_host_pipe[dev];
    if (!r.ready) {
        bool ok = cudaStreamCreateWithFlags(&r.h2d, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&r.d2h, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; ok && i < 256; ++i) ok = cudaEventCreateWithFlags(&r.events[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        r.ready = true;
    }
    *out = &r;
    return HASS_OK;
}

int hass_topk_distill_fwd_bwd_host(const void* H_t_host, const void* H_d_host, const void* W, int64_t N, int64_t d,
                                   int64_t V, int32_t K, const float* grad_loss_host, float* loss_host,
                                   int32_t* topk_idx_host, float* topk_q_host, void* dH_d_host, int dH_dtype,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    if (!H_t_host || !H_d_host || !W || !loss_host || !dH_d_host) return HASS_ERR_INVALID_ARG;
    if (dH_dtype != HASS_BF16 && dH_dtype != HASS_FP32) return HASS_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    size_t base = 0;
    rc = hass_topk_distill_workspace_bytes(N, d, V, K, &base);
    if (rc != HASS_OK) return rc;
    HostStage s;
    host_stage(N, d, V, K, dH_dtype, base, &s);
    if (workspace_bytes < s.total) return HASS_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    HostPipeResources* res = nullptr;
    rc = host_pipe_resources(&res);
    if (rc != HASS_OK) return rc;
    const float* grad_dev = nullptr;
    if (grad_loss_host) {
        if (cudaMemcpyAsync(ws + s.grad, grad_loss_host, static_cast<size_t>(N) * 4, cudaMemcpyHostToDevice, st) !=
            cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        grad_dev = reinterpret_cast<const float*>(ws + s.grad);
    }
    // The copy streams start after whatever the caller's stream still does with the workspace. The rows of a chunk
    // travel to the device while the previous chunk computes; a chunk's dH_d rows travel back while the next computes.
    ChunkPipe pipe;
    pipe.h2d = res->h2d;
    pipe.d2h = res->d2h;
    pipe.Ht_host = static_cast<const uint8_t*>(H_t_host);
    pipe.Hd_host = static_cast<const uint8_t*>(H_d_host);
    pipe.dH_host = static_cast<uint8_t*>(dH_d_host);
    pipe.in_row_bytes = static_cast<size_t>(d) * 2;
    pipe.out_row_bytes = static_cast<size_t>(d) * (dH_dtype == HASS_FP32 ? 4 : 2);
    pipe.events = res->events;
    pipe.n_events = 256;
    pipe.used = 0;
    cudaEvent_t ev_start = pipe.next();
    if (cudaEventRecord(ev_start, st) != cudaSuccess || cudaStreamWaitEvent(pipe.h2d, ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(pipe.d2h, ev_start, 0) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    rc = fused2_impl(true, ws + s.H_t, ws + s.H_d, W, N, d, V, K, grad_dev, nullptr, nullptr,
                     reinterpret_cast<float*>(ws + s.loss), reinterpret_cast<int32_t*>(ws + s.idx),
                     reinterpret_cast<float*>(ws + s.q), reinterpret_cast<float*>(ws + s.lse_t),
                     reinterpret_cast<float*>(ws + s.lse_d), ws + s.dH, dH_dtype, workspace, base, st, 0.f, nullptr, &pipe);
    if (rc == HASS_ERR_UNSUPPORTED) {
        // more row chunks than events (a very small workspace): one copy in, the call, one copy out
        const size_t hbytes = static_cast<size_t>(N) * d * 2;
        cudaStreamSynchronize(pipe.h2d);
        cudaStreamSynchronize(pipe.d2h);
        if (cudaMemcpyAsync(ws + s.H_t, H_t_host, hbytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(ws + s.H_d, H_d_host, hbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        rc = fused2_impl(true, ws + s.H_t, ws + s.H_d, W, N, d, V, K, grad_dev, nullptr, nullptr,
                         reinterpret_cast<float*>(ws + s.loss), reinterpret_cast<int32_t*>(ws + s.idx),
                         reinterpret_cast<float*>(ws + s.q), reinterpret_cast<float*>(ws + s.lse_t),
                         reinterpret_cast<float*>(ws + s.lse_d), ws + s.dH, dH_dtype, workspace, base, st);
        if (rc == HASS_OK && cudaMemcpyAsync(dH_d_host, ws + s.dH, static_cast<size_t>(N) * pipe.out_row_bytes,
                                             cudaMemcpyDeviceToHost, st) != cudaSuccess) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
    } else if (rc == HASS_OK) {
        // the caller's stream ends after the last outbound copy
        cudaEvent_t ev_out = pipe.next();
        if (!ev_out || cudaEventRecord(ev_out, pipe.d2h) != cudaSuccess || cudaStreamWaitEvent(st, ev_out, 0) != cudaSuccess) {
            cudaGetLastError();
            cudaStreamSynchronize(pipe.d2h);
        }
    }
    if (rc != HASS_OK) {
        cudaStreamSynchronize(pipe.h2d);
        cudaStreamSynchronize(pipe.d2h);
        return rc;
    }
    bool ok = cudaMemcpyAsync(loss_host, ws + s.loss, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (topk_idx_host)
        ok = ok && cudaMemcpyAsync(topk_idx_host, ws + s.idx, static_cast<size_t>(N) * K * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (topk_q_host)
        ok = ok && cudaMemcpyAsync(topk_q_host, ws + s.q, static_cast<size_t>(N) * K * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    // word 2 of the status block: the exact route ran after the chunks' dH_d rows had left; fetch them again
    unsigned int redo = 0;
    ok = cudaMemcpyAsync(&redo, ws + 8, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    rc = hass_check(workspace, cuda_stream);
    cudaStreamSynchronize(pipe.d2h);
    if (rc != HASS_OK) return rc;
    if (!ok) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    if (redo != 0u &&
        cudaMemcpy(dH_d_host, ws + s.dH, static_cast<size_t>(N) * pipe.out_row_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    return HASS_OK;
}

// ---- forward without a caller-provided workspace -------------------------------------------------
// Scratch of hass_topk_distill_fwd_static: lives in the library's device image, so every GPU that
// loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HASS_STATIC_SCRATCH_MAX_BYTES];
// Device address of g_static_scratch per device. In host code the symbol itself is only a handle
// for the runtime, never a pointer a kernel may use; the address comes from cudaGetSymbolAddress.
static void* g_static_scratch_addr[64] = {nullptr};

int hass_topk_distill_fwd_static_scratch_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes) {
    if (!bytes) return HASS_ERR_INVALID_ARG;
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    // the forward needs the statistics / candidate part of the workspace layout only
    Layout L;
    rc = make_layout(N, d, V, K, sm_count_or_default(), &L, nullptr);
    if (rc != HASS_OK) return rc;
    *bytes = L.fwd_end;
    return HASS_OK;
}

int hass_topk_distill_fwd_static(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                                 int32_t K, float* loss, int32_t* topk_idx, float* topk_q, float* lse_t,
                                 float* lse_d, unsigned int* device_status, void* cuda_stream) {
    int rc = check_sizes(N, d, V, K);
    if (rc != HASS_OK) return rc;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    size_t need = 0;
    rc = hass_topk_distill_fwd_static_scratch_bytes(N, d, V, K, &need);
    if (rc != HASS_OK) return rc;
    if (need > HASS_STATIC_SCRATCH_MAX_BYTES) {
        if (kLog)
            std::fprintf(stderr, "[hass] hass_topk_distill_fwd_static: this size needs %zu bytes of scratch, the built-in "
                         "array holds %u; use hass_topk_distill_fwd with a workspace\n", need,
                         HASS_STATIC_SCRATCH_MAX_BYTES);
        return HASS_ERR_UNSUPPORTED;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    if (!g_static_scratch_addr[dev]) {
        // once per device, with that device current
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return HASS_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = ptr;
    }
    void* scratch = g_static_scratch_addr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // forward_impl zeroes the status word (the only part of the scratch that must start at zero:
    // every statistic and candidate slot that is read has been written by the same call)
    rc = forward_impl(true, H_t, H_d, W, N, d, V, K, nullptr, nullptr, loss, topk_idx, topk_q, lse_t, lse_d, scratch,
                      HASS_STATIC_SCRATCH_MAX_BYTES, st);
    if (rc != HASS_OK) return rc;
    if (device_status &&
        cudaMemcpyAsync(device_status, scratch, sizeof(unsigned int), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    return HASS_OK;
}

int hass_hca_attention_workspace_bytes(size_t* bytes) {
    if (!bytes) return HASS_ERR_INVALID_ARG;
    *bytes = 256;
    return HASS_OK;
}

int hass_hca_attention_fwd(const void* Q, const void* K_t, const void* V_t, const void* const* K_d,
                           const void* const* V_d, int32_t m, int64_t B, int64_t T, int64_t H, int64_t Hkv, int64_t D,
                           float scale, void* O, float* lse, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
    if (!Q || !K_t || !V_t || !O) return HASS_ERR_INVALID_ARG;
    if (m < 0 || m > HASS_HCA_MAX_DRAFTS || (m > 0 && (!K_d || !V_d))) return HASS_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || H < 1 || Hkv < 1 || H % Hkv != 0 || !(scale > 0.f) || !(scale < INFINITY))
        return HASS_ERR_INVALID_ARG;
    if (D != hca::HD) return HASS_ERR_UNSUPPORTED;
    if (B > 65535 || T > (1 << 22) || H > 4096 || B * H * ((T + hca::QT - 1) / hca::QT) > INT_MAX / 2)
        return HASS_ERR_UNSUPPORTED;
    auto misaligned = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; };
    if (misaligned(Q) || misaligned(K_t) || misaligned(V_t) || (reinterpret_cast<uintptr_t>(O) & 31u) != 0)
        return HASS_ERR_INVALID_ARG;
    for (int i = 0; i < m; ++i)
        if (!K_d[i] || !V_d[i] || misaligned(K_d[i]) || misaligned(V_d[i])) return HASS_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < 256 || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    {
        hca2::Params p;
        std::memset(&p, 0, sizeof(p));
        rc = make_tmap_seq(&p.tmQ, Q, B, T, H * hca2::HD, hca2::QT);
        if (rc == HASS_OK) rc = make_tmap_seq(&p.tmK, K_t, B, T, Hkv * hca2::HD, hca2::KT);
        if (rc == HASS_OK) rc = make_tmap_seq(&p.tmV, V_t, B, T, Hkv * hca2::HD, hca2::KT);
        for (int i = 0; i < m && rc == HASS_OK; ++i) {
            rc = make_tmap_seq(&p.tmKd[i], K_d[i], B, T, Hkv * hca2::HD, hca2::KT);
            if (rc == HASS_OK) rc = make_tmap_seq(&p.tmVd[i], V_d[i], B, T, Hkv * hca2::HD, hca2::KT);
        }
        if (rc != HASS_OK) return rc;
        p.O = static_cast<__nv_bfloat16*>(O);
        p.lse = lse;
        p.B = static_cast<int>(B);
        p.T = static_cast<int>(T);
        p.H = static_cast<int>(H);
        p.Hkv = static_cast<int>(Hkv);
        p.m = m;
        p.q_tiles = static_cast<int>((T + hca2::QT - 1) / hca2::QT);
        // two query heads of one key/value group per CTA when the group size is even, else two query tiles of one head
        p.head_pairing = ((H / Hkv) % 2 == 0) ? 1 : 0;
        p.pairs = p.head_pairing ? static_cast<int>(B * (H / 2)) * p.q_tiles : static_cast<int>(B * H) * ((p.q_tiles + 1) / 2);
        p.c2 = scale * 1.4426950408889634f;
        p.status = static_cast<unsigned int*>(workspace);
        const int grid = p.pairs < di.sms ? p.pairs : di.sms;
        {
            KernelTimer kt(KIND_HCA, st);
            hca2::hca_attention_pair_kernel<<<grid, hca2::NUM_THREADS, hca2::SMEM_BYTES, st>>>(p);
        }
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
        return HASS_OK;
    }
}

// workspace of the HCA backward: status word, D [B, H, T], and the fp32 dQ accumulator [B, T, H, 128]
struct HcaBwdLayout {
    size_t D, dQacc, total;
};
static HcaBwdLayout hca_bwd_layout(int64_t B, int64_t T, int64_t H) {
    HcaBwdLayout L;
    auto up = [](size_t x) { return (x + 255) & ~static_cast<size_t>(255); };
    const size_t rows = static_cast<size_t>(B) * H * T;
    L.D = 256;
    L.dQacc = up(L.D + rows * 4);
    L.total = up(L.dQacc + rows * hca::HD * 4);
    return L;
}

int hass_hca_attention_bwd_workspace_bytes(int64_t B, int64_t T, int64_t H, int32_t m, size_t* bytes) {
    if (!bytes || B < 1 || T < 1 || H < 1 || m < 0 || m > HASS_HCA_MAX_DRAFTS) return HASS_ERR_INVALID_ARG;
    *bytes = hca_bwd_layout(B, T, H).total;
    return HASS_OK;
}

int hass_hca_attention_bwd(const void* Q, const void* K_t, const void* V_t, const void* const* K_d,
                           const void* const* V_d, int32_t m, int64_t B, int64_t T, int64_t H, int64_t Hkv, int64_t D,
                           float scale, const void* O, const float* lse, const void* dO, void* dQ, void* dK_t,
                           void* dV_t, void* const* dK_d, void* const* dV_d, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
    if (!Q || !K_t || !V_t || !O || !lse || !dO || !dQ || !dK_t || !dV_t) return HASS_ERR_INVALID_ARG;
    if (m < 0 || m > HASS_HCA_MAX_DRAFTS || (m > 0 && (!K_d || !V_d || !dK_d || !dV_d))) return HASS_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || H < 1 || Hkv < 1 || H % Hkv != 0 || !(scale > 0.f) || !(scale < INFINITY))
        return HASS_ERR_INVALID_ARG;
    if (D != hca::HD) return HASS_ERR_UNSUPPORTED;
    if (B > 65535 || T > (1 << 22) || H > 4096 || B * H * ((T + hca::QT - 1) / hca::QT) > INT_MAX / 2)
        return HASS_ERR_UNSUPPORTED;
    auto mis = [](const void* q, uintptr_t a) { return (reinterpret_cast<uintptr_t>(q) & (a - 1)) != 0; };
    if (mis(Q, 16) || mis(K_t, 16) || mis(V_t, 16) || mis(O, 16) || mis(dO, 16) || mis(lse, 4) || mis(dQ, 32) ||
        mis(dK_t, 32) || mis(dV_t, 32))
        return HASS_ERR_INVALID_ARG;
    for (int i = 0; i < m; ++i)
        if (!K_d[i] || !V_d[i] || !dK_d[i] || !dV_d[i] || mis(K_d[i], 16) || mis(V_d[i], 16) || mis(dK_d[i], 16) ||
            mis(dV_d[i], 16))
            return HASS_ERR_INVALID_ARG;
    const HcaBwdLayout L = hca_bwd_layout(B, T, H);
    if (!workspace || workspace_bytes < L.total || mis(workspace, 256)) return HASS_ERR_WORKSPACE;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    rc = get_encode();
    if (rc != HASS_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* Dv = reinterpret_cast<float*>(ws + L.D);
    float* dQacc = reinterpret_cast<float*>(ws + L.dQacc);
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    const int iB = static_cast<int>(B), iT = static_cast<int>(T), iH = static_cast<int>(H), iHkv = static_cast<int>(Hkv);
    const float c2 = scale * 1.4426950408889634f;

    hca_bwd::FusedParams k;
    std::memset(&k, 0, sizeof(k));
    rc = make_tmap_seq(&k.tmK, K_t, B, T, Hkv * hca::HD, hca_bwd::KEYS);
    if (rc == HASS_OK) rc = make_tmap_seq(&k.tmV, V_t, B, T, Hkv * hca::HD, hca_bwd::KEYS);
    if (rc == HASS_OK) rc = make_tmap_seq(&k.tmQ, Q, B, T, H * hca::HD, hca_bwd::QE);
    if (rc == HASS_OK) rc = make_tmap_seq(&k.tmdO, dO, B, T, H * hca::HD, hca_bwd::QE);
    if (rc == HASS_OK) {
        // the fp32 accumulator [B, T, H * 128]: boxes of 32 positions x one head's 128 floats, rows as they lie in memory
        cuuint64_t gdim[3] = {static_cast<cuuint64_t>(H * hca::HD), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(B)};
        cuuint64_t gstride[2] = {gdim[0] * 4, gdim[0] * 4 * gdim[1]};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(hca::HD), 32, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (g_encode(&k.tmdQ, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dQacc, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            rc = HASS_ERR_CUDA;
    }
    if (rc != HASS_OK) return rc;

    {   // D, the substituted entries and everything that follows from them, the start value of the dQ accumulator
        hca_bwd::RowsParams r;
        std::memset(&r, 0, sizeof(r));
        r.Q = static_cast<const __nv_bfloat16*>(Q);
        r.O = static_cast<const __nv_bfloat16*>(O);
        r.dO = static_cast<const __nv_bfloat16*>(dO);
        for (int i = 0; i < m; ++i) {
            r.Kd[i] = static_cast<const __nv_bfloat16*>(K_d[i]);
            r.Vd[i] = static_cast<const __nv_bfloat16*>(V_d[i]);
            r.dKd[i] = static_cast<__nv_bfloat16*>(dK_d[i]);
            r.dVd[i] = static_cast<__nv_bfloat16*>(dV_d[i]);
        }
        r.lse = lse;
        r.D = Dv;
        r.dQacc = dQacc;
        r.m = m; r.B = iB; r.T = iT; r.H = iH; r.Hkv = iHkv;
        r.c2 = c2;
        r.scale = scale;
        KernelTimer kt(KIND_HCA_BWD_ROWS, st);
        const long long halves = static_cast<long long>(B) * T * Hkv;
        hca_bwd::hca_bwd_rows_kernel<<<static_cast<unsigned>((halves * 16 + 255) / 256), 256, 0, st>>>(r);
    }
    g_launches.fetch_add(1);

    k.dK = static_cast<__nv_bfloat16*>(dK_t);
    k.dV = static_cast<__nv_bfloat16*>(dV_t);
    k.lse = lse;
    k.D = Dv;
    k.B = iB; k.T = iT; k.H = iH; k.Hkv = iHkv; k.m = m;
    k.kt_tiles = static_cast<int>((T + hca_bwd::KEYS - 1) / hca_bwd::KEYS);
    k.q_tiles64 = static_cast<int>((T + hca_bwd::QE - 1) / hca_bwd::QE);
    k.items = iB * iHkv * k.kt_tiles;
    k.c2 = c2;
    k.scale = scale;
    k.status = static_cast<unsigned int*>(workspace);
    {
        KernelTimer kt(KIND_HCA_BWD_FUSED, st);
        hca_bwd::hca_bwd_fused_kernel<<<k.items < di.sms ? k.items : di.sms, hca_bwd::NUM_THREADS, hca_bwd::F_SMEM_BYTES, st>>>(k);
    }
    g_launches.fetch_add(1);

    {
        KernelTimer kt(KIND_HCA_DQ_CONVERT, st);
        const long long n8 = static_cast<long long>(B) * T * H * (hca::HD / 8);
        hca_bwd::hca_dq_convert_kernel<<<static_cast<unsigned>((n8 + 255) / 256), 256, 0, st>>>(
            dQacc, static_cast<__nv_bfloat16*>(dQ), n8);
    }
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return HASS_ERR_CUDA;
    return HASS_OK;
}

int hass_selftest_wait_expiry(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* cuda_stream) {
    if (!workspace || workspace_bytes < 256 || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HASS_ERR_WORKSPACE;
    if (limit_ns < 1000ull || limit_ns > 100000000ull) return HASS_ERR_INVALID_ARG;      // 1 us .. 100 ms
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != HASS_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    unsigned int* words = static_cast<unsigned int*>(workspace);
    wait_expiry_selftest_kernel<<<1, 128, 0, st>>>(words, limit_ns, words + 16);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? HASS_OK : HASS_ERR_CUDA;
}

int hass_check(void* workspace, void* cuda_stream) {
    if (!workspace) return HASS_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    unsigned int word = 0;
    if (cudaMemcpy(&word, workspace, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return HASS_ERR_CUDA;
    }
    if (word != 0) {
        cudaMemset(workspace, 0, 4);
        if (kLog) std::fprintf(stderr, "[hass] device status word 0x%x\n", word);
        return (word & 0xffu) == 2u ? HASS_ERR_RANGE : HASS_ERR_TIMEOUT;
    }
    return HASS_OK;
}

}  // extern "C"
