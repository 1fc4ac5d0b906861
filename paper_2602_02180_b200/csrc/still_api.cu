// Host side of the C ABI declared in include/still.h: argument validation,
// workspace / state planning and kernel launches.  No device memory is
// allocated here and nothing falls back to the CPU.
#include "../../include/still.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>

#include "still_simt.cuh"
#include "still_tc.h"

namespace still {

static thread_local int g_launches = 0;

// Event pairs of still_profile_enable (per host thread).
static thread_local cudaEvent_t *g_prof_ev = nullptr;
static thread_local int g_prof_cap = 0, g_prof_used = 0;

void profile_mark_begin(cudaStream_t st) {
    if (g_prof_ev && g_prof_used < g_prof_cap) cudaEventRecord(g_prof_ev[2 * g_prof_used], st);
}
void profile_mark_end(cudaStream_t st) {
    if (g_prof_ev && g_prof_used < g_prof_cap) {
        cudaEventRecord(g_prof_ev[2 * g_prof_used + 1], st);
        ++g_prof_used;
    }
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline size_t esize(int dtype) { return dtype == STILL_DTYPE_FP32 ? 4 : 2; }

static int validate(const still_params_t *p) {
    if (!p) return STILL_ERR_INVALID_ARG;
    if (p->B <= 0 || p->H <= 0 || p->Hkv <= 0 || p->H % p->Hkv != 0) return STILL_ERR_INVALID_ARG;
    if (p->topk < 0 || p->topk > p->chunk) return STILL_ERR_INVALID_ARG;
    if (!(p->sm_scale > 0.f) || !(p->eps > 0.f)) return STILL_ERR_INVALID_ARG;
    if (p->max_salient < 0) return STILL_ERR_INVALID_ARG;
    if (p->dtype != STILL_DTYPE_FP32 && p->dtype != STILL_DTYPE_BF16) return STILL_ERR_UNSUPPORTED;
    if (p->d != 64 && p->d != 128) return STILL_ERR_UNSUPPORTED;
    if (p->chunk != 32 && p->chunk != 64 && p->chunk != 128) return STILL_ERR_UNSUPPORTED;
    if (p->d_f != 32 && p->d_f != 64 && p->d_f != 128) return STILL_ERR_UNSUPPORTED;
    if (p->d_f > p->d) return STILL_ERR_UNSUPPORTED;
    if (p->max_salient > 0) {
        // budget of the salient cache: whole chunks' worth of selections, on the tensor-core kernels
        if (p->topk == 0 || p->max_salient % p->topk != 0 || p->max_salient / p->topk > (1 << 20)) return STILL_ERR_UNSUPPORTED;
        if (!tc_supported(p) || !tc_la_supported(p)) return STILL_ERR_UNSUPPORTED;
    }
    return STILL_OK;
}

// The linear branch runs when a chunk can have unselected tokens, or when cached tokens can leave the cache.
static inline bool la_active(const still_params_t *p) { return p->topk < p->chunk || p->max_salient > 0; }

// Workspace plan of the prefill.
struct FwdPlan {
    size_t status, scores, sel_idx, phiQ, phiK, csum, zpre, segs, nla, dla, ypart, dpart, ksel, vsel, phiKsel, total;
    long long T, sel_rows;  // chunks; rows of the compacted salient K/V per head
    bool la, tc, tc_la;
};

static FwdPlan plan_fwd(const still_params_t *p, long long N) {
    FwdPlan w{};
    const long long T = (N + p->chunk - 1) / p->chunk;
    const size_t BH = (size_t)p->B * p->H, BHkv = (size_t)p->B * p->Hkv;
    const size_t es = esize(p->dtype), dp = 2 * (size_t)p->d_f;
    w.T = T;
    w.la = la_active(p);
    w.tc = tc_supported(p);
    w.tc_la = w.la && tc_la_supported(p);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 1024);
        return o;
    };
    w.status = take(256);
    w.scores = take(BH * (size_t)N * 4);
    w.sel_idx = take(BH * (size_t)T * (size_t)std::max(p->topk, 1) * 4);
    if (w.la) {
        w.phiK = take(BHkv * (size_t)N * dp * es);
        if (w.tc_la) {
            // tensor-core branch: phi(Q) is never stored; the branch leaves two bf16 partial results
            w.csum = take(BHkv * (size_t)T * dp * 4);
            w.zpre = take(BH * (size_t)std::max<long long>(T - 2, 1) * dp * 4);
            int seg_chunks = 0;
            const int n_seg = tc_la_segments(p, N, &seg_chunks);
            w.segs = take(BH * (size_t)std::max((n_seg - 1) * tc_la_sum_parts(seg_chunks), 1) * dp * p->d * 4);
        } else {
            w.phiQ = take(BH * (size_t)N * dp * es);
            w.nla = take(BH * (size_t)N * p->d * 4);
            w.dla = take(BH * (size_t)N * 4);
        }
        if (w.tc) {
            const int parts = w.tc_la ? 2 : 1;
            w.ypart = take(parts * BH * (size_t)N * p->d * 2);
            w.dpart = take(parts * BH * (size_t)N * 4);
        }
    }
    if (w.tc) {
        w.sel_rows = tc_sel_rows(p, N);
        if (p->topk < p->chunk) {  // with topk = chunk the salient prefix is K / V itself: no compacted copy
            w.ksel = take(BH * (size_t)w.sel_rows * p->d * es);
            w.vsel = take(BH * (size_t)w.sel_rows * p->d * es);
            // (with a budget: phi(K) of the selected rows, from which the leaving tokens enter the state)
            if (w.tc_la && p->max_salient > 0) w.phiKsel = take(BH * (size_t)w.sel_rows * dp * 2);
        }
    }
    w.total = off;
    return w;
}

static int plan_state(const still_params_t *p, long long max_tokens, still_state_layout_t *L) {
    if (max_tokens <= 0) return STILL_ERR_INVALID_ARG;
    const long long cap = (max_tokens + p->chunk - 1) / p->chunk * p->chunk;
    const size_t BH = (size_t)p->B * p->H, BHkv = (size_t)p->B * p->Hkv;
    const size_t es = esize(p->dtype), dp = 2 * (size_t)p->d_f;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 1024);
        return o;
    };
    L->capacity = cap;
    L->header = take(256);
    const size_t kvr = (size_t)state_kv_rows(p, cap);
    L->k_cache = take(BHkv * kvr * p->d * es);
    L->v_cache = take(BHkv * kvr * p->d * es);
    L->score = take(BH * (size_t)cap * 4);
    L->sel_idx = take(BH * (size_t)(cap / p->chunk) * (size_t)std::max(p->topk, 1) * 4);
    L->sel_mask = take(BH * (size_t)(cap / p->chunk) * (size_t)(p->chunk / 32) * 4);
    L->S = take(BH * dp * p->d * 4);
    L->z = take(BH * dp * 4);
    L->scratch = take(step_scratch_bytes(p, cap));
    L->total = off;
    return STILL_OK;
}

template <typename K>
static cudaError_t set_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

#define STILL_CUDA(expr)                                   \
    do {                                                   \
        cudaError_t e__ = (expr);                          \
        if (e__ != cudaSuccess) return STILL_ERR_CUDA;     \
    } while (0)

__global__ void write_header_kernel(int32_t *hdr, still_params_t p, long long cap, long long t) {
    if (threadIdx.x == 0) {
        hdr[0] = 0x5354494c;  // "STIL"
        hdr[1] = 1;
        hdr[2] = p.B; hdr[3] = p.H; hdr[4] = p.Hkv; hdr[5] = p.d; hdr[6] = p.d_f;
        hdr[7] = p.chunk; hdr[8] = p.topk; hdr[9] = p.dtype;
        hdr[10] = (int32_t)(cap & 0xffffffffll); hdr[11] = (int32_t)(cap >> 32);
        hdr[12] = (int32_t)(t & 0xffffffffll); hdr[13] = (int32_t)(t >> 32);
        hdr[14] = 0; hdr[15] = 0;
    }
}

// Selection of every chunk as bit masks for the decode state: one warp per (head, chunk); bit j of
// word w is set when position chunk * C + 32 w + j is among the chunk's selected positions.
__global__ void sel_mask_kernel(const int32_t *__restrict__ sel_idx, uint32_t *__restrict__ sel_mask, long long BH,
                                long long T, long long capT, int C, int lam) {
    const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= BH * T) return;
    const int lane = threadIdx.x & 31;
    const long long bh = wid / T, c = wid % T;
    const int32_t *si = sel_idx + (bh * T + c) * lam;
    for (int w = 0; w < C / 32; ++w) {
        const long long p0 = c * C + 32ll * w;
        uint32_t bits = 0u;
        for (int i = lane; i < lam; i += 32) {
            const long long p = si[i];
            if (p >= p0 && p < p0 + 32) bits |= 1u << (int)(p - p0);
        }
        bits = __reduce_or_sync(0xffffffffu, bits);
        if (lane == 0) sel_mask[(bh * capT + c) * (C / 32) + w] = bits;
    }
}

// ------------------------------------------------------------------ FMA path launches

template <typename T>
static int launch_score_select(const still_params_t *p, long long N, long long Tn, const T *Q,
                               const T *K, float *scores, int32_t *sel, cudaStream_t st) {
    const int C = p->chunk, d = p->d;
    size_t smem = ((size_t)2 * C * (d + 1) + (size_t)C * d + C) * 4 + (size_t)C * 4;
    STILL_CUDA(set_smem(score_select_kernel<T>, smem));
    dim3 grid((unsigned)Tn, p->H, p->B);
    score_select_kernel<T><<<grid, 256, smem, st>>>(Q, K, scores, sel, p->H, p->Hkv, N, d, C,
                                                    p->topk, p->sm_scale, p->eps);
    ++g_launches;
    STILL_CUDA(cudaGetLastError());
    return STILL_OK;
}

template <typename T>
static int launch_npmap(const still_params_t *p, long long N, int heads, const T *X, const T *W,
                        const T *bias, T *phi, cudaStream_t st) {
    size_t smem = ((size_t)p->d * p->d_f + p->d_f + 8 * (size_t)p->d) * 4;
    STILL_CUDA(set_smem(npmap_kernel<T, T>, smem));
    dim3 grid((unsigned)((N + 63) / 64), heads, p->B);
    npmap_kernel<T, T><<<grid, 256, smem, st>>>(X, W, bias, phi, heads, N, p->d, p->d_f);
    ++g_launches;
    STILL_CUDA(cudaGetLastError());
    return STILL_OK;
}

template <typename T, int FPT>
static int launch_la_scan_t(const still_params_t *p, long long N, long long Tn, const T *phiQ,
                            const T *phiK, const T *V, const T *G, const int32_t *sel, float *nla,
                            float *dla, float *S_out, float *z_out, cudaStream_t st) {
    constexpr int DP = FPT * 8;
    size_t smem = ((size_t)32 * DP + 32 * 32 + 8 * 32 * 33 + DP) * 4 + (size_t)p->chunk * 4;
    STILL_CUDA(set_smem(la_scan_kernel<T, T, FPT>, smem));
    dim3 grid(p->B * p->H, p->d / 32);
    int n_route = (int)std::max<long long>(0, Tn - 2);
    la_scan_kernel<T, T, FPT><<<grid, 256, smem, st>>>(phiQ, phiK, V, G, sel, nla, dla, S_out, z_out,
                                                       p->H, p->Hkv, N, p->d, p->chunk, p->topk,
                                                       n_route);
    ++g_launches;
    STILL_CUDA(cudaGetLastError());
    return STILL_OK;
}

template <typename T>
static int launch_la_scan(const still_params_t *p, long long N, long long Tn, const T *phiQ,
                          const T *phiK, const T *V, const T *G, const int32_t *sel, float *nla,
                          float *dla, float *S_out, float *z_out, cudaStream_t st) {
    switch (p->d_f) {
        case 32: return launch_la_scan_t<T, 8>(p, N, Tn, phiQ, phiK, V, G, sel, nla, dla, S_out, z_out, st);
        case 64: return launch_la_scan_t<T, 16>(p, N, Tn, phiQ, phiK, V, G, sel, nla, dla, S_out, z_out, st);
        default: return launch_la_scan_t<T, 32>(p, N, Tn, phiQ, phiK, V, G, sel, nla, dla, S_out, z_out, st);
    }
}

template <typename T, int RPW, int DPL>
static int launch_sa_merge_t(const still_params_t *p, long long N, long long Tn, const T *Q,
                             const T *K, const T *V, const int32_t *sel, const float *nla,
                             const float *dla, T *Y, cudaStream_t st) {
    constexpr int C = RPW * 8, d = DPL * 32;
    size_t smem = ((size_t)C * d + 32 * (d + 1) + 32 * d) * 4 + 32 * 8;
    STILL_CUDA(set_smem(sa_merge_kernel<T, RPW, DPL>, smem));
    dim3 grid((unsigned)Tn, p->H, p->B);
    sa_merge_kernel<T, RPW, DPL><<<grid, 256, smem, st>>>(Q, K, V, sel, nla, dla, Y, p->H, p->Hkv, N,
                                                          p->topk, p->sm_scale);
    ++g_launches;
    STILL_CUDA(cudaGetLastError());
    return STILL_OK;
}

template <typename T>
static int launch_sa_merge(const still_params_t *p, long long N, long long Tn, const T *Q, const T *K,
                           const T *V, const int32_t *sel, const float *nla, const float *dla, T *Y,
                           cudaStream_t st) {
#define STILL_SA_CASE(CC, DD, RPW, DPL) \
    if (p->chunk == CC && p->d == DD) return launch_sa_merge_t<T, RPW, DPL>(p, N, Tn, Q, K, V, sel, nla, dla, Y, st);
    STILL_SA_CASE(32, 64, 4, 2)
    STILL_SA_CASE(32, 128, 4, 4)
    STILL_SA_CASE(64, 64, 8, 2)
    STILL_SA_CASE(64, 128, 8, 4)
    STILL_SA_CASE(128, 64, 16, 2)
    STILL_SA_CASE(128, 128, 16, 4)
#undef STILL_SA_CASE
    return STILL_ERR_UNSUPPORTED;
}

template <typename T>
static int fwd_typed(const still_params_t *p, long long N, const T *Q, const T *K, const T *V,
                     const T *G, const T *Wq, const T *bq, const T *Wk, const T *bk, T *Y,
                     float *scores, int32_t *sel_idx, char *state, long long state_max_tokens,
                     char *ws, const FwdPlan &w, cudaStream_t st) {
    int rc;
    float *sc = scores ? scores : reinterpret_cast<float *>(ws + w.scores);
    int32_t *sel = sel_idx ? sel_idx : reinterpret_cast<int32_t *>(ws + w.sel_idx);
    STILL_CUDA(cudaMemsetAsync(ws + w.status, 0, 256, st));

    still_state_layout_t L{};
    if (state) {
        if ((rc = plan_state(p, state_max_tokens, &L)) != STILL_OK) return rc;
        if (N > L.capacity) return STILL_ERR_STATE_FULL;
    }

    // (1)+(2) Self-Saliency Score and per-chunk top-k.
    if (w.tc)
        rc = tc_score_select(p, N, Q, K, sc, sel, reinterpret_cast<int *>(ws + w.status), st, &g_launches);
    else
        rc = launch_score_select<T>(p, N, w.T, Q, K, sc, sel, st);
    if (rc != STILL_OK) return rc;

    // (3) NP-Map + linear-attention scan (skipped when no token can be in M^LA).
    float *nla = nullptr, *dla = nullptr, *dpart = nullptr;
    void *ypart = nullptr;
    int n_parts = 0;
    float *S_out = state ? reinterpret_cast<float *>(state + L.S) : nullptr;
    float *z_out = state ? reinterpret_cast<float *>(state + L.z) : nullptr;
    if (w.la) {
        T *phiK = reinterpret_cast<T *>(ws + w.phiK);
        if (w.tc_la) {
            ypart = ws + w.ypart;
            dpart = reinterpret_cast<float *>(ws + w.dpart);
            n_parts = 2;
            rc = tc_la_branch(p, N, Q, K, V, G, Wq, bq, Wk, bk, sel, phiK, reinterpret_cast<float *>(ws + w.csum),
                              reinterpret_cast<float *>(ws + w.zpre), ypart, dpart, reinterpret_cast<float *>(ws + w.segs), S_out,
                              z_out, w.phiKsel ? ws + w.phiKsel : nullptr, w.phiKsel ? ws + w.vsel : nullptr, w.sel_rows,
                              reinterpret_cast<int *>(ws + w.status), st, &g_launches);
            if (rc != STILL_OK) return rc;
        } else {
            T *phiQ = reinterpret_cast<T *>(ws + w.phiQ);
            nla = reinterpret_cast<float *>(ws + w.nla);
            dla = reinterpret_cast<float *>(ws + w.dla);
            if ((rc = launch_npmap<T>(p, N, p->H, Q, Wq, bq, phiQ, st)) != STILL_OK) return rc;
            if ((rc = launch_npmap<T>(p, N, p->Hkv, K, Wk, bk, phiK, st)) != STILL_OK) return rc;
            if ((rc = launch_la_scan<T>(p, N, w.T, phiQ, phiK, V, G, sel, nla, dla, S_out, z_out, st)) != STILL_OK)
                return rc;
            if (w.tc && Y) {   // the tensor-core attention kernel takes the linear branch as bf16 parts
                ypart = ws + w.ypart;
                dpart = reinterpret_cast<float *>(ws + w.dpart);
                n_parts = 1;
                if ((rc = tc_la_to_part(nla, dla, ypart, dpart, (long long)p->B * p->H * N, p->d, st, &g_launches)) != STILL_OK)
                    return rc;
            }
        }
    } else if (state) {
        STILL_CUDA(cudaMemsetAsync(state + L.S, 0, L.scratch - L.S, st));
    }

    // (4) softmax-attention branch + merge.
    if (Y) {
        if (w.tc) {
            rc = tc_sa_merge(p, N, Q, K, V, sel, ypart, dpart, n_parts, Y, ws + w.ksel, ws + w.vsel, w.sel_rows,
                             reinterpret_cast<int *>(ws + w.status), st, &g_launches);
        } else {
            profile_mark_begin(st);
            rc = launch_sa_merge<T>(p, N, w.T, Q, K, V, sel, nla, dla, Y, st);
            profile_mark_end(st);
        }
        if (rc != STILL_OK) return rc;
    }

    // Decode state: K/V history, scores, selection; S and z were written above.
    if (state) {
        const size_t es = sizeof(T);
        const size_t BH = (size_t)p->B * p->H, BHkv = (size_t)p->B * p->Hkv;
        // K / V history: the whole sequence, or with a budget the last kvr positions into their ring rows
        // (position q in row q % kvr: at most two contiguous runs)
        const long long kvr = state_kv_rows(p, L.capacity), first = std::max<long long>(0, N - kvr);
        const size_t row = (size_t)p->d * es;
        for (long long q0 = first; q0 < N;) {
            const long long r0 = q0 % kvr, run = std::min<long long>(N - q0, kvr - r0);
            STILL_CUDA(cudaMemcpy2DAsync(state + L.k_cache + r0 * row, kvr * row, reinterpret_cast<const char *>(K) + q0 * row,
                                         (size_t)N * row, run * row, BHkv, cudaMemcpyDeviceToDevice, st));
            STILL_CUDA(cudaMemcpy2DAsync(state + L.v_cache + r0 * row, kvr * row, reinterpret_cast<const char *>(V) + q0 * row,
                                         (size_t)N * row, run * row, BHkv, cudaMemcpyDeviceToDevice, st));
            q0 += run;
        }
        STILL_CUDA(cudaMemcpy2DAsync(state + L.score, (size_t)L.capacity * 4, sc, (size_t)N * 4,
                                     (size_t)N * 4, BH, cudaMemcpyDeviceToDevice, st));
        if (p->topk > 0)
            STILL_CUDA(cudaMemcpy2DAsync(state + L.sel_idx, (size_t)(L.capacity / p->chunk) * p->topk * 4,
                                         sel, (size_t)w.T * p->topk * 4, (size_t)w.T * p->topk * 4, BH,
                                         cudaMemcpyDeviceToDevice, st));
        if (p->topk > 0) {
            const long long units = (long long)BH * w.T;
            sel_mask_kernel<<<(unsigned)((units + 7) / 8), 256, 0, st>>>(
                sel, reinterpret_cast<uint32_t *>(state + L.sel_mask), (long long)BH, w.T, L.capacity / p->chunk,
                p->chunk, p->topk);
            ++g_launches;
            STILL_CUDA(cudaGetLastError());
        }
        write_header_kernel<<<1, 32, 0, st>>>(reinterpret_cast<int32_t *>(state + L.header), *p,
                                              L.capacity, N);
        ++g_launches;
        STILL_CUDA(cudaGetLastError());
    }
    return STILL_OK;
}

static bool misaligned(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; }

}  // namespace still

using namespace still;

extern "C" {

size_t still_workspace_bytes(const still_params_t *p, int64_t N) {
    if (validate(p) != STILL_OK || N < 0) return 0;
    return plan_fwd(p, std::max<int64_t>(N, 1)).total;
}

size_t still_state_bytes(const still_params_t *p, int64_t max_tokens) {
    still_state_layout_t L{};
    if (validate(p) != STILL_OK || plan_state(p, max_tokens, &L) != STILL_OK) return 0;
    return L.total;
}

int still_state_layout(const still_params_t *p, int64_t max_tokens, still_state_layout_t *out) {
    int rc = validate(p);
    if (rc != STILL_OK) return rc;
    if (!out) return STILL_ERR_INVALID_ARG;
    return plan_state(p, max_tokens, out);
}

int still_hybrid_attn_fwd(const still_params_t *p, int64_t N, const void *Q, const void *K,
                          const void *V, const void *G, const void *Wq, const void *bq,
                          const void *Wk, const void *bk, void *Y, float *scores, int32_t *sel_idx,
                          void *state_out, int64_t state_max_tokens, void *workspace,
                          size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0;
    int rc = validate(p);
    if (rc != STILL_OK) return rc;
    if (N < 0) return STILL_ERR_INVALID_ARG;
    if (N > (int64_t)1 << 30) return STILL_ERR_UNSUPPORTED;  // positions are int32
    if (N == 0) {
        // An empty prefill only initialises the decode state (no tokens, zero S and z).
        if (!state_out) return STILL_OK;
        if (misaligned(state_out)) return STILL_ERR_INVALID_ARG;
        still_state_layout_t L{};
        if ((rc = plan_state(p, state_max_tokens, &L)) != STILL_OK) return rc;
        cudaStream_t st0 = reinterpret_cast<cudaStream_t>(cuda_stream);
        char *s0 = reinterpret_cast<char *>(state_out);
        STILL_CUDA(cudaMemsetAsync(s0 + L.S, 0, L.scratch - L.S, st0));
        write_header_kernel<<<1, 32, 0, st0>>>(reinterpret_cast<int32_t *>(s0 + L.header), *p, L.capacity, 0);
        ++g_launches;
        STILL_CUDA(cudaGetLastError());
        return STILL_OK;
    }
    if (!Q || !K || !V || !workspace) return STILL_ERR_INVALID_ARG;
    if (!Y && !state_out && !scores && !sel_idx) return STILL_ERR_INVALID_ARG;
    const void *ptrs[] = {Q, K, V, G, Wq, bq, Wk, bk, Y, scores, sel_idx, state_out, workspace};
    for (const void *ptr : ptrs)
        if (ptr && misaligned(ptr)) return STILL_ERR_INVALID_ARG;
    FwdPlan w = plan_fwd(p, N);
    if (workspace_bytes < w.total) return STILL_ERR_WORKSPACE_TOO_SMALL;
    if (w.la && (!Wq || !Wk)) return STILL_ERR_INVALID_ARG;   // the linear branch needs both maps
    if (state_out) {
        still_state_layout_t L{};
        if ((rc = plan_state(p, state_max_tokens, &L)) != STILL_OK) return rc;
        if (N > L.capacity) return STILL_ERR_STATE_FULL;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    char *ws = reinterpret_cast<char *>(workspace);
    char *state = reinterpret_cast<char *>(state_out);
    if (p->dtype == STILL_DTYPE_FP32)
        return fwd_typed<float>(p, N, (const float *)Q, (const float *)K, (const float *)V,
                                (const float *)G, (const float *)Wq, (const float *)bq,
                                (const float *)Wk, (const float *)bk, (float *)Y, scores, sel_idx,
                                state, state_max_tokens, ws, w, st);
    using bf = __nv_bfloat16;
    return fwd_typed<bf>(p, N, (const bf *)Q, (const bf *)K, (const bf *)V, (const bf *)G,
                         (const bf *)Wq, (const bf *)bq, (const bf *)Wk, (const bf *)bk, (bf *)Y,
                         scores, sel_idx, state, state_max_tokens, ws, w, st);
}

int still_hybrid_attn_step(const still_params_t *p, void *state, int64_t state_max_tokens,
                           int64_t t_pos, const void *q, const void *k, const void *v,
                           const void *g, const void *Wq, const void *bq, const void *Wk,
                           const void *bk, void *y, void *cuda_stream) {
    g_launches = 0;
    int rc = validate(p);
    if (rc != STILL_OK) return rc;
    if (!state || !q || !k || !v || !y || t_pos < 0) return STILL_ERR_INVALID_ARG;
    const void *ptrs[] = {state, q, k, v, g, Wq, bq, Wk, bk, y};
    for (const void *ptr : ptrs)
        if (ptr && misaligned(ptr)) return STILL_ERR_INVALID_ARG;
    if (la_active(p) && (!Wq || !Wk)) return STILL_ERR_INVALID_ARG;
    still_state_layout_t L{};
    if ((rc = plan_state(p, state_max_tokens, &L)) != STILL_OK) return rc;
    if (t_pos >= L.capacity) return STILL_ERR_STATE_FULL;
    return step_launch(p, reinterpret_cast<char *>(state), &L, t_pos, q, k, v, g, Wq, bq, Wk, bk, y,
                       reinterpret_cast<cudaStream_t>(cuda_stream), &g_launches);
}

size_t still_host_arena_bytes(const still_params_t *p, int64_t N) {
    if (validate(p) != STILL_OK || N <= 0) return 0;
    const size_t es = esize(p->dtype);
    const size_t q = align_up((size_t)p->B * p->H * N * p->d * es, 1024);
    const size_t kv = align_up((size_t)p->B * p->Hkv * N * p->d * es, 1024);
    const size_t wq = align_up((size_t)p->H * (p->d + 1) * p->d_f * es, 1024);
    const size_t wk = align_up((size_t)p->Hkv * (p->d + 1) * p->d_f * es, 1024);
    const long long T = (N + p->chunk - 1) / p->chunk;
    const size_t sc = align_up((size_t)p->B * p->H * N * 4, 1024);
    const size_t si = align_up((size_t)p->B * p->H * T * std::max(p->topk, 1) * 4, 1024);
    // Q, G, Y; K, V; Wq+bq, Wk+bk (two slots each); scores; sel_idx; workspace
    return 3 * q + 2 * kv + 2 * wq + 2 * wk + sc + si + plan_fwd(p, N).total;
}

int still_hybrid_attn_fwd_host(const still_params_t *p, int64_t N, const void *hQ, const void *hK,
                               const void *hV, const void *hG, const void *hWq, const void *hbq,
                               const void *hWk, const void *hbk, void *hY, float *hscores,
                               int32_t *hsel_idx, void *arena, size_t arena_bytes,
                               void *cuda_stream) {
    int rc = validate(p);
    if (rc != STILL_OK) return rc;
    if (N <= 0 || !hQ || !hK || !hV || !hY || !arena) return STILL_ERR_INVALID_ARG;
    if (arena_bytes < still_host_arena_bytes(p, N)) return STILL_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t es = esize(p->dtype);
    const size_t qb = (size_t)p->B * p->H * N * p->d * es, kvb = (size_t)p->B * p->Hkv * N * p->d * es;
    const size_t wqb = (size_t)p->H * p->d * p->d_f * es, wkb = (size_t)p->Hkv * p->d * p->d_f * es;
    const size_t bqb = (size_t)p->H * p->d_f * es, bkb = (size_t)p->Hkv * p->d_f * es;
    const long long T = (N + p->chunk - 1) / p->chunk;
    const size_t scb = (size_t)p->B * p->H * N * 4, sib = (size_t)p->B * p->H * T * std::max(p->topk, 1) * 4;
    char *a = reinterpret_cast<char *>(arena);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char *r = a + off;
        off = align_up(off + bytes, 1024);
        return r;
    };
    const size_t wslot = align_up((size_t)p->H * (p->d + 1) * p->d_f * es, 1024);
    const size_t kslot = align_up((size_t)p->Hkv * (p->d + 1) * p->d_f * es, 1024);
    char *dQ = take(qb), *dG = take(qb), *dY = take(qb), *dK = take(kvb), *dV = take(kvb);
    char *dWq = take(wslot), *dbq = take(wslot), *dWk = take(kslot), *dbk = take(kslot);
    char *dsc = take(scb), *dsi = take(sib);
    char *ws = a + off;
    const size_t ws_bytes = arena_bytes - off;
    // Weights first, on the caller's stream.
    if (hWq) STILL_CUDA(cudaMemcpyAsync(dWq, hWq, wqb, cudaMemcpyHostToDevice, st));
    if (hbq) STILL_CUDA(cudaMemcpyAsync(dbq, hbq, bqb, cudaMemcpyHostToDevice, st));
    if (hWk) STILL_CUDA(cudaMemcpyAsync(dWk, hWk, wkb, cudaMemcpyHostToDevice, st));
    if (hbk) STILL_CUDA(cudaMemcpyAsync(dbk, hbk, bkb, cudaMemcpyHostToDevice, st));

    // The (batch, KV-head group) units are independent, so the call is cut into up to sixteen parts --
    // contiguous ranges of KV heads of one batch entry with their query heads -- and pipelined: the
    // host-to-device copies of part i+1 and the device-to-host copies of part i-1 run on two side
    // streams while part i computes (PCIe is full duplex, and the copies are as long as the compute at
    // the benchmark shapes).  What the pipeline cannot hide is the first part's copy in and the last
    // part's copy out, hence small parts; and since a small part's kernels end in a partly filled wave,
    // the parts compute alternately on the caller's stream and on a second one, each with its own
    // workspace, so that the next part's thread blocks fill that tail.
    static thread_local cudaStream_t s_in = nullptr, s_out = nullptr, s_alt = nullptr;
    if (!s_in) {
        STILL_CUDA(cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking));
        STILL_CUDA(cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking));
        STILL_CUDA(cudaStreamCreateWithFlags(&s_alt, cudaStreamNonBlocking));
    }
    const int rep = p->H / p->Hkv;
    int g = std::max(1, p->Hkv * p->B / 16);         // KV heads per part
    while (p->Hkv % g != 0) --g;
    const int parts_per_b = p->Hkv / g, n_parts = p->B * parts_per_b;
    constexpr int kMaxParts = 64;
    const size_t sc_part_bytes = (size_t)g * rep * N * 4, si_part_bytes = (size_t)g * rep * T * std::max(p->topk, 1) * 4;
    if (n_parts > kMaxParts || sc_part_bytes % 16 != 0 || si_part_bytes % 16 != 0) {
        // too many parts for the fixed event table, or a part's scores / indices would not start on a
        // 16-byte boundary (N not a multiple of 4): plain copy - compute - copy
        STILL_CUDA(cudaMemcpyAsync(dQ, hQ, qb, cudaMemcpyHostToDevice, st));
        STILL_CUDA(cudaMemcpyAsync(dK, hK, kvb, cudaMemcpyHostToDevice, st));
        STILL_CUDA(cudaMemcpyAsync(dV, hV, kvb, cudaMemcpyHostToDevice, st));
        if (hG) STILL_CUDA(cudaMemcpyAsync(dG, hG, qb, cudaMemcpyHostToDevice, st));
        rc = still_hybrid_attn_fwd(p, N, dQ, dK, dV, hG ? dG : nullptr, hWq ? dWq : nullptr, hbq ? dbq : nullptr,
                                   hWk ? dWk : nullptr, hbk ? dbk : nullptr, dY, reinterpret_cast<float *>(dsc),
                                   reinterpret_cast<int32_t *>(dsi), nullptr, 0, ws, ws_bytes, cuda_stream);
        if (rc != STILL_OK) return rc;
        STILL_CUDA(cudaMemcpyAsync(hY, dY, qb, cudaMemcpyDeviceToHost, st));
        if (hscores) STILL_CUDA(cudaMemcpyAsync(hscores, dsc, scb, cudaMemcpyDeviceToHost, st));
        if (hsel_idx && p->topk > 0) STILL_CUDA(cudaMemcpyAsync(hsel_idx, dsi, sib, cudaMemcpyDeviceToHost, st));
        STILL_CUDA(cudaStreamSynchronize(st));
        return STILL_OK;
    }
    // Events of the pipeline: created on first use per host thread and kept, like the side streams.
    static thread_local cudaEvent_t ev_start = nullptr, ev_in[kMaxParts] = {}, ev_done[kMaxParts] = {};
    if (!ev_start) STILL_CUDA(cudaEventCreateWithFlags(&ev_start, cudaEventDisableTiming));
    for (int i = 0; i < n_parts; ++i) {
        if (!ev_in[i]) STILL_CUDA(cudaEventCreateWithFlags(&ev_in[i], cudaEventDisableTiming));
        if (!ev_done[i]) STILL_CUDA(cudaEventCreateWithFlags(&ev_done[i], cudaEventDisableTiming));
    }
    // after a failure, whatever was enqueued drains before the call returns (the host buffers are the caller's)
    auto cleanup = [&]() {
        cudaStreamSynchronize(s_in);
        cudaStreamSynchronize(st);
        cudaStreamSynchronize(s_alt);
        cudaStreamSynchronize(s_out);
    };
    // the side streams start after what the caller has already enqueued (and after the weights)
    STILL_CUDA(cudaEventRecord(ev_start, st));
    STILL_CUDA(cudaStreamWaitEvent(s_in, ev_start, 0));
    STILL_CUDA(cudaStreamWaitEvent(s_alt, ev_start, 0));
    still_params_t sub = *p;
    sub.B = 1;
    sub.Hkv = g;
    sub.H = g * rep;
    // a second workspace for the alternate compute stream, if the arena's workspace holds two of a part's size
    const size_t ws_part = align_up(plan_fwd(&sub, N).total, 1024);
    const bool two_streams = n_parts > 1 && 2 * ws_part <= ws_bytes;
    const size_t q_part = (size_t)g * rep * N * p->d * es, kv_part = (size_t)g * N * p->d * es;
    const size_t sc_part = (size_t)g * rep * N * 4, si_part = (size_t)g * rep * T * std::max(p->topk, 1) * 4;
    const char *cQ = static_cast<const char *>(hQ), *cK = static_cast<const char *>(hK), *cV = static_cast<const char *>(hV);
    const char *cG = static_cast<const char *>(hG);
    for (int i = 0; i < n_parts; ++i) {
        cudaError_t e = cudaMemcpyAsync(dQ + i * q_part, cQ + i * q_part, q_part, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dK + i * kv_part, cK + i * kv_part, kv_part, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dV + i * kv_part, cV + i * kv_part, kv_part, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess && hG) e = cudaMemcpyAsync(dG + i * q_part, cG + i * q_part, q_part, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaEventRecord(ev_in[i], s_in);
        if (e != cudaSuccess) { cleanup(); return STILL_ERR_CUDA; }
    }
    for (int i = 0; i < n_parts && rc == STILL_OK; ++i) {
        const int kv0 = (i % parts_per_b) * g;   // first KV head of the part: selects its slice of the NP-Map weights
        const bool alt = two_streams && (i & 1);
        cudaStream_t cs = alt ? s_alt : st;
        char *ws_i = alt ? ws + ws_part : ws;
        const size_t ws_i_bytes = two_streams ? ws_part : ws_bytes;
        if (cudaStreamWaitEvent(cs, ev_in[i], 0) != cudaSuccess) { rc = STILL_ERR_CUDA; break; }
        rc = still_hybrid_attn_fwd(&sub, N, dQ + i * q_part, dK + i * kv_part, dV + i * kv_part,
                                   hG ? dG + i * q_part : nullptr,
                                   hWq ? dWq + (size_t)kv0 * rep * p->d * p->d_f * es : nullptr,
                                   hbq ? dbq + (size_t)kv0 * rep * p->d_f * es : nullptr,
                                   hWk ? dWk + (size_t)kv0 * p->d * p->d_f * es : nullptr,
                                   hbk ? dbk + (size_t)kv0 * p->d_f * es : nullptr, dY + i * q_part,
                                   reinterpret_cast<float *>(dsc + i * sc_part), reinterpret_cast<int32_t *>(dsi + i * si_part),
                                   nullptr, 0, ws_i, ws_i_bytes, cs);
        if (rc != STILL_OK) break;
        cudaError_t e = cudaEventRecord(ev_done[i], cs);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, ev_done[i], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(static_cast<char *>(hY) + i * q_part, dY + i * q_part, q_part, cudaMemcpyDeviceToHost, s_out);
        if (e == cudaSuccess && hscores)
            e = cudaMemcpyAsync(reinterpret_cast<char *>(hscores) + i * sc_part, dsc + i * sc_part, sc_part, cudaMemcpyDeviceToHost, s_out);
        if (e == cudaSuccess && hsel_idx && p->topk > 0)
            e = cudaMemcpyAsync(reinterpret_cast<char *>(hsel_idx) + i * si_part, dsi + i * si_part, si_part, cudaMemcpyDeviceToHost, s_out);
        if (e != cudaSuccess) rc = STILL_ERR_CUDA;
    }
    // everything enqueued has to drain before the host reads the outputs
    cudaError_t e1 = cudaStreamSynchronize(s_in), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(s_alt);
    cudaError_t e4 = cudaStreamSynchronize(s_out);
    if (rc != STILL_OK) return rc;
    if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess || e4 != cudaSuccess) return STILL_ERR_CUDA;
    return STILL_OK;
}

int still_device_status(const void *workspace_or_state, void *cuda_stream, int *status, int *detail) {
    if (!workspace_or_state || !status) return STILL_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int words[16];
    STILL_CUDA(cudaStreamSynchronize(st));
    STILL_CUDA(cudaMemcpy(words, workspace_or_state, sizeof(words), cudaMemcpyDeviceToHost));
    // A decode state keeps its status in header word 14/15, a workspace in word 0/1.
    const bool is_state = words[0] == 0x5354494c;
    *status = is_state ? words[14] : words[0];
    if (detail) *detail = is_state ? words[15] : words[1];
    return STILL_OK;
}

int still_last_launch_count(void) { return g_launches; }

int still_selftest_wait_timeout(void *status_block, int64_t limit_cycles, void *cuda_stream) {
    if (!status_block || misaligned(status_block) || limit_cycles <= 0) return STILL_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    STILL_CUDA(cudaMemsetAsync(status_block, 0, 256, st));
    return tc_selftest_wait_timeout(reinterpret_cast<int *>(status_block), limit_cycles, st);
}

int still_profile_enable(int max_records) {
    if (max_records <= 0 || g_prof_ev) return STILL_ERR_INVALID_ARG;
    g_prof_ev = new cudaEvent_t[2 * (size_t)max_records];
    for (int i = 0; i < 2 * max_records; ++i)
        if (cudaEventCreate(&g_prof_ev[i]) != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(g_prof_ev[j]);
            delete[] g_prof_ev;
            g_prof_ev = nullptr;
            return STILL_ERR_CUDA;
        }
    g_prof_cap = max_records;
    g_prof_used = 0;
    return STILL_OK;
}

int still_profile_collect(float *ms, int capacity, int *n_records) {
    if (!g_prof_ev || !ms || !n_records) return STILL_ERR_INVALID_ARG;
    int rc = STILL_OK, n = 0;
    for (int i = 0; i < g_prof_used; ++i) {
        float t = 0.f;
        if (cudaEventSynchronize(g_prof_ev[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&t, g_prof_ev[2 * i], g_prof_ev[2 * i + 1]) != cudaSuccess)
            rc = STILL_ERR_CUDA;
        else if (n < capacity)
            ms[n++] = t;
    }
    for (int i = 0; i < 2 * g_prof_cap; ++i) cudaEventDestroy(g_prof_ev[i]);
    delete[] g_prof_ev;
    g_prof_ev = nullptr;
    g_prof_cap = g_prof_used = 0;
    *n_records = n;
    return rc;
}

const char *still_strerror(int status) {
    switch (status) {
        case STILL_OK: return "ok";
        case STILL_ERR_INVALID_ARG: return "invalid argument";
        case STILL_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case STILL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case STILL_ERR_STATE_FULL: return "decode state is full";
        case STILL_ERR_CUDA: return "CUDA call failed";
        case STILL_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case STILL_ERR_STATE_MISMATCH: return "decode state does not match the parameters";
        default: return "unknown status";
    }
}

}  // extern "C"
