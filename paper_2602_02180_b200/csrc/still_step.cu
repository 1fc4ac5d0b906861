// Decode: one step of the Recurrent Form (Sec. 3.3) on the decode state.
//
//   step_append_score : appends (k_t, v_t) to the K/V history and computes the
//                       Self-Saliency Score of the new token (Sec. 3.1).
//   step_route        : when the new token opens a chunk, the chunk that has just
//                       left the two-chunk local region is routed (Eq.
//                       delayed_selection, Eq. cache_routing_sum): top-k positions
//                       into sel_idx, every other token into (S, z) through the
//                       NP-Map.
//   step_attend       : split-KV pass over the salient cache h_t (selected rows of
//                       the routed chunks + the local region), one partial
//                       (max, sum, numerator) per split; HBM-bound.
//   step_merge        : combines the partials, reads out the linear branch and
//                       applies y = (N_SA + N_LA) / (D_SA + D_LA).
#include "still_common.cuh"
#include "still_step_mma.cuh"
#include "still_tc.h"

#include <algorithm>

namespace still {

constexpr int kMaxSplits = 32;  // history splits; one more partial holds the local region

long long state_kv_rows(const still_params_t *p, long long capacity) {
    if (p->max_salient <= 0 || p->topk <= 0) return capacity;
    const long long window = p->max_salient / p->topk;   // chunks whose selections stay cached
    return std::min<long long>(capacity, (window + 3) * p->chunk);
}

size_t step_scratch_bytes(const still_params_t *p, long long) {
    return (size_t)p->B * p->H * (kMaxSplits + 1) * (p->d + 2) * sizeof(float);
}

template <int n, typename T>
__device__ __forceinline__ void load_vec(const T *p, float (&out)[n]);
template <>
__device__ __forceinline__ void load_vec<2, float>(const float *p, float (&out)[2]) {
    float2 v = *reinterpret_cast<const float2 *>(p);
    out[0] = v.x; out[1] = v.y;
}
template <>
__device__ __forceinline__ void load_vec<4, float>(const float *p, float (&out)[4]) {
    float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void load_vec<2, __nv_bfloat16>(const __nv_bfloat16 *p, float (&out)[2]) {
    float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p));
    out[0] = v.x; out[1] = v.y;
}
template <>
__device__ __forceinline__ void load_vec<4, __nv_bfloat16>(const __nv_bfloat16 *p, float (&out)[4]) {
    uint2 raw = *reinterpret_cast<const uint2 *>(p);
    float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
    float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
    out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}

// What a step expects to find in the header of the decode state.
struct StateKey {
    int32_t B, H, Hkv, d, d_f, chunk, topk, dtype;
    long long cap, t;
};

// Header words 0-13 against the call: 0 if they agree, else a detail code (1: token count, 2: not a
// state / other layout version, 3: built with other parameters or another capacity, 4: an earlier step
// has already failed).  Nothing writes these words while the first kernel of a step runs.
__device__ __forceinline__ int state_mismatch(const int32_t *hdr, const StateKey &k) {
    if (hdr[0] != 0x5354494c || hdr[1] != 1) return 2;
    if (hdr[2] != k.B || hdr[3] != k.H || hdr[4] != k.Hkv || hdr[5] != k.d || hdr[6] != k.d_f || hdr[7] != k.chunk ||
        hdr[8] != k.topk || hdr[9] != k.dtype)
        return 3;
    const long long cap = ((long long)hdr[11] << 32) | (unsigned int)hdr[10];
    if (cap != k.cap) return 3;
    if (hdr[14] != 0) return 4;
    const long long have = ((long long)hdr[13] << 32) | (unsigned int)hdr[12];
    return have != k.t ? 1 : 0;
}

// grid (H, B), 32 threads: one warp scores the new token of one query head.  This is the first kernel of a
// step: every block compares the header with the call and leaves the state untouched on a mismatch (block
// (0, 0) records it); the later kernels of the step only look at the status word.
template <typename T>
__global__ void step_append_score_kernel(T *__restrict__ kc, T *__restrict__ vc,
                                         float *__restrict__ score, int32_t *__restrict__ hdr,
                                         const T *__restrict__ q, const T *__restrict__ k,
                                         const T *__restrict__ v, StateKey key, int H, int Hkv, long long cap,
                                         long long kvr, int d, int C, long long t, float scale, float eps) {
    __shared__ float qs[128];
    const int h = blockIdx.x, b = blockIdx.y, rep = H / Hkv, kv = h / rep, lane = threadIdx.x;
    {
        const int bad = state_mismatch(hdr, key);
        if (bad != 0) {
            if (h == 0 && b == 0 && lane == 0 && bad != 4) report_status(hdr + 14, STILL_ERR_STATE_MISMATCH, bad);
            return;
        }
    }
    const T *kn = k + ((long long)b * Hkv + kv) * d;
    // K / V rows live in a ring of kvr rows per KV head (kvr = capacity unless the salient cache has a budget)
    T *krow = kc + (((long long)b * Hkv + kv) * kvr + t % kvr) * d;
    if (h % rep == 0) {
        const T *vn = v + ((long long)b * Hkv + kv) * d;
        T *vrow = vc + (((long long)b * Hkv + kv) * kvr + t % kvr) * d;
        for (int i = lane; i < d; i += 32) {
            krow[i] = kn[i];
            vrow[i] = vn[i];
        }
    }
    for (int i = lane; i < d; i += 32) qs[i] = ld_f(q + ((long long)b * H + h) * d + i);
    __syncwarp();
    const int spl = C >> 5;
    float l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        l[i] = -INFINITY;
        if (i < spl) {
            int j = lane + 32 * i;
            long long pos = t - (C - 1) + j;
            if (pos >= 0) {
                // the new key is read from the input, not from the cache row another block writes
                const T *kr = (pos == t) ? kn : kc + (((long long)b * Hkv + kv) * kvr + pos % kvr) * d;
                float acc = 0.f;
                for (int x = 0; x < d; ++x) acc = fmaf(qs[x], ld_f(kr + x), acc);
                l[i] = acc * scale;
            }
        }
    }
    float s = window_score(l, lane, spl, C, eps);
    if (lane == 0) score[((long long)b * H + h) * cap + t] = s;
}

// grid (H, B), 256 threads.  Routes chunk cr (complete, C tokens): top-k into sel_idx / sel_mask, the other tokens
// into (S, z).  With a salient-cache budget of `window` chunks the selected tokens of chunk cr - window leave the
// cache at the same moment and are folded into (S, z) as well.
template <typename T>
__global__ void __launch_bounds__(256)
step_route_kernel(const T *__restrict__ kc, const T *__restrict__ vc, const float *__restrict__ score,
                  int32_t *__restrict__ sel_idx, uint32_t *__restrict__ sel_mask, float *__restrict__ S,
                  float *__restrict__ z, const T *__restrict__ Wk, const T *__restrict__ bk, const int32_t *__restrict__ hdr,
                  int H, int Hkv, long long cap, long long kvr, int d, int df, int C, int lam, long long cr, int window,
                  int w_in_smem) {
    extern __shared__ float smem[];
    if (hdr[14] != 0) return;   // the step's first kernel found the state not to match the call
    const int dp = 2 * df;
    float *ph = smem;                 // [C][dp]
    float *vs = ph + C * dp;          // [C][d]
    float *xs = vs + C * d;           // [8][d]
    float *sc = xs + 8 * d;           // [C]
    int *flag = reinterpret_cast<int *>(sc + C);  // [C]
    T *Ws = reinterpret_cast<T *>(flag + C);      // [d][df] the head's W_k (read once per row of the chunk otherwise)
    const int h = blockIdx.x, b = blockIdx.y, kv = h / (H / Hkv);
    const long long bh = (long long)b * H + h;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < C; i += blockDim.x) {
        sc[i] = score[bh * cap + cr * C + i];
        flag[i] = 0;
    }
    __syncthreads();
    if (lam > 0) select_chunk(sc, flag, C, C, lam, cr * C, sel_idx + (bh * (cap / C) + cr) * lam);
    __syncthreads();
    if (threadIdx.x < C / 32) {  // the same selection as bit masks (read by the split-KV pass)
        uint32_t bits = 0u;
        for (int j = 0; j < 32; ++j) bits |= (flag[threadIdx.x * 32 + j] ? 1u : 0u) << j;
        sel_mask[(bh * (cap / C) + cr) * (C / 32) + threadIdx.x] = bits;
    }
    const T *Wh = Wk + (long long)kv * d * df;
    const T *bh_ = bk ? bk + (long long)kv * df : nullptr;
    float *Sh = S + bh * dp * d;
    const T *Wuse = Wh;   // W_k from shared memory when it fits beside the chunk's tiles, else from global memory
    if (w_in_smem && (lam < C || window > 0)) {
        for (int i = threadIdx.x; i < d * df; i += blockDim.x) Ws[i] = Wh[i];
        Wuse = Ws;
    }
    // pass 0: the unselected tokens of chunk cr; pass 1: the selected tokens of the chunk that leaves the cache
    for (int pass = 0; pass < 2; ++pass) {
        const long long chunk = pass == 0 ? cr : cr - window;
        if (pass == 0 ? lam >= C : (window <= 0 || chunk < 0)) continue;   // nothing to fold in this pass
        __syncthreads();
        if (pass == 1) {   // fold[r] = 1 for the tokens to fold: here the chunk's selected ones, recorded when it was routed
            for (int i = threadIdx.x; i < C; i += blockDim.x)
                flag[i] = !((sel_mask[(bh * (cap / C) + chunk) * (C / 32) + i / 32] >> (i & 31)) & 1u);
            __syncthreads();
        }
        const long long base = chunk * C;
        const T *kh = kc + (((long long)b * Hkv + kv) * kvr + base % kvr) * d;   // (a chunk never straddles the ring's end)
        const T *vh = vc + (((long long)b * Hkv + kv) * kvr + base % kvr) * d;
        for (int i = threadIdx.x; i < C * d; i += blockDim.x) vs[i] = ld_f(vh + i);
        float *xw = xs + warp * d;
        for (int r = warp; r < C; r += 8) {   // flag[r] != 0: the token stays out of this pass
            float ep[4], en[4];
            if (!flag[r]) {
                for (int i = lane; i < d; i += 32) xw[i] = ld_f(kh + (long long)r * d + i);
                __syncwarp();
                npmap_row(xw, Wuse, bh_, d, df, lane, ep, en);
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
                if (jj < (df >> 5)) {
                    int j = lane + 32 * jj;
                    // features are rounded to the storage type, as the prefill stores them
                    T a, c2;
                    st_f(&a, flag[r] ? 0.f : ep[jj]);
                    st_f(&c2, flag[r] ? 0.f : en[jj]);
                    ph[r * dp + j] = ld_f(&a);
                    ph[r * dp + df + j] = ld_f(&c2);
                }
            __syncwarp();
        }
        __syncthreads();
        // S[f][e] += sum_i phi[i][f] v[i][e]: a thread owns 4 features x 8 value columns at a time, so that a token
        // costs 3 shared-memory reads for 32 multiply-adds
        for (int blk = threadIdx.x; blk < (dp / 4) * (d / 8); blk += blockDim.x) {
            const int f0 = (blk / (d / 8)) * 4, e0 = (blk % (d / 8)) * 8;
            float acc[4][8];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[a][c] = Sh[(f0 + a) * d + e0 + c];
            for (int i = 0; i < C; ++i) {
                const float4 pf = *reinterpret_cast<const float4 *>(ph + i * dp + f0);
                const float4 v0 = *reinterpret_cast<const float4 *>(vs + i * d + e0);
                const float4 v1 = *reinterpret_cast<const float4 *>(vs + i * d + e0 + 4);
                const float pa[4] = {pf.x, pf.y, pf.z, pf.w};
                const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc[a][c] = fmaf(pa[a], vv[c], acc[a][c]);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 8; ++c) Sh[(f0 + a) * d + e0 + c] = acc[a][c];
        }
        for (int f = threadIdx.x; f < dp; f += blockDim.x) {
            float acc = z[bh * dp + f];
            for (int i = 0; i < C; ++i) acc += ph[i * dp + f];
            z[bh * dp + f] = acc;
        }
    }
}

// grid (n_splits + 1, Hkv, B), 128 threads: warp w serves query heads w, w+4, ... of the group.
// Split s < n_splits covers routed chunks [s*cps, (s+1)*cps); split n_splits is the local region.
template <typename T, int DPL>
__global__ void __launch_bounds__(128)
step_attend_kernel(const T *__restrict__ kc, const T *__restrict__ vc,
                   const int32_t *__restrict__ sel_idx, const T *__restrict__ q,
                   float *__restrict__ part, const int32_t *__restrict__ hdr, int H, int Hkv, long long cap, int C,
                   int lam, long long t, int n_splits, long long cps, long long n_routed, float scale) {
    constexpr int d = DPL * 32;
    __shared__ float qs[4][d];
    if (hdr[14] != 0) return;
    const int split = blockIdx.x, kv = blockIdx.y, b = blockIdx.z, rep = H / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *kh = kc + ((long long)b * Hkv + kv) * cap * d;
    const T *vh = vc + ((long long)b * Hkv + kv) * cap * d;
    const bool local = split == n_splits;
    const long long c_cur = t / C;
    for (int hh = warp; hh < rep; hh += 4) {
        const int h = kv * rep + hh;
        const long long bh = (long long)b * H + h;
        for (int i = lane; i < d; i += 32) qs[warp][i] = ld_f(q + bh * d + i);
        __syncwarp();
        long long n_e, loc0 = 0;
        const int32_t *si = nullptr;
        if (local) {
            loc0 = c_cur >= 1 ? (c_cur - 1) * C : 0;
            n_e = t + 1 - loc0;
        } else {
            long long c_lo = split * cps, c_hi = (c_lo + cps < n_routed) ? c_lo + cps : n_routed;
            n_e = c_hi > c_lo ? (c_hi - c_lo) * lam : 0;
            si = sel_idx + (bh * (cap / C) + c_lo) * lam;
        }
        float m = -INFINITY, l = 0.f, o[DPL];
#pragma unroll
        for (int e = 0; e < DPL; ++e) o[e] = 0.f;
        for (long long e0 = 0; e0 < n_e; e0 += 32) {
            long long e = e0 + lane;
            long long pos = -1;
            if (e < n_e) pos = local ? loc0 + e : (long long)si[e];
            float s = -INFINITY;
            if (pos >= 0) {
                const T *kr = kh + pos * d;
                float acc = 0.f;
#pragma unroll 4
                for (int x = 0; x < d; x += 4) {
                    float kk[4];
                    load_vec<4>(kr + x, kk);
                    float4 qq = *reinterpret_cast<const float4 *>(&qs[warp][x]);
                    acc = fmaf(qq.x, kk[0], acc);
                    acc = fmaf(qq.y, kk[1], acc);
                    acc = fmaf(qq.z, kk[2], acc);
                    acc = fmaf(qq.w, kk[3], acc);
                }
                s = acc * scale;
            }
            float mn = fmaxf(m, warp_max(s));
            if (mn == -INFINITY) continue;
            float alpha = expf(m - mn);
            float pj = (pos >= 0) ? expf(s - mn) : 0.f;
            l = l * alpha + warp_sum(pj);
            m = mn;
#pragma unroll
            for (int x = 0; x < DPL; ++x) o[x] *= alpha;
            const int cnt = (n_e - e0 < 32) ? (int)(n_e - e0) : 32;
            for (int j = 0; j < cnt; ++j) {
                float pb = __shfl_sync(0xffffffffu, pj, j);
                long long pp = __shfl_sync(0xffffffffu, pos, j);
                if (pp < 0) continue;
                float vv[DPL];
                load_vec<DPL>(vh + pp * d + lane * DPL, vv);
#pragma unroll
                for (int x = 0; x < DPL; ++x) o[x] = fmaf(pb, vv[x], o[x]);
            }
        }
        float *pr = part + (bh * (kMaxSplits + 1) + split) * (d + 2);
        if (lane == 0) {
            pr[0] = m;
            pr[1] = l;
        }
#pragma unroll
        for (int x = 0; x < DPL; ++x) pr[2 + lane * DPL + x] = o[x];
        __syncwarp();
    }
}

// grid (H, B), 128 threads.
template <typename T>
__global__ void __launch_bounds__(128)
step_merge_kernel(const float *__restrict__ part, const float *__restrict__ S,
                  const float *__restrict__ z, const T *__restrict__ q, const T *__restrict__ g,
                  const T *__restrict__ Wq, const T *__restrict__ bq, T *__restrict__ y,
                  int32_t *__restrict__ hdr, int H, int d, int df, int n_splits, int la,
                  long long t) {
    __shared__ float qs[128], phi[256], red[4];
    if (hdr[14] != 0) return;   // mismatch recorded by the step's first kernel: no output, token count unchanged
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long bh = (long long)b * H + h;
    const int dp = 2 * df;
    const float *pr = part + bh * (kMaxSplits + 1) * (d + 2);
    float M = -INFINITY;
    for (int s = 0; s <= n_splits; ++s) M = fmaxf(M, pr[s * (d + 2)]);
    float Lsum = 0.f, O = 0.f;
    for (int s = 0; s <= n_splits; ++s) {
        float ms = pr[s * (d + 2)];
        if (ms == -INFINITY) continue;
        float w = expf(ms - M);
        Lsum += w * pr[s * (d + 2) + 1];
        if (tid < d) O += w * pr[s * (d + 2) + 2 + tid];
    }
    float nla = 0.f, dla = 0.f;
    if (la) {
        for (int i = tid; i < d; i += blockDim.x) qs[i] = ld_f(q + bh * d + i);
        __syncthreads();
        if (warp == 0) {
            float ep[4], en[4];
            npmap_row(qs, Wq + (long long)h * d * df, bq ? bq + (long long)h * df : (const T *)nullptr, d,
                      df, lane, ep, en);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
                if (jj < (df >> 5)) {
                    T a, c2;
                    st_f(&a, ep[jj]);
                    st_f(&c2, en[jj]);
                    phi[lane + 32 * jj] = ld_f(&a);
                    phi[df + lane + 32 * jj] = ld_f(&c2);
                }
        }
        __syncthreads();
        const float *Sh = S + bh * dp * d;
        if (tid < d)
            for (int f = 0; f < dp; ++f) nla = fmaf(phi[f], Sh[(long long)f * d + tid], nla);
        float part_d = 0.f;
        for (int f = tid; f < dp; f += blockDim.x) part_d = fmaf(phi[f], z[bh * dp + f], part_d);
        part_d = warp_sum(part_d);
        if (lane == 0) red[warp] = part_d;
        __syncthreads();
        dla = red[0] + red[1] + red[2] + red[3];
        if (g && tid < d) nla *= ld_f(g + bh * d + tid);
    }
    if (tid < d) {
        float fs = 1.f, fl = 0.f;
        if (dla > 0.f) {
            float ms = fmaxf(M, 0.f);
            fs = expf(M - ms);
            fl = expf(-ms);
        }
        st_f(y + bh * d + tid, (O * fs + fl * nla) / (Lsum * fs + fl * dla));
    }
    if (h == 0 && b == 0 && tid == 0) {
        long long nt = t + 1;
        hdr[12] = (int32_t)(nt & 0xffffffffll);
        hdr[13] = (int32_t)(nt >> 32);
    }
}

#define STILL_CUDA(expr)                               \
    do {                                               \
        cudaError_t e__ = (expr);                      \
        if (e__ != cudaSuccess) return STILL_ERR_CUDA; \
    } while (0)

template <typename T>
static int step_typed(const still_params_t *p, char *state, const still_state_layout_t *L, long long t,
                      const T *q, const T *k, const T *v, const T *g, const T *Wq, const T *bq,
                      const T *Wk, const T *bk, T *y, cudaStream_t st, int *launches) {
    const int C = p->chunk, d = p->d, df = p->d_f, lam = p->topk;
    const long long cap = L->capacity, kvr = state_kv_rows(p, cap);
    T *kc = reinterpret_cast<T *>(state + L->k_cache), *vc = reinterpret_cast<T *>(state + L->v_cache);
    float *score = reinterpret_cast<float *>(state + L->score);
    int32_t *sel = reinterpret_cast<int32_t *>(state + L->sel_idx);
    uint32_t *smask = reinterpret_cast<uint32_t *>(state + L->sel_mask);
    float *S = reinterpret_cast<float *>(state + L->S), *z = reinterpret_cast<float *>(state + L->z);
    float *part = reinterpret_cast<float *>(state + L->scratch);
    int32_t *hdr = reinterpret_cast<int32_t *>(state + L->header);
    const int window = lam > 0 ? (int)(p->max_salient / lam) : 0;   // chunks whose selections the salient cache holds
    const bool la = lam < C || window > 0;

    const StateKey key{p->B, p->H, p->Hkv, p->d, p->d_f, p->chunk, p->topk, p->dtype, cap, t};
    step_append_score_kernel<T><<<dim3(p->H, p->B), 32, 0, st>>>(kc, vc, score, hdr, q, k, v, key, p->H, p->Hkv,
                                                                  cap, kvr, d, C, t, p->sm_scale, p->eps);
    ++*launches;
    STILL_CUDA(cudaGetLastError());

    const long long c_cur = t / C;
    if (t % C == 0 && c_cur >= 2) {
        size_t smem = ((size_t)C * 2 * df + (size_t)C * d + 8 * (size_t)d + C) * 4 + (size_t)C * 4;
        const int w_in_smem = smem + (size_t)d * df * sizeof(T) <= 200 * 1024 ? 1 : 0;
        if (w_in_smem) smem += (size_t)d * df * sizeof(T);
        STILL_CUDA(cudaFuncSetAttribute(step_route_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)smem));
        step_route_kernel<T><<<dim3(p->H, p->B), 256, smem, st>>>(kc, vc, score, sel, smask, S, z, Wk, bk, hdr, p->H,
                                                                  p->Hkv, cap, kvr, d, df, C, lam, c_cur - 2, window, w_in_smem);
        ++*launches;
        STILL_CUDA(cudaGetLastError());
    }

    const long long n_routed = (lam > 0 && c_cur >= 2) ? c_cur - 1 : 0;  // chunks 0..c_cur-2
    int n_splits = 1;
    if constexpr (sizeof(T) == 2) {
        // bf16: tensor-core split-KV pass, the query heads of a KV group share every K / V row read
        if (p->H / p->Hkv > 16) return STILL_ERR_UNSUPPORTED;  // the group's heads are the 16 rows of one MMA tile
        // with a budget, the routed chunks still cached are the last `window` ones before the local region
        const long long first_pos = window > 0 ? std::max<long long>(0, c_cur - 1 - window) * C : 0;
        const long long nb = (t + 32) / 32 - first_pos / 32;  // 32-position key blocks
        const long long groups = (long long)p->B * p->Hkv;
        const long long want = (6 * 148 + groups - 1) / groups;  // about six waves of CTAs
        n_splits = (int)std::max<long long>(1, std::min<long long>({want, (long long)kMaxSplits + 1, (nb + 3) / 4}));
        dim3 grid(n_splits, p->Hkv, p->B);
        const float scale_log2 = p->sm_scale * 1.4426950408889634f;
        // a topk of 0 keeps nothing of the routed chunks: the kernel then sees only the local region
        profile_mark_begin(st);
        if (d == 64) {
            STILL_CUDA(ensure_dynamic_smem((const void *)step_attend_mma_kernel<64>, AttendPlan<64>::kTotal));
            step_attend_mma_kernel<64><<<grid, 128, AttendPlan<64>::kTotal, st>>>(
                (const __nv_bfloat16 *)kc, (const __nv_bfloat16 *)vc, smask, (const __nv_bfloat16 *)q, part, hdr, p->H, p->Hkv,
                cap, kvr, C, lam, t, first_pos, n_splits, kMaxSplits + 1, scale_log2);
        } else {
            STILL_CUDA(ensure_dynamic_smem((const void *)step_attend_mma_kernel<128>, AttendPlan<128>::kTotal));
            step_attend_mma_kernel<128><<<grid, 128, AttendPlan<128>::kTotal, st>>>(
                (const __nv_bfloat16 *)kc, (const __nv_bfloat16 *)vc, smask, (const __nv_bfloat16 *)q, part, hdr, p->H, p->Hkv,
                cap, kvr, C, lam, t, first_pos, n_splits, kMaxSplits + 1, scale_log2);
        }
        profile_mark_end(st);
        ++*launches;
        STILL_CUDA(cudaGetLastError());
        n_splits -= 1;  // the merge kernel reads partials 0 .. n_splits inclusive
    } else {
        if (n_routed > 0) {
            long long want = (2048 + (long long)p->B * p->Hkv - 1) / ((long long)p->B * p->Hkv);
            n_splits = (int)std::max<long long>(1, std::min<long long>({want, (long long)kMaxSplits, n_routed}));
        }
        const long long cps = n_routed > 0 ? (n_routed + n_splits - 1) / n_splits : 1;
        dim3 grid(n_splits + 1, p->Hkv, p->B);
        profile_mark_begin(st);
        if (d == 64)
            step_attend_kernel<T, 2><<<grid, 128, 0, st>>>(kc, vc, sel, q, part, hdr, p->H, p->Hkv, cap, C, lam, t,
                                                           n_splits, cps, n_routed, p->sm_scale);
        else
            step_attend_kernel<T, 4><<<grid, 128, 0, st>>>(kc, vc, sel, q, part, hdr, p->H, p->Hkv, cap, C, lam, t,
                                                           n_splits, cps, n_routed, p->sm_scale);
        profile_mark_end(st);
        ++*launches;
        STILL_CUDA(cudaGetLastError());
    }

    step_merge_kernel<T><<<dim3(p->H, p->B), 128, 0, st>>>(part, S, z, q, g, Wq, bq, y, hdr, p->H, d, df,
                                                           n_splits, la ? 1 : 0, t);
    ++*launches;
    STILL_CUDA(cudaGetLastError());
    return STILL_OK;
}

int step_launch(const still_params_t *p, char *state, const still_state_layout_t *L, long long t_pos,
                const void *q, const void *k, const void *v, const void *g, const void *Wq,
                const void *bq, const void *Wk, const void *bk, void *y, cudaStream_t st,
                int *launches) {
    if (p->dtype == STILL_DTYPE_FP32)
        return step_typed<float>(p, state, L, t_pos, (const float *)q, (const float *)k, (const float *)v,
                                 (const float *)g, (const float *)Wq, (const float *)bq, (const float *)Wk,
                                 (const float *)bk, (float *)y, st, launches);
    using bf = __nv_bfloat16;
    return step_typed<bf>(p, state, L, t_pos, (const bf *)q, (const bf *)k, (const bf *)v, (const bf *)g,
                          (const bf *)Wq, (const bf *)bq, (const bf *)Wk, (const bf *)bk, (bf *)y, st,
                          launches);
}

}  // namespace still
