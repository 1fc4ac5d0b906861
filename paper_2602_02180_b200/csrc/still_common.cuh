// Shared device helpers of the STILL kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace still {

// Words of the 256-byte status block at the start of a workspace / decode state.
enum StatusWord { kStatusCode = 0, kStatusDetail = 1 };

__device__ __forceinline__ float ld_f(const float *p) { return *p; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st_f(float *p, float v) { *p = v; }
__device__ __forceinline__ void st_f(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Records the first device-side failure (bounded wait expired, state mismatch).
__device__ __forceinline__ void report_status(int *status, int code, int detail) {
    if (atomicCAS(status + kStatusCode, 0, code) == 0) status[kStatusDetail] = detail;
}

// ---------------------------------------------------------------------------
// Self-Saliency Score of one token from the logits of its window (Sec. 3.1).
// The warp holds the window: lane j has slots j, j+32, ... (spl = C/32 per lane),
// slot C-1 is the token itself, an absent slot holds -inf.  a_diag is the softmax
// over the window, a_nodiag the softmax over the window without the token (with
// its own max, so it cannot degenerate to 0/0), and
//   Score = sum_j a_diag_j log((a_diag_j + eps) / (a_nodiag_j + eps)).
// Returns the score in every lane.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float window_score(const float (&l)[4], int lane, int spl, int C, float eps) {
    float m_all = -INFINITY, m_nd = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (i < spl) {
            m_all = fmaxf(m_all, l[i]);
            if (lane + 32 * i != C - 1) m_nd = fmaxf(m_nd, l[i]);
        }
    m_all = warp_max(m_all);
    m_nd = warp_max(m_nd);
    float e_all[4], e_nd[4], z_all = 0.f, z_nd = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        e_all[i] = 0.f;
        e_nd[i] = 0.f;
        if (i < spl && l[i] != -INFINITY) {
            e_all[i] = expf(l[i] - m_all);
            z_all += e_all[i];
            if (lane + 32 * i != C - 1) {
                e_nd[i] = expf(l[i] - m_nd);
                z_nd += e_nd[i];
            }
        }
    }
    z_all = warp_sum(z_all);
    z_nd = warp_sum(z_nd);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (i < spl && l[i] != -INFINITY) {
            float a = e_all[i] / z_all;
            float bb = (lane + 32 * i != C - 1 && z_nd > 0.f) ? e_nd[i] / z_nd : 0.f;
            s += a * logf((a + eps) / (bb + eps));
        }
    return warp_sum(s);
}

// ---------------------------------------------------------------------------
// Top-k of one chunk (Sec. 3.3, delayed selection).  sc[0..n_c) are the scores of
// the chunk's tokens in shared memory, flag[0..C) is shared scratch.  Rank under
// (score descending, position ascending) with NaN as -inf; the k best positions
// are written to out[0..k) in ascending order, -1 padded.  Must be called by all
// threads of a block with at least C threads; flag[r] = 1 marks a selected token.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void select_chunk(const float *sc, int *flag, int n_c, int C, int lam,
                                             long long base, int32_t *out) {
    const int r = threadIdx.x;
    int selected = 0;
    if (r < C) {
        if (r < n_c) {
            float mine = sc[r];
            if (isnan(mine)) mine = -INFINITY;
            int rank = 0;
            for (int j = 0; j < n_c; ++j) {
                float o = sc[j];
                if (isnan(o)) o = -INFINITY;
                rank += (o > mine) || (o == mine && j < r);
            }
            selected = rank < lam;
        }
        flag[r] = selected;
    }
    __syncthreads();
    if (r < C) {
        int before = 0;
        for (int j = 0; j < r; ++j) before += flag[j];
        if (selected) out[before] = (int32_t)(base + r);
        int n_sel = n_c < lam ? n_c : lam;
        if (r >= n_sel && r < lam) out[r] = -1;
    }
}

// ---------------------------------------------------------------------------
// Norm-Preserved Feature Map of one row by one warp (Sec. 3.2, Eq. feature_map):
// u = f(x) ||x|| / max(||f(x)||, 1e-12), f(x) = xW + b, phi = [softmax(u),
// softmax(-u)].  xw: the row in shared memory as fp32; W [d][df] and bias [df]
// (or NULL) in any memory.  Lane j produces features j, j+32, ... of both halves:
// pos[jj] = softmax(u)_j, neg[jj] = softmax(-u)_j.
// ---------------------------------------------------------------------------
template <typename TW>
__device__ __forceinline__ void npmap_row(const float *xw, const TW *W, const TW *bias, int d, int df,
                                          int lane, float (&pos)[4], float (&neg)[4]) {
    const int jpl = df >> 5;
    float nx2 = 0.f;
    for (int i = lane; i < d; i += 32) nx2 += xw[i] * xw[i];
    nx2 = warp_sum(nx2);
    float f[4], nf2 = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) f[jj] = (jj < jpl && bias) ? ld_f(bias + lane + 32 * jj) : 0.f;
    for (int i = 0; i < d; ++i) {   // one read of x_i serves the lane's (up to) four outputs
        const float xi = xw[i];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
            if (jj < jpl) f[jj] = fmaf(xi, ld_f(W + i * df + lane + 32 * jj), f[jj]);
    }
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
        if (jj < jpl) nf2 += f[jj] * f[jj];
    nf2 = warp_sum(nf2);
    const float ratio = sqrtf(nx2) / fmaxf(sqrtf(nf2), 1e-12f);
    float umax = -INFINITY, umin = INFINITY;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
        if (jj < jpl) {
            f[jj] *= ratio;
            umax = fmaxf(umax, f[jj]);
            umin = fminf(umin, f[jj]);
        }
    umax = warp_max(umax);
    umin = warp_min(umin);
    float zp = 0.f, zn = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
        pos[jj] = neg[jj] = 0.f;
        if (jj < jpl) {
            pos[jj] = expf(f[jj] - umax);
            neg[jj] = expf(umin - f[jj]);
            zp += pos[jj];
            zn += neg[jj];
        }
    }
    zp = warp_sum(zp);
    zn = warp_sum(zn);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
        pos[jj] /= zp;
        neg[jj] /= zn;
    }
}

}  // namespace still
