// fp32 FMA kernels of the STILL layer: the path for fp32 inputs and for bf16
// shapes the tensor-core kernels do not cover.  Arithmetic is fp32 throughout;
// T is the storage type of Q/K/V/G/W/Y, TP the storage type of the NP-Map
// features kept in the workspace.
#pragma once
#include "still_common.cuh"

namespace still {

// ---------------------------------------------------------------------------
// Self-Saliency Score (Sec. 3.1) + per-chunk top-k (Sec. 3.3, delayed selection).
// One block per (chunk, head, batch).  A warp scores one token at a time: lane j
// holds the logits of window slots j, j+32, ...; slot C-1 is the token itself.
// a_diag is the softmax over the window, a_nodiag the softmax over the window
// without the token (own max, so it cannot underflow to 0/0), and
// Score = sum_j a_diag_j log((a_diag_j + eps) / (a_nodiag_j + eps)).
// Selection: rank under (score descending, position ascending), NaN as -inf;
// the k best are written in ascending position order, -1 padded.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
score_select_kernel(const T *__restrict__ Q, const T *__restrict__ K, float *__restrict__ scores,
                    int32_t *__restrict__ sel_idx, int H, int Hkv, long long N, int d, int C,
                    int lam, float scale, float eps) {
    extern __shared__ float smem[];
    const int c = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kv = h / (H / Hkv);
    const long long base = (long long)c * C;
    const int Tn = gridDim.x;
    float *kbuf = smem;                       // [2C][d+1]: previous chunk, then this chunk
    float *qbuf = kbuf + 2 * C * (d + 1);     // [C][d]
    float *sc = qbuf + C * d;                 // [C]
    int *flag = reinterpret_cast<int *>(sc + C);  // [C]
    const T *Qh = Q + ((long long)b * H + h) * N * d;
    const T *Kh = K + ((long long)b * Hkv + kv) * N * d;

    for (int i = threadIdx.x; i < 2 * C * d; i += blockDim.x) {
        int row = i / d, col = i - row * d;
        long long pos = base - C + row;
        kbuf[row * (d + 1) + col] = (pos >= 0 && pos < N) ? ld_f(Kh + pos * d + col) : 0.f;
    }
    for (int i = threadIdx.x; i < C * d; i += blockDim.x) {
        int row = i / d;
        long long pos = base + row;
        qbuf[i] = (pos < N) ? ld_f(Qh + pos * d + (i - row * d)) : 0.f;
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    const int spl = C >> 5;  // window slots per lane (C is a multiple of 32, at most 128)
    for (int r = warp; r < C; r += nwarp) {
        if (base + r >= N) {
            if (lane == 0) sc[r] = 0.f;
            continue;
        }
        float l[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            l[i] = -INFINITY;
            if (i < spl) {
                int j = lane + 32 * i;            // window slot; token position base + r - (C-1) + j
                long long pos = base + r - (C - 1) + j;
                if (pos >= 0) {
                    const float *kr = kbuf + (r + 1 + j) * (d + 1);
                    const float *qr = qbuf + r * d;
                    float acc = 0.f;
                    for (int x = 0; x < d; ++x) acc = fmaf(qr[x], kr[x], acc);
                    l[i] = acc * scale;
                }
            }
        }
        float s = window_score(l, lane, spl, C, eps);
        if (lane == 0) {
            sc[r] = s;
            if (scores) scores[((long long)b * H + h) * N + base + r] = s;
        }
    }
    __syncthreads();
    if (lam <= 0) return;

    const int n_c = (int)((N - base < C) ? (N - base) : C);
    select_chunk(sc, flag, n_c, C, lam, base, sel_idx + (((long long)b * H + h) * Tn + c) * lam);
}

// ---------------------------------------------------------------------------
// Norm-Preserved Feature Map (Sec. 3.2, Eq. feature_map) of every row of X.
// u = f(x) ||x|| / ||f(x)||, f(x) = xW + b; phi = [softmax(u), softmax(-u)].
// grid (ceil(N/64), heads, B); a warp maps one row at a time.
// ---------------------------------------------------------------------------
template <typename T, typename TP>
__global__ void __launch_bounds__(256)
npmap_kernel(const T *__restrict__ X, const T *__restrict__ W, const T *__restrict__ bias,
             TP *__restrict__ phi, int heads, long long N, int d, int df) {
    extern __shared__ float smem[];
    float *Ws = smem;             // [d][df]
    float *bs = Ws + d * df;      // [df]
    float *xs = bs + df;          // [8][d]
    const int hd = blockIdx.y, b = blockIdx.z;
    const T *Wh = W + (long long)hd * d * df;
    for (int i = threadIdx.x; i < d * df; i += blockDim.x) Ws[i] = ld_f(Wh + i);
    for (int i = threadIdx.x; i < df; i += blockDim.x) bs[i] = bias ? ld_f(bias + (long long)hd * df + i) : 0.f;
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int jpl = df >> 5;  // features per lane (df in {32, 64, 128})
    float *xw = xs + warp * d;
    for (int rr = warp; rr < 64; rr += 8) {
        long long row = (long long)blockIdx.x * 64 + rr;
        if (row >= N) break;
        const T *xr = X + (((long long)b * heads + hd) * N + row) * d;
        for (int i = lane; i < d; i += 32) xw[i] = ld_f(xr + i);
        __syncwarp();
        float ep[4], en[4];
        npmap_row(xw, Ws, bias ? bs : (const float *)nullptr, d, df, lane, ep, en);
        TP *pr = phi + (((long long)b * heads + hd) * N + row) * 2 * df;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
            if (jj < jpl) {
                int j = lane + 32 * jj;
                st_f(pr + j, ep[jj]);
                st_f(pr + df + j, en[jj]);
            }
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------
// Linear-attention branch (Algorithm 1 "Linear Attention Branch"; Eq.
// cache_routing_sum): sequential scan over chunks of one (batch, head) for a
// slice of 32 value columns.  At chunk c the state holds the LA tokens of chunks
// <= c-2:  S += sum_{i in M^LA_{c-2}} phi_k(k_i)^T v_i,  z += sum phi_k(k_i)^T;
// then N_LA = (phi_q(q) S) . g and D_LA = phi_q(q) z for the rows of chunk c.
// Thread (fg, e): fg = warp = group of FPT features, e = lane = value column.
// grid (B*H, d/32).  Final S, z go to the decode state when asked.
// ---------------------------------------------------------------------------
template <typename T, typename TP, int FPT>
__global__ void __launch_bounds__(256)
la_scan_kernel(const TP *__restrict__ phiQ, const TP *__restrict__ phiK, const T *__restrict__ V,
               const T *__restrict__ G, const int32_t *__restrict__ sel_idx,
               float *__restrict__ N_LA, float *__restrict__ D_LA, float *__restrict__ S_out,
               float *__restrict__ z_out, int H, int Hkv, long long N, int d, int C, int lam,
               int n_route /* chunks folded into the returned state */) {
    constexpr int DP = FPT * 8;
    extern __shared__ float smem[];
    float *ph = smem;                 // [32][DP] feature rows of the current sub-tile
    float *vt = ph + 32 * DP;         // [32][32]
    float *red = vt + 32 * 32;        // [8][32][33]
    float *zs = red + 8 * 32 * 33;    // [DP]
    int *keep = reinterpret_cast<int *>(zs + DP);  // [C] 1 = LA token
    const int bh = blockIdx.x, b = bh / H, h = bh % H, kv = h / (H / Hkv);
    const int e0 = blockIdx.y * 32;
    const int lane = threadIdx.x & 31, fg = threadIdx.x >> 5;
    const long long Tn = (N + C - 1) / C;
    const TP *pq = phiQ + (long long)bh * N * DP;
    const TP *pk = phiK + ((long long)b * Hkv + kv) * N * DP;
    const T *vh = V + ((long long)b * Hkv + kv) * N * d;
    float S[FPT];
#pragma unroll
    for (int i = 0; i < FPT; ++i) S[i] = 0.f;
    for (int i = threadIdx.x; i < DP; i += blockDim.x) zs[i] = 0.f;
    __syncthreads();

    const long long n_iter = (Tn > (long long)n_route + 2) ? Tn : (long long)n_route + 2;
    for (long long c = 0; c < n_iter; ++c) {
        if (c >= 2 && c - 2 < n_route) {
            const long long ub = (c - 2) * C;  // chunk c-2 is complete
            for (int i = threadIdx.x; i < C; i += blockDim.x) keep[i] = 1;
            __syncthreads();
            const int32_t *si = sel_idx + ((long long)bh * Tn + (c - 2)) * lam;
            for (int i = threadIdx.x; i < lam; i += blockDim.x) {
                int32_t p = si[i];
                if (p >= 0) keep[p - ub] = 0;
            }
            __syncthreads();
            for (int sub = 0; sub < C; sub += 32) {
                for (int i = threadIdx.x; i < 32 * DP; i += blockDim.x) {
                    int row = i / DP;
                    ph[i] = keep[sub + row] ? ld_f(pk + (ub + sub + row) * DP + (i - row * DP)) : 0.f;
                }
                for (int i = threadIdx.x; i < 32 * 32; i += blockDim.x) {
                    int row = i >> 5, col = i & 31;
                    vt[i] = ld_f(vh + (ub + sub + row) * d + e0 + col);
                }
                __syncthreads();
                for (int i = 0; i < 32; ++i) {
                    float vv = vt[i * 32 + lane];
#pragma unroll
                    for (int ii = 0; ii < FPT; ++ii) S[ii] = fmaf(ph[i * DP + fg * FPT + ii], vv, S[ii]);
                }
                if (threadIdx.x < DP) {
                    float a = zs[threadIdx.x];
                    for (int i = 0; i < 32; ++i) a += ph[i * DP + threadIdx.x];
                    zs[threadIdx.x] = a;
                }
                __syncthreads();
            }
        }
        if (c >= Tn) continue;
        const long long base = c * C;
        for (int sub = 0; sub < C; sub += 32) {
            if (base + sub >= N) break;
            for (int i = threadIdx.x; i < 32 * DP; i += blockDim.x) {
                int row = i / DP;
                long long pos = base + sub + row;
                ph[i] = (pos < N) ? ld_f(pq + pos * DP + (i - row * DP)) : 0.f;
            }
            __syncthreads();
            for (int r = 0; r < 32; ++r) {
                float acc = 0.f;
#pragma unroll
                for (int ii = 0; ii < FPT; ++ii) acc = fmaf(ph[r * DP + fg * FPT + ii], S[ii], acc);
                red[(fg * 32 + r) * 33 + lane] = acc;
            }
            __syncthreads();
            for (int i = threadIdx.x; i < 32 * 32; i += blockDim.x) {
                int r = i >> 5, e = i & 31;
                long long pos = base + sub + r;
                if (pos < N) {
                    float acc = 0.f;
#pragma unroll
                    for (int w = 0; w < 8; ++w) acc += red[(w * 32 + r) * 33 + e];
                    long long o = ((long long)bh * N + pos) * d + e0 + e;
                    if (G) acc *= ld_f(G + o);
                    N_LA[o] = acc;
                }
            }
            if (blockIdx.y == 0) {
                for (int r = fg; r < 32; r += 8) {
                    long long pos = base + sub + r;
                    float acc = 0.f;
                    for (int f = lane; f < DP; f += 32) acc = fmaf(ph[r * DP + f], zs[f], acc);
                    acc = warp_sum(acc);
                    if (lane == 0 && pos < N) D_LA[(long long)bh * N + pos] = acc;
                }
            }
            __syncthreads();
        }
    }
    if (S_out) {
#pragma unroll
        for (int ii = 0; ii < FPT; ++ii)
            S_out[((long long)bh * DP + fg * FPT + ii) * d + e0 + lane] = S[ii];
        if (blockIdx.y == 0)
            for (int i = threadIdx.x; i < DP; i += blockDim.x) z_out[(long long)bh * DP + i] = zs[i];
    }
}

// ---------------------------------------------------------------------------
// Softmax-attention branch + merge (Algorithm 1 "Softmax Attention Branch" and
// the output line; Sec. 3.3 merge equation).  One block per (chunk, head,
// batch).  The keys of chunk c are the selected tokens of chunks 0..c-2 (through
// sel_idx), all of chunk c-1 and the causal part of chunk c; they are streamed
// through shared memory 32 at a time.  A warp owns RPW query rows; per key tile a
// lane computes one logit per row, the row's running max / sum are updated
// online, and each lane accumulates DPL output columns.
// Merge: with m the running max, ms = max(m, 0):
//   y = (o e^{m-ms} + e^{-ms} N_LA) / (l e^{m-ms} + e^{-ms} D_LA).
// ---------------------------------------------------------------------------
template <typename T, int RPW, int DPL>
__global__ void __launch_bounds__(256)
sa_merge_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                const int32_t *__restrict__ sel_idx, const float *__restrict__ N_LA,
                const float *__restrict__ D_LA, T *__restrict__ Y, int H, int Hkv, long long N,
                int lam, float scale) {
    constexpr int C = RPW * 8, d = DPL * 32;
    extern __shared__ float smem[];
    float *qs = smem;                 // [C][d]
    float *ks = qs + C * d;           // [32][d+1]
    float *vs = ks + 32 * (d + 1);    // [32][d]
    long long *kpos = reinterpret_cast<long long *>(vs + 32 * d);  // [32]
    const int c = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kv = h / (H / Hkv);
    const long long Tn = gridDim.x, base = (long long)c * C, bh = (long long)b * H + h;
    const T *Qh = Q + bh * N * d;
    const T *Kh = K + ((long long)b * Hkv + kv) * N * d;
    const T *Vh = V + ((long long)b * Hkv + kv) * N * d;
    const int32_t *si = sel_idx + bh * Tn * lam;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < C * d; i += blockDim.x) {
        int row = i / d;
        long long pos = base + row;
        qs[i] = (pos < N) ? ld_f(Qh + pos * d + (i - row * d)) : 0.f;
    }
    const long long n_sel = (c >= 2) ? (long long)(c - 1) * lam : 0;
    const long long loc0 = (c >= 1) ? base - C : 0;
    const long long loc1 = (base + C < N) ? base + C : N;
    const long long L = n_sel + (loc1 - loc0);

    float m[RPW], l[RPW], o[RPW][DPL];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
#pragma unroll
        for (int e = 0; e < DPL; ++e) o[r][e] = 0.f;
    }
    for (long long t0 = 0; t0 < L; t0 += 32) {
        __syncthreads();
        if (threadIdx.x < 32) {
            long long e = t0 + threadIdx.x, p = -1;
            if (e < n_sel) p = si[e];
            else if (e < L) p = loc0 + (e - n_sel);
            kpos[threadIdx.x] = p;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < 32 * d; i += blockDim.x) {
            int row = i / d, col = i - row * d;
            long long p = kpos[row];
            ks[row * (d + 1) + col] = (p >= 0) ? ld_f(Kh + p * d + col) : 0.f;
            vs[i] = (p >= 0) ? ld_f(Vh + p * d + col) : 0.f;
        }
        __syncthreads();
        const long long p = kpos[lane];
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const long long t = base + warp * RPW + r;
            const float *qr = qs + (warp * RPW + r) * d;
            const float *kr = ks + lane * (d + 1);
            float s = 0.f;
#pragma unroll 8
            for (int x = 0; x < d; ++x) s = fmaf(qr[x], kr[x], s);
            const bool ok = (p >= 0) && (p <= t) && (t < N);
            s = ok ? s * scale : -INFINITY;
            float mn = fmaxf(m[r], warp_max(s));
            if (mn == -INFINITY) continue;  // nothing visible yet (uniform across the warp)
            float alpha = expf(m[r] - mn);
            float pj = ok ? expf(s - mn) : 0.f;
            l[r] = l[r] * alpha + warp_sum(pj);
            m[r] = mn;
#pragma unroll
            for (int e = 0; e < DPL; ++e) o[r][e] *= alpha;
            for (int j = 0; j < 32; ++j) {
                float pb = __shfl_sync(0xffffffffu, pj, j);
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[r][e] = fmaf(pb, vs[j * d + lane + 32 * e], o[r][e]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        const long long t = base + warp * RPW + r;
        if (t >= N) continue;
        float dla = D_LA ? D_LA[bh * N + t] : 0.f;
        float fs = 1.f, fl = 0.f;
        if (dla > 0.f) {
            float ms = fmaxf(m[r], 0.f);
            fs = expf(m[r] - ms);
            fl = expf(-ms);
        }
        float den = l[r] * fs + fl * dla;
#pragma unroll
        for (int e = 0; e < DPL; ++e) {
            long long oidx = (bh * N + t) * d + lane + 32 * e;
            float num = o[r][e] * fs;
            if (dla > 0.f) num += fl * N_LA[oidx];
            st_f(Y + oidx, num / den);
        }
    }
}

}  // namespace still
