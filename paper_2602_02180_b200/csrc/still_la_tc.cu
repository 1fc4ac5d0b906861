// Linear-attention branch of the prefill on tensor cores (bf16 inputs, sm_100a).
//
// npmap_tc_kernel -- Norm-Preserved Feature Map (Sec. 3.2, Eq. feature_map) of 128 rows of K per CTA,
//   fused into the load of the rows:  f = x W  on tcgen05 (x tile K-major from TMA, W MN-major from TMA,
//   accumulator in TMEM), then per row  u = (f + b) ||x|| / max(||f + b||, 1e-12),
//   phi = [softmax(u), softmax(-u)], stored as bf16 (the B operand of the bf16 state-update GEMM) once
//   per KV head, together with the column sums of every chunk.
//
// z_delta_kernel / z_scan_kernel -- the normaliser z of Eq. cache_routing_sum after every routed chunk:
//   column sums of the chunk minus the rows of its selected tokens, then a running sum over chunks.
//
// la_fused_kernel -- Algorithm 1 "Linear Attention Branch" with the state of Eq. cache_routing_sum kept
//   in tensor memory and the query-side NP-Map computed on the fly (phi(Q) never reaches HBM).  One CTA
//   owns one (batch, query head) and one half of the feature dimension (the softmax(u) features or the
//   softmax(-u) features) and walks the chunks in order.  The state half is held transposed, S^T
//   [value columns x d_f features] fp32 in TMEM.
//     update   S^T += V_c^T phi_k(K_c)   for the chunk c that has just left the two-chunk local region:
//              bf16 UMMA, A = V tile (M-major, as TMA delivers it), B = phi(K) half tile (MN-major)
//              whose rows of the tokens selected for softmax attention were zeroed;
//     map      f = Q W_q for a block of 128 query rows (UMMA), then a thread per row: norm re-injection,
//              this CTA's softmax half, written unnormalised (e_j = 2^(+-u_j - max)) as an fp32 K-major
//              tile into shared memory; D_part = (e . z_half of the chunk two back) / sum e;
//     read-out N_part^T = S^T phi_q(Q_c)^T  for the chunk c being answered: TF32 UMMA with the fp32
//              state read straight from TMEM as the A operand (10-bit mantissa instead of the 7 bits a
//              bf16 copy of the state would keep), B = the phi(Q) tile.
//   Output: y_part = N_part / D_part = (e . S) / (e . z) (times the gate) as bf16 and D_part as fp32, per feature half; the
//   merge epilogue of the attention kernel forms N_LA = sum y_part D_part, D_LA = sum D_part.
//   The lag of two chunks between update and read-out is the delayed selection of Sec. 3.3.  Work is
//   tiled in 64-token sub-chunks, so C = 128 is two sub-chunks per chunk.
//
// Roles of la_fused_kernel (384 threads): warp 0 TMA producer, warp 1 MMA issuer, warp 2 zeroes the
// selected rows of the phi(K) tiles, warps 4-7 write the output, warps 8-11 the query-side map.  Every mbarrier
// wait is bounded; on expiry the kernel records STILL_ERR_DEVICE_TIMEOUT in the status word, all roles
// leave their loops and tensor memory is freed before the CTA exits.
#include "still_tc.h"

#include <algorithm>

#include "still_tc_ptx.cuh"

namespace still {

namespace {

using namespace ptx;

// Instruction descriptor of kind::tf32 (fp32 accumulation, both operands TF32, B K-major).
__host__ __device__ constexpr uint32_t make_idesc_tf32(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem, fp32 read as TF32] * B[smem desc]
__device__ __forceinline__ void mma_ts_tf32(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// ------------------------------------------------------------------------------------------
// NP-Map
// ------------------------------------------------------------------------------------------
// Shared memory of the NP-Map kernel: the x and W tiles, later reused as the staging space of the output
// (four warps x 32 padded rows); the region is the larger of the two.
template <int D, int DF, typename TOut>
struct NpmapSmem {
    static constexpr int kHalfChunks = 32 * (int)sizeof(TOut) / 16;   // 16-byte pieces of 32 features
    static constexpr int kStageRow = 2 * kHalfChunks * 16 + 16;       // padded: conflict-free 16-byte accesses
    static constexpr int kTiles = 128 * D * 2 + D * DF * 2;
    static constexpr int kStage = 4 * 32 * kStageRow;
    static constexpr int kRegion = ((kTiles > kStage ? kTiles : kStage) + 1023) / 1024 * 1024;
    static constexpr int kTotal = kRegion + 64;
};

template <int D, int DF, typename TOut>
__global__ void __launch_bounds__(192, 3)
npmap_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                const __nv_bfloat16 *__restrict__ bias, TOut *__restrict__ phi, float *__restrict__ csum, int *status,
                int heads, int N, int C) {
    constexpr int kXBytes = 128 * D * 2, kWBytes = D * DF * 2;
    using Lay = NpmapSmem<D, DF, TOut>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *x_s = smem, *w_s = smem + kXBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + Lay::kRegion);  // [0] loads done, [1] f done
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(bars + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_base_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hd = blockIdx.y, b = blockIdx.z, R0 = blockIdx.x * 128;
    const long long row0 = ((long long)b * heads + hd) * N + R0;
    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) report_status(status, STILL_ERR_DEVICE_TIMEOUT, 98);
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 1, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, 128);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp == 0 && lane == 0) {
        mbar_expect_tx(bars, kXBytes + kWBytes);
        for (int half = 0; half < D / 64; ++half)  // x rows: K-major, 64-element atoms 128 rows apart
            tma_load_2d(x_s + half * (128 * 128), &tm_x, bars, half * 64, (int)row0);
        for (int a = 0; a < DF / 64; ++a)          // W [d rows, d_f columns]: MN-major, 64-column atoms D rows apart
            tma_load_2d(w_s + a * (D * 128), &tm_w, bars, a * 64, hd * D);
    } else if (warp == 1 && lane == 0) {
        constexpr uint32_t idesc = make_idesc(128, DF, true);
        if (mbar_wait(bars, 0, abort_flag, status, 30)) {
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t xa = smem_u32(x_s) + (k / 4) * (128 * 128) + (k % 4) * 32;
                const uint32_t wa = smem_u32(w_s) + k * (16 * 128);
                mma_ss(tmem_base, smem_desc(xa, 0), smem_desc(wa, D * 128), idesc, k > 0 ? 1u : 0u);
            }
            tc_commit(bars + 1);
        }
    } else if (warp >= 2) {
        const int wq = warp & 3, r = wq * 32 + lane;   // TMEM lane quarter of this warp; row of the tile
        const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
        bool ok = mbar_wait(bars, 0, abort_flag, status, 31);   // x tile in shared memory
        ok = __all_sync(0xffffffffu, ok);
        float nx2 = 0.f;
        if (ok) {
#pragma unroll
            for (int a = 0; a < D / 64; ++a)
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(x_s + a * (128 * 128) + r * 128 + ((c ^ (r & 7)) << 4));
                    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = __uint_as_float(w4[e] << 16), hi = __uint_as_float(w4[e] & 0xffff0000u);
                        nx2 = fmaf(lo, lo, nx2);
                        nx2 = fmaf(hi, hi, nx2);
                    }
                }
        }
        // all four epilogue warps are done reading the x tile before any of them reuses it as staging space
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok) ok = mbar_wait(bars + 1, 0, abort_flag, status, 32);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            // Three passes over the row of f in tensor memory, 32 columns at a time, so that the row is
            // never held in registers (several CTAs per SM then overlap their load / MMA / epilogue
            // phases): norms and extrema, the two softmax denominators, the features themselves.
            const __nv_bfloat16 *bh_ = bias != nullptr ? bias + (long long)hd * DF : nullptr;
            float nf2 = 0.f, fmax_ = -INFINITY, fmin_ = INFINITY;
#pragma unroll 1
            for (int q = 0; q < DF / 32; ++q) {
                uint32_t v[32];
                tmem_ld32(taddr + q * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x = __uint_as_float(v[j]);
                    if (bh_ != nullptr) x += __bfloat162float(bh_[q * 32 + j]);
                    nf2 = fmaf(x, x, nf2);
                    fmax_ = fmaxf(fmax_, x);
                    fmin_ = fminf(fmin_, x);
                }
            }
            // u = f * ratio in the log2 domain; ratio > 0, so the extrema of u are those of f
            const float ratio = sqrtf(nx2) / fmaxf(sqrtf(nf2), 1e-12f) * 1.4426950408889634f;
            const float umax = fmax_ * ratio, umin = fmin_ * ratio;
            float zp = 0.f, zn = 0.f;
#pragma unroll 1
            for (int q = 0; q < DF / 32; ++q) {
                uint32_t v[32];
                tmem_ld32(taddr + q * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x = __uint_as_float(v[j]);
                    if (bh_ != nullptr) x += __bfloat162float(bh_[q * 32 + j]);
                    const float u = x * ratio;
                    zp += ex2(u - umax);
                    zn += ex2(umin - u);
                }
            }
            const float ip = 1.f / zp, in = 1.f / zn;
            // The features leave through shared memory: a thread owns a row, but a store instruction in
            // which every lane writes to a different row touches 32 lines; staged, 8 (fp32) or 4 (bf16)
            // consecutive lanes write one 128- or 64-byte run of a row.  Each warp stages and writes its
            // own 32 rows (the x / W tiles are dead by now), 32 columns of both halves at a time.
            constexpr int kHalfChunks = Lay::kHalfChunks, kStageRow = Lay::kStageRow;
            uint8_t *stage = smem + wq * (32 * kStageRow);
            const int rows_live = min(32, N - (R0 + wq * 32));        // rows of this warp that exist
            float *csw = reinterpret_cast<float *>(smem + 4 * 32 * kStageRow) + wq * (2 * DF);   // this warp's column sums
#pragma unroll 1
            for (int q = 0; q < DF / 32; ++q) {
                uint32_t v[32];
                tmem_ld32(taddr + q * 32, v);
                tmem_wait_ld();
                uint8_t *mine = stage + lane * kStageRow;
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    float u[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float x = __uint_as_float(v[j + e]);
                        if (bh_ != nullptr) x += __bfloat162float(bh_[q * 32 + j + e]);
                        u[e] = x * ratio;
                    }
                    if constexpr (sizeof(TOut) == 4) {
                        *reinterpret_cast<float4 *>(mine + j * 4) =
                            make_float4(ex2(u[0] - umax) * ip, ex2(u[1] - umax) * ip, ex2(u[2] - umax) * ip, ex2(u[3] - umax) * ip);
                        *reinterpret_cast<float4 *>(mine + kHalfChunks * 16 + j * 4) =
                            make_float4(ex2(umin - u[0]) * in, ex2(umin - u[1]) * in, ex2(umin - u[2]) * in, ex2(umin - u[3]) * in);
                    } else {
                        *reinterpret_cast<uint2 *>(mine + j * 2) =
                            make_uint2(pack_bf16(ex2(u[0] - umax) * ip, ex2(u[1] - umax) * ip),
                                       pack_bf16(ex2(u[2] - umax) * ip, ex2(u[3] - umax) * ip));
                        *reinterpret_cast<uint2 *>(mine + kHalfChunks * 16 + j * 2) =
                            make_uint2(pack_bf16(ex2(umin - u[0]) * in, ex2(umin - u[1]) * in),
                                       pack_bf16(ex2(umin - u[2]) * in, ex2(umin - u[3]) * in));
                    }
                }
                __syncwarp();
                if constexpr (sizeof(TOut) == 2) {
                    // column sums of the stored (bf16-rounded) features over the warp's rows, in row order: lane l
                    // adds feature 32 q + l of both halves (what the normaliser z of the linear branch is made of)
                    if (csum != nullptr) {
                        float sp = 0.f, sn = 0.f;
                        for (int row = 0; row < rows_live; ++row) {
                            const uint8_t *src = stage + row * kStageRow + lane * 2;
                            sp += __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t *>(src)) << 16);
                            sn += __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t *>(src + kHalfChunks * 16)) << 16);
                        }
                        csw[q * 32 + lane] = sp;
                        csw[DF + q * 32 + lane] = sn;
                    }
                }
#pragma unroll
                for (int it = 0; it < 2 * kHalfChunks; ++it) {
                    const int id = it * 32 + lane, row = id / (2 * kHalfChunks), c = id % (2 * kHalfChunks);
                    if (row < rows_live) {
                        const uint4 val = *reinterpret_cast<const uint4 *>(stage + row * kStageRow + c * 16);
                        uint8_t *dst = reinterpret_cast<uint8_t *>(phi + (row0 + wq * 32 + row) * (2 * DF) +
                                                                   (c < kHalfChunks ? 0 : DF) + q * 32) +
                                       (c % kHalfChunks) * 16;
                        *reinterpret_cast<uint4 *>(dst) = val;
                    }
                }
                __syncwarp();
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (sizeof(TOut) == 2) {
        // per-chunk column sums: the warps of a chunk are added in warp order (fixed order: the sums are reproducible)
        if (csum != nullptr && warp >= 2 && !*abort_flag) {
            const float *csw_all = reinterpret_cast<const float *>(smem + 4 * 32 * NpmapSmem<D, DF, TOut>::kStageRow);
            const int Tn = (N + C - 1) / C, wpc = C / 32;             // warps (of 32 rows) per chunk: 2 or 4
            for (int i = threadIdx.x - 64; i < (128 / C) * 2 * DF; i += 128) {
                const int k = i / (2 * DF), f = i % (2 * DF), chunk = R0 / C + k;
                if (chunk < Tn) {
                    float acc = 0.f;
                    for (int w = 0; w < wpc; ++w)
                        if (R0 + (k * wpc + w) * 32 < N) acc += csw_all[(k * wpc + w) * (2 * DF) + f];
                    csum[(((long long)b * heads + hd) * Tn + chunk) * (2 * DF) + f] = acc;
                }
            }
        }
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// ------------------------------------------------------------------------------------------
// Normaliser prefix z (Eq. cache_routing_sum): z after chunk c = sum over the chunks 0..c of the features
// of their unselected tokens = (column sums of phi(K) over the chunk) - (rows of its selected tokens).
// ------------------------------------------------------------------------------------------
// grid (routed chunks, B*H), 2 d_f threads: zpre[bh][c][f] = csum[kv][c][f] - sum_i phi(K)[sel[bh][c][i]][f], plus,
// with a salient-cache budget of `window` chunks, the selected rows of chunk c - window, which leave the cache
// for the state when chunk c is routed.
__global__ void z_delta_kernel(const float *__restrict__ csum, const __nv_bfloat16 *__restrict__ phiK,
                               const int32_t *__restrict__ sel_idx, float *__restrict__ zpre, int H, int Hkv, long long N,
                               int Tn, int n_routed, int lam, int C, int window, int NF) {
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H, kv = b * Hkv + h / (H / Hkv), f = threadIdx.x;
    float d = 0.f;
    if (lam < C) {   // (with lam = C every token of the chunk is selected: nothing is left over)
        d = csum[((long long)kv * Tn + c) * NF + f];
        const int32_t *si = sel_idx + ((long long)bh * Tn + c) * lam;
        for (int i = 0; i < lam; ++i) {
            const int p = si[i];
            if (p >= 0) d -= __bfloat162float(phiK[((long long)kv * N + p) * NF + f]);
        }
    }
    if (window > 0 && c >= window) {
        const int32_t *si = sel_idx + ((long long)bh * Tn + (c - window)) * lam;
        for (int i = 0; i < lam; ++i) {
            const int p = si[i];
            if (p >= 0) d += __bfloat162float(phiK[((long long)kv * N + p) * NF + f]);
        }
    }
    zpre[((long long)bh * n_routed + c) * NF + f] = d;
}
// grid (B*H), 2 d_f threads: in-place running sum over the routed chunks; the last value is the state's z.
__global__ void z_scan_kernel(float *__restrict__ zpre, float *__restrict__ z_out, int n_routed, int NF) {
    const int bh = blockIdx.x, f = threadIdx.x;
    float *z = zpre + (long long)bh * n_routed * NF + f;
    float acc = 0.f;
    for (int c0 = 0; c0 < n_routed; c0 += 8) {   // eight independent loads in flight, then the running sum
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = c0 + i < n_routed ? z[(long long)(c0 + i) * NF] : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            acc += v[i];
            if (c0 + i < n_routed) z[(long long)(c0 + i) * NF] = acc;
        }
    }
    if (z_out != nullptr) z_out[(long long)bh * NF + f] = acc;
}

// ------------------------------------------------------------------------------------------
// State scan with the query-side NP-Map fused into its loads
// ------------------------------------------------------------------------------------------
// One CTA owns one (batch, query head) and one half of the feature dimension: the softmax(u) half or the
// softmax(-u) half of phi (each d_f features).  N_LA and D_LA are sums over features, so the two CTAs of a
// head produce two partial results that the merge epilogue of the attention kernel adds.
template <int D, int DF>
struct FusedPlan {
    static constexpr int kW = D * DF * 2;               // W_q, MN-major (as TMA delivers [d rows, d_f columns])
    static constexpr int kX = 128 * D * 2;              // raw Q rows of one block of 128 tokens
    static constexpr int kPhiQ = 64 * DF * 4;           // phi_q half of 64 tokens, fp32 (TF32 operand)
    static constexpr int kUTok = 32;                    // tokens per state-update tile
    static constexpr int kUStages = 4;                  // ring of update tiles (loads run this far ahead of the MMAs)
    static constexpr int kPhiK = kUTok * DF * 2;        // phi_k half of an update tile, bf16
    static constexpr int kVt = kUTok * D * 2;           // V of an update tile
    static constexpr int kUStage = kPhiK + kVt;
    static constexpr int oW = 0;
    static constexpr int oX = oW + kW;
    static constexpr int oQ = oX + kX;                  // two slots
    static constexpr int oU = oQ + 2 * kPhiQ;           // kUStages stages
    static constexpr int oDinv = oU + kUStages * kUStage;      // [8][64] 1 / D_part of the tokens of the last sub-chunks
    static constexpr int oZ = oDinv + 8 * 64 * 4;       // [4 map warps][d_f] z half of the chunk two back
    static constexpr int oStage = oZ + 4 * DF * 4;      // [64 tokens][d] bf16: the output of a sub-chunk on its way out
    static constexpr int oBar = oStage + 64 * D * 2;
    static constexpr int kNumBars = 30;
    static constexpr int oMisc = oBar + kNumBars * 8;
    static constexpr int kTotal = oMisc + 16;
};
static_assert(FusedPlan<128, 128>::kTotal <= 232448 && FusedPlan<128, 64>::kTotal <= 232448 && FusedPlan<64, 64>::kTotal <= 232448,
              "fused scan: the shared-memory plan exceeds what a CTA can have");

template <int D, int DF>
__global__ void __launch_bounds__(384, 1)
la_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_wq,
                const __grid_constant__ CUtensorMap tm_phik, const __grid_constant__ CUtensorMap tm_v,
                const __grid_constant__ CUtensorMap tm_phiks, const __grid_constant__ CUtensorMap tm_vs,
                const __nv_bfloat16 *__restrict__ bq, const __nv_bfloat16 *__restrict__ G,
                const int32_t *__restrict__ sel_idx, const float *__restrict__ zpre, __nv_bfloat16 *__restrict__ y_part,
                float *__restrict__ d_part, float *__restrict__ S_out, float *__restrict__ seg_sums, int *status, int H, int Hkv,
                int N, int C, int lam, int window, long long part_stride_y, long long part_stride_d, int seg_chunks, int n_seg,
                int sum_parts, int sums_only, int sel_rows) {
    using P = FusedPlan<D, DF>;
    constexpr int NF = 2 * DF;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + P::oBar);
    uint64_t *w_full = bars, *x_full = bars + 1, *x_empty = bars + 2;
    uint64_t *f_done = bars + 28, *f_free = bars + 3;   // [2] each: f of even / odd blocks
    uint64_t *pq_full = bars + 5, *pq_empty = bars + 7, *r_done = bars + 9, *out_free = bars + 11, *fin = bars + 13;
    uint64_t *init_done = bars + 14, *u_full = bars + 15, *u_empty = u_full + P::kUStages, *u_masked = u_empty + P::kUStages;
    constexpr int kUS = P::kUStages, kUTok = P::kUTok;
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(smem + P::oMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + P::oMisc + 8);
    float *dinv_ring = reinterpret_cast<float *>(smem + P::oDinv);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;   // (known to be the same in all lanes)
    const int bh = blockIdx.x, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int half = blockIdx.y;                // 0: features softmax(u), 1: features softmax(-u)
    const int sc = C / 64;                      // 64-token sub-chunks per chunk
    const int Tn = (N + C - 1) / C;
    const int n_routed = Tn >= 3 ? Tn - 2 : 0;  // chunks whose tokens enter the state
    // The sequence is cut into n_seg segments of seg_chunks chunks (two-level scan): segment g answers the
    // sub-chunks [u_first, NU) and performs the updates that fall between them, starting from the sum of the
    // earlier segments' updates (seg_sums, produced by a first pass of this kernel with sums_only set).
    // The first pass cuts every segment into sum_parts pieces, one CTA each (it has no scan to keep in order, and
    // the pieces fill the SMs that the n_seg - 1 summed segments alone would leave idle).
    const int seg = blockIdx.z;
    if (sums_only) seg_chunks /= sum_parts;
    const int NU_all = (N + 63) / 64;           // sub-chunks with query rows
    const int u_first = seg == 0 ? 2 * sc : seg * seg_chunks * sc;   // the first two chunks see an empty state
    const int NU = (!sums_only && seg == n_seg - 1) ? NU_all : min(NU_all, (seg + 1) * seg_chunks * sc);
    const int b_first = u_first / 2;            // blocks of 128 query rows: [b_first, NB)
    const int NB = sums_only ? b_first : (NU + 1) / 2;
    // Update tiles of kUTok tokens: per routed chunk its su tiles (selected rows zeroed) and, with a salient-cache
    // budget of `window` chunks, the su tiles of the chunk `window` back with everything but its selected rows
    // zeroed: those tokens leave the cache for the state when the chunk is routed.
    // With sel_rows > 0 the leaving tokens come from the gathered copies of their phi(K) and V rows (sel_rows rows
    // per head, lam per chunk): nl tiles per chunk instead of su, and only a last partial tile has rows to clear.
    const int su = C / kUTok;
    const int nl = sel_rows > 0 ? (lam + kUTok - 1) / kUTok : su;
    const int per_chunk = window > 0 ? su + nl : su;
    const int nu0 = (u_first / sc - 2) * per_chunk;    // first update tile of the segment
    const int n_upd = NU > u_first ? ((NU - 1) / sc - 1) * per_chunk - nu0 : 0;
    const bool has_init = !sums_only && seg > 0;
    __nv_bfloat16 *y_out = y_part + (long long)half * part_stride_y;
    float *d_out = d_part + (long long)half * part_stride_d;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) report_status(status, STILL_ERR_DEVICE_TIMEOUT, 97);
        return;
    }
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status) != 0;
    __syncthreads();
    if (*abort_flag) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_init(w_full, 1);
        mbar_init(x_full, 1);
        mbar_init(x_empty, 5);      // the f GEMM has read the rows (1) and so have the four map warps (4)
        for (int i = 0; i < 2; ++i) {
            mbar_init(f_done + i, 1);
            mbar_init(f_free + i, 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(pq_full + i, 2);   // the two map warps that own the slot's 64 rows
            mbar_init(pq_empty + i, 1);
            mbar_init(r_done + i, 1);
            mbar_init(out_free + i, 4);
        }
        for (int i = 0; i < kUS; ++i) {
            mbar_init(u_full + i, 1);
            mbar_init(u_empty + i, 1);
            mbar_init(u_masked + i, 1);
        }
        mbar_init(fin, 1);
        mbar_init(init_done, 4);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_base_slot, 0);
    // TMEM columns: S^T half [value lanes x d_f features] fp32; f = x W_q of a block [128 rows x d_f]; two read-out
    // results [value lanes x 64 tokens]
    constexpr uint32_t col_state = 0, col_f = DF, col_out = 3 * DF;   // f: two buffers of DF columns

    // Registers move from the first warpgroup (single-thread roles) to the map warps, whose threads hold a row of f
    // (per scheduler: 72 + 152 + 224 registers for its three warps, of the 3 x 168 the CTA was launched with).
    if (warp < 4) {
    reg_dec<72>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int kv_row0 = (b * Hkv + kvh) * N, q_row0 = bh * N;
            const int n_blk = NB > b_first ? NB - b_first : 0;
            if (n_blk > 0) {
                mbar_expect_tx(w_full, P::kW);
                for (int a = 0; a < DF / 64; ++a) tma_load_2d(smem + P::oW + a * (D * 128), &tm_wq, w_full, a * 64, h * D);
            }
            int nu = 0, nx = 0, spins = 0;
            long long t0 = clock64();
            while (nu < n_upd || nx < n_blk) {
                bool progressed = false;
                if (nx < n_blk && mbar_try_wait(x_empty, (nx & 1) ^ 1)) {
                    mbar_expect_tx(x_full, P::kX);
                    for (int a = 0; a < D / 64; ++a)   // K-major, 64-element atoms 128 rows apart
                        tma_load_2d(smem + P::oX + a * (128 * 128), &tm_q, x_full, a * 64, q_row0 + (b_first + nx) * 128);
                    ++nx;
                    progressed = true;
                }
                if (nu < n_upd && mbar_try_wait(u_empty + nu % kUS, ((nu / kUS) & 1) ^ 1)) {
                    uint8_t *stg = smem + P::oU + (nu % kUS) * P::kUStage;
                    // tile a = nu0 + nu: chunk a / per_chunk, then which of its tiles; a leaving-tile reads the chunk
                    // `window` back (before there is one, any valid tile: all its rows are zeroed)
                    const int a_t = nu0 + nu, cc = a_t / per_chunk, rt = a_t % per_chunk;
                    const int src = (rt >= su && cc >= window) ? cc - window : cc;
                    const bool gathered = rt >= su && sel_rows > 0;
                    // first row of the tile: in phi(K) / V of the KV head, or in the head's gathered rows
                    const int row = gathered ? bh * sel_rows + src * lam + (rt - su) * kUTok : kv_row0 + (src * su + rt % su) * kUTok;
                    const CUtensorMap *mp = gathered ? &tm_phiks : &tm_phik, *mv = gathered ? &tm_vs : &tm_v;
                    mbar_expect_tx(u_full + nu % kUS, P::kUStage);
                    for (int a = 0; a < DF / 64; ++a)  // phi(K) half: MN-major, 64-feature atoms kUTok rows apart
                        tma_load_2d(stg + a * (kUTok * 128), mp, u_full + nu % kUS, half * DF + a * 64, row);
                    for (int a = 0; a < D / 64; ++a)   // V: M-major A operand, 64-column atoms kUTok rows apart
                        tma_load_2d(stg + P::kPhiK + a * (kUTok * 128), mv, u_full + nu % kUS, a * 64, row);
                    ++nu;
                    progressed = true;
                }
                if (progressed) {
                    spins = 0;
                } else if ((++spins & 1023) == 0) {
                    if (spins == 1024) t0 = clock64();
                    if (*abort_flag) break;
                    if (clock64() - t0 > kWaitLimitCycles) {
                        *abort_flag = 1;
                        report_status(status, STILL_ERR_DEVICE_TIMEOUT, 60);
                        break;
                    }
                }
            }
            if (*abort_flag) {  // leave no copy in flight behind
                if (nu > 0) mbar_wait_drain(u_full + (nu - 1) % kUS, ((nu - 1) / kUS) & 1);
                if (nx > 0) mbar_wait_drain(x_full, (nx - 1) & 1);
                if (n_blk > 0) mbar_wait_drain(w_full, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the schedule and waits on the barriers; one elected lane issues (control flow and
        // descriptors stay the same in all lanes and can live in uniform registers, where the tensor-core
        // instructions take their operands from).  A failed wait does not leave the loops: it switches off the
        // remaining waits and instructions, and the loops run out.
        {
            const bool leader = elect_one();
            constexpr uint32_t idesc_f = make_idesc(128, DF, true);
            constexpr uint32_t idesc_upd = make_idesc(128, DF, true) | (1u << 15);  // A M-major, B MN-major
            constexpr uint32_t idesc_rd = make_idesc_tf32(128, 64);
            bool ok = true;
            int nu = 0, nq = 0, nx = 0;
            auto wait = [&](uint64_t *bar, int parity, int where) {
                if (ok) ok = mbar_wait(bar, (uint32_t)parity, abort_flag, status, where);
            };
            // descriptors as low words: a k-step adds a constant
            const uint32_t x_lo = desc_lo(smem_u32(smem + P::oX), 0), w_lo = desc_lo(smem_u32(smem + P::oW), D * 128);
            const uint32_t q_lo0 = desc_lo(smem_u32(smem + P::oQ), 0);
            const uint32_t pk_lo0 = desc_lo(smem_u32(smem + P::oU), kUTok * 128);
            const uint32_t v_lo0 = desc_lo(smem_u32(smem + P::oU + P::kPhiK), D == 128 ? kUTok * 128 : 0);
            // f = x W_q of block b_first + nx (the map warps have taken the previous f out of tensor memory)
            auto issue_f = [&]() {
                if (nx == 0) wait(w_full, 0, 61);
                wait(x_full, nx & 1, 62);
                wait(f_free + (nx & 1), ((nx >> 1) & 1) ^ 1, 63);
                tc_fence_after();
                if (leader && ok) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t xo = ((k / 4) * (128 * 128) + (k % 4) * 32) >> 4, wo = (k * (16 * 128)) >> 4;
                        if (k == 0) mma_ss_lo<idesc_f, 0>(tmem_base + col_f + (nx & 1) * DF, x_lo + xo, w_lo + wo);
                        else mma_ss_lo<idesc_f, 1>(tmem_base + col_f + (nx & 1) * DF, x_lo + xo, w_lo + wo);
                    }
                    tc_commit(f_done + (nx & 1));
                    tc_commit(x_empty);
                }
                ++nx;
            };
            if (has_init) {   // the workers have put the sum of the earlier segments into tensor memory
                wait(init_done, 0, 73);
                tc_fence_after();
            }
            auto issue_update = [&]() {
                wait(u_masked + nu % kUS, (nu / kUS) & 1, 64);
                tc_fence_after();
                const uint32_t so = (uint32_t)(nu % kUS) * (P::kUStage >> 4);
                const uint32_t acc0 = (nu > 0 || has_init) ? 1u : 0u;
                if (leader && ok) {
                    mma_ss_lo_acc<idesc_upd>(tmem_base + col_state, v_lo0 + so, pk_lo0 + so, acc0);
#pragma unroll
                    for (int k = 1; k < kUTok / 16; ++k)   // 16 tokens per step: 16 rows of 128 bytes in both operands
                        mma_ss_lo_acc<idesc_upd>(tmem_base + col_state, v_lo0 + so + k * (2048 >> 4), pk_lo0 + so + k * (2048 >> 4), 1u);
                    tc_commit(u_empty + nu % kUS);
                }
                ++nu;
            };
            if (sums_only)
                while (nu < n_upd) issue_update();
            if (NB > b_first) issue_f();
            for (int u = u_first; u < NU && !sums_only; ++u) {
                if (u % sc == 0) {
                    // the chunk that has just left the local region: sub-chunks of chunk u / sc - 2
                    for (int j = 0; j < per_chunk; ++j) issue_update();
                }
                // The next block's f = x W_q goes out as soon as its rows have arrived and the map warps have taken the
                // current f out of tensor memory: it is then ready when they finish the current block.  (Issued after
                // this block's read-out, it made the map warps wait for a round trip through this warp per block.)
                if ((u & 1) == 0 && b_first + nx < NB) issue_f();
                wait(pq_full + (u & 1), (nq >> 1) & 1, 65);
                wait(out_free + (nq & 1), ((nq >> 1) & 1) ^ 1, 66);
                tc_fence_after();
                const uint32_t q_lo = q_lo0 + (uint32_t)(u & 1) * (P::kPhiQ >> 4), d_out_t = tmem_base + col_out + (nq & 1) * 64;
                if (leader && ok) {
#pragma unroll
                    for (int k = 0; k < DF / 8; ++k) {   // 8 features per step: 32 bytes within a 32-feature atom
                        const uint32_t qo = ((k / 4) * (64 * 128) + (k % 4) * 32) >> 4;
                        if (k == 0) mma_ts_tf32_lo<idesc_rd, 0>(d_out_t, tmem_base + col_state, q_lo + qo);
                        else mma_ts_tf32_lo<idesc_rd, 1>(d_out_t, tmem_base + col_state + k * 8, q_lo + qo);
                    }
                    tc_commit(r_done + (nq & 1));
                    tc_commit(pq_empty + (u & 1));
                }
                ++nq;
            }
            // state after the last update, for the decode state; after a failure, nothing issued may still run
            if (leader) tc_commit(fin);
            if (!__all_sync(0xffffffffu, ok) && leader) mbar_wait_drain(fin, 0);
        }
    } else {
        // ------------------------------------------------------------ mask warps (2 and 3: alternate tiles)
        // Zeroes, in every phi(K) tile, the rows of the tokens kept for softmax attention: only the others enter the
        // state.  The indices of a tile's chunk are requested one tile ahead (a round trip to L2 per tile would
        // otherwise pace the whole update path), and two warps take turns.
        bool ok = true;
        // positions of the selected tokens of tile nu's chunk relative to the tile's first row (-1: none)
        auto fetch = [&](int nu, int (&r)[4]) {
            const int a_t = nu0 + nu, cc = a_t / per_chunk, rt = a_t % per_chunk, sub = rt % su;
            const int chunk = rt >= su ? cc - window : cc;       // (chunk < 0: nothing leaves yet, every row is zeroed)
            const bool need = !(rt >= su && sel_rows > 0);       // (a gathered tile needs no indices)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = lane + 32 * q;
                r[q] = (need && nu < n_upd && i < lam && chunk >= 0)
                           ? sel_idx[((long long)bh * Tn + chunk) * lam + i] - (chunk * C + sub * kUTok) : -1;
            }
        };
        auto process = [&](int nu, const int (&sel)[4]) {
            const int rt = (nu0 + nu) % per_chunk;
            const bool leaving = rt >= su;                       // tile of the tokens that leave the salient cache
            // the selected rows of the tile as a 32-bit set
            uint32_t rows = 0u;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (sel[q] >= 0 && sel[q] < kUTok) rows |= 1u << sel[q];
            rows = __reduce_or_sync(0xffffffffu, rows);
            if (leaving) rows = ~rows;                           // rows to zero: the selected ones, or all the others
            if (leaving && sel_rows > 0) {
                // gathered tile: its first `valid` rows are the chunk's leaving tokens, the rest belong to the next chunk
                const int cw = (nu0 + nu) / per_chunk - window;
                const int valid = cw < 0 ? 0 : min(kUTok, lam - (rt - su) * kUTok);
                rows = valid >= 32 ? 0u : ~((1u << valid) - 1u);
            }
            if (ok) ok = mbar_wait(u_full + nu % kUS, (nu / kUS) & 1, abort_flag, status, 67);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                // A row is 128 bytes in each 64-feature atom.  Eight lanes clear one such line (all 32 banks, no
                // conflict), so a store instruction clears the lines of four rows.
                uint8_t *tile = smem + P::oU + (nu % kUS) * P::kUStage;
#pragma unroll
                for (int it = 0; it < kUTok / 4; ++it) {
                    const int rz = it * 4 + (lane >> 3);
                    if ((rows >> rz) & 1u) {
#pragma unroll
                        for (int a = 0; a < DF / 64; ++a)
                            *reinterpret_cast<uint4 *>(tile + a * (kUTok * 128) + rz * 128 + ((lane & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                }
                fence_proxy_async();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(u_masked + nu % kUS);
        };
        // (two register sets that change roles: a copy from one to the other would wait for the loads)
        int sel_a[4], sel_b[4];
        fetch(warp - 2, sel_a);
        for (int nu = warp - 2; nu < n_upd; nu += 4) {
            fetch(nu + 2, sel_b);
            process(nu, sel_a);
            fetch(nu + 4, sel_a);
            if (nu + 2 < n_upd) process(nu + 2, sel_b);
        }
    }
    } else if (warp < 8) {
        reg_dec<152>();
        // ------------------------------------------------------------ workers: output
        const int wq = warp & 3;                     // TMEM lane quarter this warp may read
        const int e = wq * 32 + lane;                // value column (lane of S^T and of the read-out result)
        const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int tid = threadIdx.x - 128;           // 0..127
        bool ok = true;
        int nq = 0;
        // rows of the first two chunks see an empty state
        if (seg == 0 && !sums_only) {
            const int n0 = min(N, 2 * C);
            for (int i = tid; i < n0 * (D / 8); i += 128)
                reinterpret_cast<uint4 *>(y_out + (long long)bh * N * D)[i] = make_uint4(0, 0, 0, 0);
            for (int t = tid; t < n0; t += 128) d_out[(long long)bh * N + t] = 0.f;
        }
        if (has_init) {
            // S^T of this segment starts as the sum of the earlier segments' updates: lane e, column f <- sum_g P_g[f][e]
            const float *P0 = seg_sums + (((long long)bh * 2 + half) * ((n_seg - 1) * sum_parts)) * (DF * D);
            const int n_sums = seg * sum_parts;
#pragma unroll 1
            for (int q = 0; q < DF / 32; ++q) {
                uint32_t sreg[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float acc = 0.f;
                    if (e < D)
                        for (int g2 = 0; g2 < n_sums; ++g2) acc += P0[(long long)g2 * (DF * D) + (q * 32 + j) * D + e];
                    sreg[j] = __float_as_uint(acc);
                }
                tmem_st32(taddr + col_state + q * 32, sreg);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(init_done);
        }
        for (int u = u_first; u < NU && !sums_only; ++u) {
            if (ok) ok = mbar_wait(r_done + (nq & 1), (nq >> 1) & 1, abort_flag, status, 68);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                // y_part[t][e] = N_part / D_part (times the gate): the read-out scaled by 1 / (e . z) of its token.  A thread holds one value column of 64 tokens, but
                // the rows of y_part are token-major and a store loop over tokens costs about a hundred clocks per
                // instruction; so the tile is transposed through shared memory and leaves in 16-byte pieces.  Two
                // rolled rounds of 32 tokens keep the instruction stream short; the scales of a round are loaded
                // before its first store (shared-memory loads are kept behind earlier stores).
                const float4 *dinv = reinterpret_cast<const float4 *>(dinv_ring + (u & 7) * 64);
                __nv_bfloat16 *stg = reinterpret_cast<__nv_bfloat16 *>(smem + P::oStage);
#pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t o[32];
                    tmem_ld32(taddr + col_out + (nq & 1) * 64 + hf * 32, o);
                    float4 sc4[8];
#pragma unroll
                    for (int t4 = 0; t4 < 8; ++t4) sc4[t4] = dinv[hf * 8 + t4];
                    tmem_wait_ld();
                    if (e < D) {
#pragma unroll
                        for (int t4 = 0; t4 < 8; ++t4) {
                            __nv_bfloat16 *dst = stg + (hf * 32 + 4 * t4) * D + e;
                            dst[0] = __float2bfloat16_rn(__uint_as_float(o[4 * t4]) * sc4[t4].x);
                            dst[D] = __float2bfloat16_rn(__uint_as_float(o[4 * t4 + 1]) * sc4[t4].y);
                            dst[2 * D] = __float2bfloat16_rn(__uint_as_float(o[4 * t4 + 2]) * sc4[t4].z);
                            dst[3 * D] = __float2bfloat16_rn(__uint_as_float(o[4 * t4 + 3]) * sc4[t4].w);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(out_free + (nq & 1));
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");   // the four worker warps (always, whatever `ok`)
            if (ok) {
                const int base = u * 64;
                constexpr int kPiecesPerRow = D / 8;
#pragma unroll 2
                for (int it = 0; it < 64 * kPiecesPerRow / 128; ++it) {
                    const int id = it * 128 + tid, t = id / kPiecesPerRow, c = id % kPiecesPerRow;
                    if (base + t < N) {
                        uint4 v = *reinterpret_cast<const uint4 *>(smem + P::oStage + (t * D + c * 8) * 2);
                        const long long off = ((long long)bh * N + base + t) * D + c * 8;
                        if (G != nullptr) {
                            const uint4 gg = *reinterpret_cast<const uint4 *>(G + off);
                            const uint32_t vw[4] = {v.x, v.y, v.z, v.w}, gw[4] = {gg.x, gg.y, gg.z, gg.w};
                            uint32_t rw[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                rw[q] = pack_bf16(__uint_as_float(vw[q] << 16) * __uint_as_float(gw[q] << 16),
                                                  __uint_as_float(vw[q] & 0xffff0000u) * __uint_as_float(gw[q] & 0xffff0000u));
                            v = make_uint4(rw[0], rw[1], rw[2], rw[3]);
                        }
                        *reinterpret_cast<uint4 *>(y_out + off) = v;
                    }
                }
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");   // the staging tile has been read before the next one is written
            ++nq;
        }
        // the state after the segment's last update: the segment's own sum for the second pass (sums_only), or,
        // from the last segment, S [2 d_f, d] of the decode state (this CTA's features)
        float *S_dst = nullptr;
        if (sums_only) S_dst = seg_sums + (((long long)bh * 2 + half) * ((n_seg - 1) * sum_parts) + seg) * (DF * D);
        else if (S_out != nullptr && seg == n_seg - 1) S_dst = S_out + ((long long)bh * NF + half * DF) * D;
        if (S_dst != nullptr) {
            if (n_upd > 0 || has_init) {
                if (ok) ok = mbar_wait(fin, 0, abort_flag, status, 69);
                ok = __all_sync(0xffffffffu, ok);
                if (ok) {
                    tc_fence_after();
#pragma unroll 1
                    for (int q = 0; q < DF / 32; ++q) {
                        uint32_t sreg[32];
                        tmem_ld32(taddr + col_state + q * 32, sreg);
                        tmem_wait_ld();
                        if (e < D) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) S_dst[(q * 32 + j) * D + e] = __uint_as_float(sreg[j]);
                        }
                    }
                }
            } else {
                for (int i = tid; i < DF * D; i += 128) S_dst[i] = 0.f;
            }
        }
    } else {
        reg_inc<224>();
        // ------------------------------------------------------------ map warps: phi_q of a block of 128 rows
        // A thread owns one row: u = (f + b) ||x|| / max(||f + b||, 1e-12); this CTA's half of phi is softmax(u) or
        // softmax(-u) over all d_f features.  The row goes to the slot of its 64-token sub-chunk as fp32, K-major
        // with the 128-byte swizzle the UMMA descriptor expects; D_part = phi_half . z_half of the chunk two back.
        const int wq = warp & 3, r = wq * 32 + lane;   // TMEM lane quarter; row of the block
        const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
        const __nv_bfloat16 *bias = bq != nullptr ? bq + (long long)h * DF : nullptr;
        float *zs = reinterpret_cast<float *>(smem + P::oZ) + (warp - 8) * DF;   // this warp's copy of the z row
        bool ok = true;
        int nx = 0;
        for (int blk = b_first; blk < NB; ++blk, ++nx) {
            const int u = 2 * blk + (r >> 6);            // this row's sub-chunk; its slot is u & 1 = r >> 6
            const int slot = r >> 6, rr = r & 63;
            // z half of the chunk two back (every row of the warp dots its features with it): requested now,
            // placed in shared memory when it is needed
            float4 zreg = make_float4(0.f, 0.f, 0.f, 0.f);
            {
                const int chunk = min((u * 64) / C, Tn - 1);   // (a sub-chunk past the end of a ragged last block has no chunk)
                const float *zrow = zpre + ((long long)bh * n_routed + (chunk - 2)) * NF + half * DF;
                if (lane < DF / 4) zreg = reinterpret_cast<const float4 *>(zrow)[lane];
            }
            if (ok) ok = mbar_wait(x_full, nx & 1, abort_flag, status, 70);
            ok = __all_sync(0xffffffffu, ok);
            float nx2 = 0.f;
            if (ok) {
                float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int a = 0; a < D / 64; ++a)
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(smem + P::oX + a * (128 * 128) + r * 128 + ((c ^ (r & 7)) << 4));
                        const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float lo = __uint_as_float(w4[q] << 16), hi = __uint_as_float(w4[q] & 0xffff0000u);
                            s4[q] = fmaf(lo, lo, s4[q]);
                            s4[q] = fmaf(hi, hi, s4[q]);
                        }
                    }
                nx2 = (s4[0] + s4[1]) + (s4[2] + s4[3]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(x_empty);
            if (lane < DF / 4) reinterpret_cast<float4 *>(zs)[lane] = zreg;
            // f of this block is read from tensor memory twice, 32 columns at a time, in loops that stay rolled: the
            // warp's instruction stream per block is then a few kilobytes.  (With the row held in 128 registers and
            // everything unrolled, instruction fetch was the first stall reason of the kernel.)  f has a buffer per
            // block parity, so the next block's GEMM does not wait for this second reading.
            const uint32_t faddr = taddr + col_f + (nx & 1) * DF;
            if (ok) ok = mbar_wait(f_done + (nx & 1), (nx >> 1) & 1, abort_flag, status, 71);
            ok = __all_sync(0xffffffffu, ok);
            float sgn = 0.f, shift = 0.f;
            if (ok) {
                tc_fence_after();
                // (packed arithmetic and four independent chains each; this CTA's half needs only one extremum:
                // max f for softmax(u), min f for softmax(-u))
                float2 n2[4];
                float ex[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    n2[q] = make_float2(0.f, 0.f);
                    ex[q] = half == 0 ? -INFINITY : INFINITY;
                }
#pragma unroll 1
                for (int q = 0; q < DF / 32; ++q) {
                    float fv[32];
                    tmem_ld32(faddr + q * 32, reinterpret_cast<uint32_t *>(fv));
                    tmem_wait_ld();
                    if (bias != nullptr) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) fv[j] += __bfloat162float(bias[q * 32 + j]);
                    }
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float2 v = make_float2(fv[j + 2 * c], fv[j + 2 * c + 1]);
                            n2[c] = __ffma2_rn(v, v, n2[c]);
                            ex[c] = half == 0 ? max3(ex[c], v.x, v.y) : min3(ex[c], v.x, v.y);
                        }
                    }
                }
                const float nf2 = ((n2[0].x + n2[0].y) + (n2[1].x + n2[1].y)) + ((n2[2].x + n2[2].y) + (n2[3].x + n2[3].y));
                const float unit = half == 0 ? 1.f : -1.f;
                const float extreme = half == 0 ? fmaxf(fmaxf(ex[0], ex[1]), fmaxf(ex[2], ex[3]))
                                                : -fminf(fminf(ex[0], ex[1]), fminf(ex[2], ex[3]));   // max of +-f
                // u = f * ratio in the log2 domain; the exponent of this half is +-u - max(+-u) <= 0
                const float ratio = sqrtf(nx2) / fmaxf(sqrtf(nf2), 1e-12f) * 1.4426950408889634f;
                sgn = unit * ratio;
                shift = -extreme * ratio;
            }
            // the slot is written only after the read-out that used it last has completed (every block fills both
            // slots once)
            if (ok) ok = mbar_wait(pq_empty + slot, (nx & 1) ^ 1, abort_flag, status, 72);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                // The features go into the tile unnormalised, e_j = 2^(+-u_j - max): with D_part = (e . z) / sum e and
                // N_part = (e . S) / sum e the output N_part / D_part = (e . S) / (e . z) does not need the sum, so the
                // row is written as it is computed.  The z values of a block of 32 features are loaded before the
                // block's stores (shared-memory loads are kept behind earlier stores).
                uint8_t *tile = smem + P::oQ + slot * P::kPhiQ;
                float2 zs2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)}, ds2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                const float2 sgn2 = make_float2(sgn, sgn), shift2 = make_float2(shift, shift);
#pragma unroll 1
                for (int q = 0; q < DF / 32; ++q) {          // 32 features: one swizzle atom of the tile
                    float fv[32];
                    tmem_ld32(faddr + q * 32, reinterpret_cast<uint32_t *>(fv));
                    float4 zc[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) zc[i] = *reinterpret_cast<const float4 *>(zs + 32 * q + 4 * i);
                    tmem_wait_ld();
                    if (bias != nullptr) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) fv[j] += __bfloat162float(bias[q * 32 + j]);
                    }
                    uint8_t *row = tile + q * (64 * 128) + rr * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int j = 4 * i;
                        const float2 a0 = __ffma2_rn(make_float2(fv[j], fv[j + 1]), sgn2, shift2);
                        const float2 a1 = __ffma2_rn(make_float2(fv[j + 2], fv[j + 3]), sgn2, shift2);
                        float4 ev;
                        ev.x = ex2(a0.x);
                        ev.y = ex2(a0.y);
                        ev.z = ex2(a1.x);
                        ev.w = ex2(a1.y);
                        zs2[0] = __fadd2_rn(zs2[0], make_float2(ev.x, ev.y));
                        zs2[1] = __fadd2_rn(zs2[1], make_float2(ev.z, ev.w));
                        ds2[0] = __ffma2_rn(make_float2(ev.x, ev.y), make_float2(zc[i].x, zc[i].y), ds2[0]);
                        ds2[1] = __ffma2_rn(make_float2(ev.z, ev.w), make_float2(zc[i].z, zc[i].w), ds2[1]);
                        // features 4 i .. 4 i + 3 of the atom: 16-byte piece i, swizzled by the row
                        *reinterpret_cast<float4 *>(row + ((i ^ (rr & 7)) << 4)) = ev;
                    }
                }
                tc_fence_before();
                const float zsum = (zs2[0].x + zs2[0].y) + (zs2[1].x + zs2[1].y), draw = (ds2[0].x + ds2[0].y) + (ds2[1].x + ds2[1].y);
                const int t = u * 64 + rr;
                if (t < N) d_out[(long long)bh * N + t] = draw / zsum;     // D_part
                dinv_ring[(u & 7) * 64 + rr] = draw > 0.f ? 1.f / draw : 0.f;
                fence_proxy_async();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(f_free + (nx & 1));
            __syncwarp();
            if (lane == 0) mbar_arrive(pq_full + slot);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Rows of phi(K) [2 d_f] and V [d] of the selected tokens, per query head, in selection order (row j of a head is
// token sel_idx[j]; -1 entries and the padding up to sel_rows are zero): with a salient-cache budget the tokens
// that leave the cache enter the state from these copies, lam rows per chunk.  One warp per row.
template <int D, int DF>
__global__ void __launch_bounds__(256)
gather_selected_kernel(const __nv_bfloat16 *__restrict__ phiK, const __nv_bfloat16 *__restrict__ V,
                       const int32_t *__restrict__ sel_idx, __nv_bfloat16 *__restrict__ phiKsel,
                       __nv_bfloat16 *__restrict__ Vsel, int H, int Hkv, long long N, long long n_idx, long long sel_rows) {
    const int bh = blockIdx.y, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long j = (long long)blockIdx.x * 8 + warp;
    if (j >= sel_rows) return;
    long long pos = -1;
    if (j < n_idx) pos = sel_idx[(long long)bh * n_idx + j];
    constexpr int kPhiVec = 2 * DF / 8, kVVec = D / 8;   // uint4 per row
    uint4 pp = make_uint4(0, 0, 0, 0), vv = pp;
    const long long src = ((long long)b * Hkv + kvh) * N + pos;
    if (pos >= 0) {
        if (lane < kPhiVec) pp = reinterpret_cast<const uint4 *>(phiK + src * (2 * DF))[lane];
        if (lane < kVVec) vv = reinterpret_cast<const uint4 *>(V + src * D)[lane];
    }
    const long long dst = (long long)bh * sel_rows + j;
    if (lane < kPhiVec) reinterpret_cast<uint4 *>(phiKsel + dst * (2 * DF))[lane] = pp;
    if (lane < kVVec) reinterpret_cast<uint4 *>(Vsel + dst * D)[lane] = vv;
}

// ------------------------------------------------------------------------------------------ host side

template <int D, int DF, typename TOut>
int launch_npmap(const void *X, const void *W, const void *bias, void *phi, float *csum, int B, int heads, long long N,
                 int C, int *status, cudaStream_t st, int *launches) {
    CUtensorMap tx, tw;
    if (!make_map_2d(&tx, X, (unsigned long long)B * heads * N, D, 128, false) ||
        !make_map_2d(&tw, W, (unsigned long long)heads * D, DF, D, false))
        return STILL_ERR_CUDA;
    constexpr int kSmem = NpmapSmem<D, DF, TOut>::kTotal;
    if (ensure_dynamic_smem((const void *)npmap_tc_kernel<D, DF, TOut>, kSmem) != cudaSuccess) return STILL_ERR_CUDA;
    dim3 grid((unsigned)((N + 127) / 128), (unsigned)heads, (unsigned)B);
    npmap_tc_kernel<D, DF, TOut><<<grid, 192, kSmem, st>>>(tx, tw, (const __nv_bfloat16 *)bias, (TOut *)phi, csum, status, heads,
                                                          (int)N, C);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

template <int D, int DF>
int launch_fused(const still_params_t *p, long long N, const void *Q, const void *V, const void *G, const void *Wq,
                 const void *bq, const int32_t *sel_idx, const void *phiK, const float *zpre, void *y_part, float *d_part,
                 float *S_out, float *seg_sums, void *phiK_sel, void *v_sel, long long sel_rows, int *status, cudaStream_t st,
                 int *launches) {
    using bf = __nv_bfloat16;
    CUtensorMap tq, tw, tk, tv, tks, tvs;
    const unsigned long long BH = (unsigned long long)p->B * p->H, BHkv = (unsigned long long)p->B * p->Hkv;
    if (!make_map_2d(&tq, Q, BH * N, D, 128, false) || !make_map_2d(&tw, Wq, (unsigned long long)p->H * D, DF, D, false) ||
        !make_map_2d(&tk, phiK, BHkv * N, 2 * DF, FusedPlan<D, DF>::kUTok, false) ||
        !make_map_2d(&tv, V, BHkv * N, D, FusedPlan<D, DF>::kUTok, false))
        return STILL_ERR_CUDA;
    // With a salient-cache budget and topk < chunk the leaving tokens are read from gathered copies of their rows
    // (otherwise every token of a chunk is selected and the chunk's own tiles are the leaving tiles).
    const bool gathered = p->max_salient > 0 && p->topk < p->chunk && phiK_sel != nullptr && v_sel != nullptr;
    tks = tk;
    tvs = tv;
    if (gathered) {
        if (BH * (unsigned long long)sel_rows >= (1ull << 31)) return STILL_ERR_UNSUPPORTED;   // TMA row coordinate
        const long long Tn = (N + p->chunk - 1) / p->chunk;
        dim3 ggrid((unsigned)((sel_rows + 7) / 8), (unsigned)BH);
        gather_selected_kernel<D, DF><<<ggrid, 256, 0, st>>>((const bf *)phiK, (const bf *)V, sel_idx, (bf *)phiK_sel, (bf *)v_sel,
                                                           p->H, p->Hkv, N, Tn * p->topk, sel_rows);
        ++*launches;
        if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
        if (!make_map_2d(&tks, phiK_sel, BH * (unsigned long long)sel_rows, 2 * DF, FusedPlan<D, DF>::kUTok, false) ||
            !make_map_2d(&tvs, v_sel, BH * (unsigned long long)sel_rows, D, FusedPlan<D, DF>::kUTok, false))
            return STILL_ERR_CUDA;
    }
    using Plan = FusedPlan<D, DF>;
    if (ensure_dynamic_smem((const void *)la_fused_kernel<D, DF>, Plan::kTotal) != cudaSuccess) return STILL_ERR_CUDA;
    int seg_chunks = 0;
    const int n_seg = tc_la_segments(p, N, &seg_chunks), parts = tc_la_sum_parts(seg_chunks);
    for (int pass = n_seg > 1 ? 0 : 1; pass < 2; ++pass) {
        // pass 0 (only with several segments): the sum of every segment's own updates; pass 1: the scan proper
        dim3 grid((unsigned)BH, 2, (unsigned)(pass == 0 ? (n_seg - 1) * parts : n_seg));   // head, feature half, segment (piece)
        la_fused_kernel<D, DF><<<grid, 384, Plan::kTotal, st>>>(tq, tw, tk, tv, tks, tvs, (const bf *)bq, (const bf *)G, sel_idx, zpre,
                                                               (bf *)y_part, d_part, S_out, seg_sums, status, p->H, p->Hkv, (int)N,
                                                               p->chunk, p->topk, p->topk > 0 ? (int)(p->max_salient / p->topk) : 0,
                                                               (long long)BH * N * D, (long long)BH * N,
                                                               seg_chunks, n_seg, parts, pass == 0 ? 1 : 0, gathered ? (int)sel_rows : 0);
        ++*launches;
        if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
    }
    return STILL_OK;
}

}  // namespace

bool tc_la_supported(const still_params_t *p) {
    return tc_supported(p) && (p->d_f == 64 || p->d_f == 128) && p->d_f <= p->d;
}

// Two-level scan: with few (batch, head) units the sequence is cut into segments that run side by side, each
// starting from the sum of the earlier segments' state updates.  Segments are whole, even numbers of chunks, at
// least eight of them, and as many as fill the SMs once (two CTAs per head and segment).
int tc_la_segments(const still_params_t *p, long long N, int *seg_chunks) {
    const long long Tn = (N + p->chunk - 1) / p->chunk, ctas = 2ll * p->B * p->H;
    int n_seg = 1;
    while (n_seg < 4 && ctas * (n_seg * 2) <= 148 && Tn / (n_seg * 2) >= 8) n_seg *= 2;
    long long sc = (Tn + n_seg - 1) / n_seg;
    sc += sc & 1;
    if (seg_chunks) *seg_chunks = (int)sc;
    return n_seg;
}

// Pieces per segment in the first pass of the two-level scan (each at least two chunks long).
int tc_la_sum_parts(int seg_chunks) {
    return (seg_chunks % 4 == 0 && seg_chunks >= 8) ? 4 : (seg_chunks % 2 == 0 && seg_chunks >= 4) ? 2 : 1;
}

int tc_la_branch(const still_params_t *p, long long N, const void *Q, const void *K, const void *V, const void *G,
                 const void *Wq, const void *bq, const void *Wk, const void *bk, const int32_t *sel_idx, void *phiK,
                 float *csum, float *zpre, void *y_part, float *d_part, float *seg_sums, float *S_out, float *z_out,
                 void *phiK_sel, void *v_sel, long long sel_rows, int *status_words, cudaStream_t st, int *launches) {
    using bf = __nv_bfloat16;
    if ((long long)p->B * p->H * N >= (1ll << 31)) return STILL_ERR_UNSUPPORTED;  // TMA row coordinate
    const int NF = 2 * p->d_f, C = p->chunk;
    const long long Tn = (N + C - 1) / C, BH = (long long)p->B * p->H;
    const int n_routed = Tn >= 3 ? (int)(Tn - 2) : 0;
    // phi(K) once per KV head (bf16; the B operand of the state update), with the column sums of every chunk
    int rc;
    if (p->d == 64 && p->d_f == 64)
        rc = launch_npmap<64, 64, bf>(K, Wk, bk, phiK, csum, p->B, p->Hkv, N, C, status_words, st, launches);
    else if (p->d == 128 && p->d_f == 64)
        rc = launch_npmap<128, 64, bf>(K, Wk, bk, phiK, csum, p->B, p->Hkv, N, C, status_words, st, launches);
    else
        rc = launch_npmap<128, 128, bf>(K, Wk, bk, phiK, csum, p->B, p->Hkv, N, C, status_words, st, launches);
    if (rc != STILL_OK) return rc;
    // z after every routed chunk (per query head: the selection is per query head)
    if (n_routed > 0) {
        z_delta_kernel<<<dim3((unsigned)n_routed, (unsigned)BH), NF, 0, st>>>(csum, (const bf *)phiK, sel_idx, zpre, p->H, p->Hkv,
                                                                                N, (int)Tn, n_routed, p->topk, C,
                                                                                p->topk > 0 ? (int)(p->max_salient / p->topk) : 0, NF);
        ++*launches;
        if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
    }
    if (n_routed > 0 || z_out != nullptr) {
        z_scan_kernel<<<(unsigned)BH, NF, 0, st>>>(zpre, z_out, n_routed, NF);
        ++*launches;
        if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
    }
    if (p->d == 64 && p->d_f == 64)
        return launch_fused<64, 64>(p, N, Q, V, G, Wq, bq, sel_idx, phiK, zpre, y_part, d_part, S_out, seg_sums, phiK_sel, v_sel, sel_rows,
                                   status_words, st, launches);
    if (p->d == 128 && p->d_f == 64)
        return launch_fused<128, 64>(p, N, Q, V, G, Wq, bq, sel_idx, phiK, zpre, y_part, d_part, S_out, seg_sums, phiK_sel, v_sel, sel_rows,
                                   status_words, st, launches);
    return launch_fused<128, 128>(p, N, Q, V, G, Wq, bq, sel_idx, phiK, zpre, y_part, d_part, S_out, seg_sums, phiK_sel, v_sel, sel_rows,
                                   status_words, st, launches);
}

}  // namespace still
