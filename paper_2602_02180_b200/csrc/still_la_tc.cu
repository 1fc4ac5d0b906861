// Linear-attention branch of the prefill on tensor cores (bf16 inputs, sm_100a).
//
// Two kernels:
//
// npmap_tc_kernel -- Norm-Preserved Feature Map (Sec. 3.2, Eq. feature_map) of 128 rows of Q or K
//   per CTA, fused into the load of the rows:  f = x W  on tcgen05 (x tile K-major from TMA, W
//   MN-major from TMA, accumulator in TMEM), then per row  u = (f + b) ||x|| / max(||f + b||, 1e-12),
//   phi = [softmax(u), softmax(-u)].  phi(K) is stored as bf16 (it is the B operand of the bf16
//   state-update GEMM), phi(Q) as fp32 (B operand of the TF32 read-out GEMM).
//
// la_scan_tc_kernel -- Algorithm 1 "Linear Attention Branch" with the state of Eq.
//   cache_routing_sum kept in tensor memory.  One CTA owns one (batch, query head) and 64 of the d
//   value columns and walks the chunks in order.  The state is held transposed, S^T [128 x d']
//   fp32 in TMEM: lanes 0-63 are the 64 value columns, lane 64 is the normaliser z (the A operand
//   of the update has a second 64-row atom whose first row is all ones), lanes 65-127 are zero.
//     update   S^T += [V_c^T ; 1] phi_k(K_c)   for the chunk c that has just left the two-chunk
//              local region: bf16 UMMA, A = V tile (M-major, as TMA delivers it), B = phi(K) tile
//              (MN-major) whose rows of the tokens selected for softmax attention were zeroed;
//     read-out [N_LA^T ; D_LA] = S^T phi_q(Q_c)^T  for the chunk c being answered: TF32 UMMA with
//              the fp32 state read straight from TMEM as the A operand (no conversion pass; 10-bit
//              mantissa instead of the 7 bits a bf16 copy of the state would keep), B = phi(Q)
//              tile (K-major fp32).
//   The lag of two chunks between update and read-out is the delayed selection of Sec. 3.3.
//   Work is tiled in 64-token sub-chunks, so C = 128 is two sub-chunks per chunk.
//
// Roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 zero the selected rows of
// the phi(K) tiles and run the epilogue (N_LA times the gate, D_LA, final state).  Every mbarrier
// wait is bounded; on expiry the kernel records STILL_ERR_DEVICE_TIMEOUT in the status word, all
// roles leave their loops and tensor memory is freed before the CTA exits.
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
                const __nv_bfloat16 *__restrict__ bias, TOut *__restrict__ phi, int *status, int heads, int N) {
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
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// ------------------------------------------------------------------------------------------
// State scan
// ------------------------------------------------------------------------------------------
template <int NF>  // feature dim d' = 2 d_f: 128 or 256
struct ScanPlan {
    static constexpr int kPhiK = 64 * NF * 2;          // phi(K) tile of 64 tokens, bf16
    static constexpr int kVt = 64 * 64 * 2;            // V tile: 64 tokens x 64 value columns, bf16
    static constexpr int kUStage = kPhiK + kVt;
    static constexpr int kPhiQ = 64 * NF * 4;          // phi(Q) tile of 64 tokens, fp32
    static constexpr int kU = 0;                       // two update stages
    static constexpr int kQ = kU + 2 * kUStage;        // two read-out stages
    static constexpr int kOnes = kQ + 2 * kPhiQ;       // second M atom of the update's A operand
    static constexpr int kBar = kOnes + 64 * 128;
    static constexpr int kNumBars = 2 + 2 + 2 + 2 + 2 + 5;  // u_full, u_empty, u_masked, q_full, q_empty, r_done[2], out_free[2], fin
    static constexpr int kMisc = kBar + kNumBars * 8;
    static constexpr int kTotal = kMisc + 16;
};
static_assert(ScanPlan<128>::kTotal <= 232448 && ScanPlan<256>::kTotal <= 232448,
              "state scan: the shared-memory plan exceeds what a CTA can have");

template <int NF>
__global__ void __launch_bounds__(192, 1)
la_scan_tc_kernel(const __grid_constant__ CUtensorMap tm_phik, const __grid_constant__ CUtensorMap tm_v,
                  const __grid_constant__ CUtensorMap tm_phiq, const __nv_bfloat16 *__restrict__ G,
                  const int32_t *__restrict__ sel_idx, float *__restrict__ N_LA, float *__restrict__ D_LA,
                  float *__restrict__ S_out, float *__restrict__ z_out, int *status, int H, int Hkv, int N, int d,
                  int C, int lam) {
    using P = ScanPlan<NF>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + P::kBar);
    uint64_t *u_full = bars, *u_empty = bars + 2, *u_masked = bars + 4, *q_full = bars + 6, *q_empty = bars + 8;
    uint64_t *r_done = bars + 10, *out_free = bars + 12, *fin = bars + 14;
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(smem + P::kMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + P::kMisc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.x, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int e0 = blockIdx.y * 64;            // first value column of this CTA
    const int sc = C / 64;                      // 64-token sub-chunks per chunk
    const int Tn = (N + C - 1) / C;             // chunks
    const int NU = (N + 63) / 64;               // sub-chunks with query rows
    const int n_upd = Tn >= 3 ? (Tn - 2) * sc : 0;   // update tiles: sub-chunks of chunks 0 .. Tn-3
    const int u_first = 2 * sc;                 // first sub-chunk whose read-out sees a non-empty state

    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) report_status(status, STILL_ERR_DEVICE_TIMEOUT, 97);
        return;
    }
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status) != 0;
    __syncthreads();
    if (*abort_flag) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(u_full + i, 1);
            mbar_init(u_empty + i, 1);
            mbar_init(u_masked + i, 4);
            mbar_init(q_full + i, 1);
            mbar_init(q_empty + i, 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(r_done + i, 1);
            mbar_init(out_free + i, 4);
        }
        mbar_init(fin, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    // The "ones" atom: 64 token rows of 128 bytes; value column 0 (i.e. M index 64 of the A operand)
    // is 1 for every token, everything else 0.  With the 128-byte swizzle, element 0 of row t sits in
    // the 16-byte chunk (0 xor (t mod 8)).
    for (int i = threadIdx.x; i < 64 * 128 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(smem + P::kOnes)[i] = 0u;
    __syncthreads();
    if (threadIdx.x < 64) {
        const int t = threadIdx.x;
        *reinterpret_cast<uint16_t *>(smem + P::kOnes + t * 128 + ((t & 7) << 4)) = 0x3f80;  // bf16 1.0
    }
    fence_proxy_async();
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    const uint32_t col_state = 0, col_out = NF;   // S^T [128 x NF] fp32; two read-out results [128 x 64] fp32, so that
                                                  // the epilogue of one sub-chunk overlaps the MMAs of the next

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int kv_row0 = (b * Hkv + kvh) * N, q_row0 = bh * N;
            int nu = 0, nq = 0;   // tiles requested so far
            const int n_q = NU > u_first ? NU - u_first : 0;
            int spins = 0;
            long long t0 = clock64();
            while (nu < n_upd || nq < n_q) {
                bool progressed = false;
                if (nu < n_upd && mbar_try_wait(u_empty + (nu & 1), ((nu >> 1) & 1) ^ 1)) {
                    uint8_t *stg = smem + P::kU + (nu & 1) * P::kUStage;
                    mbar_expect_tx(u_full + (nu & 1), P::kUStage);
                    for (int a = 0; a < NF / 64; ++a)   // phi(K): MN-major, 64-feature atoms 64 rows apart
                        tma_load_2d(stg + a * (64 * 128), &tm_phik, u_full + (nu & 1), a * 64, kv_row0 + nu * 64);
                    tma_load_2d(stg + P::kPhiK, &tm_v, u_full + (nu & 1), e0, kv_row0 + nu * 64);
                    ++nu;
                    progressed = true;
                }
                if (nq < n_q && mbar_try_wait(q_empty + (nq & 1), ((nq >> 1) & 1) ^ 1)) {
                    uint8_t *stg = smem + P::kQ + (nq & 1) * P::kPhiQ;
                    mbar_expect_tx(q_full + (nq & 1), P::kPhiQ);
                    for (int a = 0; a < NF / 32; ++a)   // phi(Q): K-major fp32, 32-feature atoms 64 rows apart
                        tma_load_2d(stg + a * (64 * 128), &tm_phiq, q_full + (nq & 1), a * 32, q_row0 + (u_first + nq) * 64);
                    ++nq;
                    progressed = true;
                }
                if (progressed) {
                    spins = 0;
                } else if ((++spins & 1023) == 0) {
                    if (spins == 1024) t0 = clock64();
                    if (*abort_flag) break;
                    if (clock64() - t0 > kWaitLimitCycles) {
                        *abort_flag = 1;
                        report_status(status, STILL_ERR_DEVICE_TIMEOUT, 40);
                        break;
                    }
                }
            }
            if (*abort_flag) {  // leave no copy in flight behind
                if (nu > 0) mbar_wait_drain(u_full + ((nu - 1) & 1), ((nu - 1) >> 1) & 1);
                if (nq > 0) mbar_wait_drain(q_full + ((nq - 1) & 1), ((nq - 1) >> 1) & 1);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_upd = make_idesc(128, NF, true) | (1u << 15);  // A M-major, B MN-major
            constexpr uint32_t idesc_rd = make_idesc_tf32(128, 64);
            bool ok = true;
            int nu = 0, nq = 0;
            for (int u = u_first; u < NU && ok; ++u) {
                if (u % sc == 0) {
                    // the chunk that has just left the local region: sub-chunks of chunk u / sc - 2
                    for (int j = 0; j < sc && ok; ++j, ++nu) {
                        ok = mbar_wait(u_masked + (nu & 1), (nu >> 1) & 1, abort_flag, status, 41);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t stg = smem_u32(smem + P::kU + (nu & 1) * P::kUStage);
                        const uint32_t v_addr = stg + P::kPhiK, ones = smem_u32(smem + P::kOnes);
#pragma unroll
                        for (int k = 0; k < 4; ++k)   // 16 tokens per step: 16 rows of 128 bytes in both operands
                            mma_ss(tmem_base + col_state, smem_desc(v_addr + k * 2048, ones - v_addr),
                                   smem_desc(stg + k * 2048, 64 * 128), idesc_upd, (nu > 0 || k > 0) ? 1u : 0u);
                        tc_commit(u_empty + (nu & 1));
                    }
                    if (!ok) break;
                }
                ok = mbar_wait(q_full + (nq & 1), (nq >> 1) & 1, abort_flag, status, 42);
                if (ok) ok = mbar_wait(out_free + (nq & 1), ((nq >> 1) & 1) ^ 1, abort_flag, status, 43);
                if (!ok) break;
                tc_fence_after();
                const uint32_t qs = smem_u32(smem + P::kQ + (nq & 1) * P::kPhiQ);
#pragma unroll
                for (int k = 0; k < NF / 8; ++k)   // 8 features per step: 32 bytes within a 32-feature atom
                    mma_ts_tf32(tmem_base + col_out + (nq & 1) * 64, tmem_base + col_state + k * 8,
                                smem_desc(qs + (k / 4) * (64 * 128) + (k % 4) * 32, 0), idesc_rd, k > 0 ? 1u : 0u);
                tc_commit(r_done + (nq & 1));
                ++nq;
            }
            // state after the last update (chunks 0 .. Tn-3), for the decode state
            if (ok) tc_commit(fin);
            if (!ok) {
                tc_commit(fin);
                mbar_wait_drain(fin, 0);
            }
        }
    } else {
        // ------------------------------------------------------------ workers: mask, epilogue
        const int wq = warp & 3;                     // TMEM lane quarter this warp may read
        const int e = wq * 32 + lane;                // lane of S^T / of the read-out result
        const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int tid = threadIdx.x - 64;            // 0..127
        bool ok = true;
        int nu = 0, nq = 0;
        // zero the rows of the tokens kept for softmax attention in update tile nu
        auto mask_tile = [&]() {
            if (ok) ok = mbar_wait(u_full + (nu & 1), (nu >> 1) & 1, abort_flag, status, 44);
            ok = __all_sync(0xffffffffu, ok);
            if (ok && lam > 0) {
                const int chunk = nu / sc, sub = nu % sc;
                const int32_t *si = sel_idx + ((long long)bh * Tn + chunk) * lam;
                uint8_t *tile = smem + P::kU + (nu & 1) * P::kUStage;
                // one token row = NF / 64 atoms x eight 16-byte pieces; a thread zeroes one piece at a time
                constexpr int kPieces = NF / 8;
                for (int i = tid; i < lam * kPieces; i += 128) {
                    const int p = si[i / kPieces] - (chunk * C + sub * 64);   // row within this 64-token tile
                    const int piece = i % kPieces;
                    if (p >= 0 && p < 64)
                        *reinterpret_cast<uint4 *>(tile + (piece >> 3) * (64 * 128) + p * 128 + ((piece & 7) << 4)) =
                            make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(u_masked + (nu & 1));
            ++nu;
        };
        // rows of the first two chunks see an empty state
        for (int i = tid; i < min(N, u_first * 64) * 64; i += 128) {
            const int t = i >> 6, col = i & 63;
            N_LA[((long long)bh * N + t) * d + e0 + col] = 0.f;
        }
        if (blockIdx.y == 0)
            for (int t = tid; t < min(N, u_first * 64); t += 128) D_LA[(long long)bh * N + t] = 0.f;

        for (int j = 0; j < sc && nu < n_upd; ++j) mask_tile();       // tiles of the first update
        for (int u = u_first; u < NU; ++u) {
            if ((u + 1) % sc == 0)                                     // tiles of the next chunk's update
                for (int j = 0; j < sc && nu < n_upd; ++j) mask_tile();
            if (ok) ok = mbar_wait(r_done + (nq & 1), (nq >> 1) & 1, abort_flag, status, 45);
            ok = __all_sync(0xffffffffu, ok);
            // The result leaves through shared memory (the phi(Q) stage this read-out has just consumed is free
            // until the workers release it): a thread holds one value column of 64 tokens, but the rows of
            // N_LA are token-major, and a column-wise store loop costs over a hundred clocks per instruction.
            float *stg = reinterpret_cast<float *>(smem + P::kQ + (nq & 1) * P::kPhiQ);   // [64 tokens][64 columns], then D_LA [64]
            const int base = u * 64;
            if (ok) {
                tc_fence_after();
                uint32_t o[64];
                tmem_ld32(taddr + col_out + (nq & 1) * 64, o);
                tmem_ld32(taddr + col_out + (nq & 1) * 64 + 32, o + 32);
                tmem_wait_ld();
                tc_fence_before();
                if (e < 64) {
#pragma unroll
                    for (int t = 0; t < 64; ++t) stg[t * 64 + e] = __uint_as_float(o[t]);
                } else if (e == 64) {
#pragma unroll
                    for (int t = 0; t < 64; ++t) stg[64 * 64 + t] = __uint_as_float(o[t]);
                }
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");   // the four worker warps (always, whatever `ok`)
            if (ok) {
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int id = it * 128 + tid, t = id >> 4, c = id & 15;
                    if (base + t < N) {
                        float4 v = *reinterpret_cast<const float4 *>(stg + t * 64 + c * 4);
                        const long long off = ((long long)bh * N + base + t) * d + e0 + c * 4;
                        if (G != nullptr) {
                            const uint2 gg = *reinterpret_cast<const uint2 *>(G + off);
                            v.x *= __uint_as_float(gg.x << 16);
                            v.y *= __uint_as_float(gg.x & 0xffff0000u);
                            v.z *= __uint_as_float(gg.y << 16);
                            v.w *= __uint_as_float(gg.y & 0xffff0000u);
                        }
                        *reinterpret_cast<float4 *>(N_LA + off) = v;
                    }
                }
                if (blockIdx.y == 0 && tid < 64 && base + tid < N) D_LA[(long long)bh * N + base + tid] = stg[64 * 64 + tid];
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");   // staging space read by all before the stage is released
            if (lane == 0) {
                mbar_arrive(out_free + (nq & 1));
                mbar_arrive(q_empty + (nq & 1));
            }
            ++nq;
        }
        // final state for the decode state: S [d', d] and z [d']
        if (S_out != nullptr) {
            if (n_upd > 0) {
                if (ok) ok = mbar_wait(fin, 0, abort_flag, status, 46);
                ok = __all_sync(0xffffffffu, ok);
                if (ok) {
                    tc_fence_after();
#pragma unroll 1
                    for (int q = 0; q < NF / 32; ++q) {
                        uint32_t sreg[32];
                        tmem_ld32(taddr + col_state + q * 32, sreg);
                        tmem_wait_ld();
                        if (e < 64) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                S_out[((long long)bh * NF + q * 32 + j) * d + e0 + e] = __uint_as_float(sreg[j]);
                        } else if (e == 64 && blockIdx.y == 0) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) z_out[(long long)bh * NF + q * 32 + j] = __uint_as_float(sreg[j]);
                        }
                    }
                }
            } else {
                for (int i = tid; i < NF * 64; i += 128) S_out[((long long)bh * NF + (i >> 6)) * d + e0 + (i & 63)] = 0.f;
                if (blockIdx.y == 0)
                    for (int i = tid; i < NF; i += 128) z_out[(long long)bh * NF + i] = 0.f;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ host side

template <int D, int DF, typename TOut>
int launch_npmap(const void *X, const void *W, const void *bias, void *phi, int B, int heads, long long N, int *status,
                 cudaStream_t st, int *launches) {
    CUtensorMap tx, tw;
    if (!make_map_2d(&tx, X, (unsigned long long)B * heads * N, D, 128, false) ||
        !make_map_2d(&tw, W, (unsigned long long)heads * D, DF, D, false))
        return STILL_ERR_CUDA;
    constexpr int kSmem = NpmapSmem<D, DF, TOut>::kTotal;
    if (ensure_dynamic_smem((const void *)npmap_tc_kernel<D, DF, TOut>, kSmem) !=
        cudaSuccess)
        return STILL_ERR_CUDA;
    dim3 grid((unsigned)((N + 127) / 128), (unsigned)heads, (unsigned)B);
    npmap_tc_kernel<D, DF, TOut><<<grid, 192, kSmem, st>>>(tx, tw, (const __nv_bfloat16 *)bias, (TOut *)phi, status, heads,
                                                          (int)N);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

template <typename TOut>
int launch_npmap_any(const still_params_t *p, const void *X, const void *W, const void *bias, void *phi, int heads,
                     long long N, int *status, cudaStream_t st, int *launches) {
    if (p->d == 64 && p->d_f == 64) return launch_npmap<64, 64, TOut>(X, W, bias, phi, p->B, heads, N, status, st, launches);
    if (p->d == 128 && p->d_f == 64) return launch_npmap<128, 64, TOut>(X, W, bias, phi, p->B, heads, N, status, st, launches);
    if (p->d == 128 && p->d_f == 128) return launch_npmap<128, 128, TOut>(X, W, bias, phi, p->B, heads, N, status, st, launches);
    return STILL_ERR_UNSUPPORTED;
}

template <int NF>
int launch_scan(const still_params_t *p, long long N, const void *phiQ, const void *phiK, const void *V, const void *G,
                const int32_t *sel_idx, float *nla, float *dla, float *S_out, float *z_out, int *status, cudaStream_t st,
                int *launches) {
    CUtensorMap tk, tv, tq;
    const unsigned long long BH = (unsigned long long)p->B * p->H, BHkv = (unsigned long long)p->B * p->Hkv;
    if (!make_map_2d(&tk, phiK, BHkv * N, NF, 64, false) || !make_map_2d(&tv, V, BHkv * N, p->d, 64, false) ||
        !make_map_2d(&tq, phiQ, BH * N, NF, 64, true))
        return STILL_ERR_CUDA;
    if (ensure_dynamic_smem((const void *)la_scan_tc_kernel<NF>, ScanPlan<NF>::kTotal) !=
        cudaSuccess)
        return STILL_ERR_CUDA;
    dim3 grid((unsigned)BH, (unsigned)(p->d / 64));
    la_scan_tc_kernel<NF><<<grid, 192, ScanPlan<NF>::kTotal, st>>>(tk, tv, tq, (const __nv_bfloat16 *)G, sel_idx, nla, dla,
                                                                  S_out, z_out, status, p->H, p->Hkv, (int)N, p->d,
                                                                  p->chunk, p->topk);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

}  // namespace

bool tc_la_supported(const still_params_t *p) {
    return tc_supported(p) && (p->d_f == 64 || p->d_f == 128) && p->d_f <= p->d;
}

int tc_la_branch(const still_params_t *p, long long N, const void *Q, const void *K, const void *V, const void *G,
                 const void *Wq, const void *bq, const void *Wk, const void *bk, const int32_t *sel_idx, void *phiQ,
                 void *phiK, float *nla, float *dla, float *S_out, float *z_out, int *status_words, cudaStream_t st,
                 int *launches) {
    if ((long long)p->B * p->H * N >= (1ll << 31)) return STILL_ERR_UNSUPPORTED;  // TMA row coordinate
    int rc = launch_npmap_any<float>(p, Q, Wq, bq, phiQ, p->H, N, status_words, st, launches);
    if (rc != STILL_OK) return rc;
    rc = launch_npmap_any<__nv_bfloat16>(p, K, Wk, bk, phiK, p->Hkv, N, status_words, st, launches);
    if (rc != STILL_OK) return rc;
    if (p->d_f == 64)
        return launch_scan<128>(p, N, phiQ, phiK, V, G, sel_idx, nla, dla, S_out, z_out, status_words, st, launches);
    return launch_scan<256>(p, N, phiQ, phiK, V, G, sel_idx, nla, dla, S_out, z_out, status_words, st, launches);
}

}  // namespace still
