// Tensor-core prefill path for bf16 (sm_100a): salient K/V compaction and the
// softmax-attention + merge kernel on tcgen05 / TMEM / TMA.
//
// Softmax Attention Branch of Algorithm 1 + the merge equation of Sec. 3.3.
// For a query in chunk c the keys are: the selected tokens of chunks 0..c-2, all
// of chunk c-1, and chunk c up to the query itself.  The selected rows of every
// chunk are first compacted per query head into K_sel / V_sel ([B*H, sel_rows, d],
// ascending position), so that "selected tokens of chunks 0..c-2" is the prefix
// [0, (c-1)*lambda) of a contiguous array that TMA can tile.
//
// One CTA owns 256 consecutive query rows of one (batch, head): two query tiles
// A and B of 128 rows, each with its own S accumulator (128 fp32 columns of TMEM)
// and O accumulator (d columns).  The key stream of the CTA is a sequence of
// 128-key tiles: SEL tiles j (rows [128j, 128j+128) of K_sel / V_sel) followed by
// the three LOC tiles (rows of K / V at positions [128m, 128m+128), m = m0-1, m0,
// m0+1 with m0 = first row / 128).  Which columns of a tile a query row sees is a
// per-row column interval, applied as a mask in the softmax.
//
// Warp roles (384 threads):
//   warp 0     TMA producer: Q tiles once, then K and V tiles through mbarrier rings
//   warp 1     MMA issuer (one elected thread): S_X = Q_X K^T (operands in shared
//              memory, SWIZZLE_128B K-major), O_X += P_X V (P_X read from TMEM, V in
//              shared memory MN-major); tcgen05.commit signals the softmax warps and
//              frees the ring stages
//   warps 4-7  softmax of tile A: one thread per query row (tcgen05.ld of the S row),
//              online softmax in the log2 domain with lazy rescaling of O, P written
//              back to TMEM as bf16 over S
//   warps 8-11 the same for tile B
//   The softmax warps also run the epilogue: O / l merged with the linear branch
//   (N_LA, D_LA) under one denominator and stored as bf16.
//
// Every mbarrier wait is bounded: on expiry the kernel records
// STILL_ERR_DEVICE_TIMEOUT in the status word, all roles leave their loops, and
// tensor memory is freed before the CTA exits.
#include "still_tc.h"

#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "still_common.cuh"
#include "still_tc_ptx.cuh"

// Column pairs out of every four whose exponential is computed on the FMA pipes (see softmax_role); measured
// best at one: two and three were slower on both head dims.
#ifndef STILL_POLY_OF4
#define STILL_POLY_OF4 1
#endif

namespace still {

namespace {

constexpr int kBlockM = 128;   // query rows per tile
constexpr int kBlockN = 128;   // keys per tile
constexpr int kThreads = 384;
using namespace ptx;

// ----------------------------------------------------------------- shared memory plan

template <int D>
struct SmemPlan {
    static constexpr int kTileBytes = kBlockN * D * 2;        // one K or V or Q tile
    static constexpr int kKStages = (D == 128) ? 3 : 4;
    static constexpr int kVStages = (D == 128) ? 2 : 3;
    static constexpr int kQ = 0;                               // two Q tiles
    static constexpr int kK = kQ + 2 * kTileBytes;
    static constexpr int kV = kK + kKStages * kTileBytes;
    static constexpr int kBar = kV + kVStages * kTileBytes;    // mbarriers
    static constexpr int kNumBars = 1 + 2 * kKStages + 2 * kVStages + 9;
    static constexpr int kMisc = kBar + kNumBars * 8;          // tmem base, abort flag
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kAlloc = kTotal + 1024;               // slack to align the base to 1024
};

constexpr int kMaxDynamicSmem = 232448;   // 227 KiB: the most a CTA can be given on sm_100
static_assert(SmemPlan<64>::kAlloc <= kMaxDynamicSmem && SmemPlan<128>::kAlloc <= kMaxDynamicSmem,
              "attention kernel: the shared-memory plan exceeds what a CTA can have");
// every operand descriptor of the attention kernel addresses a whole tile inside its ring
static_assert(SmemPlan<128>::kK == SmemPlan<128>::kQ + 2 * SmemPlan<128>::kTileBytes &&
              SmemPlan<128>::kBar == SmemPlan<128>::kV + SmemPlan<128>::kVStages * SmemPlan<128>::kTileBytes,
              "attention kernel: rings must follow each other without gaps");

// Per-CTA description of the key stream.
struct Stream {
    int sel_first;          // first SEL tile of the stream (0 unless the salient cache has a budget)
    int n_sel_a, n_sel_b;   // SEL tiles used by tile A / tile B, counted from sel_first
    int m0;                 // first LOC tile index of interest is m0 - 1
    int has_prev;           // m0 > 0
    int has_b;              // tile B has rows below N
    int n_tiles;            // stream length
    // stream index i: [0, n_sel_b) SEL(i); then LOC(m0-1) (if has_prev), LOC(m0), LOC(m0+1) (if has_b)
    __device__ __forceinline__ bool is_sel(int i) const { return i < n_sel_b; }
    __device__ __forceinline__ int loc_m(int i) const { return m0 - has_prev + (i - n_sel_b); }
    __device__ __forceinline__ bool used_by(int x, int i) const {
        if (i < n_sel_b) return x == 0 ? (i < n_sel_a) : true;
        int m = loc_m(i);
        return x == 0 ? (m <= m0) : (m >= m0);
    }
};

__device__ __forceinline__ int sel_limit(long long pos, int C, int lam) {  // end of the visible range of K_sel
    long long c = pos / C;
    return c >= 2 ? (int)((c - 1) * lam) : 0;
}
// Start of the visible range: 0, or with a salient-cache budget of `budget` tokens per head (a multiple of lam;
// the oldest cached tokens have left for the linear state) the last `budget` entries before the end.
__device__ __forceinline__ int sel_start(int limit, int budget) { return budget > 0 ? max(limit - budget, 0) : 0; }

// ---------------------------------------------------------------------------
// Softmax warps of the attention kernels (one warpgroup per query tile, a thread per query row) and the
// merge epilogue.  `st` describes the CTA's (or the CTA pair's) key stream, x is the query tile (0: A, 1: B),
// tile_row0 the position of the tile's first row, stage_tile the tile's Q region in shared memory (the
// epilogue's staging space).  The barriers are this CTA's, except that in a CTA pair the two halves of P
// are announced on the first CTA's p_half barriers (p_half_cluster: their address in the cluster window).
// ---------------------------------------------------------------------------
template <int D, int kKStages, int kVStages, bool kPair, int kPolyOf4, class StreamT>
__device__ __forceinline__ void softmax_role(const StreamT &st, const int x, const int tile_row0, const uint32_t tmem_base,
                                             uint64_t *s_full, uint64_t *k_empty, uint64_t *v_empty, uint64_t *p_half,
                                             const uint32_t p_half_cluster, uint64_t *o_final, volatile int *abort_flag,
                                             int *status, uint8_t *stage_tile, const __nv_bfloat16 *__restrict__ y_part,
                                             const float *__restrict__ d_part, const int n_parts, const long long part_stride_y,
                                             const long long part_stride_d, __nv_bfloat16 *__restrict__ Y, const int bh,
                                             const int N, const int C, const int lam, const int budget,
                                             const float scale_log2) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto col_s = [](int xx) -> uint32_t { return (uint32_t)xx * 128u; };
    auto col_o = [](int xx) -> uint32_t { return 256u + (uint32_t)xx * (uint32_t)D; };
    auto arrive_p = [&](int half) {
        if constexpr (kPair) mbar_arrive_cluster(p_half_cluster + (uint32_t)(2 * x + half) * 8u);
        else mbar_arrive(p_half + 2 * x + half);
    };
        const int row_in_tile = ((warp & 3) << 5) | lane;
    const int t = tile_row0 + row_in_tile;         // this thread's query position
    const bool tile_present = (x == 0) || st.has_b;   // (a tile without rows below N still runs in a pair)
    if (tile_present) {
        const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const int tq = min(t, N - 1);              // rows past N mimic the last row (never stored)
        const int c = tq / C;
        const int lim_sel = c >= 2 ? (c - 1) * lam : 0, lo_sel = sel_start(lim_sel, budget);
        const int loc_lo = c >= 1 ? (c - 1) * C : 0;
        float m_used = -INFINITY, l_sum = 0.f;     // log2 domain
        int n_seen = 0, prev_i = -1;
        bool ok = true;
        for (int i = 0; i < st.n_tiles && ok; ++i) {
            if (!st.used_by(x, i)) continue;
            // visible column interval [lo, hi] of this row in stream tile i
            int lo, hi;
            if (st.is_sel(i)) {
                lo = lo_sel - (st.sel_first + i) * kBlockN;
                hi = lim_sel - (st.sel_first + i) * kBlockN - 1;
            } else {
                const int p0 = st.loc_m(i) * kBlockN;
                lo = loc_lo - p0;
                hi = tq - p0;
            }
            lo = max(lo, 0);
            hi = min(hi, kBlockN - 1);
            const bool need_mask = __any_sync(0xffffffffu, lo > 0 || hi < kBlockN - 1);
            ok = mbar_wait(s_full + x, n_seen & 1, abort_flag, status, 8);
            if (!ok) break;
            tc_fence_after();
            if (row_in_tile == 0) {
                // S_x of tile i is complete, and so is everything the MMA warp issued before it (each
                // tcgen05.commit costs the tensor pipe a bubble, so the ring stages are released here
                // instead): tile x is done with this K stage and with the V stage of its previous tile.
                mbar_arrive(k_empty + i % kKStages);
                if (prev_i >= 0) mbar_arrive(v_empty + prev_i % kVStages);
            }
            prev_i = i;
            uint32_t sr[128];
            tmem_ld32(lane_addr + col_s(x) + 0, sr + 0);
            tmem_ld32(lane_addr + col_s(x) + 32, sr + 32);
            tmem_ld32(lane_addr + col_s(x) + 64, sr + 64);
            tmem_ld32(lane_addr + col_s(x) + 96, sr + 96);
            tmem_wait_ld();
            float *s = reinterpret_cast<float *>(sr);
            if (need_mask) {
#pragma unroll
                for (int j = 0; j < 128; ++j)
                    if (j < lo || j > hi) s[j] = -INFINITY;
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int j = 0; j < 128; j += 8) {
                mx0 = max3(mx0, s[j], s[j + 1]);
                mx1 = max3(mx1, s[j + 2], s[j + 3]);
                mx2 = max3(mx2, s[j + 4], s[j + 5]);
                mx3 = max3(mx3, s[j + 6], s[j + 7]);
            }
            const float mt = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale_log2;
            // lazy rescale: keep the old reference unless the new maximum exceeds it by 2^8
            const bool grow = mt > m_used + 8.f;
            float alpha = 1.f;
            if (grow) {
                alpha = (m_used == -INFINITY) ? 0.f : ex2(m_used - mt);
                m_used = mt;
            }
            if (n_seen > 0 && __any_sync(0xffffffffu, grow)) {
                // S of this tile was committed after the previous P V product: O is quiescent
#pragma unroll
                for (int q = 0; q < D / 32; ++q) {
                    uint32_t orow[32];
                    tmem_ld32(lane_addr + col_o(x) + q * 32, orow);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * alpha);
                    tmem_st32(lane_addr + col_o(x) + q * 32, orow);
                }
            }
            l_sum *= alpha;
            const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
            const float2 scale2 = make_float2(scale_log2, scale_log2), negm2 = make_float2(neg_m, neg_m);
            float2 acc = make_float2(0.f, 0.f);
            // P = 2^(s * scale - m) as bf16 over S, in two halves of 64 columns; the MMA warp starts on the first
            // half while the second is computed.  The MUFU unit (one warp instruction per eight cycles) would need
            // 1024 cycles for a warp's 128 exponentials of a tile, which is as long as the tensor pipe needs for the
            // tile's two products; so kPolyOf4 of every four column pairs take 2^x from the FMA pipes instead (see
            // exp2_fma2), interleaved with the others so that both units work at the same time.
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t pk[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float2 sv = make_float2(s[q * 64 + 2 * j], s[q * 64 + 2 * j + 1]);
                    const float2 xv = __ffma2_rn(sv, scale2, negm2);
                    const float2 pr = (j % 4) < kPolyOf4 ? exp2_fma2(xv) : make_float2(ex2(xv.x), ex2(xv.y));
                    acc = __fadd2_rn(acc, pr);
                    pk[j] = pack_bf16(pr.x, pr.y);
                    if (q == 1 && j == 12) {
                        // the first half of P has had time to land: hand it to the MMA warp
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) arrive_p(0);
                    }
                }
                tmem_st32(lane_addr + col_s(x) + q * 32, pk);
            }
            l_sum += acc.x + acc.y;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) arrive_p(1);
            ++n_seen;
        }
        // ---- epilogue: y = (O e^{m-ms} + e^{-ms} N_LA) / (l e^{m-ms} + e^{-ms} D_LA), ms = max(m, 0)
        // The linear branch arrives as up to two partial results (one per feature half): y_p = N_p / D_p as bf16
        // and D_p, so N_LA = sum y_p D_p and D_LA = sum D_p.  A thread owns a row, but loads / stores in which
        // every lane touches a different row cost a memory instruction per 16 bytes and row; so the y_p come in
        // and Y goes out through shared memory with 16 consecutive lanes per row.  The staging space is this
        // warp's 32 rows of the tile's Q region (one row = D bf16 = 2 D bytes: D / 2 columns of both parts), free
        // once the tile's last Q K^T has completed; 16-byte pieces are swizzled by the row so that row-wise and
        // piece-wise accesses avoid bank conflicts.
        if (ok) ok = mbar_wait(o_final + x, 0, abort_flag, status, 9);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            constexpr int kRowBytes = D * 2, kPieces = kRowBytes / 16;   // pieces of 16 bytes per staged row
            constexpr int kPartPieces = kPieces / 2;                     // pieces of one part (D / 2 columns)
            uint8_t *stg = stage_tile + (warp & 3) * 32 * kRowBytes;
            const int t0 = tile_row0 + (warp & 3) * 32;                    // first row of this warp
            float fs = 1.f, fa = 0.f, fb = 0.f, dla = 0.f;
            if (n_parts > 0 && t < N) {
                const float da = d_part[(long long)bh * N + t];
                const float db = n_parts > 1 ? d_part[part_stride_d + (long long)bh * N + t] : 0.f;
                dla = da + db;
                if (dla > 0.f) {
                    const float m_nat = m_used * 0.6931471805599453f;
                    const float ms = fmaxf(m_nat, 0.f);
                    fs = __expf(m_nat - ms);
                    const float fl = __expf(-ms);
                    fa = fl * da;
                    fb = fl * db;
                }
            }
            const float inv = 1.f / (l_sum * fs + fa + fb);
            const bool with_la = (n_parts > 0) && __any_sync(0xffffffffu, dla > 0.f);
            uint32_t out[D / 2];   // the row as packed bf16
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {   // halves of D / 2 columns
                if (with_la) {
                    __syncwarp();
#pragma unroll
                    for (int it = 0; it < kPieces; ++it) {
                        const int id = it * 32 + lane, row = id / kPieces, c = id % kPieces;
                        const int part = c / kPartPieces, cc = c % kPartPieces;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (t0 + row < N && part < n_parts)
                            v = *reinterpret_cast<const uint4 *>(y_part + part * part_stride_y + ((long long)bh * N + t0 + row) * D +
                                                                 hh * (D / 2) + cc * 8);
                        *reinterpret_cast<uint4 *>(stg + row * kRowBytes + ((c ^ (row & (kPieces - 1))) << 4)) = v;
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int q = 0; q < D / 64; ++q) {
                    uint32_t orow[32];
                    tmem_ld32(lane_addr + col_o(x) + hh * (D / 2) + q * 32, orow);
                    tmem_wait_ld();
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        uint4 pa = make_uint4(0, 0, 0, 0), pb = pa;
                        if (with_la) {
                            const int ca = q * 4 + j8, cb = kPartPieces + ca;
                            pa = *reinterpret_cast<const uint4 *>(stg + lane * kRowBytes + ((ca ^ (lane & (kPieces - 1))) << 4));
                            pb = *reinterpret_cast<const uint4 *>(stg + lane * kRowBytes + ((cb ^ (lane & (kPieces - 1))) << 4));
                        }
                        const uint32_t wa[4] = {pa.x, pa.y, pa.z, pa.w}, wb[4] = {pb.x, pb.y, pb.z, pb.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {   // two columns per 32-bit word
                            const float la0 = fmaf(fa, __uint_as_float(wa[e] << 16), fb * __uint_as_float(wb[e] << 16));
                            const float la1 = fmaf(fa, __uint_as_float(wa[e] & 0xffff0000u), fb * __uint_as_float(wb[e] & 0xffff0000u));
                            const float a0 = fmaf(__uint_as_float(orow[8 * j8 + 2 * e]), fs, la0);
                            const float a1 = fmaf(__uint_as_float(orow[8 * j8 + 2 * e + 1]), fs, la1);
                            out[hh * (D / 4) + q * 16 + 4 * j8 + e] = pack_bf16(a0 * inv, a1 * inv);
                        }
                    }
                }
            }
            // Y: own row into the staging space, then the warp writes its 32 rows piece-wise
            __syncwarp();
#pragma unroll
            for (int c = 0; c < kPieces; ++c)
                *reinterpret_cast<uint4 *>(stg + lane * kRowBytes + ((c ^ (lane & (kPieces - 1))) << 4)) =
                    make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
            __syncwarp();
#pragma unroll
            for (int it = 0; it < kPieces; ++it) {
                const int id = it * 32 + lane, row = id / kPieces, c = id % kPieces;
                if (t0 + row < N)
                    *reinterpret_cast<uint4 *>(Y + ((long long)bh * N + t0 + row) * D + c * 8) =
                        *reinterpret_cast<const uint4 *>(stg + row * kRowBytes + ((c ^ (row & (kPieces - 1))) << 4));
            }
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
sa_merge_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_ksel,
                   const __grid_constant__ CUtensorMap tm_vsel, const __nv_bfloat16 *__restrict__ y_part,
                   const float *__restrict__ d_part, int n_parts, __nv_bfloat16 *__restrict__ Y, int *status, int H, int Hkv,
                   int N, int C, int lam, int budget, int sel_rows, int sel_identity, float scale_log2, int n_qblocks) {
    using P = SmemPlan<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + P::kBar);
    uint64_t *q_full = bars;
    uint64_t *k_full = bars + 1, *k_empty = k_full + P::kKStages;
    uint64_t *v_full = k_empty + P::kKStages, *v_empty = v_full + P::kVStages;
    uint64_t *s_full = v_empty + P::kVStages;  // [2]
    uint64_t *p_half = s_full + 2;             // [2][2]: columns [0,64) / [64,128) of P_X are in TMEM
    uint64_t *o_final = p_half + 4;            // [2]
    uint64_t *drain = o_final + 2;             // MMA warp: everything issued has completed (failure path)
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(smem + P::kMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + P::kMisc + 8);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;   // (known to be the same in all lanes)
    const int qb = n_qblocks - 1 - blockIdx.x;  // heavy blocks first
    const int bh = blockIdx.y, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int R0 = qb * 2 * kBlockM;

    Stream st;
    st.m0 = R0 / kBlockN;
    st.has_prev = st.m0 > 0;
    st.has_b = (R0 + kBlockM) < N;
    {
        int last_a = min(R0 + kBlockM - 1, N - 1), last_b = min(R0 + 2 * kBlockM - 1, N - 1);
        st.sel_first = sel_start(sel_limit(R0, C, lam), budget) / kBlockN;   // the CTA's first row sees the oldest entries
        st.n_sel_a = max((sel_limit(last_a, C, lam) + kBlockN - 1) / kBlockN - st.sel_first, 0);
        st.n_sel_b = st.has_b ? max((sel_limit(last_b, C, lam) + kBlockN - 1) / kBlockN - st.sel_first, 0) : st.n_sel_a;
    }
    st.n_tiles = st.n_sel_b + st.has_prev + 1 + st.has_b;

    // A CTA that starts after another one has reported a failure does nothing.
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status) != 0;
    __syncthreads();
    if (*abort_flag) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < P::kKStages; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 2); }
        for (int i = 0; i < P::kVStages; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 2); }
        for (int i = 0; i < 2; ++i) { mbar_init(s_full + i, 1); mbar_init(o_final + i, 1); }
        for (int i = 0; i < 4; ++i) mbar_init(p_half + i, 4);  // one arrival per softmax warp
        mbar_init(drain, 1);
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
    // TMEM columns: S_A [0,128), S_B [128,256), O_A [256,256+D), O_B [256+D, 256+2D); P_X overlays S_X.
    auto col_s = [](int x) -> uint32_t { return (uint32_t)x * 128u; };
    auto col_o = [](int x) -> uint32_t { return 256u + (uint32_t)x * (uint32_t)D; };

    // The softmax threads keep a whole 128-column row in registers: move registers from the
    // load / MMA warpgroup to the two softmax warpgroups (128 * 64 + 256 * 216 <= 384 * 168).
    if (warp < 4) {
    reg_dec<64>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int q_row = bh * N + R0;
            mbar_expect_tx(q_full, (st.has_b ? 2 : 1) * P::kTileBytes);
            for (int x = 0; x < (st.has_b ? 2 : 1); ++x)
                for (int half = 0; half < D / 64; ++half)
                    tma_load_2d(smem + P::kQ + x * P::kTileBytes + half * (kBlockM * 128), &tm_q, q_full, half * 64,
                                q_row + x * kBlockM);
            // With topk = chunk every token is selected and the compacted arrays would be copies of K / V:
            // the salient prefix is then read from K / V themselves (tm_ksel / tm_vsel alias tm_k / tm_v).
            const int sel_base = sel_identity ? (b * Hkv + kvh) * N : bh * sel_rows;
            // K and V rings advance independently, each as far ahead as its free stages allow.
            bool ok = true;
            int armed_k = 0, armed_v = 0, spins = 0;
            long long t0 = clock64();
            while (armed_k < st.n_tiles || armed_v < st.n_tiles) {
                bool progressed = false;
                if (armed_k < st.n_tiles) {
                    const int i = armed_k, ks = i % P::kKStages;
                    if (mbar_try_wait(k_empty + ks, ((i / P::kKStages) & 1) ^ 1)) {
                        const bool sel = st.is_sel(i);
                        const int row = sel ? sel_base + (st.sel_first + i) * kBlockN : (b * Hkv + kvh) * N + st.loc_m(i) * kBlockN;
                        mbar_expect_tx(k_full + ks, P::kTileBytes);
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_2d(smem + P::kK + ks * P::kTileBytes + half * (kBlockN * 128), sel ? &tm_ksel : &tm_k,
                                        k_full + ks, half * 64, row);
                        ++armed_k;
                        progressed = true;
                    }
                }
                if (armed_v < st.n_tiles) {
                    const int i = armed_v, vs = i % P::kVStages;
                    if (mbar_try_wait(v_empty + vs, ((i / P::kVStages) & 1) ^ 1)) {
                        const bool sel = st.is_sel(i);
                        const int row = sel ? sel_base + (st.sel_first + i) * kBlockN : (b * Hkv + kvh) * N + st.loc_m(i) * kBlockN;
                        mbar_expect_tx(v_full + vs, P::kTileBytes);
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_2d(smem + P::kV + vs * P::kTileBytes + half * (kBlockN * 128), sel ? &tm_vsel : &tm_v,
                                        v_full + vs, half * 64, row);
                        ++armed_v;
                        progressed = true;
                    }
                }
                if (progressed) {
                    spins = 0;
                } else if ((++spins & 1023) == 0) {
                    if (spins == 1024) t0 = clock64();
                    if (*abort_flag) { ok = false; break; }
                    if (clock64() - t0 > kWaitLimitCycles) {
                        *abort_flag = 1;
                        report_status(status, STILL_ERR_DEVICE_TIMEOUT, 1);
                        ok = false;
                        break;
                    }
                }
            }
            if (!ok) {
                // leave no copy in flight behind: wait (bounded) for the loads already issued
                if (armed_k > 0) {
                    int i = armed_k - 1;
                    mbar_wait_drain(k_full + i % P::kKStages, (i / P::kKStages) & 1);
                }
                if (armed_v > 0) {
                    int i = armed_v - 1;
                    mbar_wait_drain(v_full + i % P::kVStages, (i / P::kVStages) & 1);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the stream and waits on the barriers; one elected lane issues (control flow and
        // descriptors stay the same in all lanes and can live in uniform registers, where the tensor-core
        // instructions take their operands from).  A failed wait does not leave the loop: it switches off the
        // remaining waits and instructions, and the loop runs out.
        {
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = make_idesc(kBlockM, kBlockN, false);
            constexpr uint32_t idesc_pv = make_idesc(kBlockM, D, true);
            bool ok = mbar_wait(q_full, 0, abort_flag, status, 4);
            tc_fence_after();
            // descriptors as low words: a k-step adds a constant
            const uint32_t q_lo0 = desc_lo(smem_u32(smem + P::kQ), 0);
            const uint32_t k_lo0 = desc_lo(smem_u32(smem + P::kK), 0);
            const uint32_t v_lo0 = desc_lo(smem_u32(smem + P::kV), kBlockN * 128);
            int pending[2] = {-1, -1};   // stream tile whose P V product is still to be issued
            int n_done[2] = {0, 0};      // tiles processed per query tile (phase of p_full)
            auto wait = [&](uint64_t *bar, int parity, int where) {
                if (ok) ok = mbar_wait(bar, (uint32_t)parity, abort_flag, status, where);
            };
            auto issue_pv = [&](int x, int ip) {
                const int vs = ip % P::kVStages;
                // (V has normally arrived long ago: checking it first hides the check behind the wait for P)
                wait(v_full + vs, (ip / P::kVStages) & 1, 6);
                wait(p_half + 2 * x, n_done[x] & 1, 5);
                tc_fence_after();
                const uint32_t v_lo = v_lo0 + vs * (P::kTileBytes >> 4);
                const uint32_t d_o = tmem_base + col_o(x), a_p = tmem_base + col_s(x);
                const uint32_t acc0 = n_done[x] > 0 ? 1u : 0u;
                if (leader && ok) {
                    mma_ts_lo<idesc_pv>(d_o, a_p, v_lo, acc0);
#pragma unroll
                    for (int k = 1; k < kBlockN / 32; ++k)
                        mma_ts_lo<idesc_pv>(d_o, a_p + k * 8, v_lo + k * (16 * 128 >> 4), 1u);
                }
                wait(p_half + 2 * x + 1, n_done[x] & 1, 5);
                tc_fence_after();
                if (leader && ok) {
#pragma unroll
                    for (int k = kBlockN / 32; k < kBlockN / 16; ++k)
                        mma_ts_lo<idesc_pv>(d_o, a_p + k * 8, v_lo + k * (16 * 128 >> 4), 1u);
                }
                ++n_done[x];
            };
            for (int i = 0; i < st.n_tiles; ++i) {
                const int ks = i % P::kKStages;
                wait(k_full + ks, (i / P::kKStages) & 1, 7);
                tc_fence_after();
                const uint32_t k_lo = k_lo0 + ks * (P::kTileBytes >> 4);
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const bool present = (x == 0) || st.has_b;
                    if (present && st.used_by(x, i)) {
                        if (pending[x] >= 0) {
                            const int ip = pending[x];
                            issue_pv(x, ip);
                            // a V stage is released by two arrivals: pay the other tile's share if it skipped ip
                            if (leader && ok && !(((1 - x) == 0 || st.has_b) && st.used_by(1 - x, ip)))
                                mbar_arrive(v_empty + ip % P::kVStages);
                        }
                        const uint32_t q_lo = q_lo0 + x * (P::kTileBytes >> 4), d_s = tmem_base + col_s(x);
                        if (leader && ok) {
                            mma_ss_lo<idesc_qk, 0>(d_s, q_lo, k_lo);
#pragma unroll
                            for (int k = 1; k < D / 16; ++k) {
                                // k-step of 16 elements: 32 bytes within a 64-element swizzle atom, atoms 128 rows apart
                                const uint32_t off = ((k / 4) * (kBlockM * 128) + (k % 4) * 32) >> 4;
                                mma_ss_lo<idesc_qk, 1>(d_s, q_lo + off, k_lo + off);
                            }
                            tc_commit(s_full + x);
                        }
                        pending[x] = i;
                    } else if (leader && ok) {
                        mbar_arrive(k_empty + ks);  // the share of a tile that skips this stream tile
                    }
                }
            }
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (pending[x] >= 0) {
                    issue_pv(x, pending[x]);
                    if (leader && ok) tc_commit(o_final + x);
                }
            }
            if (!__all_sync(0xffffffffu, ok) && leader) {  // no MMA may still be running when tensor memory is freed
                tc_commit(drain);
                mbar_wait_drain(drain, 0);
            }
        }
    }
    } else {
        reg_inc<216>();
        // ------------------------------------------------------------ softmax + epilogue
        const int x = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
        softmax_role<D, P::kKStages, P::kVStages, false, STILL_POLY_OF4>(st, x, R0 + x * kBlockM, tmem_base, s_full, k_empty, v_empty, p_half, 0u,
                                                         o_final, abort_flag, status, smem + P::kQ + x * P::kTileBytes, y_part,
                                                         d_part, n_parts, (long long)gridDim.y * N * D, (long long)gridDim.y * N,
                                                         Y, bh, N, C, lam, budget, scale_log2);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------
// The same branch on CTA pairs (head dim 128): two CTAs of a cluster work on 512 consecutive query rows of
// one (batch, head) with UMMAs of the cta_group::2 form.  Query tile X of the pair is 256 rows -- rows
// [R0 + 256 X + 128 r, + 128) belong to the CTA of cluster rank r -- and one instruction, issued by a thread
// of rank 0, computes S_X = Q_X K^T (or O_X += P_X V) for both CTAs.  Each CTA keeps only its half of every
// key tile in shared memory: 64 of the 128 keys of K (the B operand of Q K^T is split along N) and 64 of the
// 128 value columns of V (likewise for P V); the tensor cores of both SMs read both halves.  Per FLOP a CTA
// therefore pulls half the K / V bytes from L2 and reads a quarter less shared memory than a CTA working
// alone, and the rings hold five stages each.
//
// Who signals whom.  K / V / Q tiles: every CTA loads its halves into its own shared memory with plain TMA
// loads (no multicast) whose byte counts complete on the full-barriers of rank 0, where the issuing thread
// waits.  S_X ready, O_X final: one tcgen05.commit arrives on the barrier of both CTAs.  P_X written: the
// softmax warps of both CTAs arrive on rank 0's p_half barriers (eight arrivals).  Ring stages are released
// locally: when a CTA's softmax warps see S_X of stream tile i, the pair's instruction has completed in both
// CTAs.  Everything else -- stream, masks, online softmax, merge epilogue -- is as in the kernel above.
// ---------------------------------------------------------------------------
template <int D>
struct PairPlan {
    static constexpr int kQTile = kBlockM * D * 2;             // one Q tile of this CTA (128 rows)
    static constexpr int kKHalf = (kBlockN / 2) * D * 2;       // 64 keys of a K tile
    static constexpr int kVHalf = kBlockN * (D / 2) * 2;       // 128 keys x D / 2 value columns
    static constexpr int kKStages = 5, kVStages = 5;
    static constexpr int kQ = 0;
    static constexpr int kK = kQ + 2 * kQTile;
    static constexpr int kV = kK + kKStages * kKHalf;
    static constexpr int kBar = kV + kVStages * kVHalf;
    static constexpr int kNumBars = 1 + 2 * kKStages + 2 * kVStages + 9;
    static constexpr int kMisc = kBar + kNumBars * 8;          // tmem base, abort flag, "a CTA has failed before"
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kAlloc = kTotal + 1024;
};
static_assert(PairPlan<128>::kAlloc <= kMaxDynamicSmem, "pair attention kernel: the shared-memory plan exceeds what a CTA can have");

// Key stream of a CTA pair (same in both CTAs): SEL tiles, then the LOC tiles m_first .. m_last.
struct PairStream {
    int sel_first, n_sel_a, n_sel_b, m0, m_first, has_b, n_tiles;   // SEL tiles are counted from sel_first
    __device__ __forceinline__ bool is_sel(int i) const { return i < n_sel_b; }
    __device__ __forceinline__ int loc_m(int i) const { return m_first + (i - n_sel_b); }
    __device__ __forceinline__ bool used_by(int x, int i) const {
        if (i < n_sel_b) return x == 0 ? (i < n_sel_a) : true;
        const int m = loc_m(i);
        return x == 0 ? (m <= m0 + 1) : (m >= m0 + 1);
    }
};

template <int D>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
sa_merge_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_ksel,
                     const __grid_constant__ CUtensorMap tm_vsel, const __nv_bfloat16 *__restrict__ y_part,
                     const float *__restrict__ d_part, int n_parts, __nv_bfloat16 *__restrict__ Y, int *status, int H, int Hkv, int N,
                     int C, int lam, int budget, int sel_rows, int sel_identity, float scale_log2, int n_pairs) {
    using P = PairPlan<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + P::kBar);
    uint64_t *q_full = bars;
    uint64_t *k_full = bars + 1, *k_empty = k_full + P::kKStages;
    uint64_t *v_full = k_empty + P::kKStages, *v_empty = v_full + P::kVStages;
    uint64_t *s_full = v_empty + P::kVStages;  // [2]
    uint64_t *p_half = s_full + 2;             // [2][2]
    uint64_t *o_final = p_half + 4;            // [2]
    uint64_t *drain = o_final + 2;
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(smem + P::kMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + P::kMisc + 4);
    volatile int *failed_before = reinterpret_cast<volatile int *>(smem + P::kMisc + 8);

    // (warp index and cluster rank through a shuffle / from the block index: values the compiler knows to be
    // the same in all lanes)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const uint32_t rank = blockIdx.x & 1u, peer = rank ^ 1u;
    const int pb = n_pairs - 1 - (int)(blockIdx.x >> 1);  // heavy blocks first
    const int bh = blockIdx.y, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int R0 = pb * 4 * kBlockM;

    PairStream st;
    st.m0 = R0 / kBlockN;
    st.m_first = st.m0 - (st.m0 > 0 ? 1 : 0);
    st.has_b = (R0 + 2 * kBlockM) < N;
    {
        const int last_a = min(R0 + 2 * kBlockM - 1, N - 1), last_b = min(R0 + 4 * kBlockM - 1, N - 1);
        st.sel_first = sel_start(sel_limit(R0, C, lam), budget) / kBlockN;   // the pair's first row sees the oldest entries
        st.n_sel_a = max((sel_limit(last_a, C, lam) + kBlockN - 1) / kBlockN - st.sel_first, 0);
        st.n_sel_b = st.has_b ? max((sel_limit(last_b, C, lam) + kBlockN - 1) / kBlockN - st.sel_first, 0) : st.n_sel_a;
        const int m_last = min(st.m0 + (st.has_b ? 3 : 1), (N - 1) / kBlockN);
        st.n_tiles = st.n_sel_b + (m_last - st.m_first + 1);
    }

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < P::kKStages; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 2); }
        for (int i = 0; i < P::kVStages; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 2); }
        for (int i = 0; i < 2; ++i) { mbar_init(s_full + i, 1); mbar_init(o_final + i, 1); }
        for (int i = 0; i < 4; ++i) mbar_init(p_half + i, 8);  // one arrival per softmax warp of either CTA
        mbar_init(drain, 1);
        *abort_flag = 0;
        *failed_before = 0;
        fence_barrier_init();
    }
    // The peer's barriers exist and its shared memory may be written from here on.
    cluster_sync_all();
    // A pair that starts after some CTA has reported a failure does nothing; rank 0 decides for both.
    if (threadIdx.x == 0 && rank == 0) {
        const int seen = *reinterpret_cast<volatile int *>(status) != 0;
        *failed_before = seen;
        st_cluster_u32(mapa(smem_u32(const_cast<int *>(failed_before)), 1), (uint32_t)seen);
    }
    cluster_sync_all();
    if (*failed_before) return;
    if (warp == 1) {
        tmem_alloc_pair(tmem_base_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();   // both CTAs hold their tensor memory before the first instruction of the pair
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_base_slot, 0);
    auto col_s = [](int x) -> uint32_t { return (uint32_t)x * 128u; };
    auto col_o = [](int x) -> uint32_t { return 256u + (uint32_t)x * (uint32_t)D; };
    // a role that gives up tells the other CTA, whose waits would otherwise run to their own limit
    auto tell_peer = [&]() { st_cluster_u32(mapa(smem_u32(const_cast<int *>(abort_flag)), peer), 1u); };

    if (warp < 4) {
    reg_dec<72>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            const uint32_t q_full0 = mapa(smem_u32(q_full), 0), k_full0 = mapa(smem_u32(k_full), 0),
                           v_full0 = mapa(smem_u32(v_full), 0);
            const int n_q = st.has_b ? 2 : 1;
            const int q_row = bh * N + R0 + (int)rank * kBlockM;
            if (rank == 0) mbar_expect_tx(q_full, 2 * n_q * P::kQTile);   // both CTAs' tiles
            for (int x = 0; x < n_q; ++x)
                for (int half = 0; half < D / 64; ++half)
                    tma_load_2d_pair(smem + P::kQ + x * P::kQTile + half * (kBlockM * 128), &tm_q, q_full0, half * 64,
                                     q_row + x * 2 * kBlockM);
            const int sel_base = sel_identity ? (b * Hkv + kvh) * N : bh * sel_rows;
            bool ok = true;
            int armed_k = 0, armed_v = 0, spins = 0;
            long long t0 = clock64();
            while (armed_k < st.n_tiles || armed_v < st.n_tiles) {
                bool progressed = false;
                if (armed_k < st.n_tiles) {
                    const int i = armed_k, ks = i % P::kKStages;
                    if (mbar_try_wait(k_empty + ks, ((i / P::kKStages) & 1) ^ 1)) {
                        const bool sel = st.is_sel(i);
                        const int row = (sel ? sel_base + (st.sel_first + i) * kBlockN : (b * Hkv + kvh) * N + st.loc_m(i) * kBlockN) +
                                        (int)rank * (kBlockN / 2);   // this CTA's 64 keys
                        if (rank == 0) mbar_expect_tx(k_full + ks, 2 * P::kKHalf);
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_2d_pair(smem + P::kK + ks * P::kKHalf + half * ((kBlockN / 2) * 128), sel ? &tm_ksel : &tm_k,
                                             k_full0 + ks * 8, half * 64, row);
                        ++armed_k;
                        progressed = true;
                    }
                }
                if (armed_v < st.n_tiles) {
                    const int i = armed_v, vs = i % P::kVStages;
                    if (mbar_try_wait(v_empty + vs, ((i / P::kVStages) & 1) ^ 1)) {
                        const bool sel = st.is_sel(i);
                        const int row = sel ? sel_base + (st.sel_first + i) * kBlockN : (b * Hkv + kvh) * N + st.loc_m(i) * kBlockN;
                        if (rank == 0) mbar_expect_tx(v_full + vs, 2 * P::kVHalf);
                        for (int q = 0; q < D / 128; ++q)           // this CTA's D / 2 value columns, 64 at a time
                            tma_load_2d_pair(smem + P::kV + vs * P::kVHalf + q * (kBlockN * 128), sel ? &tm_vsel : &tm_v,
                                             v_full0 + vs * 8, (int)rank * (D / 2) + q * 64, row);
                        ++armed_v;
                        progressed = true;
                    }
                }
                if (progressed) {
                    spins = 0;
                } else if ((++spins & 1023) == 0) {
                    if (spins == 1024) t0 = clock64();
                    if (*abort_flag) { ok = false; break; }
                    if (clock64() - t0 > kWaitLimitCycles) {
                        *abort_flag = 1;
                        report_status(status, STILL_ERR_DEVICE_TIMEOUT, 51);
                        ok = false;
                        break;
                    }
                }
            }
            if (!ok) {
                tell_peer();
                // leave no copy in flight behind: rank 0 waits (bounded) for the last stages armed, which count
                // both CTAs' bytes; rank 1, whose copies complete on rank 0's barriers, waits out a fixed
                // stretch that is long against a tile load
                if (rank == 0) {
                    if (armed_k > 0) mbar_wait_drain(k_full + (armed_k - 1) % P::kKStages, ((armed_k - 1) / P::kKStages) & 1);
                    if (armed_v > 0) mbar_wait_drain(v_full + (armed_v - 1) % P::kVStages, ((armed_v - 1) / P::kVStages) & 1);
                } else {
                    const long long t1 = clock64();
                    while (clock64() - t1 < 200000) {}
                }
            }
        }
    } else if (warp == 1 && rank == 0) {
        // ------------------------------------------------------------ MMA issuer (rank 0 only)
        // The whole warp walks the stream and waits on the barriers; one elected lane issues.  Kept this way,
        // control flow and every descriptor are the same in all lanes, which lets them live in the warp's
        // uniform registers, where the tensor-core instructions take their operands from.  (With a single lane
        // in a divergent branch each instruction cost that lane 55 - 80 cycles of operand marshalling, whatever
        // the instruction's size, and the tensor pipe starved behind it.)  A failed wait does not leave the loop:
        // it switches off the remaining waits and instructions, and the loop runs out.
        {
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = make_idesc(2 * kBlockM, kBlockN, false);
            constexpr uint32_t idesc_pv = make_idesc(2 * kBlockM, D, true);
            bool ok = mbar_wait(q_full, 0, abort_flag, status, 54);
            tc_fence_after();
            const uint32_t q_lo0 = desc_lo(smem_u32(smem + P::kQ), 0);
            const uint32_t k_lo0 = desc_lo(smem_u32(smem + P::kK), 0);
            const uint32_t v_lo0 = desc_lo(smem_u32(smem + P::kV), kBlockN * 128);
            const uint32_t k_empty1 = mapa(smem_u32(k_empty), 1), v_empty1 = mapa(smem_u32(v_empty), 1);
            int pending[2] = {-1, -1};
            int n_done[2] = {0, 0};
            auto wait = [&](uint64_t *bar, int parity, int where) {
                if (ok) ok = mbar_wait(bar, (uint32_t)parity, abort_flag, status, where);
            };
            auto issue_pv = [&](int x, int ip) {
                const int vs = ip % P::kVStages;
                wait(v_full + vs, (ip / P::kVStages) & 1, 56);
                wait(p_half + 2 * x, n_done[x] & 1, 55);
                tc_fence_after();
                const uint32_t v_lo = v_lo0 + vs * (P::kVHalf >> 4);
                const uint32_t d_o = tmem_base + col_o(x), a_p = tmem_base + col_s(x);
                const uint32_t acc0 = n_done[x] > 0 ? 1u : 0u;
                if (leader && ok) {
                    mma_ts_lo_pair<idesc_pv>(d_o, a_p, v_lo, acc0);
#pragma unroll
                    for (int k = 1; k < kBlockN / 32; ++k)
                        mma_ts_lo_pair<idesc_pv>(d_o, a_p + k * 8, v_lo + k * (16 * 128 >> 4), 1u);
                }
                wait(p_half + 2 * x + 1, n_done[x] & 1, 55);
                tc_fence_after();
                if (leader && ok) {
#pragma unroll
                    for (int k = kBlockN / 32; k < kBlockN / 16; ++k)
                        mma_ts_lo_pair<idesc_pv>(d_o, a_p + k * 8, v_lo + k * (16 * 128 >> 4), 1u);
                }
                ++n_done[x];
            };
            for (int i = 0; i < st.n_tiles; ++i) {
                const int ks = i % P::kKStages;
                wait(k_full + ks, (i / P::kKStages) & 1, 57);
                tc_fence_after();
                const uint32_t k_lo = k_lo0 + ks * (P::kKHalf >> 4);
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const bool present = (x == 0) || st.has_b;
                    if (present && st.used_by(x, i)) {
                        if (pending[x] >= 0) {
                            const int ip = pending[x];
                            issue_pv(x, ip);
                            // a V stage is released by two arrivals per CTA: pay the other tile's share if it skipped ip
                            if (leader && ok && !(((1 - x) == 0 || st.has_b) && st.used_by(1 - x, ip))) {
                                mbar_arrive(v_empty + ip % P::kVStages);
                                mbar_arrive_cluster(v_empty1 + (ip % P::kVStages) * 8);
                            }
                        }
                        const uint32_t q_lo = q_lo0 + x * (P::kQTile >> 4), d_s = tmem_base + col_s(x);
                        if (leader && ok) {
                            mma_ss_lo_pair<idesc_qk, 0>(d_s, q_lo, k_lo);
#pragma unroll
                            for (int k = 1; k < D / 16; ++k) {
                                // k-step of 16 elements: 32 bytes within a 64-element swizzle atom; atoms are 128
                                // rows apart in a Q tile, 64 rows apart in a CTA's half of a K tile
                                const uint32_t off_q = ((k / 4) * (kBlockM * 128) + (k % 4) * 32) >> 4;
                                const uint32_t off_k = ((k / 4) * ((kBlockN / 2) * 128) + (k % 4) * 32) >> 4;
                                mma_ss_lo_pair<idesc_qk, 1>(d_s, q_lo + off_q, k_lo + off_k);
                            }
                            tc_commit_pair(s_full + x, 3);
                        }
                        pending[x] = i;
                    } else if (leader && ok) {
                        mbar_arrive(k_empty + ks);  // the share of a tile that skips this stream tile, in both CTAs
                        mbar_arrive_cluster(k_empty1 + ks * 8);
                    }
                }
            }
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (pending[x] >= 0) {
                    issue_pv(x, pending[x]);
                    if (leader && ok) tc_commit_pair(o_final + x, 3);
                }
            }
            if (!__all_sync(0xffffffffu, ok) && leader) {  // no MMA may still be running when tensor memory is freed
                tell_peer();
                tc_commit_pair_local(drain);
                mbar_wait_drain(drain, 0);
            }
        }
    }
    } else {
        reg_inc<216>();
        // ------------------------------------------------------------ softmax + epilogue (both CTAs)
        const int x = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
        softmax_role<D, P::kKStages, P::kVStages, true, STILL_POLY_OF4>(st, x, R0 + x * 2 * kBlockM + (int)rank * kBlockM, tmem_base, s_full,
                                                        k_empty, v_empty, p_half, mapa(smem_u32(p_half), 0), o_final,
                                                        abort_flag, status, smem + P::kQ + x * P::kQTile, y_part, d_part, n_parts,
                                                        (long long)gridDim.y * N * D, (long long)gridDim.y * N, Y, bh, N, C, lam,
                                                        budget, scale_log2);
        if (*abort_flag) tell_peer();
    }
    // Nobody touches the peer's shared memory or tensor memory after this point.
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------
// Self-Saliency Score (Sec. 3.1; Algorithm 1 "Compute Self-Saliency Score") and
// per-chunk top-k (Sec. 3.3, delayed selection) on tensor cores.
// One CTA scores 128 consecutive query rows of one (batch, head): one UMMA of
// shape 128 x 256 x d gives the logits of those rows against the 256 keys at
// positions [R0-128, R0+128) -- s_prev and s_in of Algorithm 1 side by side.  A
// thread owns one row; its window is the last C keys up to itself, i.e. the
// elements j in [lane+1, lane+C] of the C+32 columns its warp reads from TMEM
// (element lane+C is the token itself).  With e_j = exp(l_j - max), Z = sum e_j,
// Z' = sum_{j != t} e_j:  a_diag_j = e_j / Z,  a_nodiag_j = e_j / Z' (0 at j = t),
// Score = sum_j a_diag_j log((a_diag_j + eps) / (a_nodiag_j + eps)).
// The kernel is persistent: a CTA (one per SM) walks over tiles n = blockIdx.x, blockIdx.x + gridDim.x, ...
// (tile n = head n / n_row_blocks, rows 128 (n % n_row_blocks) ...) with two stages of shared memory and two
// TMEM accumulators, so that the loads of tile n+1 and its UMMA run under the row epilogue of tile n.
// Warps: 0 TMA producer, 1 MMA issuer, 2-5 score group 0 (even tiles of the CTA), 6-9 score group 1 (odd
// tiles); TMEM lane quarter = warp % 4.
// ---------------------------------------------------------------------------
template <int D>
struct ScoreSmem {
    static constexpr int kQBytes = kBlockM * D * 2, kKBytes = 2 * kBlockN * D * 2;
    static constexpr int kStage = kQBytes + kKBytes;
    static constexpr int kBar = 2 * kStage;          // full[2], mma_done[2], smem_free[2], tmem_free[2]
    static constexpr int kMisc = kBar + 8 * 8;       // tmem base, abort flag
    static constexpr int kSc = kMisc + 16;           // [2][128] scores of the group's tile (16-byte aligned)
    static constexpr int kBallot = kSc + 2 * kBlockM * 4;   // [2][4]
    static constexpr int kTotal = kBallot + 2 * 4 * 4;
    static constexpr int kAlloc = kTotal + 1024;     // slack to align the base to 1024
};

static_assert(ScoreSmem<64>::kAlloc <= kMaxDynamicSmem && ScoreSmem<128>::kAlloc <= kMaxDynamicSmem,
              "score kernel: two stages must fit one CTA's shared memory");

template <int D, int C>
__global__ void __launch_bounds__(320, 1)
score_select_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       float *__restrict__ scores, int32_t *__restrict__ sel_idx, int *status, int H, int Hkv,
                       int N, int lam, float scale_log2, float eps, int n_row_blocks, int n_tiles) {
    using P = ScoreSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + P::kBar);
    uint64_t *mma_done = full + 2, *smem_free = full + 4, *tmem_free = full + 6;
    uint32_t *tmem_base_slot = reinterpret_cast<uint32_t *>(smem + P::kMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + P::kMisc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int Tn = (N + C - 1) / C;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(full + s, 1);
            mbar_init(mma_done + s, 1);
            mbar_init(smem_free + s, 1);
            mbar_init(tmem_free + s, 4);   // one arrival per warp of the score group
        }
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
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int n = blockIdx.x; n < n_tiles; n += gridDim.x, ++it) {
                const int s = it & 1, ph = (it >> 1) & 1;
                if (!mbar_wait(smem_free + s, ph ^ 1, abort_flag, status, 22)) break;
                const int bh = n / n_row_blocks, R0 = (n - bh * n_row_blocks) * kBlockM;
                const int b = bh / H, h = bh - b * H, kvh = h / (H / Hkv);
                uint8_t *q_s = smem + s * P::kStage, *k_s = q_s + P::kQBytes;
                mbar_expect_tx(full + s, P::kQBytes + P::kKBytes);
                // rows before the start of K or of the previous head are masked by position in the epilogue
                const int k_row = (b * Hkv + kvh) * N + R0 - kBlockN;
                for (int half = 0; half < D / 64; ++half) {
                    tma_load_2d(q_s + half * (kBlockM * 128), &tm_q, full + s, half * 64, bh * N + R0);
                    // K-major operand of 256 rows: per 64-column half, rows 0..255 contiguous
                    tma_load_2d(k_s + half * (2 * kBlockN * 128), &tm_k, full + s, half * 64, k_row);
                    tma_load_2d(k_s + half * (2 * kBlockN * 128) + kBlockN * 128, &tm_k, full + s, half * 64, k_row + kBlockN);
                }
            }
            // leave no copy in flight behind: every armed stage is waited for by the MMA warp in the normal
            // course; after a failure wait (bounded) for the last one armed
            if (*abort_flag && it > 0) mbar_wait_drain(full + ((it - 1) & 1), ((it - 1) >> 1) & 1);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(kBlockM, 2 * kBlockN, false);
            int it = 0;
            bool ok = true;
            for (int n = blockIdx.x; n < n_tiles; n += gridDim.x, ++it) {
                const int s = it & 1, ph = (it >> 1) & 1;
                ok = mbar_wait(full + s, ph, abort_flag, status, 20) &&
                     mbar_wait(tmem_free + s, ph ^ 1, abort_flag, status, 23);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_a = smem_u32(smem + s * P::kStage), k_a = q_a + P::kQBytes;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t qa = q_a + (k / 4) * (kBlockM * 128) + (k % 4) * 32;
                    const uint32_t ka = k_a + (k / 4) * (2 * kBlockN * 128) + (k % 4) * 32;
                    mma_ss(tmem_base + s * 256, smem_desc(qa, 0), smem_desc(ka, 0), idesc, k > 0 ? 1u : 0u);
                }
                tc_commit(mma_done + s);
            }
            // no MMA may still be running when tensor memory is freed: after a failure wait (bounded) for the
            // last group issued (its commit covers everything before it)
            if (!ok && it > 0) mbar_wait_drain(mma_done + ((it - 1) & 1), ((it - 1) >> 1) & 1);
        }
    } else {
        const int g = (warp - 2) >> 2;                 // score group = stage = TMEM accumulator
        const int wq = warp & 3;                       // TMEM lane quarter this warp may read
        const int r = wq * 32 + lane;                  // row of the tile owned by this thread
        float *sc = reinterpret_cast<float *>(smem + P::kSc) + g * kBlockM;
        uint32_t *ballots = reinterpret_cast<uint32_t *>(smem + P::kBallot) + g * 4;
        const uint32_t taddr = tmem_base + g * 256 + ((uint32_t)(wq * 32) << 16) + (uint32_t)(wq * 32 + kBlockN - C);
        const int group_bar = 1 + g;
        int it = g, j = 0;
        for (int n = blockIdx.x + g * gridDim.x; n < n_tiles; n += 2 * gridDim.x, it += 2, ++j) {
            const int ph = j & 1;
            const int bh = n / n_row_blocks, R0 = (n - bh * n_row_blocks) * kBlockM;
            const int t = R0 + r;
            bool ok = mbar_wait(mma_done + g, ph, abort_flag, status, 21);
            // the group leaves the loop together
            {
                uint32_t all_ok;
                asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 p, %1, 0;\nbarrier.cta.red.and.pred q, %2, 128, p;\nselp.b32 %0, 1, 0, q;\n}"
                             : "=r"(all_ok) : "r"((uint32_t)ok), "r"(group_bar) : "memory");
                ok = all_ok != 0;
            }
            if (!ok) break;
            tc_fence_after();
            if (r == 0) mbar_arrive(smem_free + g);    // the logits are complete: the stage's operands are free
            float score = 0.f;
            {
                // Element j of the warp's C+32 columns is the key at position R0 + 32 wq - C + j, and the window of
                // the row in lane l is j in [l+1, l+C].  Columns [32, C) lie in every lane's window; of columns jj
                // and C + jj (jj < 32) exactly one does (the first if jj > l).  So the first and the last block of
                // 32 columns fold into one, and a row becomes C values without gaps: block 0 is the folded one (the
                // token itself sits at jj = l), blocks 1 .. C/32-1 are columns [32 q, 32 q + 32).  Keys at negative
                // positions (first tile of a sequence only) are set to -inf, which the exponential turns into 0.
                constexpr int kBlocks = C / 32;
                const bool first_tile = R0 == 0;
                auto load_block = [&](int q, uint32_t (&v)[32]) {
                    tmem_ld32(taddr + q * 32, v);
                    if (q == 0) {
                        uint32_t w[32];
                        tmem_ld32(taddr + C, w);
                        tmem_wait_ld();
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) v[jj] = (jj > lane) ? v[jj] : w[jj];
                    } else {
                        tmem_wait_ld();
                    }
                    if (first_tile) {
                        const int n_neg = C - wq * 32;   // columns below n_neg are before the start of the sequence
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj)
                            if (q * 32 + jj < n_neg && (q > 0 || jj > lane)) v[jj] = 0xff800000u;
                    }
                };
                auto tmem_read_done = [&]() {   // the accumulator may be overwritten by the UMMA of the tile after next
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tmem_free + g);
                };
                if constexpr (kBlocks == 2) {
                    // the row fits the register file: one read of tensor memory, exponentials kept in place
                    uint32_t v0[32], v1[32];
                    load_block(0, v0);
                    load_block(1, v1);
                    tmem_read_done();
                    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2) {
                        mx0 = max3(mx0, __uint_as_float(v0[jj]), __uint_as_float(v0[jj + 1]));
                        mx1 = max3(mx1, __uint_as_float(v1[jj]), __uint_as_float(v1[jj + 1]));
                    }
                    const float neg_m = -fmaxf(mx0, mx1) * scale_log2;
                    float z0 = 0.f, z1 = 0.f, e_self = 0.f;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const float e0 = ex2(fmaf(__uint_as_float(v0[jj]), scale_log2, neg_m));
                        const float e1 = ex2(fmaf(__uint_as_float(v1[jj]), scale_log2, neg_m));
                        v1[jj] = __float_as_uint(e1);
                        z1 += e1;
                        if (jj == lane) e_self = e0;
                        else z0 += e0;                    // the sum without the token itself is formed directly
                        v0[jj] = __float_as_uint(e0);
                    }
                    const float z_nd = z0 + z1, z_all = z_nd + e_self;
                    const float inv_all = 1.f / z_all, inv_nd = z_nd > 0.f ? 1.f / z_nd : 0.f;
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        // a * ln((a + eps) / (b + eps)); a masked key has a = b = 0 and adds nothing
                        const float e0 = __uint_as_float(v0[jj]), e1 = __uint_as_float(v1[jj]);
                        const float a0 = e0 * inv_all, a1 = e1 * inv_all;
                        const float b0 = (jj == lane) ? 0.f : e0 * inv_nd, b1 = e1 * inv_nd;
                        s0 += a0 * (__log2f(a0 + eps) - __log2f(b0 + eps));
                        s1 += a1 * (__log2f(a1 + eps) - __log2f(b1 + eps));
                    }
                    score = s0 + s1;
                } else {
                    float mx = -INFINITY;
#pragma unroll 1
                    for (int q = 0; q < kBlocks; ++q) {
                        uint32_t v[32];
                        load_block(q, v);
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) mx = max3(mx, __uint_as_float(v[jj]), __uint_as_float(v[jj + 1]));
                    }
                    const float neg_m = -mx * scale_log2;
                    float z_nd = 0.f, e_self = 0.f;
#pragma unroll 1
                    for (int q = 0; q < kBlocks; ++q) {
                        uint32_t v[32];
                        load_block(q, v);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            const float e = ex2(fmaf(__uint_as_float(v[jj]), scale_log2, neg_m));
                            if (q == 0 && jj == lane) e_self = e;
                            else z_nd += e;
                        }
                    }
                    const float z_all = z_nd + e_self;
                    const float inv_all = 1.f / z_all, inv_nd = z_nd > 0.f ? 1.f / z_nd : 0.f;
#pragma unroll 1
                    for (int q = 0; q < kBlocks; ++q) {
                        uint32_t v[32];
                        load_block(q, v);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            const float e = ex2(fmaf(__uint_as_float(v[jj]), scale_log2, neg_m));
                            const float a = e * inv_all;
                            const float bb = (q == 0 && jj == lane) ? 0.f : e * inv_nd;
                            score += a * (__log2f(a + eps) - __log2f(bb + eps));
                        }
                    }
                    tmem_read_done();
                }
                score *= 0.6931471805599453f;
            }
            sc[r] = score;
            if (t < N && scores != nullptr) scores[(long long)bh * N + t] = score;
            asm volatile("bar.sync %0, 128;" ::"r"(group_bar) : "memory");
            if (lam > 0) {
                // top-k of each chunk of the tile: rank under (score descending, position ascending), NaN as -inf
                const int cc = r / C, rr = r - cc * C;
                const int n_c = min(C, N - (R0 + cc * C));   // tokens of this row's chunk (<= 0: past the end)
                bool selected = false;
                if (rr < n_c) {
                    float mine = sc[r];
                    if (isnan(mine)) mine = -INFINITY;
                    int rank = 0;
                    for (int jx = 0; jx < n_c; ++jx) {
                        float o = sc[cc * C + jx];
                        if (isnan(o)) o = -INFINITY;
                        rank += (o > mine) || (o == mine && jx < rr);
                    }
                    selected = rank < lam;
                }
                // place of a selected row in the ascending output = selected rows before it in its chunk
                const uint32_t votes = __ballot_sync(0xffffffffu, selected);
                if (lane == 0) ballots[wq] = votes;
                asm volatile("bar.sync %0, 128;" ::"r"(group_bar) : "memory");
                if (n_c > 0) {
                    int32_t *out = sel_idx + ((long long)bh * Tn + (R0 / C + cc)) * lam;
                    int before = __popc(votes & ((1u << lane) - 1u));
                    for (int w = cc * (C / 32); w < wq; ++w) before += __popc(ballots[w]);
                    if (selected) out[before] = R0 + cc * C + rr;
                    const int n_sel = n_c < lam ? n_c : lam;
                    if (rr >= n_sel && rr < lam) out[rr] = -1;
                }
            }
            // sc / ballots are written again in the group's next tile
            asm volatile("bar.sync %0, 128;" ::"r"(group_bar) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// K_sel / V_sel [B*H, sel_rows, d]: row j < n_valid is row sel_idx[j] of the head's K / V
// (a -1 entry, or a row of the padding, is zero).  One warp per row.
template <int D>
__global__ void __launch_bounds__(256)
compact_kernel(const __nv_bfloat16 *__restrict__ K, const __nv_bfloat16 *__restrict__ V,
               const int32_t *__restrict__ sel_idx, __nv_bfloat16 *__restrict__ Ksel,
               __nv_bfloat16 *__restrict__ Vsel, int H, int Hkv, long long N, long long n_idx, long long sel_rows) {
    const int bh = blockIdx.y, b = bh / H, h = bh % H, kvh = h / (H / Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long j = (long long)blockIdx.x * 8 + warp;
    if (j >= sel_rows) return;
    long long p = -1;
    if (j < n_idx) p = sel_idx[(long long)bh * n_idx + j];
    constexpr int kVec = D / 8;  // uint4 per row
    uint4 kk = make_uint4(0, 0, 0, 0), vv = kk;
    if (lane < kVec && p >= 0) {
        kk = reinterpret_cast<const uint4 *>(K + (((long long)b * Hkv + kvh) * N + p) * D)[lane];
        vv = reinterpret_cast<const uint4 *>(V + (((long long)b * Hkv + kvh) * N + p) * D)[lane];
    }
    if (lane < kVec) {
        reinterpret_cast<uint4 *>(Ksel + ((long long)bh * sel_rows + j) * D)[lane] = kk;
        reinterpret_cast<uint4 *>(Vsel + ((long long)bh * sel_rows + j) * D)[lane] = vv;
    }
}

// The bounded wait of the kernels above, alone: one warp, one mbarrier that expects an arrival which never
// comes.  No TMA, no tensor memory, no MMA: when the limit has passed the kernel records the timeout and ends.
__global__ void wait_timeout_selftest_kernel(int *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) (void)mbar_wait_limit(&bar, 0, abort_flag, status, 99, limit_cycles);
    __syncthreads();
}

// ----------------------------------------------------------------- host side

// 2-D bf16 tensor [rows, d] tiled in boxes of [128 rows, 64 columns] with 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *base, unsigned long long rows, int d) {
    return make_map_2d(m, base, rows, (unsigned long long)d, 128, false);
}

template <int D>
int launch_tc(const still_params_t *p, long long N, const void *Q, const void *K, const void *V,
              const int32_t *sel_idx, const void *y_part, const float *d_part, int n_parts, void *Y, void *k_sel, void *v_sel,
              long long sel_rows, int *status, cudaStream_t st, int *launches) {
    using bf = __nv_bfloat16;
    const long long T = (N + p->chunk - 1) / p->chunk, BH = (long long)p->B * p->H;
    const long long n_idx = T * p->topk;
    const bool identity = p->topk == p->chunk;  // the selection of every chunk is the chunk itself
    if (!identity) {
        dim3 grid((unsigned)((sel_rows + 7) / 8), (unsigned)BH);
        compact_kernel<D><<<grid, 256, 0, st>>>((const bf *)K, (const bf *)V, sel_idx, (bf *)k_sel, (bf *)v_sel, p->H,
                                               p->Hkv, N, n_idx, sel_rows);
        ++*launches;
        if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
    }
    const unsigned long long kv_rows = (unsigned long long)p->B * p->Hkv * N;
    const unsigned long long sel_total = identity ? kv_rows : (unsigned long long)BH * sel_rows;
    constexpr bool kPair = D == 128;   // head dim 128 runs on CTA pairs, each CTA holding 64 keys of a K tile
    CUtensorMap tq, tk, tv, tks, tvs;
    if (!make_map(&tq, Q, (unsigned long long)BH * N, D) ||
        !make_map_2d(&tk, K, kv_rows, D, kPair ? kBlockN / 2 : kBlockN, false) || !make_map(&tv, V, kv_rows, D) ||
        !make_map_2d(&tks, identity ? K : k_sel, sel_total, D, kPair ? kBlockN / 2 : kBlockN, false) ||
        !make_map(&tvs, identity ? V : v_sel, sel_total, D))
        return STILL_ERR_CUDA;
    const float scale_log2 = p->sm_scale * 1.4426950408889634f;
    if constexpr (kPair) {
        const int n_pairs = (int)((N + 4 * kBlockM - 1) / (4 * kBlockM));
        if (ensure_dynamic_smem((const void *)sa_merge_pair_kernel<D>, PairPlan<D>::kAlloc) != cudaSuccess) return STILL_ERR_CUDA;
        dim3 grid((unsigned)(2 * n_pairs), (unsigned)BH);   // clusters of two along x
        profile_mark_begin(st);
        sa_merge_pair_kernel<D><<<grid, kThreads, PairPlan<D>::kAlloc, st>>>(
            tq, tk, tv, tks, tvs, (const bf *)y_part, d_part, n_parts, (bf *)Y, status, p->H, p->Hkv, (int)N, p->chunk, p->topk, (int)p->max_salient, (int)sel_rows,
            identity ? 1 : 0, scale_log2, n_pairs);
        profile_mark_end(st);
    } else {
        const int n_qblocks = (int)((N + 2 * kBlockM - 1) / (2 * kBlockM));
        if (ensure_dynamic_smem((const void *)sa_merge_tc_kernel<D>, SmemPlan<D>::kAlloc) != cudaSuccess) return STILL_ERR_CUDA;
        dim3 grid((unsigned)n_qblocks, (unsigned)BH);
        profile_mark_begin(st);
        sa_merge_tc_kernel<D><<<grid, kThreads, SmemPlan<D>::kAlloc, st>>>(
            tq, tk, tv, tks, tvs, (const bf *)y_part, d_part, n_parts, (bf *)Y, status, p->H, p->Hkv, (int)N, p->chunk, p->topk, (int)p->max_salient, (int)sel_rows,
            identity ? 1 : 0, scale_log2, n_qblocks);
        profile_mark_end(st);
    }
    ++*launches;
    if (cudaGetLastError() != cudaSuccess) return STILL_ERR_CUDA;
    return STILL_OK;
}

template <int D, int C>
int launch_score_tc(const still_params_t *p, long long N, const void *Q, const void *K, float *scores,
                    int32_t *sel_idx, int *status, cudaStream_t st, int *launches) {
    CUtensorMap tq, tk;
    const long long BH = (long long)p->B * p->H;
    if (!make_map(&tq, Q, (unsigned long long)BH * N, D) ||
        !make_map(&tk, K, (unsigned long long)p->B * p->Hkv * N, D))
        return STILL_ERR_CUDA;
    constexpr int kSmem = ScoreSmem<D>::kAlloc;
    if (ensure_dynamic_smem((const void *)score_select_tc_kernel<D, C>, kSmem) !=
        cudaSuccess)
        return STILL_ERR_CUDA;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm <= 0)
        return STILL_ERR_CUDA;
    const long long n_row_blocks = (N + kBlockM - 1) / kBlockM, n_tiles = n_row_blocks * BH;
    if (n_tiles >= (1ll << 31)) return STILL_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)std::min<long long>(n_tiles, n_sm);   // one persistent CTA per SM
    score_select_tc_kernel<D, C><<<grid, 320, kSmem, st>>>(tq, tk, scores, sel_idx, status, p->H, p->Hkv, (int)N,
                                                           p->topk, p->sm_scale * 1.4426950408889634f, p->eps,
                                                           (int)n_row_blocks, (int)n_tiles);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

}  // namespace

int tc_score_select(const still_params_t *p, long long N, const void *Q, const void *K, float *scores,
                    int32_t *sel_idx, int *status_words, cudaStream_t st, int *launches) {
    if ((long long)p->B * p->H * N >= (1ll << 31)) return STILL_ERR_UNSUPPORTED;
    if (p->d == 64 && p->chunk == 64) return launch_score_tc<64, 64>(p, N, Q, K, scores, sel_idx, status_words, st, launches);
    if (p->d == 64 && p->chunk == 128) return launch_score_tc<64, 128>(p, N, Q, K, scores, sel_idx, status_words, st, launches);
    if (p->d == 128 && p->chunk == 64) return launch_score_tc<128, 64>(p, N, Q, K, scores, sel_idx, status_words, st, launches);
    return launch_score_tc<128, 128>(p, N, Q, K, scores, sel_idx, status_words, st, launches);
}

// N_LA / D_LA of the fp32-accumulating FMA kernels as one bf16 part: y = N_LA / D_LA, d = D_LA.
__global__ void la_to_part_kernel(const float *__restrict__ N_LA, const float *__restrict__ D_LA, __nv_bfloat16 *__restrict__ y,
                                  float *__restrict__ dp, long long rows, int d) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * d) return;
    const long long r = i / d;
    const float dd = D_LA[r];
    y[i] = __float2bfloat16_rn(dd > 0.f ? N_LA[i] / dd : 0.f);
    if (i == r * d) dp[r] = dd;
}

int tc_la_to_part(const float *N_LA, const float *D_LA, void *y_part, float *d_part, long long rows, int d, cudaStream_t st,
                  int *launches) {
    const long long n = rows * d;
    la_to_part_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(N_LA, D_LA, (__nv_bfloat16 *)y_part, d_part, rows, d);
    ++*launches;
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

int tc_selftest_wait_timeout(int *status_words, long long limit_cycles, cudaStream_t st) {
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(status_words, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? STILL_OK : STILL_ERR_CUDA;
}

bool tc_supported(const still_params_t *p) {
    return p->dtype == STILL_DTYPE_BF16 && (p->d == 64 || p->d == 128) && (p->chunk == 64 || p->chunk == 128);
}

long long tc_sel_rows(const still_params_t *p, long long N) {
    const long long T = (N + p->chunk - 1) / p->chunk;
    return (T * p->topk + kBlockN - 1) / kBlockN * kBlockN + kBlockN;
}

int tc_sa_merge(const still_params_t *p, long long N, const void *Q, const void *K, const void *V,
                const int32_t *sel_idx, const void *y_part, const float *d_part, int n_parts, void *Y, void *k_sel, void *v_sel,
                long long sel_rows, int *status_words, cudaStream_t st, int *launches) {
    if ((long long)p->B * p->H * std::max(N, sel_rows) >= (1ll << 31)) return STILL_ERR_UNSUPPORTED;  // TMA row coordinate
    if (p->d == 64)
        return launch_tc<64>(p, N, Q, K, V, sel_idx, y_part, d_part, n_parts, Y, k_sel, v_sel, sel_rows, status_words, st, launches);
    return launch_tc<128>(p, N, Q, K, V, sel_idx, y_part, d_part, n_parts, Y, k_sel, v_sel, sel_rows, status_words, st, launches);
}

}  // namespace still
