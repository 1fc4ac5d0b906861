// Split-KV pass of the decode step for bf16 (Sec. 3.3: N_SA, D_SA over the salient cache h_t).
//
// HBM-bound: every step reads the K and V history once.  One CTA serves one (batch, KV head) and a
// range of 32-position key blocks; the query heads of the group (at most 16) are the rows of one
// m16n8k16 tensor-core tile, so the K / V rows are read once for the whole group.  Which rows a
// query head sees is a per-head membership mask: for a position in a routed chunk, whether the
// head's selection (the sel_mask words of the decode state) contains it; for the two-chunk local region, every position up to the
// new token.  Key blocks are streamed by 16-byte cp.async into padded shared-memory rows, two stages per
// warp; a row is read from memory only if some head of the group selected it (the union of the group's
// salient caches, read once for the group rather than once per head) and gets weight zero for the heads
// that did not; with topk = chunk that is every row.
// Each warp runs its own online softmax over its blocks; the four warps are merged through shared
// memory and the CTA writes one partial (max, sum, numerator) per head and split.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace still {

__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src, bool valid) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    const int bytes = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *p) {
    const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p));
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void *p) {
    const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p));
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int D>
struct AttendPlan {
    static constexpr int kRow = D * 2 + 16;          // padded row: ldmatrix without bank conflicts
    static constexpr int kTile = 32 * kRow;          // 32 keys
    static constexpr int kStage = 2 * kTile;         // K and V
    static constexpr int kWarp = 2 * kStage;         // two stages
    static constexpr int kTotal = 4 * kWarp;
};

// grid (n_splits, Hkv, B), 128 threads.  first_pos: a multiple of the chunk size.  part: [B*H][max_splits][D + 2] = running max (natural
// log units), sum, numerator.
template <int D>
__global__ void __launch_bounds__(128)
step_attend_mma_kernel(const __nv_bfloat16 *__restrict__ kc, const __nv_bfloat16 *__restrict__ vc,
                       const uint32_t *__restrict__ sel_mask, const __nv_bfloat16 *__restrict__ q,
                       float *__restrict__ part, const int32_t *__restrict__ hdr, int H, int Hkv, long long cap, long long kvr, int C,
                       int lam, long long t, long long first_pos, int n_splits, int max_splits, float scale_log2) {
    using P = AttendPlan<D>;
    extern __shared__ __align__(16) uint8_t attend_smem[];
    if (hdr[14] != 0) return;   // the step's first kernel found the state not to match the call
    uint8_t *smem = attend_smem;
    const int split = blockIdx.x, kv = blockIdx.y, b = blockIdx.z, rep = H / Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;          // fragment row (and row + 8), column pair
    // K / V rows live in a ring of kvr rows per KV head (position p in row p % kvr; kvr is a multiple of the chunk
    // size, so a 32-position block never straddles the end)
    const __nv_bfloat16 *kh = kc + ((long long)b * Hkv + kv) * kvr * D;
    const __nv_bfloat16 *vh = vc + ((long long)b * Hkv + kv) * kvr * D;
    uint8_t *my = smem + warp * P::kWarp;

    const long long c_cur = t / C;
    const long long loc0 = c_cur >= 1 ? (c_cur - 1) * C : 0;   // first position of the local region
    const int n_chunk_cap = (int)(cap / C);
    // key blocks covering positions first_pos..t (first_pos > 0 with a salient-cache budget: older chunks have
    // left the cache for the linear state)
    const int kb0 = (int)(first_pos / 32), nb = (int)((t + 32) / 32);
    const int per = (nb - kb0 + n_splits - 1) / n_splits;
    const int kb_lo = kb0 + split * per, kb_hi = min(nb, kb_lo + per);

    // Q fragments of the group's heads (rows >= rep are zero)
    uint32_t qa[D / 16][4];
    {
        const long long hq = (long long)b * H + (long long)kv * rep;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int col = ks * 16 + tig * 2;
            qa[ks][0] = g < rep ? *reinterpret_cast<const uint32_t *>(q + (hq + g) * D + col) : 0u;
            qa[ks][1] = g + 8 < rep ? *reinterpret_cast<const uint32_t *>(q + (hq + g + 8) * D + col) : 0u;
            qa[ks][2] = g < rep ? *reinterpret_cast<const uint32_t *>(q + (hq + g) * D + col + 8) : 0u;
            qa[ks][3] = g + 8 < rep ? *reinterpret_cast<const uint32_t *>(q + (hq + g + 8) * D + col + 8) : 0u;
        }
    }
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // rows g and g + 8, log2 domain

    // Rows of a block that no query head of the group sees are not read from memory (a zero-filling copy with
    // no source bytes): with topk < chunk only the union of the group's selections crosses HBM.
    auto load_block = [&](int kb, int stage, uint32_t rows_needed) {
        uint8_t *ks = my + stage * P::kStage, *vs = ks + P::kTile;
        constexpr int kChunksPerRow = D / 8;
        const long long p0 = (long long)kb * 32;
        const long long r0 = p0 % kvr;   // ring row of the block's first position (one division per block)
#pragma unroll
        for (int i = lane; i < 32 * kChunksPerRow; i += 32) {
            const int row = i / kChunksPerRow, ch = i % kChunksPerRow;
            const bool valid = (rows_needed >> row) & 1u;
            const long long src = (valid ? r0 + row : 0) * D + ch * 8;
            cp_async16(ks + row * P::kRow + ch * 16, kh + src, valid);
            cp_async16(vs + row * P::kRow + ch * 16, vh + src, valid);
        }
    };
    // Membership word of block kb for the head in this lane (lanes >= group size: 0): bit j = position 32 kb + j is
    // visible to the head.  Local region: every position up to the new token; routed chunks: the head's selection
    // (bit masks written when the chunk was routed), all of it when topk = chunk.
    auto member_word = [&](int kb) -> uint32_t {
        if (kb >= kb_hi || lane >= rep) return 0u;
        const long long p0 = (long long)kb * 32;
        if (p0 >= loc0) {
            const long long last = t - p0;   // positions up to the new token
            return last >= 31 ? 0xffffffffu : ((1u << (int)(last + 1)) - 1u);
        }
        if (lam >= C) return 0xffffffffu;
        if (lam <= 0) return 0u;
        const int chunk = (int)(p0 / C), word = (int)((p0 % C) / 32);
        return sel_mask[(((long long)b * H + (long long)kv * rep + lane) * n_chunk_cap + chunk) * (C / 32) + word];
    };

    // The membership words run two blocks ahead of the compute and one ahead of the copies they steer.
    const int first = kb_lo + warp;
    uint32_t m_cur = member_word(first), m_next = member_word(first + 4);
    if (first < kb_hi) load_block(first, 0, __reduce_or_sync(0xffffffffu, m_cur));
    cp_async_commit();
    int it = 0;
    for (int kb = first; kb < kb_hi; kb += 4, ++it) {
        const int stage = it & 1;
        const uint32_t m_after = member_word(kb + 8);
        if (kb + 4 < kb_hi) load_block(kb + 4, stage ^ 1, __reduce_or_sync(0xffffffffu, m_next));
        cp_async_commit();

        // membership of the block's 32 positions for rows g and g + 8 (bit j: position 32 kb + j)
        uint32_t vis[2];
        vis[0] = __shfl_sync(0xffffffffu, m_cur, g);
        vis[1] = __shfl_sync(0xffffffffu, m_cur, g + 8);
        m_cur = m_next;
        m_next = m_after;
        cp_async_wait<1>();
        __syncwarp();
        const uint8_t *ks = my + stage * P::kStage, *vs = ks + P::kTile;

        // S = Q K^T for 32 keys: 4 n-tiles of 8 keys
        float s[4][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int ks16 = 0; ks16 < D / 16; ++ks16) {
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                // matrices: (keys 16 np .. +8, d lo), (same keys, d hi), (keys 16 np + 8 .., d lo), (.., d hi)
                uint32_t bfr[4];
                const int key = np * 16 + ((lane >> 4) << 3) + (lane & 7);
                const int dcol = ks16 * 16 + (((lane >> 3) & 1) << 3);
                ldmatrix_x4(bfr, ks + key * P::kRow + dcol * 2);
                mma_16816(s[np * 2], qa[ks16], bfr[0], bfr[1]);
                mma_16816(s[np * 2 + 1], qa[ks16], bfr[2], bfr[3]);
            }
        }
        // mask, scale, online softmax (rows g and g + 8; a thread holds columns 8 nt + 2 tig + {0, 1})
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int col = nt * 8 + tig * 2 + (e & 1), hr = e >> 1;
                const bool on = (vis[hr] >> col) & 1u;
                s[nt][e] = on ? s[nt][e] * scale_log2 : -INFINITY;
                mx[hr] = fmaxf(mx[hr], s[nt][e]);
            }
        float alpha[2];
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
            mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 1));
            mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 2));
            const float mn = fmaxf(m_run[hr], mx[hr]);
            alpha[hr] = (mn == -INFINITY) ? 1.f : ex2_approx(m_run[hr] - mn);
            m_run[hr] = mn;
        }
        float ls[2] = {0.f, 0.f};
        uint32_t pa[2][4];   // P as A fragments of the two 16-key k-steps
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            float pv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hr = e >> 1;
                pv[e] = (m_run[hr] == -INFINITY) ? 0.f : ex2_approx(s[nt][e] - m_run[hr]);
                ls[hr] += pv[e];
            }
            pa[nt >> 1][(nt & 1) * 2 + 0] = pack2_bf16(pv[0], pv[1]);   // row g
            pa[nt >> 1][(nt & 1) * 2 + 1] = pack2_bf16(pv[2], pv[3]);   // row g + 8
        }
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
            ls[hr] += __shfl_xor_sync(0xffffffffu, ls[hr], 1);
            ls[hr] += __shfl_xor_sync(0xffffffffu, ls[hr], 2);
            l_run[hr] = l_run[hr] * alpha[hr] + ls[hr];
        }
#pragma unroll
        for (int dt = 0; dt < D / 8; ++dt) {
            o[dt][0] *= alpha[0];
            o[dt][1] *= alpha[0];
            o[dt][2] *= alpha[1];
            o[dt][3] *= alpha[1];
        }
        // O += P V: k-steps of 16 keys, n-tiles of 8 value columns
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                // matrices (transposed on load): (keys 16 kk .. +8, d 16 dp ..), (keys + 8, same d),
                // (keys, d + 8), (keys + 8, d + 8)
                uint32_t bfr[4];
                const int key = kk * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                const int dcol = dp * 16 + ((lane >> 4) << 3);
                ldmatrix_x4_trans(bfr, vs + key * P::kRow + dcol * 2);
                mma_16816(o[dp * 2], pa[kk], bfr[0], bfr[1]);
                mma_16816(o[dp * 2 + 1], pa[kk], bfr[2], bfr[3]);
            }
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    __syncthreads();

    // merge the four warps: smem [4 warps][16 rows][D + 2]
    float *mg = reinterpret_cast<float *>(smem);
    constexpr int kStride = D + 2;
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
        const int row = g + hr * 8;
        float *dst = mg + (warp * 16 + row) * kStride;
        if (tig == 0) {
            dst[0] = m_run[hr];
            dst[1] = l_run[hr];
        }
#pragma unroll
        for (int dt = 0; dt < D / 8; ++dt) {
            dst[2 + dt * 8 + tig * 2] = o[dt][hr * 2];
            dst[2 + dt * 8 + tig * 2 + 1] = o[dt][hr * 2 + 1];
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < rep * kStride; idx += blockDim.x) {
        const int row = idx / kStride, col = idx % kStride;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, mg[(w * 16 + row) * kStride]);
        float acc = 0.f;
        if (col == 0) {
            acc = M * 0.6931471805599453f;   // the merge kernel works in natural-log units
        } else {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float mw = mg[(w * 16 + row) * kStride];
                if (mw != -INFINITY) acc += ex2_approx(mw - M) * mg[(w * 16 + row) * kStride + col];
            }
        }
        const long long bh = (long long)b * H + (long long)kv * rep + row;
        part[(bh * max_splits + split) * kStride + col] = acc;
    }
}

}  // namespace still
