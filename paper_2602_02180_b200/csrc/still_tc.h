// Internal interfaces between the host API (still_api.cu), the tensor-core
// prefill kernels (still_tc.cu) and the decode-step kernels (still_step.cu).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/still.h"

namespace still {

// cudaFuncAttributeMaxDynamicSharedMemorySize, set once per kernel and device instead of on every call.
inline cudaError_t ensure_dynamic_smem(const void *func, int bytes) {
    struct Done {
        const void *func;
        int dev;
    };
    constexpr int kSlots = 64;
    static thread_local Done done[kSlots] = {};
    static thread_local int n_done = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    for (int i = 0; i < n_done; ++i)
        if (done[i].func == func && done[i].dev == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && n_done < kSlots) done[n_done++] = Done{func, dev};
    return e;
}

// ---- timing of the dominant kernel (still_profile_enable / still_profile_collect) ----
void profile_mark_begin(cudaStream_t st);
void profile_mark_end(cudaStream_t st);

// ---- tensor-core (tcgen05) prefill path, bf16 only --------------------------------
// True when the softmax-attention branch of these parameters runs on the tcgen05 kernel.
bool tc_supported(const still_params_t *p);
// Rows per head of the compacted salient K/V copies (selected rows of all chunks plus tile padding).
long long tc_sel_rows(const still_params_t *p, long long N);
// Self-Saliency Score + per-chunk top-k on tensor cores (scores may be NULL).
int tc_score_select(const still_params_t *p, long long N, const void *Q, const void *K, float *scores,
                    int32_t *sel_idx, int *status_words, cudaStream_t st, int *launches);
// Compacts the selected K/V rows and runs the softmax-attention + merge kernel.
// The linear branch arrives as n_parts (0, 1 or 2) partial results: y_part [n_parts][B,H,N,d] bf16 = N_part /
// D_part and d_part [n_parts][B,H,N] fp32; N_LA = sum y_part d_part, D_LA = sum d_part.
int tc_sa_merge(const still_params_t *p, long long N, const void *Q, const void *K, const void *V,
                const int32_t *sel_idx, const void *y_part, const float *d_part, int n_parts, void *Y, void *k_sel,
                void *v_sel, long long sel_rows, int *status_words, cudaStream_t st, int *launches);
// fp32 N_LA / D_LA of the FMA kernels as one such part (y = N_LA / D_LA, d = D_LA).
int tc_la_to_part(const float *N_LA, const float *D_LA, void *y_part, float *d_part, long long rows, int d,
                  cudaStream_t st, int *launches);

// One CTA whose only act is a bounded mbarrier wait on a barrier that nothing arrives on: the wait runs
// out after limit_cycles, the kernel records STILL_ERR_DEVICE_TIMEOUT (detail 99) in status_words and
// returns.  Exercises the expiry path of the waits every tcgen05 kernel uses.
int tc_selftest_wait_timeout(int *status_words, long long limit_cycles, cudaStream_t st);

// ---- tensor-core linear-attention branch of the prefill, bf16 only --------------------
// True when NP-Map and the chunk-wise state scan of these parameters run on the tcgen05 kernels.
bool tc_la_supported(const still_params_t *p);
// NP-Map of K (bf16 features into phiK [B,Hkv,N,2 d_f], chunk column sums into csum [B,Hkv,T,2 d_f]), the
// normaliser z after every routed chunk (zpre [B,H,T-2,2 d_f]), then the state scan with the query-side NP-Map
// fused in: y_part [2][B,H,N,d] bf16 = N_part / D_part (gated), d_part [2][B,H,N] fp32, one part per feature
// half; S_out / z_out (optional) receive the state after the chunks that have left the local region.
int tc_la_branch(const still_params_t *p, long long N, const void *Q, const void *K, const void *V, const void *G,
                 const void *Wq, const void *bq, const void *Wk, const void *bk, const int32_t *sel_idx, void *phiK,
                 float *csum, float *zpre, void *y_part, float *d_part, float *seg_sums, float *S_out, float *z_out,
                 void *phiK_sel, void *v_sel, long long sel_rows, int *status_words, cudaStream_t st, int *launches);
// Segments of the two-level state scan for these parameters (1 = plain scan); *seg_chunks = chunks per segment.
// seg_sums holds (segments - 1) partial states [2 d_f, d] fp32 per (batch, head).
int tc_la_segments(const still_params_t *p, long long N, int *seg_chunks);
int tc_la_sum_parts(int seg_chunks);

// ---- decode step ----------------------------------------------------------------------
size_t step_scratch_bytes(const still_params_t *p, long long capacity);
// Rows of the K / V store per KV head in a decode state of that capacity: the capacity itself, or, with a
// salient-cache budget, a ring that holds the cached chunks, the two-chunk local region and the chunk being routed.
long long state_kv_rows(const still_params_t *p, long long capacity);
int step_launch(const still_params_t *p, char *state, const still_state_layout_t *L, long long t_pos,
                const void *q, const void *k, const void *v, const void *g, const void *Wq,
                const void *bq, const void *Wk, const void *bk, void *y, cudaStream_t st,
                int *launches);

}  // namespace still
