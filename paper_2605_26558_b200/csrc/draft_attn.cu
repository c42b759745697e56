// Log-sum-exp merge of the attention kernels' partial results, and the dispatch of the draft attention (Sec. 4.1 draft
// inference over the compressed KV cache of Sec. 4.2; the kernel itself is in draft_attn_tc.cu).
#include "kernels.cuh"

namespace cass {

// Merge the chunk partials of every (row, query head): out = sum_c e^{m_c - M} o_c / sum_c e^{m_c - M} l_c.
// Row r (the (r % rps)-th of sequence r / rps) sees positions < len + (draft: inflight + 1 | verify: r % rps + 1);
// chunks hold `chunk_tokens` positions.
// The reductions run in a fixed order that depends on the number of visible chunks only.
constexpr int kMergeThreads = 256;
constexpr int kMergeWarps = kMergeThreads / 32;

__global__ void __launch_bounds__(kMergeThreads) k_attn_merge(AttnScratch sc, int n_chunks_alloc, int chunk_tokens, int rps, int n_q, int d,
                                                              const DevState* __restrict__ st, int draft_mode, int draft_units,
                                                              uint16_t* __restrict__ out) {
    extern __shared__ __align__(16) float w_s[];    // [n_chunks_alloc] weights e^{m_c - M}, then [kMergeWarps][d] partial outputs
    __shared__ float s_red[kMergeWarps];
    pdl_early<3>();
    pdl_wait();
    const int hq = blockIdx.x, r = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int seq = r / rps;
    const int vis = st->len[seq] + (draft_mode ? st->inflight[seq] + 1 : r % rps + 1);
    if (draft_units < 0) chunk_tokens = tc_run_tokens(vis, -draft_units);     // the draft attention's runs follow the visible length
    const int n_ch = ceil_div(vis, chunk_tokens);
    const size_t pair = (size_t)r * n_q + hq;
    const float* mp = sc.m + pair * n_chunks_alloc;
    const float* lp = sc.l + pair * n_chunks_alloc;
    float* part_s = w_s + ((n_chunks_alloc + 3) & ~3);
    // What the first round of every loop below needs is requested here, before any of it is used: the statistics of
    // chunk tid and the partial outputs of this warp's first two chunks share one round trip to L2.
    const float* op = sc.o + pair * n_chunks_alloc * d;
    const bool has0 = tid < n_ch;
    const float m_first = has0 ? __ldcg(mp + tid) : -INFINITY, l_first = has0 ? __ldcg(lp + tid) : 0.f;
    const int dim0 = lane * 4;
    float4 o_first[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int c = warp + k * kMergeWarps;
        o_first[k] = (c < n_ch && dim0 < d) ? __ldcg(reinterpret_cast<const float4*>(op + (size_t)c * d + dim0)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float M = m_first;
    for (int c = tid + kMergeThreads; c < n_ch; c += kMergeThreads) M = fmaxf(M, mp[c]);
    M = warp_max(M);
    if (lane == 0) s_red[warp] = M;
    __syncthreads();
    M = s_red[0];
#pragma unroll
    for (int w = 1; w < kMergeWarps; ++w) M = fmaxf(M, s_red[w]);
    __syncthreads();
    float L = 0.f;
    if (has0) {
        const float w = expf(m_first - M);
        w_s[tid] = w;
        L += w * l_first;
    }
    for (int c = tid + kMergeThreads; c < n_ch; c += kMergeThreads) {
        const float w = expf(mp[c] - M);
        w_s[c] = w;
        L += w * lp[c];
    }
    L = warp_sum(L);
    if (lane == 0) s_red[warp] = L;
    __syncthreads();
    L = s_red[0];
#pragma unroll
    for (int w = 1; w < kMergeWarps; ++w) L += s_red[w];
    // warp w adds the chunks w, w + 8, ... (four dims per lane, 16-byte loads); the warps' sums are then added in warp
    // order: the order of every addition depends on the number of visible chunks only
    for (int dim = dim0; dim < d; dim += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int c = warp;
        if (dim == dim0) {
#pragma unroll
            for (int k = 0; k < 2; ++k, c += kMergeWarps) {
                if (c < n_ch) {
                    const float w = w_s[c];
                    const float4 o = o_first[k];
                    acc.x = fmaf(w, o.x, acc.x); acc.y = fmaf(w, o.y, acc.y); acc.z = fmaf(w, o.z, acc.z); acc.w = fmaf(w, o.w, acc.w);
                }
            }
        }
#pragma unroll 4
        for (; c < n_ch; c += kMergeWarps) {
            const float w = w_s[c];
            const float4 o = *reinterpret_cast<const float4*>(op + (size_t)c * d + dim);
            acc.x = fmaf(w, o.x, acc.x); acc.y = fmaf(w, o.y, acc.y); acc.z = fmaf(w, o.z, acc.z); acc.w = fmaf(w, o.w, acc.w);
        }
        *reinterpret_cast<float4*>(part_s + warp * d + dim) = acc;
    }
    __syncthreads();
    for (int dim = tid; dim < d; dim += kMergeThreads) {
        float acc = part_s[dim];
#pragma unroll
        for (int w = 1; w < kMergeWarps; ++w) acc += part_s[w * d + dim];
        out[((size_t)r * n_q + hq) * d + dim] = float_to_bf16_bits(acc / L);
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int rps, int n_q, int d,
                      const DevState* st, int draft_mode, int draft_units, uint16_t* out, cudaStream_t s) {
    if (d % 4) return CASS_ERR_UNSUPPORTED;
    dim3 grid(n_q, rows);
    const size_t smem = ((size_t)((n_chunks_alloc + 3) & ~3) + (size_t)kMergeWarps * d) * 4;
    if (smem > 200 * 1024) return CASS_ERR_CAPACITY;
    static size_t attr = 48 * 1024;
    if (smem > attr) {
        CASS_CUDA_CHECK(cudaFuncSetAttribute(k_attn_merge, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr = smem;
    }
    CASS_PDL_LAUNCH(k_attn_merge, grid, dim3(kMergeThreads), smem, s, sc, n_chunks_alloc, chunk_tokens, rps, n_q, d, st, draft_mode,
                    draft_units, out);
    return CASS_OK;
}

bool draft_attn_tc_supported(const KvGeom& g, int n_q);
int launch_draft_attn_tc(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                         int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s);

// Both record formats, truncations t = 0 and 4, up to 8 query heads per KV head, head sizes that are multiples of 32.
int launch_draft_attn(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                      int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    if (!draft_attn_tc_supported(g, n_q)) return CASS_ERR_UNSUPPORTED;
    return launch_draft_attn_tc(g, ck, cv, qkv, qkv_stride, n_q, n_seq, st, sc, out, s);
}

}  // namespace cass
