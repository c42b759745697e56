// Verification attention (Sec. 2.2): causal grouped-query attention of the gamma+1 new rows over the bf16 KV
// cache, split over the sequence in fixed 64-token chunks.  One CTA = one (KV head, chunk): the chunk's K and V
// tiles are staged once in shared memory and reused by all rows and by the query heads of the group.  The work of
// one (row, head, chunk) never depends on the other rows of the call, so verification with one row reproduces plain
// autoregressive decoding bit for bit.
#include "kernels.cuh"

namespace cass {

constexpr int kVaThreads = 128;
constexpr int kVaRowBatch = 2;
constexpr int kVaMaxGroup = 8;
constexpr int kVaMaxPairs = kVaRowBatch * kVaMaxGroup;      // (row, query head) pairs handled at a time
constexpr int kVaHalfPairs = kVaMaxPairs / 2;

// grid (chunk, KV head, sequence); `rows` = rows of each sequence in this call.
__global__ void __launch_bounds__(kVaThreads) k_verify_attn(KvGeom g, const uint16_t* __restrict__ k_cache0,
                                                            const uint16_t* __restrict__ v_cache0, const uint16_t* __restrict__ qkv0,
                                                            int rows, int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                            int n_chunks_alloc) {
    extern __shared__ __align__(16) uint8_t smem[];
    pdl_early<4>();
    pdl_wait();
    const int chunk = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    const int len = st->len[seq];
    const uint16_t* __restrict__ k_cache = of_seq(k_cache0, seq, g.seq_stride);
    const uint16_t* __restrict__ v_cache = of_seq(v_cache0, seq, g.seq_stride);
    const int t0 = chunk * kAttnChunk;
    if (t0 >= len + rows) return;
    const int d = g.d, G = n_q / g.n_kv, ks = d + 8;                  // padded K row stride (elements)
    const int qkv_dim = (n_q + 2 * g.n_kv) * d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint16_t* __restrict__ qkv = qkv0 + (size_t)seq * rows * qkv_dim;     // this sequence's rows
    uint16_t* k_s = reinterpret_cast<uint16_t*>(smem);                         // [64][d+8]
    uint16_t* v_s = k_s + kAttnChunk * ks;                                      // [64][d]
    float* q_s = reinterpret_cast<float*>(v_s + kAttnChunk * d);                // [pairs][d]
    float* s_s = q_s + kVaMaxPairs * d;                                         // [pairs][64]

    const int n_tok = min(kAttnChunk, len + rows - t0);
    const int vec_per_row = d / 8;
    for (int i = tid; i < kAttnChunk * vec_per_row; i += kVaThreads) {
        int t = i / vec_per_row, c = i % vec_per_row;
        uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
        if (t < n_tok) {
            size_t src = ((size_t)(t0 + t) * g.n_kv + head) * d + c * 8;
            kv = *reinterpret_cast<const uint4*>(k_cache + src);
            vv = *reinterpret_cast<const uint4*>(v_cache + src);
        }
        *reinterpret_cast<uint4*>(k_s + (size_t)t * ks + c * 8) = kv;
        *reinterpret_cast<uint4*>(v_s + (size_t)t * d + c * 8) = vv;
    }
    const float scale = rsqrtf((float)d);

    const int row_batch = kVaMaxPairs / G;                            // rows whose (row, query head) pairs fit one pass
    for (int r0 = 0; r0 < rows; r0 += row_batch) {
        const int nr = min(row_batch, rows - r0);
        if (t0 >= len + r0 + nr) continue;                              // no row of this batch sees the chunk (later rows may)
        const int P = nr * G;
        __syncthreads();
        for (int i = tid; i < P * d; i += kVaThreads) {
            int p = i / d, dim = i % d, r = r0 + p / G, gi = p % G;
            q_s[i] = bf16_bits_to_float(qkv[(size_t)r * qkv_dim + (size_t)(head * G + gi) * d + dim]);
        }
        __syncthreads();
        // scores: thread = (token, half of the pairs); the dot product of one (token, pair) runs over d in a fixed order
        {
            const int t = tid & (kAttnChunk - 1), p_lo = tid / kAttnChunk;      // this thread's pairs: p_lo, p_lo + 2, ...
            float acc[kVaHalfPairs];
#pragma unroll
            for (int p = 0; p < kVaHalfPairs; ++p) acc[p] = 0.f;
            for (int dd = 0; dd < d; dd += 8) {
                const uint4 kv = *reinterpret_cast<const uint4*>(k_s + (size_t)t * ks + dd);
                const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
                float kf[8];
#pragma unroll
                for (int q = 0; q < 4; ++q) { kf[2 * q] = __uint_as_float(kw[q] << 16); kf[2 * q + 1] = __uint_as_float(kw[q] & 0xFFFF0000u); }
#pragma unroll
                for (int p = 0; p < kVaHalfPairs; ++p) {
                    if (p_lo + 2 * p < P) {
                        const float4 qa = *reinterpret_cast<const float4*>(q_s + (p_lo + 2 * p) * d + dd);
                        const float4 qb = *reinterpret_cast<const float4*>(q_s + (p_lo + 2 * p) * d + dd + 4);
                        acc[p] = fmaf(kf[0], qa.x, acc[p]); acc[p] = fmaf(kf[1], qa.y, acc[p]);
                        acc[p] = fmaf(kf[2], qa.z, acc[p]); acc[p] = fmaf(kf[3], qa.w, acc[p]);
                        acc[p] = fmaf(kf[4], qb.x, acc[p]); acc[p] = fmaf(kf[5], qb.y, acc[p]);
                        acc[p] = fmaf(kf[6], qb.z, acc[p]); acc[p] = fmaf(kf[7], qb.w, acc[p]);
                    }
                }
            }
#pragma unroll
            for (int p = 0; p < kVaHalfPairs; ++p) {
                if (p_lo + 2 * p < P) {
                    int r = r0 + (p_lo + 2 * p) / G;
                    bool vis = (t0 + t) <= len + r;                       // causal: row r sits at position len + r
                    s_s[(p_lo + 2 * p) * kAttnChunk + t] = vis ? acc[p] * scale : -INFINITY;
                }
            }
        }
        __syncthreads();
        // per pair: chunk softmax and P.V; warp w takes pairs w, w+4, ...
        for (int p = warp; p < P; p += kVaThreads / 32) {
            const int r = r0 + p / G, gi = p % G;
            if (t0 > len + r) continue;                                  // chunk entirely in the future of this row
            float a = s_s[p * kAttnChunk + lane], b = s_s[p * kAttnChunk + 32 + lane];
            const float m = warp_max(fmaxf(a, b));
            a = expf(a - m);
            b = expf(b - m);
            s_s[p * kAttnChunk + lane] = a;
            s_s[p * kAttnChunk + 32 + lane] = b;
            const float l = warp_sum(a + b);
            __syncwarp();
            const size_t pair = ((size_t)seq * rows + r) * n_q + head * G + gi;
            for (int dim = lane * 4; dim < d; dim += 128) {             // four dims per lane, tokens in order
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
                for (int t = 0; t < n_tok; ++t) {
                    const float pr = s_s[p * kAttnChunk + t];
                    const uint2 vv = *reinterpret_cast<const uint2*>(v_s + (size_t)t * d + dim);
                    a0 = fmaf(pr, __uint_as_float(vv.x << 16), a0);
                    a1 = fmaf(pr, __uint_as_float(vv.x & 0xFFFF0000u), a1);
                    a2 = fmaf(pr, __uint_as_float(vv.y << 16), a2);
                    a3 = fmaf(pr, __uint_as_float(vv.y & 0xFFFF0000u), a3);
                }
                *reinterpret_cast<float4*>(sc.o + (pair * n_chunks_alloc + chunk) * d + dim) = make_float4(a0, a1, a2, a3);
            }
            if (lane == 0) {
                sc.m[pair * n_chunks_alloc + chunk] = m;
                sc.l[pair * n_chunks_alloc + chunk] = l;
            }
        }
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int rps, int n_q, int d,
                      const DevState* st, int draft_mode, int draft_units, uint16_t* out, cudaStream_t s);

int launch_verify_attn(const KvGeom& g, const uint16_t* k_cache, const uint16_t* v_cache, const uint16_t* qkv, int n_seq,
                       int rps, int n_q, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    const int G = n_q / g.n_kv;
    if (G > kVaMaxGroup || g.d % 8) return CASS_ERR_UNSUPPORTED;
    static_assert(kAttnChunk == 64 && kVaThreads == 2 * kAttnChunk, "thread = (token, half of the pairs)");
    const int n_chunks = ceil_div(g.max_seq, kAttnChunk);
    size_t smem = (size_t)kAttnChunk * (g.d + 8) * 2 + (size_t)kAttnChunk * g.d * 2 + (size_t)kVaMaxPairs * g.d * 4 +
                  (size_t)kVaMaxPairs * kAttnChunk * 4;
    static size_t attr = 0;
    if (smem > attr) {
        CASS_CUDA_CHECK(cudaFuncSetAttribute(k_verify_attn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr = smem;
    }
    dim3 grid(n_chunks, g.n_kv, n_seq);
    CASS_PDL_LAUNCH(k_verify_attn, grid, dim3(kVaThreads), smem, s, g, k_cache, v_cache, qkv, rps, n_q, st, sc, n_chunks);
    return launch_attn_merge(sc, n_chunks, kAttnChunk, n_seq * rps, rps, n_q, g.d, st, 0, 0, out, s);
}

}  // namespace cass
