// Verification attention (Sec. 2.2): causal grouped-query attention of the gamma+1 new rows over the bf16 KV
// cache, split over the sequence in fixed 256-token chunks.  The work of one (row, head, chunk) never depends on
// the other rows of the call, so verification with one row reproduces plain autoregressive decoding bit for bit.
#include "kernels.cuh"

namespace cass {

constexpr int kVaRowBatch = 2;
constexpr int kVaMaxGroup = 8;
constexpr int kVaMaxPairs = kVaRowBatch * kVaMaxGroup;

__global__ void __launch_bounds__(256) k_verify_attn(KvGeom g, const uint16_t* __restrict__ k_cache,
                                                     const uint16_t* __restrict__ v_cache, const uint16_t* __restrict__ qkv,
                                                     int rows, int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                     int n_chunks_alloc) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int chunk = blockIdx.x, head = blockIdx.y;
    const int len = st->len;
    const int t0 = chunk * kAttnChunk;
    if (t0 >= len + rows) return;
    const int d = g.d, G = n_q / g.n_kv, ks = d + 8;                  // padded K row stride (elements)
    const int qkv_dim = (n_q + 2 * g.n_kv) * d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint16_t* k_s = reinterpret_cast<uint16_t*>(smem);                         // [256][d+8]
    uint16_t* v_s = k_s + kAttnChunk * ks;                                      // [256][d]
    float* q_s = reinterpret_cast<float*>(v_s + kAttnChunk * d);                // [pairs][d]
    float* s_s = q_s + kVaMaxPairs * d;                                         // [pairs][256]

    const int n_tok = min(kAttnChunk, len + rows - t0);
    const int vec_per_row = d / 8;
    for (int i = tid; i < kAttnChunk * vec_per_row; i += 256) {
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

    for (int r0 = 0; r0 < rows; r0 += kVaRowBatch) {
        const int nr = min(kVaRowBatch, rows - r0);
        if (t0 >= len + r0 + nr) continue;                              // no row of this batch sees the chunk (later rows may)
        const int P = nr * G;
        __syncthreads();
        for (int i = tid; i < P * d; i += 256) {
            int p = i / d, dim = i % d, r = r0 + p / G, gi = p % G;
            q_s[i] = bf16_bits_to_float(qkv[(size_t)r * qkv_dim + (size_t)(head * G + gi) * d + dim]);
        }
        __syncthreads();
        // scores: thread = token
        {
            const int t = tid;
            float acc[kVaMaxPairs];
#pragma unroll
            for (int p = 0; p < kVaMaxPairs; ++p) acc[p] = 0.f;
            for (int dd = 0; dd < d; dd += 8) {
                const uint4 kv = *reinterpret_cast<const uint4*>(k_s + (size_t)t * ks + dd);
                const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
                float kf[8];
#pragma unroll
                for (int q = 0; q < 4; ++q) { kf[2 * q] = __uint_as_float(kw[q] << 16); kf[2 * q + 1] = __uint_as_float(kw[q] & 0xFFFF0000u); }
#pragma unroll
                for (int p = 0; p < kVaMaxPairs; ++p) {
                    if (p < P) {
                        const float4 qa = *reinterpret_cast<const float4*>(q_s + p * d + dd);
                        const float4 qb = *reinterpret_cast<const float4*>(q_s + p * d + dd + 4);
                        acc[p] = fmaf(kf[0], qa.x, acc[p]); acc[p] = fmaf(kf[1], qa.y, acc[p]);
                        acc[p] = fmaf(kf[2], qa.z, acc[p]); acc[p] = fmaf(kf[3], qa.w, acc[p]);
                        acc[p] = fmaf(kf[4], qb.x, acc[p]); acc[p] = fmaf(kf[5], qb.y, acc[p]);
                        acc[p] = fmaf(kf[6], qb.z, acc[p]); acc[p] = fmaf(kf[7], qb.w, acc[p]);
                    }
                }
            }
#pragma unroll
            for (int p = 0; p < kVaMaxPairs; ++p) {
                if (p < P) {
                    int r = r0 + p / G;
                    bool vis = (t0 + t) <= len + r;                       // causal: row r sits at position len + r
                    s_s[p * kAttnChunk + t] = vis ? acc[p] * scale : -INFINITY;
                }
            }
        }
        __syncthreads();
        // per pair: chunk softmax and P.V; warp w takes pairs w, w+8, ...
        for (int p = warp; p < P; p += 8) {
            const int r = r0 + p / G, gi = p % G;
            if (t0 > len + r) continue;                                  // chunk entirely in the future of this row
            float m = -INFINITY;
            for (int i = lane; i < kAttnChunk; i += 32) m = fmaxf(m, s_s[p * kAttnChunk + i]);
            m = warp_max(m);
            float l = 0.f;
            for (int i = lane; i < kAttnChunk; i += 32) {
                float pr = expf(s_s[p * kAttnChunk + i] - m);
                s_s[p * kAttnChunk + i] = pr;
                l += pr;
            }
            l = warp_sum(l);
            __syncwarp();
            const size_t pair = (size_t)r * n_q + head * G + gi;
            for (int dim = lane; dim < d; dim += 32) {
                float acc = 0.f;
                for (int t = 0; t < n_tok; ++t)
                    acc = fmaf(s_s[p * kAttnChunk + t], bf16_bits_to_float(v_s[(size_t)t * d + dim]), acc);
                sc.o[(pair * n_chunks_alloc + chunk) * d + dim] = acc;
            }
            if (lane == 0) {
                sc.m[pair * n_chunks_alloc + chunk] = m;
                sc.l[pair * n_chunks_alloc + chunk] = l;
            }
        }
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int n_q, int d,
                      const DevState* st, int draft_mode, uint16_t* out, cudaStream_t s);

int launch_verify_attn(const KvGeom& g, const uint16_t* k_cache, const uint16_t* v_cache, const uint16_t* qkv, int rows,
                       int n_q, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    const int G = n_q / g.n_kv;
    if (G > kVaMaxGroup || g.d % 8) return CASS_ERR_UNSUPPORTED;
    const int n_chunks = ceil_div(g.max_seq, kAttnChunk);
    size_t smem = (size_t)kAttnChunk * (g.d + 8) * 2 + (size_t)kAttnChunk * g.d * 2 + (size_t)kVaMaxPairs * g.d * 4 +
                  (size_t)kVaMaxPairs * kAttnChunk * 4;
    static size_t attr = 0;
    if (smem > attr) {
        CASS_CUDA_CHECK(cudaFuncSetAttribute(k_verify_attn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr = smem;
    }
    dim3 grid(n_chunks, g.n_kv);
    k_verify_attn<<<grid, 256, smem, s>>>(g, k_cache, v_cache, qkv, rows, n_q, st, sc, n_chunks);
    CASS_LAUNCH_CHECK();
    return launch_attn_merge(sc, n_chunks, kAttnChunk, rows, n_q, g.d, st, 0, out, s);
}

}  // namespace cass
