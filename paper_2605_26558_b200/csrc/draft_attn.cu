// Draft decode attention over the compressed KV cache (Sec. 4.1 draft inference; KV speculation data of
// Sec. 4.2): grouped-query attention of one query row, split over the sequence in fixed 256-token chunks
// with a log-sum-exp merge.  Lane = token: every lane walks its own token's record (bitmap, fields, unary
// codes) and accumulates q.k for all query heads of the group; V records are decoded into a dense bf16 tile in
// shared memory and multiplied by the chunk's probabilities.
#include "kernels.cuh"

namespace cass {

constexpr int kDaWarps = kAttnChunk / 32;     // 8 warps, 32 tokens each
constexpr int kDaUnaStage = 24;               // staged unary words per token; longer records are read in place
constexpr int kMaxGroup = 8;                  // query heads per KV head

// Sequential decode of one token's record.  fix: bitmap then field words with stride fs; una: words with stride us.
template <class Emit>
__device__ __forceinline__ void kv_decode_token(const uint32_t* fix, int fs, const uint32_t* una, int us, uint32_t n_una,
                                                int bm_words, int t, const uint8_t* __restrict__ r2e, Emit&& emit) {
    const int F = 8 - t, per = 32 / F;
    uint32_t ub = 0;
    const uint32_t limit = n_una * 32u;
    int k = 0;
    for (int w = 0; w < bm_words; ++w) {
        uint32_t bm = fix[w * fs];
        while (bm) {
            int s = __clz(bm);
            bm &= ~(0x80000000u >> s);
            uint32_t fword = fix[(bm_words + k / per) * fs];
            int rank = 0;
            while (ub < limit) {
                uint32_t v = una[(ub >> 5) * us] << (ub & 31);
                int avail = 32 - (int)(ub & 31);
                if (v) { int z = __clz(v); rank += z; ub += z + 1; break; }
                rank += avail;
                ub += avail;
            }
            uint32_t e = r2e[rank & 255];
            uint32_t bits = field_sign_mant_bf16(fword, k % per, t) | (e << 7);
            emit(w * 32 + s, bits);
            ++k;
        }
    }
}

struct DaSmem {
    // carved from dynamic shared memory by the kernel
};

__global__ void __launch_bounds__(256) k_draft_attn(KvGeom g, KvComp ck, KvComp cv, const uint16_t* __restrict__ qkv,
                                                    int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                    int n_chunks_alloc) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int chunk = blockIdx.x, head = blockIdx.y;
    const int cur_len = st->len + st->inflight + 1;            // positions visible to the drafted token
    const int t0 = chunk * kAttnChunk;
    if (t0 >= cur_len) return;
    const int G = n_q / g.n_kv, d = g.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    float* q_s = reinterpret_cast<float*>(smem);                              // [G][d]
    float* sc_s = q_s + kMaxGroup * d;                                        // [G][256] scores -> probabilities
    float* ml_s = sc_s + kMaxGroup * kAttnChunk;                              // [G][2]
    uint32_t* fix_s = reinterpret_cast<uint32_t*>(ml_s + 2 * kMaxGroup);      // [8 warps][wpt][32]
    uint32_t* una_s = fix_s + kDaWarps * g.wpt * 32;                          // [8 warps][kDaUnaStage][32]
    uint16_t* v_s = reinterpret_cast<uint16_t*>(una_s + kDaWarps * kDaUnaStage * 32);   // [256][d] bf16
    uint8_t* r2e_s = reinterpret_cast<uint8_t*>(v_s + kAttnChunk * d);        // [2][256]

    const float scale = rsqrtf((float)d);
    for (int i = tid; i < G * d; i += 256) q_s[i] = bf16_bits_to_float(qkv[(size_t)head * G * d + i]);
    for (int i = tid; i < 256; i += 256) { r2e_s[i] = ck.rank_to_exp[i]; r2e_s[256 + i] = cv.rank_to_exp[i]; }
    for (int i = tid; i < kAttnChunk * d / 2; i += 256) reinterpret_cast<uint32_t*>(v_s)[i] = 0u;
    __syncthreads();

    const int tok = t0 + warp * 32 + lane;
    const bool valid = tok < cur_len;
    const int blk = tok / 32;                                               // same for the whole warp
    uint32_t* my_fix = fix_s + warp * g.wpt * 32 + lane;
    uint32_t* my_una = una_s + warp * kDaUnaStage * 32 + lane;

    for (int kind = 0; kind < 2; ++kind) {
        const KvComp& c = kind ? cv : ck;
        const uint32_t* fixed = c.fixed + ((size_t)head * g.n_blocks + blk) * g.wpt * 32;
        const uint32_t* off = c.off + (size_t)head * (g.max_seq + 1);
        const uint32_t* arena = c.arena + (size_t)head * g.arena_words;
        __syncwarp();
        for (int w = 0; w < g.wpt; ++w) my_fix[w * 32] = fixed[w * 32 + lane];         // coalesced block copy
        uint32_t o0 = 0, n_una = 0;
        if (valid) { o0 = off[tok]; n_una = off[tok + 1] - o0; }
        const bool staged = n_una <= (uint32_t)kDaUnaStage;
        if (staged) for (uint32_t w = 0; w < n_una; ++w) my_una[w * 32] = arena[o0 + w];
        __syncwarp();
        const uint32_t* una = staged ? my_una : arena + o0;
        const int us = staged ? 32 : 1;
        if (kind == 0) {
            float acc[kMaxGroup];
#pragma unroll
            for (int gi = 0; gi < kMaxGroup; ++gi) acc[gi] = 0.f;
            if (valid) {
                kv_decode_token(my_fix, 32, una, us, n_una, g.bm_words, g.t, r2e_s, [&](int col, uint32_t bits) {
                    float kvv = bf16_bits_to_float(bits);
#pragma unroll
                    for (int gi = 0; gi < kMaxGroup; ++gi)
                        if (gi < G) acc[gi] = fmaf(kvv, q_s[gi * d + col], acc[gi]);
                });
            }
#pragma unroll
            for (int gi = 0; gi < kMaxGroup; ++gi)
                if (gi < G) sc_s[gi * kAttnChunk + warp * 32 + lane] = valid ? acc[gi] * scale : -INFINITY;
        } else {
            if (valid) {
                uint16_t* vrow = v_s + (size_t)(warp * 32 + lane) * d;
                kv_decode_token(my_fix, 32, una, us, n_una, g.bm_words, g.t, r2e_s + 256,
                                [&](int col, uint32_t bits) { vrow[col] = (uint16_t)bits; });
            }
        }
    }
    __syncthreads();
    // chunk softmax statistics: warp gi handles query head gi of the group
    if (warp < G) {
        float m = -INFINITY;
        for (int i = lane; i < kAttnChunk; i += 32) m = fmaxf(m, sc_s[warp * kAttnChunk + i]);
        m = warp_max(m);
        float l = 0.f;
        for (int i = lane; i < kAttnChunk; i += 32) {
            float p = expf(sc_s[warp * kAttnChunk + i] - m);          // exp(-inf) = 0 for tokens beyond the end
            sc_s[warp * kAttnChunk + i] = p;
            l += p;
        }
        l = warp_sum(l);
        if (lane == 0) { ml_s[warp * 2] = m; ml_s[warp * 2 + 1] = l; }
    }
    __syncthreads();
    // o[gi][dim] = sum_t p[gi][t] * v[t][dim]
    const int n_tok = min(kAttnChunk, cur_len - t0);
    for (int item = tid; item < G * d; item += 256) {
        int gi = item / d, dim = item % d;
        float acc = 0.f;
        for (int t = 0; t < n_tok; ++t) acc = fmaf(sc_s[gi * kAttnChunk + t], bf16_bits_to_float(v_s[(size_t)t * d + dim]), acc);
        int hq = head * G + gi;
        sc.o[((size_t)hq * n_chunks_alloc + chunk) * d + dim] = acc;
    }
    if (tid < G) {
        int hq = head * G + tid;
        sc.m[(size_t)hq * n_chunks_alloc + chunk] = ml_s[tid * 2];
        sc.l[(size_t)hq * n_chunks_alloc + chunk] = ml_s[tid * 2 + 1];
    }
}

// Merge the chunk partials of every (row, query head): out = sum_c e^{m_c - M} o_c / sum_c e^{m_c - M} l_c.
// Row r sees positions < len + (draft: inflight + 1 | verify: r + 1).
__global__ void k_attn_merge(AttnScratch sc, int n_chunks_alloc, int n_q, int d, const DevState* __restrict__ st,
                             int draft_mode, uint16_t* __restrict__ out) {
    const int hq = blockIdx.x, r = blockIdx.y;
    const int vis = st->len + (draft_mode ? st->inflight + 1 : r + 1);
    const int n_ch = ceil_div(vis, kAttnChunk);
    const size_t pair = (size_t)r * n_q + hq;
    float M = -INFINITY;
    for (int c = 0; c < n_ch; ++c) M = fmaxf(M, sc.m[pair * n_chunks_alloc + c]);
    float L = 0.f;
    for (int c = 0; c < n_ch; ++c) L += expf(sc.m[pair * n_chunks_alloc + c] - M) * sc.l[pair * n_chunks_alloc + c];
    for (int dim = threadIdx.x; dim < d; dim += blockDim.x) {
        float acc = 0.f;
        for (int c = 0; c < n_ch; ++c)
            acc += expf(sc.m[pair * n_chunks_alloc + c] - M) * sc.o[(pair * n_chunks_alloc + c) * d + dim];
        out[((size_t)r * n_q + hq) * d + dim] = float_to_bf16_bits(acc / L);
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int rows, int n_q, int d, const DevState* st,
                      int draft_mode, uint16_t* out, cudaStream_t s) {
    dim3 grid(n_q, rows);
    k_attn_merge<<<grid, 128, 0, s>>>(sc, n_chunks_alloc, n_q, d, st, draft_mode, out);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

int launch_draft_attn(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int n_q,
                      const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    const int G = n_q / g.n_kv;
    if (G > kMaxGroup || g.d > 256 || g.d % 32) return CASS_ERR_UNSUPPORTED;
    const int n_chunks = ceil_div(g.max_seq, kAttnChunk);
    size_t smem = (size_t)kMaxGroup * g.d * 4 + (size_t)kMaxGroup * kAttnChunk * 4 + 2 * kMaxGroup * 4 +
                  (size_t)kDaWarps * g.wpt * 32 * 4 + (size_t)kDaWarps * kDaUnaStage * 32 * 4 +
                  (size_t)kAttnChunk * g.d * 2 + 512;
    static size_t attr = 0;
    if (smem > attr) {
        CASS_CUDA_CHECK(cudaFuncSetAttribute(k_draft_attn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr = smem;
    }
    dim3 grid(n_chunks, g.n_kv);
    k_draft_attn<<<grid, 256, smem, s>>>(g, ck, cv, qkv, n_q, st, sc, n_chunks);
    CASS_LAUNCH_CHECK();
    return launch_attn_merge(sc, n_chunks, 1, n_q, g.d, st, 1, out, s);
}

}  // namespace cass
