// Online KV encoder (Sec. 4.2: per-token magnitude pruning of K and V, mantissa truncation, unary exponent
// code; Sec. 5.1 encoder): one warp formats one (token, KV head, K|V) record; records are appended to the
// compressed cache and, on request, the raw bf16 rows go to the target's cache.
#include "kernels.cuh"

namespace cass {

constexpr int kKvMaxPerLane = 8;       // head_dim <= 256
constexpr int kKvStageWords = 64;      // exponent staging per token: 2048 bits (a unary stream takes at most 1023, raw bytes 8 per value)
constexpr int kKvWarps = 8;
constexpr int kKvFixMax = 76;        // head_dim 256, no truncation: 3 entry + 8 bitmap + 64 field words (+ 2 exponent words in mode 2)

// Per-token selection: lane holds elements c = lane + 32 j.  keep[j] is set for the d - n_prune largest
// |x| (ties: the lower channel is pruned first).  Key = (|x| bits << 8) | channel is unique, so the kept set is
// {key >= T} where T is the largest value with at most n_prune keys below it; T is found two bits at a time: the three
// candidates of a step are counted in one packed word, so a step costs one warp reduction and the chain of dependent
// reductions is half that of a bit-by-bit search.
__device__ __forceinline__ void kv_select(const uint32_t (&bits)[kKvMaxPerLane], int nj, int n_prune, int lane,
                                          bool (&keep)[kKvMaxPerLane]) {
    uint32_t key[kKvMaxPerLane];
#pragma unroll
    for (int j = 0; j < kKvMaxPerLane; ++j)
        key[j] = j < nj ? (((bits[j] & 0x7FFFu) << 8) | (uint32_t)(lane + 32 * j)) : 0xFFFFFFFFu;
    uint32_t thr = 0;
    if (n_prune > 0) {
        {                                                                        // 23 key bits: the top one alone
            int c = 0;
#pragma unroll
            for (int j = 0; j < kKvMaxPerLane; ++j) c += key[j] < (1u << 22);
            if ((int)__reduce_add_sync(0xffffffffu, c) <= n_prune) thr = 1u << 22;
        }
#pragma unroll 1
        for (int bit = 20; bit >= 0; bit -= 2) {
            const uint32_t c1 = thr | (1u << bit), c2 = thr | (2u << bit), c3 = thr | (3u << bit);
            uint32_t c = 0;                                   // three counts of at most 256 each in one word: one reduction per step
#pragma unroll
            for (int j = 0; j < kKvMaxPerLane; ++j)
                c += (uint32_t)(key[j] < c1) + ((uint32_t)(key[j] < c2) << 10) + ((uint32_t)(key[j] < c3) << 20);
            c = __reduce_add_sync(0xffffffffu, c);
            const int n1 = (int)(c & 1023u), n2 = (int)((c >> 10) & 1023u), n3 = (int)(c >> 20);      // n1 <= n2 <= n3
            thr = n3 <= n_prune ? c3 : (n2 <= n_prune ? c2 : (n1 <= n_prune ? c1 : thr));
        }
    }
#pragma unroll
    for (int j = 0; j < kKvMaxPerLane; ++j) keep[j] = j < nj && key[j] >= thr;
}

__global__ void __launch_bounds__(256) k_kv_hist(KvGeom g, KvComp ck, KvComp cv, const uint16_t* __restrict__ k_cache,
                                                 const uint16_t* __restrict__ v_cache, int n_tokens) {
    __shared__ unsigned int s_hist[256];
    const int head = blockIdx.x, kind = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint16_t* cache = kind ? v_cache : k_cache;
    s_hist[threadIdx.x] = 0;
    __syncthreads();
    const int nj = g.d / 32;
    for (int t = blockIdx.z * kKvWarps + warp; t < n_tokens; t += gridDim.z * kKvWarps) {
        uint32_t bits[kKvMaxPerLane];
        bool keep[kKvMaxPerLane];
        const uint16_t* src = cache + ((size_t)t * g.n_kv + head) * g.d;
#pragma unroll
        for (int j = 0; j < kKvMaxPerLane; ++j) bits[j] = j < nj ? src[lane + 32 * j] : 0;
        kv_select(bits, nj, g.n_prune, lane, keep);
#pragma unroll
        for (int j = 0; j < kKvMaxPerLane; ++j)
            if (keep[j]) atomicAdd(&s_hist[(bits[j] >> 7) & 0xFF], 1u);
    }
    __syncthreads();
    unsigned long long* hist = kind ? cv.hist : ck.hist;
    if (s_hist[threadIdx.x]) atomicAdd(&hist[threadIdx.x], (unsigned long long)s_hist[threadIdx.x]);
}

__global__ void k_kv_rank(KvComp ck, KvComp cv) {
    __shared__ unsigned long long s[256];
    KvComp c = blockIdx.x ? cv : ck;
    int e = threadIdx.x;
    s[e] = c.hist[e];
    __syncthreads();
    unsigned long long mine = s[e];
    int rank = 0;
    for (int o = 0; o < 256; ++o) rank += (s[o] > mine) || (s[o] == mine && o < e);
    c.rank_to_exp[rank] = (uint8_t)e;
    c.exp_to_rank[e] = (uint8_t)rank;
}

// grid (n_kv, 2): block of 8 warps walks the n_new tokens in batches of 8; offsets into the unary arena are
// assigned sequentially by one thread per batch, so records stay densely packed in token order.
// What the fused form of the encoder needs on top: the projection's fp32 split-K parts (the q, k, v features of every
// row), the rotary tables and the bf16 qkv rows to write.
struct RopeSrc {
    Partials pp;
    const float *cos_t, *sin_t;
    uint16_t* qkv;          // [rows][(n_q + 2 n_kv) d]
    int n_q;
};

// grid.z = sequence of the call; its rows start at row blockIdx.z * n_new of the source.
// FUSED: the source is the qkv projection's split-K parts: this kernel adds them, rounds to bf16, rotates q and k
// (RoPE, Sec. 2.1) and writes the qkv rows; the K and V records are then formed from the rotated values as in the
// plain form.  Blocks with blockIdx.x >= n_kv rotate the query heads; head_dim must be a multiple of 64 so that a
// rotation pair (c, c + d/2) sits in one lane.
template <bool FUSED>
__global__ void __launch_bounds__(256) k_kv_append(KvGeom g, KvComp ck, KvComp cv, uint16_t* __restrict__ k_cache,
                                                   uint16_t* __restrict__ v_cache, const uint16_t* __restrict__ src_k,
                                                   const uint16_t* __restrict__ src_v, int row_stride, int start_pos_arg,
                                                   int use_inflight, int n_new, int flags, DevState* st, int seq0, RopeSrc rs) {
    __shared__ uint32_t s_fix[kKvWarps][kKvFixMax];          // bitmap (<= 8) + field words (<= 64)
    __shared__ uint32_t s_una[kKvWarps][kKvStageWords];
    __shared__ uint32_t s_nw[kKvWarps], s_off[kKvWarps];
    __shared__ uint8_t s_e2r[256];                           // exponent -> rank of this (head, K|V): frozen with the codebook
    const int head = blockIdx.x, kind = blockIdx.y, seq = seq0 + blockIdx.z;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // The codebook tables were written when the codebook was frozen, long before this launch's predecessor: they may be
    // read ahead of the wait, which hides their latency.
    if ((flags & CASS_KV_COMPRESSED) && (!FUSED || head < g.n_kv) && threadIdx.x < 256)
        s_e2r[threadIdx.x] = of_seq((kind ? cv : ck).exp_to_rank, seq, g.seq_stride)[threadIdx.x];
    pdl_early<1>();
    pdl_wait();
    __syncthreads();
    if (FUSED && head >= g.n_kv) {
        // ---- query heads: q[r][h][j], q[r][h][j + d/2] rotated by the row's position ----
        if (kind != 0) return;
        const int start = st->len[seq] + (use_inflight ? st->inflight[seq] : 0);
        const int half = g.d / 2, qkv_dim = (rs.n_q + 2 * g.n_kv) * g.d;
        const int per_row = rs.n_q * half, n_items = n_new * per_row;
        const Partials& pp = rs.pp;
        for (int it = (head - g.n_kv) * blockDim.x + threadIdx.x; it < n_items; it += (gridDim.x - g.n_kv) * blockDim.x) {
            const int i = it / per_row, e = it % per_row, hq = e / half, j = e % half;
            const size_t r = (size_t)blockIdx.z * n_new + i;
            const int ia = hq * g.d + j, ib = ia + half;
            const size_t ti = (size_t)(start + i) * half + j;
            const float c = __ldg(rs.cos_t + ti), sn = __ldg(rs.sin_t + ti);      // travel together with the parts
            const size_t offs[2] = {r * pp.row_stride + ia, r * pp.row_stride + ib};
            const bool on2[2] = {true, true};
            float ab[2];
            parts_sum_n<2>(pp, offs, on2, ab);
            const float a = round_bf16(ab[0]), b = round_bf16(ab[1]);
            rs.qkv[r * qkv_dim + ia] = float_to_bf16_bits(a * c - b * sn);
            rs.qkv[r * qkv_dim + ib] = float_to_bf16_bits(b * c + a * sn);
        }
        return;
    }
    const KvComp& c0 = kind ? cv : ck;                       // sequence 0's; shifted to this sequence below
    const uint8_t* exp_to_rank = of_seq(c0.exp_to_rank, seq, g.seq_stride);
    const uint16_t* src = (kind ? src_v : src_k) + (size_t)blockIdx.z * n_new * row_stride;
    uint16_t* cache = of_seq(kind ? v_cache : k_cache, seq, g.seq_stride);
    const int start_pos = start_pos_arg >= 0 ? start_pos_arg : st->len[seq] + (use_inflight ? st->inflight[seq] : 0);
    const int nj = g.d / 32, t_bits = g.t, F = 8 - t_bits, per = 32 / F;
    uint32_t* off = of_seq(c0.off, seq, g.seq_stride) + (size_t)head * (g.max_seq + 1);
    uint32_t* arena = of_seq(c0.arena, seq, g.seq_stride) + (size_t)head * g.arena_words;
    uint32_t* fixed = of_seq(c0.fixed, seq, g.seq_stride) + (size_t)head * g.n_blocks * g.wpt * 32;

    for (int base = 0; base < n_new; base += kKvWarps) {
        const int i = base + warp;
        const bool active = i < n_new && start_pos + i < g.max_seq;
        const int pos = start_pos + i;
        uint32_t bits[kKvMaxPerLane];
        bool keep[kKvMaxPerLane];
        uint32_t n_words = 0;
        if (active) {
            if (FUSED) {
                const int qkv_dim = (rs.n_q + 2 * g.n_kv) * g.d, half = g.d / 2, hj = nj / 2;
                const size_t r = (size_t)blockIdx.z * n_new + i;
                const int base = (rs.n_q + (kind ? g.n_kv : 0) + head) * g.d;
                const Partials& pp = rs.pp;
                float val[kKvMaxPerLane];
                float rc[kKvMaxPerLane / 2], rsn[kKvMaxPerLane / 2];      // the position's rotation, fetched while the parts travel
#pragma unroll
                for (int j = 0; j < kKvMaxPerLane / 2; ++j) {
                    const bool rot = kind == 0 && j < hj;
                    const size_t ti = (size_t)pos * half + lane + 32 * j;
                    rc[j] = rot ? __ldg(rs.cos_t + ti) : 1.f;
                    rsn[j] = rot ? __ldg(rs.sin_t + ti) : 0.f;
                }
                {
                    size_t offs[kKvMaxPerLane];
                    bool on[kKvMaxPerLane];
#pragma unroll
                    for (int j = 0; j < kKvMaxPerLane; ++j) { offs[j] = r * pp.row_stride + base + lane + 32 * j; on[j] = j < nj; }
                    parts_sum_n<kKvMaxPerLane>(pp, offs, on, val);
#pragma unroll
                    for (int j = 0; j < kKvMaxPerLane; ++j) val[j] = j < nj ? round_bf16(val[j]) : 0.f;
                }
                if (kind == 0) {                         // K: rotate the pairs (c, c + d/2), both held by this lane
#pragma unroll
                    for (int j = 0; j < kKvMaxPerLane / 2; ++j) {
                        if (j < hj) {
                            const float c = rc[j], sn = rsn[j];
                            const float a = val[j], b = val[j + hj];
                            val[j] = bf16_bits_to_float(float_to_bf16_bits(a * c - b * sn));
                            val[j + hj] = bf16_bits_to_float(float_to_bf16_bits(b * c + a * sn));
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < kKvMaxPerLane; ++j) {
                    bits[j] = j < nj ? float_to_bf16_bits(val[j]) : 0;
                    if (j < nj) rs.qkv[r * qkv_dim + base + lane + 32 * j] = (uint16_t)bits[j];
                }
            } else {
                const uint16_t* row = src + (size_t)i * row_stride + (size_t)head * g.d;
#pragma unroll
                for (int j = 0; j < kKvMaxPerLane; ++j) bits[j] = j < nj ? row[lane + 32 * j] : 0;
            }
            if (flags & CASS_KV_BF16) {
                uint16_t* dst = cache + ((size_t)pos * g.n_kv + head) * g.d;
#pragma unroll
                for (int j = 0; j < kKvMaxPerLane; ++j)
                    if (j < nj) dst[lane + 32 * j] = (uint16_t)bits[j];
            }
        }
        if (flags & CASS_KV_COMPRESSED) {
            uint32_t off_first = 0;                          // arena offset of this round's first token: fetched while the record is formed
            if (threadIdx.x == 0 && start_pos + base < g.max_seq) off_first = off[start_pos + base];
            if (active) {
                kv_select(bits, nj, g.n_prune, lane, keep);
                for (int w = lane; w < kKvFixMax; w += 32) s_fix[warp][w] = 0;
                for (int w = lane; w < kKvStageWords; w += 32) s_una[warp][w] = 0;
                __syncwarp();
                if (g.mode == 2) {
                    // ---- Cassandra-2 record: bitmap | fields (sign, magnitude >> t; packed from the top) | slice exponents ----
                    uint32_t kbase = 0;
#pragma unroll
                    for (int j = 0; j < kKvMaxPerLane; ++j) {
                        if (j < nj) {
                            const uint32_t bm = __brev(__ballot_sync(0xffffffffu, keep[j]));
                            const uint32_t e = (bits[j] >> 7) & 0xFFu;
                            const uint32_t E = __reduce_max_sync(0xffffffffu, keep[j] ? e : 0u);   // the slice's shared exponent
                            if (lane == 0) {
                                s_fix[warp][j] = bm;
                                atomicOr(&s_fix[warp][g.bm_words + g.f_words + j / 4], E << (24 - 8 * (j % 4)));
                            }
                            if (keep[j]) {
                                const uint32_t sh = 1u + E - e;
                                const uint32_t m7 = (sh < 8u && e > 0u && E >= 7u) ? ((0x80u | (bits[j] & 0x7Fu)) >> sh) : 0u;
                                const uint32_t field = ((bits[j] >> 15) << (7 - t_bits)) | (m7 >> t_bits);
                                const uint32_t k = kbase + (lane ? __popc(bm >> (32 - lane)) : 0u);
                                atomicOr(&s_fix[warp][g.bm_words + k / per], field << (32 - F * (k % per + 1)));
                            }
                            kbase += __popc(bm);
                        }
                    }
                    n_words = 0;
                } else {
                    // ---- Cassandra-1 record: entry words | bitmap | fields; exponent stream staged in s_una ----
                    const int ew = g.e_words;
                    uint32_t kbase = 0, ubase = 0;
#pragma unroll
                    for (int j = 0; j < kKvMaxPerLane; ++j) {
                        if (j < nj) {
                            // entry point of slice j: code bits of all kept values in lower channels
                            if (j > 0 && lane == 0) s_fix[warp][(j - 1) / 3] |= (ubase & 0x3FFu) << (20 - 10 * ((j - 1) % 3));
                            uint32_t bm = __brev(__ballot_sync(0xffffffffu, keep[j]));   // channel c at bit 31 - c%32
                            if (lane == 0) s_fix[warp][ew + j] = bm;
                            uint32_t len = keep[j] ? (uint32_t)s_e2r[(bits[j] >> 7) & 0xFF] + 1u : 0u;
                            uint32_t incl = len;
#pragma unroll
                            for (int o = 1; o < 32; o <<= 1) {
                                uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                                if (lane >= o) incl += v;
                            }
                            if (keep[j]) {
                                uint32_t k = kbase + (lane ? __popc(bm >> (32 - lane)) : 0u);
                                uint32_t field = ((bits[j] >> 15) << (7 - t_bits)) | ((bits[j] & 0x7Fu) >> t_bits);
                                atomicOr(&s_fix[warp][ew + nj + k / per], field_bits_in_word(field, k % per, t_bits));
                                uint32_t p = ubase + incl - 1;
                                if ((p >> 5) < (uint32_t)kKvStageWords) atomicOr(&s_una[warp][p >> 5], 0x80000000u >> (p & 31));
                            }
                            kbase += __popc(bm);
                            ubase += __shfl_sync(0xffffffffu, incl, 31);
                        }
                    }
                    n_words = (ubase + 31) / 32;
                    if (ubase > (uint32_t)kv_code_budget(g.kept)) {
                        // the codewords take more room than raw exponents would (or their offsets leave the entry
                        // words): store the kept exponents as bytes instead and flag the record
                        __syncwarp();
                        for (int w = lane; w < kKvStageWords; w += 32) s_una[warp][w] = 0;
                        for (int w = lane; w < ew; w += 32) s_fix[warp][w] = w == 0 ? kKvRawFlag : 0u;
                        __syncwarp();
                        uint32_t kb2 = 0;
#pragma unroll
                        for (int j = 0; j < kKvMaxPerLane; ++j) {
                            if (j < nj) {
                                const uint32_t bm = __brev(__ballot_sync(0xffffffffu, keep[j]));
                                if (keep[j]) {
                                    const uint32_t k = kb2 + (lane ? __popc(bm >> (32 - lane)) : 0u);
                                    if ((k >> 2) < (uint32_t)kKvStageWords)
                                        atomicOr(&s_una[warp][k >> 2], ((bits[j] >> 7) & 0xFFu) << (24 - 8 * (k & 3)));
                                }
                                kb2 += __popc(bm);
                            }
                        }
                        n_words = (uint32_t)ceil_div(g.kept, 4);
                    }
                    if (n_words > (uint32_t)kKvStageWords) {          // cannot happen for head_dim <= 256
                        if (lane == 0) atomicCAS(&st->status, 0, CASS_ERR_CAPACITY);
                        n_words = kKvStageWords;
                    }
                }
            }
            if (lane == 0) s_nw[warp] = active ? n_words : 0u;
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t o = off_first;
                for (int w = 0; w < kKvWarps; ++w) {
                    int p = start_pos + base + w;
                    if (base + w >= n_new || p >= g.max_seq) break;
                    uint32_t nw = s_nw[w];
                    if (o + nw > (uint32_t)g.arena_words) {           // arena full: keep offsets valid, drop the codes
                        atomicCAS(&st->status, 0, CASS_ERR_CAPACITY);
                        nw = 0;
                        s_nw[w] = 0;
                    }
                    s_off[w] = o;
                    o += nw;
                    off[p + 1] = o;
                }
            }
            __syncthreads();
            if (active) {
                uint32_t* blk = fixed + (size_t)(pos / 32) * g.wpt * 32 + (pos % 32);
                for (int w = lane; w < g.wpt; w += 32) blk[w * 32] = s_fix[warp][w];
                uint32_t o = s_off[warp], nw = s_nw[warp];
                for (uint32_t w = lane; w < nw; w += 32) arena[o + w] = s_una[warp][w];
            }
            __syncthreads();
        }
    }
}

int launch_kv_append(const KvGeom& g, const KvComp& ck, const KvComp& cv, uint16_t* k_cache, uint16_t* v_cache,
                     const uint16_t* src_k, const uint16_t* src_v, int row_stride, int start_pos, int use_inflight,
                     int n_new, int flags, DevState* st, int seq0, int n_seq, cudaStream_t s) {
    if (n_new <= 0 || n_seq <= 0) return CASS_OK;
    dim3 grid(g.n_kv, 2, n_seq);
    CASS_PDL_LAUNCH(k_kv_append<false>, grid, dim3(256), 0, s, g, ck, cv, k_cache, v_cache, src_k, src_v, row_stride, start_pos,
                    use_inflight, n_new, flags, st, seq0, RopeSrc{});
    return CASS_OK;
}

bool rope_kv_fusable(const KvGeom& g) { return g.d % 64 == 0; }

int launch_rope_kv_append(const KvGeom& g, const KvComp& ck, const KvComp& cv, uint16_t* k_cache, uint16_t* v_cache,
                          Partials pp, const float* cos_t, const float* sin_t, uint16_t* qkv, int n_q, int use_inflight,
                          int rps, int flags, DevState* st, int n_seq, cudaStream_t s) {
    if (rps <= 0 || n_seq <= 0) return CASS_OK;
    if (!rope_kv_fusable(g) || !pp.p) return CASS_ERR_UNSUPPORTED;
    const int q_blocks = ceil_div(n_q * (g.d / 2), 256);
    dim3 grid(g.n_kv + q_blocks, 2, n_seq);
    CASS_PDL_LAUNCH(k_kv_append<true>, grid, dim3(256), 0, s, g, ck, cv, k_cache, v_cache, (const uint16_t*)nullptr,
                    (const uint16_t*)nullptr, 0, -1, use_inflight, rps, flags, st, 0, RopeSrc{pp, cos_t, sin_t, qkv, n_q});
    return CASS_OK;
}

int launch_kv_codebook(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* k_cache,
                       const uint16_t* v_cache, int n_tokens, cudaStream_t s) {
    CASS_CUDA_CHECK(cudaMemsetAsync(ck.hist, 0, 256 * 8, s));
    CASS_CUDA_CHECK(cudaMemsetAsync(cv.hist, 0, 256 * 8, s));
    if (n_tokens > 0) {
        dim3 grid(g.n_kv, 2, min(64, ceil_div(n_tokens, kKvWarps)));
        k_kv_hist<<<grid, 256, 0, s>>>(g, ck, cv, k_cache, v_cache, n_tokens);
        CASS_LAUNCH_CHECK();
    }
    k_kv_rank<<<2, 256, 0, s>>>(ck, cv);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

}  // namespace cass
