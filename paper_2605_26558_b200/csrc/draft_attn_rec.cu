// Draft decode attention over Cassandra-1 KV records, whole-record form, for long caches (Sec. 4.1 draft inference; KV
// speculation data of Sec. 4.2): fixed 64-token chunks with a log-sum-exp merge.  One CTA = one (KV head, chunk): warps
// 0-1 decode the K records of 32 tokens each (lane = token, the whole record by one lane) and form q.k for all query
// heads of the group, warps 2-3 decode the V records of the same tokens into a dense bf16 tile in shared memory; then
// the chunk's probabilities multiply the tile.  Every lane has the same number of values, so no issue slot is idle:
// per value this costs about half the instructions of the slice-parallel kernel (draft_attn.cu), whose shorter
// dependency chains win only while the cache is short and the grid small.  Records are walked like the weight
// streams: 8 kept values per 32-bit bitmap window, 4 codewords per 32-bit unary window, with a careful walk for the
// rare group that does not fit its windows, for records longer than the staging and for records with raw exponents.
#include <type_traits>

#include "kernels.cuh"

namespace cass {

constexpr int kDrTok = kAttnChunk;            // tokens per CTA
constexpr int kDrThreads = 128;
constexpr int kDrUnaStage = 12;               // staged unary words per token (a typical record has 5-8); longer records are read in place
constexpr int kDrMaxGroup = 8;                  // query heads per KV head

__device__ __forceinline__ uint32_t dr_shl(uint32_t v, uint32_t s) {
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
}
__device__ __forceinline__ uint32_t dr_lds(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// What happens to a decoded value.  K: multiply with the query tile; V: store into the token's dense row.
// GQ = query heads the tile has room for (4 or 8): q_s[col][GQ] floats.
template <int GQ>
struct RecEmitK {
    float acc[GQ], g[GQ];
    uint32_t q_a;
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < GQ; ++i) g[i] = 0.f;
    }
    __device__ __forceinline__ void fma_into(float (&dst)[GQ], uint32_t off, uint32_t wb) {
        const float w = __uint_as_float(wb);
        float4 a;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "r"(q_a + off));
        dst[0] = fmaf(w, a.x, dst[0]); dst[1] = fmaf(w, a.y, dst[1]); dst[2] = fmaf(w, a.z, dst[2]); dst[3] = fmaf(w, a.w, dst[3]);
        if constexpr (GQ > 4) {
            float4 b;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+16];" : "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "r"(q_a + off));
            dst[4] = fmaf(w, b.x, dst[4]); dst[5] = fmaf(w, b.y, dst[5]); dst[6] = fmaf(w, b.z, dst[6]); dst[7] = fmaf(w, b.w, dst[7]);
        }
    }
    template <int E>
    __device__ __forceinline__ void elem(uint32_t off, uint32_t wb, bool valid) { if (valid) fma_into(g, off, wb); }
    __device__ __forceinline__ void commit(int) {
#pragma unroll
        for (int i = 0; i < GQ; ++i) acc[i] += g[i];
    }
    __device__ __forceinline__ void direct(uint32_t off, uint32_t wb) { fma_into(acc, off, wb); }
    __device__ __forceinline__ void restart() {
#pragma unroll
        for (int i = 0; i < GQ; ++i) acc[i] = 0.f;
    }
};

struct RecEmitV {
    uint32_t row_a;                      // shared address of the token's dense row
    uint32_t off[kGroupCols], wb[kGroupCols];
    __device__ __forceinline__ void reset() {}
    template <int E>
    __device__ __forceinline__ void elem(uint32_t o, uint32_t w, bool) { off[E] = o; wb[E] = w; }
    __device__ __forceinline__ void commit(int cnt) {
#pragma unroll
        for (int e = 0; e < kGroupCols; ++e)
            if (e < cnt) asm volatile("st.shared.u16 [%0], %1;" ::"r"(row_a + off[e]), "h"((uint16_t)(wb[e] >> 16)));
    }
    __device__ __forceinline__ void direct(uint32_t o, uint32_t w) {
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(row_a + o), "h"((uint16_t)(w >> 16)));
    }
    __device__ __forceinline__ void restart() {}
};

// Careful walk of `count` kept values from column bpos / code bit upos on.  bm/fl: this token's words, `fs` words
// apart; un: unary words `us` apart.  STRIDE: bytes per column on the emitter's side.
template <int T, int STRIDE, class Emit>
__device__ __forceinline__ void kv_rec_group_slow(const uint32_t* bm, const uint32_t* fl, int fs, const uint32_t* un, int us,
                                           int count, uint32_t& bpos, uint32_t& upos, uint32_t bpos_lim, uint32_t upos_lim,
                                           const uint32_t* lut, Emit& em, bool raw = false, uint32_t k0 = 0) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));
    for (int e = 0; e < count; ++e) {
        bool found = false;
        while (bpos < bpos_lim) {
            uint32_t w = bm[(bpos >> 5) * fs] << (bpos & 31);
            if (w) { bpos += __clz(w); found = true; break; }
            bpos = (bpos | 31u) + 1u;
        }
        if (!found) break;
        const uint32_t col = bpos;
        bpos += 1;
        uint32_t eb;
        if (raw) {                                           // exponents stored as bytes, value k at byte k
            const uint32_t k = k0 + (uint32_t)e;
            eb = ((un[(k >> 2) * us] >> (24 - 8 * (k & 3))) & 0xFFu) << 23;
        } else {
            int rank = 0;
            while (upos < upos_lim) {
                uint32_t v = un[(upos >> 5) * us] << (upos & 31);
                int avail = 32 - (int)(upos & 31);
                if (v) { int z = __clz(v); rank += z; upos += z + 1; break; }
                rank += avail;
                upos += avail;
            }
            eb = lut[rank & 255];
        }
        const uint32_t fword = fl[(e / PER) * fs];
        const uint32_t a = __funnelshift_l(fword, fword, (F * (e % PER)) & 31);
        em.direct(col * STRIDE, (a & MASK) | eb);
    }
}

// Walk of one record by one lane; `active` lanes emit, the others only keep the warp in step.
// bm_a / fl_a / un_a: shared addresses of this lane's first bitmap / field / unary word (words 128 bytes apart).
template <int T, int STRIDE, class Emit>
__device__ __forceinline__ void kv_rec_walk(const uint32_t* bmP, const uint32_t* flP, const uint32_t* unP, uint32_t lut_a,
                                               const uint32_t* lutP, int kept, int d, uint32_t una_bits, bool active, Emit& em) {
    constexpr int F = 8 - T, PER = 32 / F, NFW = kGroupCols / PER;
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));
    const uint32_t bm_a = smem_u32(bmP), un_a = smem_u32(unP);
    uint32_t fl_a = smem_u32(flP);
    uint32_t bpos = 0, upos = 0;
    const uint32_t bpos_lim = (uint32_t)d, upos_lim = (uint32_t)kDrUnaStage * 32u;
    const int n_groups = ceil_div(kept, kGroupCols);
    for (int grp = 0; grp < n_groups; ++grp) {
        const int cnt = min(kGroupCols, kept - grp * kGroupCols);
        const bool tail = cnt < kGroupCols;
        const uint32_t bpos0 = bpos, upos0 = upos;
        const uint32_t ba = bm_a + (bpos >> 5) * 128u;
        uint32_t bv = __funnelshift_l(dr_lds(ba + 128u), dr_lds(ba), bpos);
        const uint32_t x0 = bpos * STRIDE;
        uint32_t xa = x0;
        uint32_t fwd[NFW];
        fwd[0] = dr_lds(fl_a);
        if (NFW > 1) fwd[NFW - 1] = dr_lds(fl_a + 128u);
        uint32_t dry = 0, umax = 0;
        em.reset();
#pragma unroll
        for (int half = 0; half < kGroupCols / kGroupCodes; ++half) {
            const uint32_t ua = un_a + (upos >> 5) * 128u;
            uint32_t uv = __funnelshift_l(dr_lds(ua + 128u), dr_lds(ua), upos);
            uint32_t usum = 0;
            auto elem = [&](auto ec) {
                constexpr int e = decltype(ec)::value;
                const uint32_t s = __clz(bv);
                xa += s * STRIDE;
                bv = dr_shl(dr_shl(bv, s), 1);
                const uint32_t tt = __clz(uv);
                const uint32_t eb = dr_lds(lut_a + tt * 4u);
                uv = dr_shl(dr_shl(uv, tt), 1);
                usum += tt;
                const uint32_t fword = fwd[e / PER];
                const uint32_t a = __funnelshift_l(fword, fword, (F * (e % PER)) & 31);
                const bool valid = active && (!tail || e < cnt);
                em.template elem<e>(xa + e * STRIDE, (a & MASK) | eb, valid);
                if (tail && e < cnt) dry |= s | tt;
            };
            if (half == 0) {
                elem(std::integral_constant<int, 0>{}); elem(std::integral_constant<int, 1>{});
                elem(std::integral_constant<int, 2>{}); elem(std::integral_constant<int, 3>{});
            } else {
                elem(std::integral_constant<int, 4>{}); elem(std::integral_constant<int, 5>{});
                elem(std::integral_constant<int, 6>{}); elem(std::integral_constant<int, 7>{});
            }
            upos = min(upos + usum + kGroupCodes, upos_lim);
            umax = max(umax, usum);
        }
        const uint32_t adv = (xa - x0) / STRIDE;
        bpos = min(bpos + adv + kGroupCols, bpos_lim);
        if (!tail) dry = (adv + kGroupCols > 32u || umax + kGroupCodes > 32u) ? 32u : 0u;
        if (active) {
            if (dry & 32u) {                           // a window ran dry: redo this group one value at a time
                bpos = bpos0; upos = upos0;
                kv_rec_group_slow<T, STRIDE>(bmP, flP + grp * NFW * 32, 32, unP, 32, cnt, bpos, upos, bpos_lim, min(una_bits, upos_lim),
                                         lutP, em);
            } else {
                em.commit(cnt);
            }
        }
        fl_a += NFW * 128u;
    }
}

template <int T, int GQ>
__global__ void __launch_bounds__(kDrThreads) k_draft_attn_rec(KvGeom g, KvComp ck0, KvComp cv0, const uint16_t* __restrict__ qkv,
                                                           int qkv_stride, int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                           int n_chunks_alloc) {
    extern __shared__ __align__(16) uint8_t smem[];
    pdl_early<2>();
    pdl_wait();
    const int chunk = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    const int cur_len = st->len[seq] + st->inflight[seq] + 1;  // positions visible to the drafted token
    const int t0 = chunk * kDrTok;
    if (t0 >= cur_len) return;
    const int G = n_q / g.n_kv, d = g.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    qkv += (size_t)seq * qkv_stride;

    constexpr int kQStride = GQ * 4;                                          // bytes per column of the query tile
    float* q_s = reinterpret_cast<float*>(smem);                              // [d][GQ]
    float* sc_s = q_s + d * GQ;                                               // [GQ][64] scores -> probabilities
    float* ml_s = sc_s + GQ * kDrTok;                                         // [GQ][2]
    uint32_t* lut_s = reinterpret_cast<uint32_t*>(ml_s + 2 * GQ);             // [2][256] rank -> exponent << 23
    uint32_t* fix_s = lut_s + 512;                                            // [4 warps][wpt + 1][32]
    uint32_t* una_s = fix_s + 4 * (g.wpt + 1) * 32;                           // [4 warps][kDrUnaStage + 2][32]
    uint16_t* v_s = reinterpret_cast<uint16_t*>(una_s + 4 * (kDrUnaStage + 2) * 32);   // [64][d] bf16

    const float scale = rsqrtf((float)d);
    for (int i = tid; i < d * GQ; i += kDrThreads) {
        int col = i / GQ, gi = i % GQ;
        q_s[i] = gi < G ? bf16_bits_to_float(qkv[(size_t)(head * G + gi) * d + col]) : 0.f;
    }
    {
        const uint8_t *rk = of_seq(ck0.rank_to_exp, seq, g.seq_stride), *rv = of_seq(cv0.rank_to_exp, seq, g.seq_stride);
        for (int i = tid; i < 512; i += kDrThreads) lut_s[i] = (uint32_t)(i < 256 ? rk[i] : rv[i - 256]) << 23;
    }
    for (int i = tid; i < kDrTok * d / 2; i += kDrThreads) reinterpret_cast<uint32_t*>(v_s)[i] = 0u;

    // stage this warp's 32 records: warps 0,1 -> K of tokens t0 + 32 w .., warps 2,3 -> V of the same tokens
    const int kind = warp >> 1, tw = warp & 1;
    const int tok = t0 + tw * 32 + lane;
    const bool valid = tok < cur_len;
    const KvComp& c = kind ? cv0 : ck0;                      // sequence 0's; shifted to this sequence where used
    uint32_t* my_fix = fix_s + warp * (g.wpt + 1) * 32;
    uint32_t* my_una = una_s + warp * (kDrUnaStage + 2) * 32;
    {
        const uint32_t* fixed = of_seq(c.fixed, seq, g.seq_stride) + ((size_t)head * g.n_blocks + tok / 32) * g.wpt * 32;
        for (int w = 0; w < g.wpt; ++w) my_fix[w * 32 + lane] = fixed[w * 32 + lane];          // coalesced block copy
        my_fix[g.wpt * 32 + lane] = 0u;
    }
    const uint32_t* off = of_seq(c.off, seq, g.seq_stride) + (size_t)head * (g.max_seq + 1);
    const uint32_t* arena = of_seq(c.arena, seq, g.seq_stride) + (size_t)head * g.arena_words;
    uint32_t o0 = 0, n_una = 0;
    if (valid) { o0 = off[tok]; n_una = off[tok + 1] - o0; }
    const bool raw = (my_fix[lane] & kKvRawFlag) != 0;        // entry word 0 of this token's record
    const bool staged = n_una <= (uint32_t)kDrUnaStage && !raw;
    for (int w = 0; w < kDrUnaStage + 2; ++w) my_una[w * 32 + lane] = (staged && (uint32_t)w < n_una) ? arena[o0 + w] : 0u;
    __syncthreads();

    const uint32_t* lutP = lut_s + kind * 256;
    if (kind == 0) {
        RecEmitK<GQ> em;
        em.q_a = smem_u32(q_s);
        em.restart();
        kv_rec_walk<T, kQStride>(my_fix + g.e_words * 32 + lane, my_fix + (g.e_words + g.bm_words) * 32 + lane, my_una + lane, smem_u32(lutP), lutP, g.kept, d,
                                    n_una * 32u, valid && staged, em);
        if (valid && !staged) {                                               // very long record: walk it in place
            uint32_t bpos = 0, upos = 0;
            em.restart();
            for (int grp = 0; grp * kGroupCols < g.kept; ++grp)
                kv_rec_group_slow<T, kQStride>(my_fix + g.e_words * 32 + lane, my_fix + (g.e_words + g.bm_words + grp * (kGroupCols * (8 - T) / 32)) * 32 + lane, 32,
                                           arena + o0, 1, min(kGroupCols, g.kept - grp * kGroupCols), bpos, upos, (uint32_t)d,
                                           n_una * 32u, lutP, em, raw, (uint32_t)(grp * kGroupCols));
        }
#pragma unroll
        for (int gi = 0; gi < GQ; ++gi)
            if (gi < G) sc_s[gi * kDrTok + tw * 32 + lane] = valid ? em.acc[gi] * scale : -INFINITY;
    } else {
        RecEmitV em;
        em.row_a = smem_u32(v_s + (size_t)(tw * 32 + lane) * d);
        kv_rec_walk<T, 2>(my_fix + g.e_words * 32 + lane, my_fix + (g.e_words + g.bm_words) * 32 + lane, my_una + lane, smem_u32(lutP), lutP, g.kept, d,
                             n_una * 32u, valid && staged, em);
        if (valid && !staged) {
            uint32_t bpos = 0, upos = 0;
            for (int grp = 0; grp * kGroupCols < g.kept; ++grp)
                kv_rec_group_slow<T, 2>(my_fix + g.e_words * 32 + lane, my_fix + (g.e_words + g.bm_words + grp * (kGroupCols * (8 - T) / 32)) * 32 + lane, 32,
                                    arena + o0, 1, min(kGroupCols, g.kept - grp * kGroupCols), bpos, upos, (uint32_t)d,
                                    n_una * 32u, lutP, em, raw, (uint32_t)(grp * kGroupCols));
        }
    }
    __syncthreads();
    // chunk softmax statistics: warp w handles query heads w, w + 4
    for (int gi = warp; gi < G; gi += kDrThreads / 32) {
        float a = sc_s[gi * kDrTok + lane], b = sc_s[gi * kDrTok + 32 + lane];
        const float m = warp_max(fmaxf(a, b));
        a = expf(a - m);                                              // exp(-inf) = 0 for tokens beyond the end
        b = expf(b - m);
        sc_s[gi * kDrTok + lane] = a;
        sc_s[gi * kDrTok + 32 + lane] = b;
        const float l = warp_sum(a + b);
        if (lane == 0) { ml_s[gi * 2] = m; ml_s[gi * 2 + 1] = l; }
    }
    __syncthreads();
    // o[gi][dim] = sum_t p[gi][t] * v[t][dim]
    const int n_tok = min(kDrTok, cur_len - t0);
    for (int dim = tid; dim < d; dim += kDrThreads) {
        float acc[GQ];
#pragma unroll
        for (int gi = 0; gi < GQ; ++gi) acc[gi] = 0.f;
#pragma unroll 4
        for (int t = 0; t < n_tok; ++t) {
            const float v = bf16_bits_to_float(v_s[(size_t)t * d + dim]);
#pragma unroll
            for (int gi = 0; gi < GQ; ++gi)
                if (gi < G) acc[gi] = fmaf(sc_s[gi * kDrTok + t], v, acc[gi]);
        }
#pragma unroll
        for (int gi = 0; gi < GQ; ++gi)
            if (gi < G) sc.o[(((size_t)seq * n_q + head * G + gi) * n_chunks_alloc + chunk) * d + dim] = acc[gi];
    }
    if (tid < G) {
        const size_t pair = (size_t)seq * n_q + head * G + tid;
        sc.m[pair * n_chunks_alloc + chunk] = ml_s[tid * 2];
        sc.l[pair * n_chunks_alloc + chunk] = ml_s[tid * 2 + 1];
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int rps, int n_q, int d,
                      const DevState* st, int draft_mode, int draft_units, uint16_t* out, cudaStream_t s);

size_t draft_attn_rec_smem_bytes(const KvGeom& g, int gq) {
    return (size_t)g.d * gq * 4 + (size_t)gq * kDrTok * 4 + 2 * gq * 4 + 512 * 4 +
           (size_t)4 * (g.wpt + 1) * 32 * 4 + (size_t)4 * (kDrUnaStage + 2) * 32 * 4 + (size_t)kDrTok * g.d * 2 + 64;
}

int launch_draft_attn_rec(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                      int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    const int G = n_q / g.n_kv;
    if (G > kDrMaxGroup || g.d > 256 || g.d % 32) return CASS_ERR_UNSUPPORTED;
    const int n_chunks = ceil_div(g.max_seq, kDrTok);
    const int gq = G <= 4 ? 4 : 8;
    const size_t smem = draft_attn_rec_smem_bytes(g, gq);
    dim3 grid(n_chunks, g.n_kv, n_seq);
#define CASS_DR_LAUNCH(TT, GG)                                                                                         \
    do {                                                                                                             \
        static size_t attr = 0;                                                                                      \
        if (smem > attr) {                                                                                           \
            CASS_CUDA_CHECK(cudaFuncSetAttribute((k_draft_attn_rec<TT, GG>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
            attr = smem;                                                                                             \
        }                                                                                                            \
        CASS_PDL_LAUNCH((k_draft_attn_rec<TT, GG>), grid, dim3(kDrThreads), smem, s, g, ck, cv, qkv, qkv_stride, n_q, st, sc, n_chunks);     \
    } while (0)
    if (g.t == 4 && gq == 4) CASS_DR_LAUNCH(4, 4);
    else if (g.t == 4) CASS_DR_LAUNCH(4, 8);
    else if (g.t == 0 && gq == 4) CASS_DR_LAUNCH(0, 4);
    else if (g.t == 0) CASS_DR_LAUNCH(0, 8);
    else return CASS_ERR_UNSUPPORTED;
#undef CASS_DR_LAUNCH
    CASS_LAUNCH_CHECK();
    return launch_attn_merge(sc, n_chunks, kDrTok, n_seq, 1, n_q, g.d, st, 1, 0, out, s);
}

}  // namespace cass
