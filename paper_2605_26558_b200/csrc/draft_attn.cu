// Draft decode attention over the compressed KV cache (Sec. 4.1 draft inference; KV speculation data of
// Sec. 4.2): grouped-query attention of one query row per sequence, split over the sequence with a log-sum-exp
// merge.  One CTA = one (KV head, run of 32..256 tokens); it walks its run in passes of 32 tokens (one block of the
// cache's fixed part) with a running softmax.  Inside a pass a record (token, K|V) is decoded by d/32 lanes side by
// side, one per 32-channel slice: warp (kind, slice) has lane = token, so every stream read is conflict free; a
// slice enters the record through its bitmap word, the popcount of the lower bitmap words (field index) and, for
// Cassandra-1 records, the code-bit offset its entry word holds -- the software form of the per-section cursors
// of Sec. 5.3.  K slices leave partial dot products with the group's query heads, V slices a dense bf16 tile; then
// the pass's probabilities multiply the tile.
#include <type_traits>

#include "kernels.cuh"

namespace cass {

constexpr int kDaSub = 32;                    // tokens per pass
constexpr int kDaUnaStageMax = 32;            // staged exponent words per token (records up to 1023 code bits fit)
constexpr int kMaxGroup = 8;                  // query heads per KV head

__device__ __forceinline__ uint32_t da_shl(uint32_t v, uint32_t s) {          // shift counts >= 32 give 0
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
}
__device__ __forceinline__ uint32_t da_bfind(uint32_t v) {                    // most significant set bit, 0xFFFFFFFF if none
    uint32_t r;
    asm("bfind.u32 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t da_lds(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// What happens to a decoded value of channel `col` (0..31 inside the slice).
// K: multiply with the query tile q_s[channel][GQ]; V: store into the token's dense row.
template <int GQ>
struct EmitK {
    float acc[GQ];
    uint32_t q_a;                        // shared address of the slice's first channel in the query tile
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int i = 0; i < GQ; ++i) acc[i] = 0.f;
    }
    __device__ __forceinline__ void put(uint32_t col, float w) {
        float4 a;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "r"(q_a + col * (GQ * 4)));
        acc[0] = fmaf(w, a.x, acc[0]); acc[1] = fmaf(w, a.y, acc[1]); acc[2] = fmaf(w, a.z, acc[2]); acc[3] = fmaf(w, a.w, acc[3]);
        if constexpr (GQ > 4) {
            float4 b;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+16];" : "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "r"(q_a + col * (GQ * 4)));
            acc[4] = fmaf(w, b.x, acc[4]); acc[5] = fmaf(w, b.y, acc[5]); acc[6] = fmaf(w, b.z, acc[6]); acc[7] = fmaf(w, b.w, acc[7]);
        }
    }
};

struct EmitV {
    uint32_t row_a;                      // shared address of the slice's first channel in the token's dense row
    __device__ __forceinline__ void init() {}
    __device__ __forceinline__ void put(uint32_t col, float w) {
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(row_a + col * 2u), "h"((uint16_t)(__float_as_uint(w) >> 16)));
    }
};

// ---- Cassandra-1 slice -------------------------------------------------------------------------------------------
// Careful walk of a slice's values [e_from, n): any codeword length, raw exponents too.  `un` points at the record's
// first exponent word, words `us` apart.
// The emitter travels by value (in registers): a reference would pin it to local memory in the fast path too.
template <int T, class Emit>
__device__ __noinline__ Emit kv_slice_slow(uint32_t bv, const uint32_t* fl, uint32_t fi, const uint32_t* un, int us,
                                           uint32_t upos, uint32_t upos_lim, bool raw, int n, const uint32_t* lut, Emit em) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));
    for (int e = 0; e < n && bv; ++e, ++fi) {
        const uint32_t p = da_bfind(bv);
        bv &= ~(1u << p);
        uint32_t eb;
        if (raw) {
            eb = ((un[(fi >> 2) * us] >> (24 - 8 * (fi & 3))) & 0xFFu) << 23;
        } else {
            int rank = 0;
            while (upos < upos_lim) {
                const uint32_t v = un[(upos >> 5) * us] << (upos & 31);
                const int avail = 32 - (int)(upos & 31);
                if (v) { const int z = __clz(v); rank += z; upos += z + 1; break; }
                rank += avail;
                upos += avail;
            }
            eb = lut[rank & 255];
        }
        const uint32_t fword = fl[(fi / PER) * 32];
        const uint32_t a = __funnelshift_l(fword, fword, (F * (fi % PER)) & 31);
        em.put(31u - p, __uint_as_float((a & MASK) | eb));
    }
    return em;
}

// One slice of a Cassandra-1 record per lane.  B: the slice's bitmap word; fi: index of its first field; upos: bit
// offset of its first codeword in the staged stream (words 128 bytes apart from un_a); n: its kept values (0 for
// lanes that only keep the warp in step).  Groups of 4 values = one 32-bit code window; a window that runs dry sends
// that lane through the careful walk for the rest of its slice.
template <int T, class Emit>
__device__ __forceinline__ void kv_slice_walk(uint32_t B, uint32_t fi, uint32_t upos, int n, uint32_t fl_a, const uint32_t* flP,
                                              uint32_t un_a, const uint32_t* unP, uint32_t upos_lim, uint32_t lut_a,
                                              const uint32_t* lutP, Emit& em) {
    constexpr int F = 8 - T, PER = 32 / F, GS = kGroupCodes;
    static_assert(GS <= PER, "a group's fields lie in two consecutive words");
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));
    const int n_groups = ceil_div(__reduce_max_sync(0xffffffffu, n), GS);
    uint32_t bv = B;
    bool slow = false;
    for (int grp = 0; grp < n_groups; ++grp) {
        const int rem = n - grp * GS;                                         // values this lane still has (may be <= 0)
        const uint32_t fw_a = fl_a + (fi / PER) * 128u, j0 = fi % PER;
        const uint32_t f0 = da_lds(fw_a), f1 = da_lds(fw_a + 128u);
        const uint32_t bv0 = bv, upos0 = upos;
        const uint32_t ua = un_a + (upos >> 5) * 128u;
        uint32_t uv = __funnelshift_l(da_lds(ua + 128u), da_lds(ua), upos);                // 32 code bits from upos on
        uint32_t la = lut_a + 124u, q = 0, dry = 0;
        uint32_t cols[GS], wbs[GS];
#pragma unroll
        for (int e = 0; e < GS; ++e) {
            const uint32_t p = da_bfind(bv);
            bv &= ~da_shl(1u, p);
            q = da_bfind(uv);
            const uint32_t eb = da_lds(la - (q & 31u) * 4u);                               // lut[previous - q - 1]
            la = lut_a - 4u + (q & 31u) * 4u;
            uv &= ~da_shl(1u, q);
            const uint32_t jj = j0 + e;                                                    // field jj of the two words
            const uint32_t fword = jj >= (uint32_t)PER ? f1 : f0;
            const uint32_t a = __funnelshift_l(fword, fword, (F * jj) & 31);
            cols[e] = 31u - (p & 31u);
            wbs[e] = (a & MASK) | eb;
            if (e < rem) dry |= q;                                                         // sign bit set: the window ran dry
        }
        upos = min(upos + 32u - (q & 31u), upos_lim);
        if (rem > 0 && !slow) {
            if ((int32_t)dry < 0) {
                slow = true;                             // finish this slice one value at a time, from the group's start
                em = kv_slice_slow<T>(bv0, flP, fi, unP, 32, upos0, upos_lim, false, rem, lutP, em);
            } else {
#pragma unroll
                for (int e = 0; e < GS; ++e)
                    if (e < rem) em.put(cols[e], __uint_as_float(wbs[e]));
            }
        }
        fi += GS;
    }
}

// ---- Cassandra-2 slice: fields = sign + magnitude, one shared exponent per slice ------------------------------------
// vlut: float value of every field pattern, +-(magnitude << t); scale = 2^(E - 133).
template <int T, class Emit>
__device__ __forceinline__ void kv_slice_walk_mx(uint32_t B, uint32_t fi, int n, uint32_t fl_a, uint32_t vlut_a, float scale,
                                                 Emit& em) {
    constexpr int F = 8 - T, PER = 32 / F;
    const int n_groups = ceil_div(__reduce_max_sync(0xffffffffu, n), 4);
    uint32_t bv = B;
    for (int grp = 0; grp < n_groups; ++grp) {
        const int rem = n - grp * 4;
        const uint32_t fw_a = fl_a + (fi / PER) * 128u;
        const uint32_t comb = __funnelshift_l(da_lds(fw_a + 128u), da_lds(fw_a), (F * (fi % PER)) & 31);   // 4 fields from the top
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t p = da_bfind(bv);
            bv &= ~da_shl(1u, p);
            const uint32_t f = (comb >> (32 - F * (e + 1))) & ((1u << F) - 1u);
            const float v = __uint_as_float(da_lds(vlut_a + f * 4u)) * scale;
            if (e < rem) em.put(31u - (p & 31u), v);
        }
        fi += 4;
    }
}

// 4-byte asynchronous copy global -> shared; `take` false writes a zero instead (nothing is read).
__device__ __forceinline__ void da_cp_async4(uint32_t dst, const void* src, bool take) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(take ? 4 : 0) : "memory");
}
__device__ __forceinline__ void da_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void da_cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <int MODE, int T, int GQ>
__global__ void __launch_bounds__(512, 2) k_draft_attn(KvGeom g, KvComp ck0, KvComp cv0, const uint16_t* __restrict__ qkv,
                                                       int qkv_stride, int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                       int n_chunks_alloc, int stage, uint16_t* __restrict__ out) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ int s_last;
    pdl_early<2>();
    pdl_wait();
    const int head = blockIdx.y, seq = blockIdx.z;
    const int cur_len = st->len[seq] + st->inflight[seq] + 1;  // positions visible to the drafted token
    const int tpc = da_tokens_per_cta(cur_len, g.n_kv * (int)gridDim.z);
    const int t_begin = blockIdx.x * tpc;
    if (t_begin >= cur_len) return;
    const int t_end = min(cur_len, t_begin + tpc);
    const int G = n_q / g.n_kv, d = g.d, S = d / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_thr = blockDim.x;
    qkv += (size_t)seq * qkv_stride;

    const int vrow = d + 2;                                                   // halfwords per row of the V tile (padded)
    const int fsz = (g.wpt + 2) * 32, usz = (stage + 2) * 32;
    float* q_s = reinterpret_cast<float*>(smem);                              // [d][GQ]
    float* part_s = q_s + d * GQ;                                             // [S][GQ][32] partial q.k of the slices
    float* sc_s = part_s + S * GQ * kDaSub;                                   // [32][GQ] probabilities of the pass
    float* run_s = sc_s + GQ * kDaSub;                                        // [GQ][4]: running max, running sum, rescale factor
    uint32_t* lut_s = reinterpret_cast<uint32_t*>(run_s + 4 * GQ);            // mode 1: [2][256] rank -> exponent << 23; mode 2: [256] field values
    uint32_t* meta_s = lut_s + 512;                                           // [2 buffers][2 kinds][34]: arena offsets of 32 tokens + the next
    uint32_t* fix_s = meta_s + 2 * 2 * 34;                                    // [2 buffers][2 kinds][wpt + 2][32]
    uint32_t* una_s = fix_s + 2 * 2 * fsz;                                    // [2 buffers][2 kinds][stage + 2][32] (mode 1)
    uint16_t* v_s = reinterpret_cast<uint16_t*>(una_s + (MODE == 1 ? 2 * 2 * usz : 0));   // [32][vrow] bf16

    const float scale = rsqrtf((float)d);
    for (int i = tid; i < d * GQ; i += n_thr) {
        const int col = i / GQ, gi = i % GQ;
        q_s[i] = gi < G ? bf16_bits_to_float(qkv[(size_t)(head * G + gi) * d + col]) : 0.f;
    }
    if (MODE == 1) {
        const uint8_t *rk = of_seq(ck0.rank_to_exp, seq, g.seq_stride), *rv = of_seq(cv0.rank_to_exp, seq, g.seq_stride);
        for (int i = tid; i < 512; i += n_thr) lut_s[i] = (uint32_t)(i < 256 ? rk[i] : rv[i - 256]) << 23;
    } else {
        constexpr int NF = 1 << (8 - T);
        for (int i = tid; i < NF; i += n_thr) {
            const float mag = (float)((i & (NF / 2 - 1)) << T);
            lut_s[i] = __float_as_uint((i & (NF / 2)) ? -mag : mag);
        }
    }
    if (tid < 4 * GQ) run_s[tid] = (tid & 3) == 0 ? -INFINITY : 0.f;
    for (int i = tid; i < 2 * 2 * 2 * 32; i += n_thr) fix_s[(i / 64) * fsz + g.wpt * 32 + (i % 64)] = 0u;   // the two slack rows of every block stay zero
    if (MODE == 1) for (int i = tid; i < 2 * 2 * 2 * 32; i += n_thr) una_s[(i / 64) * usz + stage * 32 + (i % 64)] = 0u;

    const int kind = warp / S, slice = warp % S;                              // warps 0..S-1: K slices, S..2S-1: V slices
    const uint32_t* fixed_kv[2] = {of_seq(ck0.fixed, seq, g.seq_stride) + (size_t)head * g.n_blocks * g.wpt * 32,
                                   of_seq(cv0.fixed, seq, g.seq_stride) + (size_t)head * g.n_blocks * g.wpt * 32};
    const uint32_t* off_kv[2] = {of_seq(ck0.off, seq, g.seq_stride) + (size_t)head * (g.max_seq + 1),
                                 of_seq(cv0.off, seq, g.seq_stride) + (size_t)head * (g.max_seq + 1)};
    const uint32_t* arena_kv[2] = {of_seq(ck0.arena, seq, g.seq_stride) + (size_t)head * g.arena_words,
                                   of_seq(cv0.arena, seq, g.seq_stride) + (size_t)head * g.arena_words};
    const int n_warps = n_thr / 32;

    // Staging runs ahead of the decode through asynchronous copies: the arena offsets of a pass two passes early, its
    // fixed-part blocks and exponent words one pass early, into the buffer the pass before the last has left.  A warp
    // copies whole rows (word w of the 32 tokens), lane = token.
    auto stage_meta = [&](int t0, int buf) {               // offsets off[t0 .. t0 + 32] of both kinds
        if (MODE == 1 && warp < 2) {
            const bool in_run = t0 < t_end;
            const bool take = in_run && t0 + lane <= cur_len;
            da_cp_async4(smem_u32(meta_s + (buf * 2 + warp) * 34 + lane), off_kv[warp] + (take ? t0 + lane : 0), take);
            if (lane == 0) {
                const bool take2 = in_run && t0 + 32 <= cur_len;
                da_cp_async4(smem_u32(meta_s + (buf * 2 + warp) * 34 + 32), off_kv[warp] + (take2 ? t0 + 32 : 0), take2);
            }
        }
    };
    auto stage_records = [&](int t0, int buf) {
        if (t0 >= t_end) return;
        const size_t blk = (size_t)(t0 / 32) * g.wpt * 32;
        for (int row = warp; row < 2 * g.wpt; row += n_warps) {
            const int kd = row >= g.wpt, w = row - kd * g.wpt;
            da_cp_async4(smem_u32(fix_s + (buf * 2 + kd) * fsz + w * 32 + lane), fixed_kv[kd] + blk + w * 32 + lane, true);
        }
        if (MODE == 1) {
            const bool tok_ok = t0 + lane < cur_len;
            uint32_t o0[2], nw[2];
#pragma unroll
            for (int kd = 0; kd < 2; ++kd) {
                const uint32_t* m = meta_s + (buf * 2 + kd) * 34 + lane;
                o0[kd] = m[0];
                nw[kd] = m[1] - m[0];
                if (!tok_ok || nw[kd] > (uint32_t)stage) nw[kd] = 0;          // longer records are read in place
            }
            for (int row = warp; row < 2 * stage; row += n_warps) {
                const int kd = row >= stage, w = row - kd * stage;
                const bool take = (uint32_t)w < nw[kd];
                da_cp_async4(smem_u32(una_s + (buf * 2 + kd) * usz + w * 32 + lane), arena_kv[kd] + (take ? o0[kd] + w : 0), take);
            }
        }
    };
    stage_meta(t_begin, 0);
    stage_meta(t_begin + kDaSub, 1);
    da_cp_async_wait_all();
    __syncthreads();
    stage_records(t_begin, 0);
    da_cp_async_wait_all();
    __syncthreads();

    float o_acc[GQ];
#pragma unroll
    for (int gi = 0; gi < GQ; ++gi) o_acc[gi] = 0.f;

    int pass = 0;
    for (int t0 = t_begin; t0 < t_end; t0 += kDaSub, ++pass) {
        const int buf = pass & 1;
        stage_records(t0 + kDaSub, buf ^ 1);               // the next pass's records travel while this pass is decoded
        // ---- decode: warp (kind, slice), lane = token ----
        if (warp < 2 * S) {
            const int tok = t0 + lane;
            const bool valid = tok < cur_len;
            const uint32_t* fx = fix_s + (buf * 2 + kind) * fsz + lane;          // word w of this token at fx[w * 32]
            const int bm0 = MODE == 1 ? g.e_words : 0;
            const uint32_t B = fx[(bm0 + slice) * 32];
            uint32_t fi = 0;
            for (int s2 = 0; s2 < slice; ++s2) fi += __popc(fx[(bm0 + s2) * 32]);
            const int n = valid ? __popc(B) : 0;
            const uint32_t fl_a = smem_u32(fx + (bm0 + g.bm_words) * 32);
            EmitK<GQ> ek;
            EmitV ev;
            ek.q_a = smem_u32(q_s + (size_t)slice * 32 * GQ);
            ev.row_a = smem_u32(v_s + (size_t)lane * vrow + slice * 32);
            ek.init();
            if (kind == 1) {                              // a V lane owns its token's 32 channels of the tile: clear them first
#pragma unroll
                for (int i = 0; i < 16; ++i) asm volatile("st.shared.u32 [%0], %1;" ::"r"(ev.row_a + 4u * i), "r"(0u));
            }
            if (MODE == 1) {
                const uint32_t e0 = fx[0];
                const bool raw = (e0 & kKvRawFlag) != 0;
                const uint32_t upos = slice == 0 ? 0u : (fx[((slice - 1) / 3) * 32] >> (20 - 10 * ((slice - 1) % 3))) & 0x3FFu;
                const uint32_t* m = meta_s + (buf * 2 + kind) * 34 + lane;
                const uint32_t o0 = m[0], nw = valid ? m[1] - m[0] : 0u;
                const bool staged = nw <= (uint32_t)stage;
                const bool fast = valid && !raw && staged;
                const uint32_t* lutP = lut_s + kind * 256;
                const uint32_t* unP = una_s + (buf * 2 + kind) * usz + lane;
                const uint32_t upos_lim = (uint32_t)stage * 32u;
                if (kind == 0) kv_slice_walk<T>(B, fi, upos, fast ? n : 0, fl_a, fx + (bm0 + g.bm_words) * 32, smem_u32(unP), unP, upos_lim,
                                                smem_u32(lutP), lutP, ek);
                else kv_slice_walk<T>(B, fi, upos, fast ? n : 0, fl_a, fx + (bm0 + g.bm_words) * 32, smem_u32(unP), unP, upos_lim,
                                      smem_u32(lutP), lutP, ev);
                if (valid && !fast) {                     // raw exponents, or a record longer than the staging: read it in place
                    const uint32_t* un = arena_kv[kind] + o0;
                    if (kind == 0) ek = kv_slice_slow<T>(B, fx + (bm0 + g.bm_words) * 32, fi, un, 1, upos, nw * 32u, raw, n, lutP, ek);
                    else ev = kv_slice_slow<T>(B, fx + (bm0 + g.bm_words) * 32, fi, un, 1, upos, nw * 32u, raw, n, lutP, ev);
                }
            } else {
                const uint32_t xw = fx[(g.bm_words + g.f_words + slice / 4) * 32];
                const uint32_t eb = (xw >> (24 - 8 * (slice % 4))) & 0xFFu;
                const float sc2 = __uint_as_float(eb >= 7u ? (eb - 6u) << 23 : 0u);     // 2^(E - 133)
                if (kind == 0) kv_slice_walk_mx<T>(B, fi, n, fl_a, smem_u32(lut_s), sc2, ek);
                else kv_slice_walk_mx<T>(B, fi, n, fl_a, smem_u32(lut_s), sc2, ev);
            }
            if (kind == 0) {
#pragma unroll
                for (int gi = 0; gi < GQ; ++gi) part_s[(slice * GQ + gi) * kDaSub + lane] = ek.acc[gi];
            }
        }
        __syncthreads();
        // this pass's offsets are no longer needed: fetch those of the pass after the next into their place
        stage_meta(t0 + 2 * kDaSub, buf);
        // ---- running softmax: warp gi handles query head gi of the group, lane = token ----
        for (int gi = warp; gi < G; gi += n_thr / 32) {
            float sdot = 0.f;
            for (int s2 = 0; s2 < S; ++s2) sdot += part_s[(s2 * GQ + gi) * kDaSub + lane];
            const bool valid = t0 + lane < cur_len;
            const float sv = valid ? sdot * scale : -INFINITY;
            const float m_old = run_s[gi * 4], l_old = run_s[gi * 4 + 1];
            const float m_new = fmaxf(m_old, warp_max(sv));                   // finite: the pass has at least one visible token
            const float pr = valid ? expf(sv - m_new) : 0.f;
            const float alpha = expf(m_old - m_new);                          // exp(-inf) = 0 on the first pass
            sc_s[lane * GQ + gi] = pr;
            const float l_new = l_old * alpha + warp_sum(pr);
            __syncwarp();
            if (lane == 0) { run_s[gi * 4] = m_new; run_s[gi * 4 + 1] = l_new; run_s[gi * 4 + 2] = alpha; }
        }
        __syncthreads();
        // ---- o[gi][dim] = alpha o + sum_t p[gi][t] v[t][dim]; thread = dim ----
        if (tid < d) {
            const int n_tok = min(kDaSub, cur_len - t0);
#pragma unroll
            for (int gi = 0; gi < GQ; ++gi) o_acc[gi] *= run_s[gi * 4 + 2];
#pragma unroll 4
            for (int t = 0; t < n_tok; ++t) {
                const float v = bf16_bits_to_float(v_s[(size_t)t * vrow + tid]);
                const float4 pa = *reinterpret_cast<const float4*>(sc_s + t * GQ);         // the pass's probabilities [token][GQ]
                o_acc[0] = fmaf(pa.x, v, o_acc[0]); o_acc[1] = fmaf(pa.y, v, o_acc[1]);
                o_acc[2] = fmaf(pa.z, v, o_acc[2]); o_acc[3] = fmaf(pa.w, v, o_acc[3]);
                if constexpr (GQ > 4) {
                    const float4 pb = *reinterpret_cast<const float4*>(sc_s + t * GQ + 4);
                    o_acc[4] = fmaf(pb.x, v, o_acc[4]); o_acc[5] = fmaf(pb.y, v, o_acc[5]);
                    o_acc[6] = fmaf(pb.z, v, o_acc[6]); o_acc[7] = fmaf(pb.w, v, o_acc[7]);
                }
            }
        }
        da_cp_async_wait_all();                            // the next pass's records (and the offsets beyond) have landed
        __syncthreads();                                   // and the pass's tile and probabilities are free again
    }
    const int chunk = blockIdx.x;
    const int n_act = ceil_div(cur_len, tpc);                                 // CTAs of this (sequence, head) that have tokens
    if (n_act == 1) {
        // the whole visible range in one CTA: normalise and write the output rows directly
        if (tid < d) {
#pragma unroll
            for (int gi = 0; gi < GQ; ++gi)
                if (gi < G) out[((size_t)seq * n_q + head * G + gi) * d + tid] = float_to_bf16_bits(o_acc[gi] / run_s[gi * 4 + 1]);
        }
        return;
    }
    if (tid < d) {
#pragma unroll
        for (int gi = 0; gi < GQ; ++gi)
            if (gi < G) sc.o[(((size_t)seq * n_q + head * G + gi) * n_chunks_alloc + chunk) * d + tid] = o_acc[gi];
    }
    if (tid < G) {
        const size_t pair = (size_t)seq * n_q + head * G + tid;
        sc.m[pair * n_chunks_alloc + chunk] = run_s[tid * 4];
        sc.l[pair * n_chunks_alloc + chunk] = run_s[tid * 4 + 1];
    }
    // ---- the CTA that finishes last merges the runs of its (sequence, head): a fixed order, whoever does it ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int* cnt = sc.cnt + seq * g.n_kv + head;
        const int done = atomicAdd(cnt, 1);
        s_last = done == n_act - 1;
        if (s_last) *cnt = 0;                                                 // ready for the next launch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // warp gi: weights of query head gi's runs (lane-parallel over the runs); then thread (gi, dim) adds the runs in order
    float* w_s = reinterpret_cast<float*>(fix_s);                             // [G][n_act] weights e^{m_c - M} (the record buffers are free; size checked at launch)
    float* L_s = sc_s;                                                        // [GQ]
    for (int gi = warp; gi < G; gi += n_thr / 32) {
        const size_t pair = (size_t)seq * n_q + head * G + gi;
        const float* mp = sc.m + pair * n_chunks_alloc;
        const float* lp = sc.l + pair * n_chunks_alloc;
        float M = -INFINITY;
        for (int c = lane; c < n_act; c += 32) M = fmaxf(M, __ldcg(mp + c));
        M = warp_max(M);
        float L = 0.f;
        for (int c0 = 0; c0 < n_act; c0 += 32) {          // sums of 32 runs at a time, in run order
            const int c = c0 + lane;
            float w = 0.f, wl = 0.f;
            if (c < n_act) { w = expf(__ldcg(mp + c) - M); wl = w * __ldcg(lp + c); w_s[gi * n_act + c] = w; }
            L += warp_sum(wl);
        }
        if (lane == 0) L_s[gi] = L;
    }
    __syncthreads();
    for (int i = tid; i < G * d; i += n_thr) {
        const int gi = i / d, dim = i % d;
        const float* op = sc.o + ((size_t)seq * n_q + head * G + gi) * n_chunks_alloc * d + dim;
        float acc = 0.f;
#pragma unroll 4
        for (int c = 0; c < n_act; ++c) acc = fmaf(w_s[gi * n_act + c], __ldcg(op + (size_t)c * d), acc);
        out[((size_t)seq * n_q + head * G + gi) * d + dim] = float_to_bf16_bits(acc / L_s[gi]);
    }
}

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
    if (draft_units > 0) chunk_tokens = da_tokens_per_cta(vis, draft_units);  // runs whose length follows the visible length
    if (draft_units < 0) chunk_tokens = tc_run_tokens(vis, -draft_units);     // the same for the dense-tile kernel
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

static int draft_attn_stage(const KvGeom& g) { return g.rec_words_max < kDaUnaStageMax ? g.rec_words_max : kDaUnaStageMax; }

size_t draft_attn_smem_bytes(const KvGeom& g, int gq) {
    const int S = g.d / 32, stage = draft_attn_stage(g);
    return (size_t)g.d * gq * 4 + (size_t)S * gq * kDaSub * 4 + (size_t)gq * kDaSub * 4 + 4 * gq * 4 + 512 * 4 + 2 * 2 * 34 * 4 +
           (size_t)4 * (g.wpt + 2) * 32 * 4 + (g.mode == 1 ? (size_t)4 * (stage + 2) * 32 * 4 : 0) +
           (size_t)kDaSub * (g.d + 2) * 2 + 64;
}

// Cassandra-1 records go to the dense-tile kernel (draft_attn_tc.cu: whole record per lane, products on mma.sync) where
// its shape limits hold; Cassandra-2 records, and the shapes it leaves out, take the slice-parallel kernel below.
bool draft_attn_tc_supported(const KvGeom& g, int n_q);
int launch_draft_attn_tc(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                         int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s);

int launch_draft_attn(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                      int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    if (draft_attn_tc_supported(g, n_q)) {
        const int rc = launch_draft_attn_tc(g, ck, cv, qkv, qkv_stride, n_q, n_seq, st, sc, out, s);
        if (rc != CASS_ERR_UNSUPPORTED) return rc;
    }
    const int G = n_q / g.n_kv;
    if (G > kMaxGroup || g.d > 256 || g.d % 32) return CASS_ERR_UNSUPPORTED;
    const int gq = G <= 4 ? 4 : 8;
    // the most CTAs a head can need: runs of 32 tokens while that keeps the grid below the target, of 256 at most
    int n_chunks = 592 / (g.n_kv * n_seq) + 1;
    if (ceil_div(g.max_seq, 256) > n_chunks) n_chunks = ceil_div(g.max_seq, 256);
    if (ceil_div(g.max_seq, kDaSub) < n_chunks) n_chunks = ceil_div(g.max_seq, kDaSub);
    if (G * n_chunks > 4 * (g.wpt + 2) * 32) return CASS_ERR_UNSUPPORTED;        // the merge keeps one weight per (query head, run) in shared memory
    const size_t smem = draft_attn_smem_bytes(g, gq);
    const int stage = draft_attn_stage(g);
    const int threads = 2 * (g.d / 32) * 32;
    dim3 grid(n_chunks, g.n_kv, n_seq);
#define CASS_DA_LAUNCH(MM, TT, GG)                                                                                     \
    do {                                                                                                             \
        static size_t attr = 0;                                                                                      \
        if (smem > attr) {                                                                                           \
            CASS_CUDA_CHECK(cudaFuncSetAttribute((k_draft_attn<MM, TT, GG>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
            attr = smem;                                                                                             \
        }                                                                                                            \
        CASS_PDL_LAUNCH((k_draft_attn<MM, TT, GG>), grid, dim3(threads), smem, s, g, ck, cv, qkv, qkv_stride, n_q, st, sc, n_chunks, stage, out); \
    } while (0)
#define CASS_DA_LAUNCH_T(MM)                                                                                          \
    do {                                                                                                             \
        if (g.t == 4 && gq == 4) CASS_DA_LAUNCH(MM, 4, 4);                                                           \
        else if (g.t == 4) CASS_DA_LAUNCH(MM, 4, 8);                                                                 \
        else if (g.t == 0 && gq == 4) CASS_DA_LAUNCH(MM, 0, 4);                                                      \
        else if (g.t == 0) CASS_DA_LAUNCH(MM, 0, 8);                                                                 \
        else return CASS_ERR_UNSUPPORTED;                                                                            \
    } while (0)
    if (g.mode == 2) CASS_DA_LAUNCH_T(2);
    else CASS_DA_LAUNCH_T(1);
#undef CASS_DA_LAUNCH_T
#undef CASS_DA_LAUNCH
    CASS_LAUNCH_CHECK();
    return CASS_OK;                                       // the last CTA of every (sequence, head) has merged its runs
}

}  // namespace cass
