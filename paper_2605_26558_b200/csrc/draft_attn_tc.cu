// Draft decode attention over the compressed KV cache, Cassandra-1 and Cassandra-2 records (Sec. 4.1 draft inference; KV speculation data of
// Sec. 4.2), dense-tile form: the decoders feed matrix units, as the paper's decoder array feeds the tensor cores
// (Sec. 5.1, 5.2).  One CTA = one (KV head, run of 64-token chunks).  Per chunk, warps 0-1 decode the K records of 32 tokens each
// (lane = token, the whole record by one lane) into a dense bf16 tile [token][channel] in shared memory, pruned channels
// zero; warps 2-3 do the same for the V records.  Then q.K^T for all query heads of the group and P.V are small
// mma.sync products over the two tiles (the group's <= 8 query heads are the N = 8 operand).  A decoded value costs its
// bit searches, one table look-up and one 16-bit store: no multiply, no gather of q, and the probabilities meet the
// values on the tensor pipe.  P is split into two bf16 terms (p = hi + lo) so that the product keeps fp32-level
// accuracy; K, V and q are bf16 by definition, so the operands are exact.
// Records are walked like the weight streams: 8 kept values per 32-bit bitmap window, 4 codewords per 32-bit unary
// window, positions by bfind with the used bit cleared; a careful walk redoes the rare group that does not fit its
// windows and reads records with raw exponents or more code words than the staging holds.
// Decoding a record with d/32 lanes (one per 32-channel slice, 16 warps per CTA) into the same tiles was measured and
// dropped: 11.6 / 27.7 / 155 us at 600 / 4096 / 32768 positions against 11.0 / 16.7 / 75.4 us for the whole record per
// lane -- the slices' uneven value counts and per-slice entry cost more than the shorter chains and the extra warps win.
#include <type_traits>

#include "kernels.cuh"

namespace cass {

constexpr int kTcTok = kAttnChunk;            // tokens per CTA
constexpr int kTcThreads = 128;
// Staged exponent words per token: room for 5 code bits per kept value (a typical record takes 2-3), the whole code
// budget at most; longer records and records with raw exponents are read in place.  A warp's staging has two rows more:
// a window reads the word of its cursor and the next.
__host__ __device__ inline int tc_una_stage(const KvGeom& g) {
    int w = ceil_div(5 * g.kept, 32);
    if (w > g.rec_words_max) w = g.rec_words_max;
    return w < 4 ? 4 : w;
}
constexpr int kTcHeads = 8;                   // query heads per KV head the N = 8 operand holds
constexpr int kTcPad = 8;                     // halfwords of padding per tile row: rows 16 bytes apart modulo 128

__device__ __forceinline__ uint32_t tc_shl(uint32_t v, uint32_t s) {          // shift counts >= 32 give 0
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
}
__device__ __forceinline__ uint32_t tc_bfind(uint32_t v) {                    // most significant set bit, 0xFFFFFFFF if none
    uint32_t r;
    asm("bfind.u32 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t tc_lds(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint32_t tc_lds_off(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
__device__ __forceinline__ uint32_t tc_mad(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ void tc_sts16(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((uint16_t)v));
}
__device__ __forceinline__ void tc_ldmatrix_x4(uint32_t (&r)[4], uint32_t a) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void tc_ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t a) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void tc_ldmatrix_x2(uint32_t (&r)[2], uint32_t a) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(a));
}
// D (16 x 8, fp32) += A (16 x 16, bf16, row-major fragment) * B (16 x 8, bf16, column-major fragment)
__device__ __forceinline__ void tc_mma(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Careful walk of the kept values k0 .. k0 + count - 1 of one record from column bpos / code bit upos on: any gap, any
// codeword length, bounded by the record.  bm / fl: this token's bitmap and field words (32 words apart); un: its
// exponent words, `us` words apart (code bits, or raw exponent bytes when `raw`).  r2e: rank -> exponent (global table).
// Values go to the token's dense row at shared address row_a; nothing is stored beyond channel d - 1.
template <int T>
__device__ __noinline__ void tc_walk_slow(const uint32_t* bm, const uint32_t* fl, const uint32_t* un, int us, bool raw, int k0, int count,
                                          uint32_t bpos, uint32_t upos, uint32_t d, uint32_t upos_lim, const uint8_t* r2e,
                                          uint32_t row_a) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr uint32_t MASK16 = 0x8000u | (((1u << (7 - T)) - 1u) << T);
    for (int e = 0; e < count; ++e) {
        bool found = false;
        while (bpos < d) {
            const uint32_t w = bm[(bpos >> 5) * 32] << (bpos & 31);
            if (w) { bpos += __clz(w); found = true; break; }
            bpos = (bpos | 31u) + 1u;
        }
        if (!found || bpos >= d) break;                       // corrupt record: stop inside the row
        const uint32_t col = bpos;
        bpos += 1;
        const uint32_t k = (uint32_t)(k0 + e);
        uint32_t eb;
        if (raw) {                                            // exponents stored as bytes, value k at byte k
            eb = ((un[(size_t)(k >> 2) * us] >> (24 - 8 * (k & 3))) & 0xFFu) << 7;
        } else {
            int rank = 0;
            while (upos < upos_lim) {
                const uint32_t v = un[(size_t)(upos >> 5) * us] << (upos & 31);
                const int avail = 32 - (int)(upos & 31);
                if (v) { const int z = __clz(v); rank += z; upos += z + 1; break; }
                rank += avail;
                upos += avail;
            }
            eb = (uint32_t)r2e[rank & 255] << 7;
        }
        const uint32_t fword = fl[(k / PER) * 32];
        const uint32_t a = __funnelshift_l(fword, fword, (F * (k % PER) + 16) & 31);
        tc_sts16(row_a + col * 2u, (a & MASK16) | eb);
    }
}

// Walk of one staged record by one lane: `kept` values go to the dense row at row_a (bf16, column c at row_a + 2 c).
// bm_a / fl_a / un_a: shared addresses of this lane's first bitmap / field / unary word (words 128 bytes apart);
// lut_a: shared address of the rank -> (exponent << 7) table.  A group whose 8 columns span more than 32 columns, or
// whose 4 codewords take more than 32 bits, shows up as a bit search that found nothing; that lane stores nothing for
// the group and redoes it with the careful walk.  `emit` = false: the lane only keeps the warp in step.
template <int T>
__device__ __forceinline__ void tc_walk(const uint32_t* bmP, const uint32_t* flP, const uint32_t* unP, const uint32_t* lutP, const uint8_t* r2e,
                                        int kept, int d, uint32_t una_bits, uint32_t row_a, bool emit, int stage) {
    constexpr int F = 8 - T, PER = 32 / F, NFW = kGroupCols / PER;
    constexpr uint32_t MASK16 = 0x8000u | (((1u << (7 - T)) - 1u) << T);
    static_assert(PER == 4 || PER == 8, "fields tile a word");
    const uint32_t bm_a = smem_u32(bmP), un_a = smem_u32(unP), lut_a = smem_u32(lutP);
    uint32_t fl_a = smem_u32(flP);
    uint32_t bpos = 0, upos = 0;
    const int n_full = kept / kGroupCols, rem = kept % kGroupCols;

    auto group = [&](int grp, auto tail_c) {
        constexpr bool tail = decltype(tail_c)::value;
        const uint32_t bpos0 = bpos, upos0 = upos;
        const uint32_t ba = bm_a + (bpos >> 5) * 128u;
        uint32_t bv = __funnelshift_l(tc_lds_off<128>(ba), tc_lds(ba), bpos);        // 32 columns from bpos on
        const uint32_t xg = row_a + bpos * 2u + 62u;                                 // address of column bpos + 31
        uint32_t fwd[NFW];
        fwd[0] = tc_lds(fl_a);
        if (NFW > 1) fwd[NFW - 1] = tc_lds_off<128>(fl_a);
        uint32_t addr[kGroupCols], val[kGroupCols];
        uint32_t dry = 0, p = 0;
#pragma unroll
        for (int half = 0; half < kGroupCols / kGroupCodes; ++half) {
            const uint32_t ua = un_a + (upos >> 5) * 128u;
            uint32_t uv = __funnelshift_l(tc_lds_off<128>(ua), tc_lds(ua), upos);    // 32 code bits from upos on
            uint32_t la = lut_a + 124u;             // lut + 4 * (position of the previous terminator - 1); none yet: 32
            uint32_t q = 0;
#pragma unroll
            for (int j = 0; j < kGroupCodes; ++j) {
                const int e = half * kGroupCodes + j;
                p = tc_bfind(bv);                                     // next kept column: bpos + 31 - p
                addr[e] = tc_mad(p, 0xFFFFFFFEu, xg);
                bv &= ~tc_shl(1u, p);
                q = tc_bfind(uv);                                     // next terminator
                const uint32_t eb = tc_lds(tc_mad(q, 0xFFFFFFFCu, la));              // lut[previous - q - 1]
                la = tc_mad(q, 4u, lut_a - 4u);
                uv &= ~tc_shl(1u, q);
                const uint32_t fword = fwd[e / PER];
                val[e] = (__funnelshift_l(fword, fword, (F * (e % PER) + 16) & 31) & MASK16) | eb;
                if (tail && e < rem) dry |= p | q;
            }
            upos += 32u - q;                                          // bits up to and including the last terminator
            if (!tail) dry |= q;                                      // a search that failed fails from then on
        }
        bpos += 32u - p;
        if (!tail) dry |= p;
        const bool ok = (int32_t)dry >= 0;
        if (emit && ok) {                                             // one branch per group: the stores themselves are unconditional
#pragma unroll
            for (int e = 0; e < kGroupCols; ++e)
                if (!tail || e < rem) tc_sts16(addr[e], val[e]);
        } else if (emit) {
            // redo the group value by value, then put the cursors behind it
            const int cnt = tail ? rem : kGroupCols;
            tc_walk_slow<T>(bmP, flP, unP, 32, false, grp * kGroupCols, cnt, bpos0, upos0, (uint32_t)d, una_bits, r2e, row_a);
            uint32_t b = bpos0, u = upos0;
            for (int e = 0; e < cnt; ++e) {
                while (b < (uint32_t)d) {
                    const uint32_t w = bmP[(b >> 5) * 32] << (b & 31);
                    if (w) { b += __clz(w) + 1; break; }
                    b = (b | 31u) + 1u;
                }
                while (u < una_bits) {
                    const uint32_t v = unP[(u >> 5) * 32] << (u & 31);
                    if (v) { u += __clz(v) + 1; break; }
                    u += 32u - (u & 31u);
                }
            }
            bpos = b; upos = u;
        }
        bpos = min(bpos, (uint32_t)d);                                // a walk that lost its way stays inside the staging
        upos = min(upos, (uint32_t)stage * 32u);
        fl_a += NFW * 128u;
    };
    for (int grp = 0; grp < n_full; ++grp) group(grp, std::false_type{});
    if (rem) group(n_full, std::true_type{});
}

// ---- Cassandra-2 (MX) records: fields = sign + magnitude >> t, one exponent byte E per 32-channel slice -------------
// A value is (-1)^s (mag << t) 2^(E - 133).  With p the leading bit of mag << t its bf16 pattern is sign, exponent
// E + p - 6, mantissa the bits below p: lut[field] = {sign | p << 7 | mantissa, mask}, and the pattern is
// lut.x + (((E - 6) << 7) & lut.y) with mask 0 for a zero magnitude (and for slices with E < 7, whose fields are all zero).
__device__ __forceinline__ uint2 tc_lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}

// Careful walk of the kept values k0 .. k0 + count - 1 of an MX record from column bpos on.  eb: the lane's slice table
// ((E - 6) << 7 per slice, rows 32 words apart); lut: field -> {pattern, mask}.
template <int T>
__device__ __noinline__ void tc_walk_mx_slow(const uint32_t* bm, const uint32_t* fl, const uint32_t* eb, const uint2* lut, int k0, int count,
                                             uint32_t bpos, uint32_t d, uint32_t row_a) {
    constexpr int F = 8 - T, PER = 32 / F;
    for (int e = 0; e < count; ++e) {
        bool found = false;
        while (bpos < d) {
            const uint32_t w = bm[(bpos >> 5) * 32] << (bpos & 31);
            if (w) { bpos += __clz(w); found = true; break; }
            bpos = (bpos | 31u) + 1u;
        }
        if (!found || bpos >= d) break;                       // corrupt record: stop inside the row
        const uint32_t col = bpos;
        bpos += 1;
        const uint32_t k = (uint32_t)(k0 + e);
        const uint32_t f = (fl[(k / PER) * 32] >> (32 - F * (k % PER + 1))) & ((1u << F) - 1u);
        const uint2 lm = lut[f];
        tc_sts16(row_a + col * 2u, lm.x + (eb[(col >> 5) * 32] & lm.y));
    }
}

// Walk of one staged MX record by one lane, 8 kept values per 32-bit bitmap window; the window's columns lie in at most
// two slices, whose exponents are fetched once per group.  xP: the record's exponent words; ebP: room for the lane's
// slice table (d / 32 + 2 rows).
template <int T>
__device__ __forceinline__ void tc_walk_mx(const uint32_t* bmP, const uint32_t* flP, const uint32_t* xP, uint32_t* ebP, const uint2* lutP,
                                           int kept, int d, uint32_t row_a) {
    constexpr int F = 8 - T, PER = 32 / F, NFW = kGroupCols / PER;
    static_assert(PER == 4 || PER == 8, "fields tile a word");
    const int S = d / 32;
    for (int sl = 0; sl < S; ++sl) {
        const uint32_t E = (xP[(sl >> 2) * 32] >> (24 - 8 * (sl & 3))) & 0xFFu;
        ebP[sl * 32] = E >= 7u ? (E - 6u) << 7 : 0u;
    }
    ebP[S * 32] = 0u;
    ebP[(S + 1) * 32] = 0u;
    __syncwarp();
    const uint32_t bm_a = smem_u32(bmP), eb_a = smem_u32(ebP), lut_a = smem_u32(lutP);
    uint32_t fl_a = smem_u32(flP);
    uint32_t bpos = 0;
    const int n_full = kept / kGroupCols, rem = kept % kGroupCols;
    auto group = [&](int grp, auto tail_c) {
        constexpr bool tail = decltype(tail_c)::value;
        const uint32_t bpos0 = bpos;
        const uint32_t ba = bm_a + (bpos >> 5) * 128u;
        uint32_t bv = __funnelshift_l(tc_lds_off<128>(ba), tc_lds(ba), bpos);        // 32 columns from bpos on
        const uint32_t xg = row_a + bpos * 2u + 62u;                                 // address of column bpos + 31
        const uint32_t ea = eb_a + (bpos >> 5) * 128u;
        const uint32_t eb0 = tc_lds(ea), eb1 = tc_lds_off<128>(ea);                  // this slice's exponent and the next one's
        const int pb = (int)(bpos & 31u) - 1;                                        // window bits <= pb lie in the next slice
        uint32_t fwd[NFW];
        fwd[0] = tc_lds(fl_a);
        if (NFW > 1) fwd[NFW - 1] = tc_lds_off<128>(fl_a);
        uint32_t addr[kGroupCols], val[kGroupCols];
        uint32_t dry = 0, p = 0;
#pragma unroll
        for (int e = 0; e < kGroupCols; ++e) {
            p = tc_bfind(bv);                                         // next kept column: bpos + 31 - p
            addr[e] = tc_mad(p, 0xFFFFFFFEu, xg);
            bv &= ~tc_shl(1u, p);
            const uint32_t f = (fwd[e / PER] >> (32 - F * (e % PER + 1))) & ((1u << F) - 1u);
            const uint2 lm = tc_lds64(lut_a + f * 8u);
            const uint32_t eb = (int)p <= pb ? eb1 : eb0;
            val[e] = lm.x + (eb & lm.y);
            if (tail && e < rem) dry |= p;
        }
        bpos += 32u - p;
        if (!tail) dry |= p;                                          // a search that failed fails from then on
        const bool ok = (int32_t)dry >= 0;
        if (ok) {                                                     // one branch per group: the stores themselves are unconditional
#pragma unroll
            for (int e = 0; e < kGroupCols; ++e)
                if (!tail || e < rem) tc_sts16(addr[e], val[e]);
        } else {
            const int cnt = tail ? rem : kGroupCols;
            tc_walk_mx_slow<T>(bmP, flP, ebP, lutP, grp * kGroupCols, cnt, bpos0, (uint32_t)d, row_a);
            uint32_t b = bpos0;
            for (int e = 0; e < cnt; ++e) {
                while (b < (uint32_t)d) {
                    const uint32_t w = bmP[(b >> 5) * 32] << (b & 31);
                    if (w) { b += __clz(w) + 1; break; }
                    b = (b | 31u) + 1u;
                }
            }
            bpos = b;
        }
        bpos = min(bpos, (uint32_t)d);
        fl_a += NFW * 128u;
    };
    for (int grp = 0; grp < n_full; ++grp) group(grp, std::false_type{});
    if (rem) group(n_full, std::true_type{});
}


__device__ __forceinline__ void tc_cp_async4(uint32_t dst, const void* src, bool take) {      // take = false: zero fill
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(take ? 4 : 0) : "memory");
}
__device__ __forceinline__ void tc_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tc_cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Words of the record staging; the scores and probabilities take its place once the records are decoded.
__host__ __device__ inline int tc_fix_words(const KvGeom& g) {
    const int rec = 4 * (g.wpt + 1) * 32;
    const int post = (2 * kTcHeads * (kTcTok + kTcPad) * 2 + kTcHeads * kTcTok * 4 + 2 * kTcHeads * 4) / 4;
    return rec > post ? rec : post;
}

// grid = (runs, KV heads, sequences).  A CTA handles a run of consecutive 64-token chunks (tc_run_tokens positions: the
// longer the visible cache, the longer the run, so that the grid stays near four CTAs per SM and the merge short) with a
// running softmax: per chunk it stages and decodes the records, forms the scores, rescales what it has and adds P.V.
__host__ __device__ inline int tc_lut_words(const KvGeom& g) { return g.mode == 1 ? 64 : 2 << (8 - g.t); }
__host__ __device__ inline int tc_una_rows(const KvGeom& g) { return g.mode == 1 ? tc_una_stage(g) + 2 : g.d / 32 + 2; }

template <int MODE, int T>
__global__ void __launch_bounds__(kTcThreads) k_draft_attn_tc(KvGeom g, KvComp ck0, KvComp cv0, const uint16_t* __restrict__ qkv,
                                                              int qkv_stride, int n_q, const DevState* __restrict__ st, AttnScratch sc,
                                                              int n_chunks_alloc) {
    extern __shared__ __align__(16) uint8_t smem[];
    pdl_early<2>();
    pdl_wait();
    const int run = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    const int cur_len = st->len[seq] + st->inflight[seq] + 1;  // positions visible to the drafted token
    const int run_tokens = tc_run_tokens(cur_len, g.n_kv * (int)gridDim.z);
    const int t_begin = run * run_tokens;
    if (t_begin >= cur_len) return;
    const int t_end = min(cur_len, t_begin + run_tokens);
    const int G = n_q / g.n_kv, d = g.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    qkv += (size_t)seq * qkv_stride;

    const int ks = d + kTcPad;                                                // halfwords per tile row
    uint16_t* kt_s = reinterpret_cast<uint16_t*>(smem);                       // [64][ks] dense K, bf16
    uint16_t* vt_s = kt_s + kTcTok * ks;                                      // [64][ks] dense V
    uint16_t* q_s = vt_s + kTcTok * ks;                                       // [8][ks] query heads of the group (unused heads zero)
    uint32_t* fix_s = reinterpret_cast<uint32_t*>(q_s + kTcHeads * ks);       // [4 warps][wpt + 1][32] records; after the walk:
    uint16_t* p_s = reinterpret_cast<uint16_t*>(fix_s);                       //   [2][8][64 + 8] probabilities, high and low bf16 term
    float* sc_s = reinterpret_cast<float*>(p_s + 2 * kTcHeads * (kTcTok + kTcPad));   //   [8][64] scores
    const int stage = MODE == 1 ? tc_una_stage(g) : 0, una_rows = MODE == 1 ? stage + 2 : d / 32 + 2;
    uint32_t* una_s = fix_s + tc_fix_words(g);                                // [4 warps][una_rows][32]: exponent words (MODE 1) | slice tables (MODE 2)
    uint32_t* lut_s = una_s + 4 * una_rows * 32;                              // MODE 1: [2][32] rank -> exponent << 7; MODE 2: field -> {pattern, mask}
    float* run_s = reinterpret_cast<float*>(lut_s + tc_lut_words(g));         // [8][3]: running max, running sum, rescale factor of the chunk

    // warps 0,1 -> K records of tokens t0 + 32 w .., warps 2,3 -> V records of the same tokens
    const int kind = warp >> 1, tw = warp & 1;
    const KvComp& c = kind ? cv0 : ck0;                                       // sequence 0's; shifted to this sequence where used
    uint32_t* my_fix = fix_s + warp * (g.wpt + 1) * 32;
    uint32_t* my_una = una_s + warp * una_rows * 32;
    const uint32_t* fixed_h = of_seq(c.fixed, seq, g.seq_stride) + (size_t)head * g.n_blocks * g.wpt * 32;
    const uint32_t* off_h = of_seq(c.off, seq, g.seq_stride) + (size_t)head * (g.max_seq + 1);
    const uint32_t* arena = of_seq(c.arena, seq, g.seq_stride) + (size_t)head * g.arena_words;
    const uint8_t* r2e = of_seq(c.rank_to_exp, seq, g.seq_stride);
    // Tokens beyond the visible length take the last visible token's record (their probabilities are zero).
    auto load_off = [&](int t0, uint32_t& o0, uint32_t& n_una) {
        o0 = 0; n_una = 0;
        if (MODE != 1) return;                                                // Cassandra-2 records have no exponent stream
        const int n_here = min(32, cur_len - (t0 + tw * 32));
        if (t0 < t_end && n_here > 0) {
            const int tok = t0 + tw * 32 + min(lane, n_here - 1);
            o0 = __ldg(off_h + tok);
            n_una = __ldg(off_h + tok + 1) - o0;
        }
    };

    // Everything the first chunk needs from global memory is requested before any of it is used: the first records'
    // arena offsets, the rank tables and the query rows share one round trip.
    uint32_t o0, n_una, o0_next, nu_next;
    load_off(t_begin, o0_next, nu_next);
    uint32_t lut_v = 0;
    if (MODE == 1 && tid < 64) {
        const uint8_t *rk = of_seq(ck0.rank_to_exp, seq, g.seq_stride), *rv = of_seq(cv0.rank_to_exp, seq, g.seq_stride);
        lut_v = tid < 32 ? rk[tid] : rv[tid - 32];
    }
    constexpr int kQIter = 4;                                                 // query words per thread and batch
    const int n_qw = G * d / 2;
    for (int i = tid; i < kTcHeads * ks / 2; i += kTcThreads) reinterpret_cast<uint32_t*>(q_s)[i] = 0u;   // unused heads stay zero
    if (tid < 3 * kTcHeads) run_s[tid] = tid % 3 == 0 ? -INFINITY : 0.f;
    __syncthreads();
    for (int i0 = tid; i0 < n_qw; i0 += kTcThreads * kQIter) {                // the query heads of the group, bf16 as they are
        uint32_t qv[kQIter];
#pragma unroll
        for (int u = 0; u < kQIter; ++u) {
            const int i = i0 + u * kTcThreads;
            qv[u] = i < n_qw ? __ldg(reinterpret_cast<const uint32_t*>(qkv + (size_t)(head * G + i / (d / 2)) * d) + i % (d / 2)) : 0u;
        }
#pragma unroll
        for (int u = 0; u < kQIter; ++u) {
            const int i = i0 + u * kTcThreads;
            if (i < n_qw) reinterpret_cast<uint32_t*>(q_s + (i / (d / 2)) * ks)[i % (d / 2)] = qv[u];
        }
    }
    if (MODE == 1) {
        if (tid < 64) lut_s[tid] = lut_v << 7;
    } else {
        constexpr int NF = 1 << (8 - T);
        for (int f = tid; f < NF; f += kTcThreads) {
            const uint32_t sgn = (uint32_t)f >> (7 - T), mag = ((uint32_t)f & ((1u << (7 - T)) - 1u)) << T;
            uint2 lm = make_uint2(0u, 0u);
            if (mag) {
                const uint32_t pl = 31u - (uint32_t)__clz(mag);               // leading bit of the 7-bit magnitude
                lm.x = (sgn << 15) | (pl << 7) | ((mag << (7u - pl)) & 0x7Fu);
                lm.y = 0xFFFFFFFFu;
            }
            reinterpret_cast<uint2*>(lut_s)[f] = lm;
        }
    }
    constexpr int kMaxMt = 4;                                                 // 16-channel tiles of the output per warp (head_dim <= 256)
    float o_acc[kMaxMt][4];
#pragma unroll
    for (int j = 0; j < kMaxMt; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) o_acc[j][i] = 0.f;
    const float scale = rsqrtf((float)d);

    for (int t0 = t_begin; t0 < t_end; t0 += kTcTok) {
        o0 = o0_next; n_una = nu_next;
        const int n_here = min(32, cur_len - (t0 + tw * 32));                 // visible tokens of this warp's block (may be <= 0)
        if (n_here > 0) {
            const int src_lane = min(lane, n_here - 1);
            const uint32_t* fixed = fixed_h + (size_t)((t0 + tw * 32) / 32) * g.wpt * 32;
            const uint32_t fa = smem_u32(my_fix + lane);
            for (int w = 0; w < g.wpt; ++w) tc_cp_async4(fa + w * 128, fixed + w * 32 + src_lane, true);      // coalesced block copy
            my_fix[g.wpt * 32 + lane] = 0u;
            if (MODE == 1) {
                const uint32_t ua = smem_u32(my_una + lane);
                const bool fits = n_una <= (uint32_t)stage;
#pragma unroll 4
                for (int w = 0; w < una_rows; ++w) {
                    const bool take = fits && (uint32_t)w < n_una;
                    tc_cp_async4(ua + w * 128, arena + (take ? o0 + w : 0), take);
                }
            }
        }
        load_off(t0 + kTcTok, o0_next, nu_next);                              // the next chunk's offsets travel meanwhile
        {   // zero the two tiles (pruned channels stay zero); 16 bytes per store
            uint4* z = reinterpret_cast<uint4*>(kt_s);
            const int n16 = 2 * kTcTok * ks / 8;
            for (int i = tid; i < n16; i += kTcThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        tc_cp_async_wait_all();
        __syncthreads();
        if (n_here > 0) {
            const uint32_t row_a = smem_u32((kind ? vt_s : kt_s) + (size_t)(tw * 32 + lane) * ks);
            const uint32_t* bmP = my_fix + g.e_words * 32 + lane;
            const uint32_t* flP = bmP + g.bm_words * 32;
            if (MODE == 1) {
                const bool raw = (my_fix[lane] & kKvRawFlag) != 0;            // entry word 0 of this token's record
                const bool staged = n_una <= (uint32_t)stage && !raw;
                const uint32_t* lutP = lut_s + kind * 32;
                tc_walk<T>(bmP, flP, my_una + lane, lutP, r2e, g.kept, d, n_una * 32u, row_a, staged, stage);
                if (!staged)                                                  // raw exponents or a very long record: read it in place
                    tc_walk_slow<T>(bmP, flP, arena + o0, 1, raw, 0, g.kept, 0u, 0u, (uint32_t)d, n_una * 32u, r2e, row_a);
            } else {
                tc_walk_mx<T>(bmP, flP, flP + g.f_words * 32, my_una + lane, reinterpret_cast<const uint2*>(lut_s), g.kept, d, row_a);
            }
        }
        __syncthreads();

        // ---- scores: S[token][head] = K[token][:] . q[head][:]; warp w takes tokens 16 w .. 16 w + 15 ----
        {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t a_base = smem_u32(kt_s + (size_t)(warp * 16 + (lane & 15)) * ks + (lane >> 4) * 8);
            const uint32_t b_base = smem_u32(q_s + (size_t)(lane & 7) * ks + ((lane >> 3) & 1) * 8);
            for (int kk = 0; kk < d / 16; ++kk) {
                uint32_t a[4], b[2];
                tc_ldmatrix_x4(a, a_base + kk * 32);
                tc_ldmatrix_x2(b, b_base + kk * 32);
                tc_mma(acc, a, b);
            }
            const int r0 = warp * 16 + (lane >> 2), h0 = (lane & 3) * 2;
            const int n_tok = cur_len - t0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = r0 + (i >> 1) * 8, h = h0 + (i & 1);
                sc_s[h * kTcTok + r] = r < n_tok ? acc[i] * scale : -INFINITY;
            }
        }
        __syncthreads();
        // ---- running softmax: warp w handles query heads w, w + 4; p = hi + lo in bf16 ----
        for (int gi = warp; gi < kTcHeads; gi += kTcThreads / 32) {
            float a = sc_s[gi * kTcTok + lane], b = sc_s[gi * kTcTok + 32 + lane];
            const float m_old = run_s[gi * 3];
            const float m = fmaxf(m_old, warp_max(fmaxf(a, b)));              // finite: the chunk has a visible token
            a = expf(a - m);                                                  // exp(-inf) = 0 for tokens beyond the end
            b = expf(b - m);
            const float l = warp_sum(a + b);
            __syncwarp();
            if (lane == 0) {
                const float alpha = expf(m_old - m);                          // 0 for the first chunk
                run_s[gi * 3] = m;
                run_s[gi * 3 + 1] = run_s[gi * 3 + 1] * alpha + l;
                run_s[gi * 3 + 2] = alpha;
            }
            uint16_t* ph = p_s + gi * (kTcTok + kTcPad);
            uint16_t* pl = ph + kTcHeads * (kTcTok + kTcPad);
            const uint16_t ah = float_to_bf16_bits(a), bh = float_to_bf16_bits(b);
            ph[lane] = ah;
            ph[32 + lane] = bh;
            pl[lane] = float_to_bf16_bits(a - bf16_bits_to_float(ah));
            pl[32 + lane] = float_to_bf16_bits(b - bf16_bits_to_float(bh));
        }
        __syncthreads();
        // ---- O^T[channel][head] = alpha O^T + V^T[channel][token] . P^T[token][head]; warp w: 16-channel tiles w, w + 4, ... ----
        {
            const int h0 = (lane & 3) * 2;
            const float al0 = run_s[h0 * 3 + 2], al1 = run_s[(h0 + 1) * 3 + 2];
            const uint32_t b_base = smem_u32(p_s + (size_t)(lane & 7) * (kTcTok + kTcPad) + ((lane >> 3) & 1) * 8);
#pragma unroll
            for (int j = 0; j < kMaxMt; ++j) {
                const int mt = warp + j * (kTcThreads / 32);
                if (mt < d / 16) {
                    o_acc[j][0] *= al0; o_acc[j][1] *= al1; o_acc[j][2] *= al0; o_acc[j][3] *= al1;
                    const uint32_t a_base = smem_u32(vt_s + (size_t)((lane >> 4) * 8 + (lane & 7)) * ks + mt * 16 + ((lane >> 3) & 1) * 8);
#pragma unroll
                    for (int kk = 0; kk < kTcTok / 16; ++kk) {
                        uint32_t a[4], bh[2], bl[2];
                        tc_ldmatrix_x4_trans(a, a_base + kk * 16 * ks * 2);
                        tc_ldmatrix_x2(bh, b_base + kk * 32);
                        tc_ldmatrix_x2(bl, b_base + kk * 32 + kTcHeads * (kTcTok + kTcPad) * 2);
                        tc_mma(o_acc[j], a, bl);
                        tc_mma(o_acc[j], a, bh);
                    }
                }
            }
        }
        __syncthreads();                                                      // tiles, records and probabilities may be overwritten
    }
    {
        const int h0 = (lane & 3) * 2;
#pragma unroll
        for (int j = 0; j < kMaxMt; ++j) {
            const int mt = warp + j * (kTcThreads / 32);
            if (mt < d / 16) {
                const int c0 = mt * 16 + (lane >> 2);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int ch = c0 + (i >> 1) * 8, h = h0 + (i & 1);
                    if (h < G) sc.o[(((size_t)seq * n_q + head * G + h) * n_chunks_alloc + run) * d + ch] = o_acc[j][i];
                }
            }
        }
    }
    if (tid < G) {
        const size_t pair = (size_t)seq * n_q + head * G + tid;
        sc.m[pair * n_chunks_alloc + run] = run_s[tid * 3];
        sc.l[pair * n_chunks_alloc + run] = run_s[tid * 3 + 1];
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int rps, int n_q, int d,
                      const DevState* st, int draft_mode, int draft_units, uint16_t* out, cudaStream_t s);

size_t draft_attn_tc_smem_bytes(const KvGeom& g) {
    const size_t ks = (size_t)g.d + kTcPad;
    return (2 * kTcTok + kTcHeads) * ks * 2 + (size_t)tc_fix_words(g) * 4 + (size_t)4 * tc_una_rows(g) * 32 * 4 + (size_t)tc_lut_words(g) * 4 + 3 * kTcHeads * 4 + 64;
}

bool draft_attn_tc_supported(const KvGeom& g, int n_q) {
    const int G = n_q / g.n_kv;
    return (g.mode == 1 || g.mode == 2) && (g.t == 4 || g.t == 0) && G >= 1 && G <= kTcHeads && g.d % 16 == 0 && g.d >= 32 && g.d <= 256;
}

int launch_draft_attn_tc(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                         int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s) {
    if (!draft_attn_tc_supported(g, n_q)) return CASS_ERR_UNSUPPORTED;
    const int n_chunks = ceil_div(g.max_seq, kTcTok);
    const size_t smem = draft_attn_tc_smem_bytes(g);
    if (smem > 227 * 1024) return CASS_ERR_UNSUPPORTED;
    dim3 grid(n_chunks, g.n_kv, n_seq);
#define CASS_TC_LAUNCH(MM, TT)                                                                                           \
    do {                                                                                                             \
        static size_t attr = 0;                                                                                      \
        if (smem > attr) {                                                                                           \
            CASS_CUDA_CHECK(cudaFuncSetAttribute((k_draft_attn_tc<MM, TT>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
            attr = smem;                                                                                             \
        }                                                                                                            \
        CASS_PDL_LAUNCH((k_draft_attn_tc<MM, TT>), grid, dim3(kTcThreads), smem, s, g, ck, cv, qkv, qkv_stride, n_q, st, sc, n_chunks);      \
    } while (0)
    if (g.mode == 1 && g.t == 4) CASS_TC_LAUNCH(1, 4);
    else if (g.mode == 1) CASS_TC_LAUNCH(1, 0);
    else if (g.t == 4) CASS_TC_LAUNCH(2, 4);
    else CASS_TC_LAUNCH(2, 0);
#undef CASS_TC_LAUNCH
    CASS_LAUNCH_CHECK();
    // the runs of every (sequence, query head) are merged by a kernel of their own: one CTA per head with the runs spread
    // over its warps (a merge by the last CTA of a KV head, as the slice-parallel kernel does it, is one CTA adding up to
    // 74 runs for the whole group in sequence: measured 32.6 instead of 16.7 us at 4096 positions)
    return launch_attn_merge(sc, n_chunks, kTcTok, n_seq, 1, n_q, g.d, st, 1, -g.n_kv * n_seq, out, s);
}

}  // namespace cass
