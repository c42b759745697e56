// Draft GEMV: y = decode(speculation data) * x with the decode done in registers (Sec. 4.1 draft inference;
// the software form of the decoder dataflow of Sec. 5.1: bitmap de-sparsification, unary exponent decode
// through a rank->exponent table, sign/mantissa concatenation).
//
// Work unit = one superblock (32 rows x one column segment).  A CTA owns one column segment (its slice of x
// stays in shared memory as fp32) and walks the row blocks assigned to it; a superblock arrives by one bulk
// asynchronous copy (contiguous reads, as Sec. 5.3 asks) into the CTA's single stage; the CTAs that share an SM
// overlap each other's copies and decodes.  Warp c decodes chunk c with lane = row: every lane
// walks its own bitmap, field and unary streams, which are interleaved word by word over the 32 rows so that
// all shared-memory reads of the streams are conflict free.
#include <type_traits>

#include "wblob.cuh"
#include "kernels.cuh"

namespace cass {

constexpr int kGemvStages = 1;         // stages of the copy ring per CTA; several CTAs share an SM, so their copies and decodes overlap
constexpr int kXSlack = 288;           // readable floats after the x slice: a window walk may run up to 8 x 32 + 8 columns past its start

static size_t gemv_stage_bytes(const cass_blob_info& bi) { return align_up((size_t)bi.max_superblock_bytes + 256, 128); }

// Bytes per column of the x slice in shared memory: one vector is kept as fp32, several as packed bf16 [col][nb].
__host__ __device__ constexpr int x_col_bytes(int nb) { return nb == 1 ? 4 : 2 * nb; }

size_t gemv_smem_bytes(const cass_blob_info& bi, int nb) {
    const int n_ch = ceil_div(bi.seg_cols, bi.chunk_cols);
    return kGemvStages * gemv_stage_bytes(bi) + (size_t)(bi.seg_cols + kXSlack) * x_col_bytes(nb) + 256 * 4 +
           (size_t)(nb < 2 ? 2 : nb) * n_ch * 32 * 4 + 64;
}

__device__ __forceinline__ uint32_t shl_sat(uint32_t v, uint32_t s) {      // shift counts >= 32 give 0
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
}

__device__ __forceinline__ uint32_t bfind_u32(uint32_t v) {         // index of the most significant one, -1 if none
    uint32_t r;
    asm("bfind.u32 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t mad_lo(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

// Sign and kept mantissa bits of a field at their binary32 positions, for truncations whose fields do not tile a
// word (8 - t = 7, 6, 5, 3): the field is packed from the most significant end, floor(32 / (8 - t)) per word.
template <int T>
__device__ __forceinline__ uint32_t packed_field_f32(uint32_t word, uint32_t j) {
    constexpr int F = 8 - T;
    const uint32_t f = (word >> (32u - (uint32_t)F * (j + 1u))) & ((1u << F) - 1u);
    return ((f >> (F - 1)) << 31) | ((f & ((1u << (F - 1)) - 1u)) << (16 + T));
}

template <int NB>
struct WalkState {
    float acc[NB];
    uint32_t bpos, upos;
};

// The NB values of x at one column: raw words as they sit in shared memory, and their use in the accumulators.
template <int NB>
struct XRaw { uint32_t w[NB == 1 ? 1 : NB / 2]; };

template <int NB>
__device__ __forceinline__ XRaw<NB> x_load(uint32_t addr) {
    XRaw<NB> r;
    if constexpr (NB <= 2) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(r.w[0]) : "r"(addr));
    else if constexpr (NB == 4) asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(r.w[0]), "=r"(r.w[1]) : "r"(addr));
    else asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]) : "r"(addr));
    return r;
}

template <int NB>
__device__ __forceinline__ void x_fma(const XRaw<NB>& r, uint32_t wb, float (&acc)[NB]) {
    const float w = __uint_as_float(wb);
    if constexpr (NB == 1) {
        acc[0] = fmaf(w, __uint_as_float(r.w[0]), acc[0]);
    } else {
#pragma unroll
        for (int i = 0; i < NB / 2; ++i) {
            acc[2 * i] = fmaf(w, __uint_as_float(r.w[i] << 16), acc[2 * i]);
            acc[2 * i + 1] = fmaf(w, __uint_as_float(r.w[i] & 0xFFFF0000u), acc[2 * i + 1]);
        }
    }
}

// Careful walk of `count` (<= 8) kept values of one row from column bpos / code bit upos on: any gap between
// kept columns, any codeword length.  Used for the rare groups that do not fit the 32-bit windows.
// flC: the segment's first field word of this row; k0: index (inside the segment) of the group's first value.
template <int T, int NB>
__device__ __noinline__ WalkState<NB> group_slow(const uint32_t* bmS, const uint32_t* unS, const uint32_t* flC, uint32_t k0, int count,
                                                 WalkState<NB> st, uint32_t bpos_lim, uint32_t upos_lim, const float* xs,
                                                 const uint32_t* lut) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));
    for (int e = 0; e < count; ++e) {
        bool found = false;
        while (st.bpos < bpos_lim) {
            uint32_t w = bmS[(st.bpos >> 5) * 32] << (st.bpos & 31);
            if (w) { st.bpos += __clz(w); found = true; break; }
            st.bpos = (st.bpos | 31u) + 1u;
        }
        if (!found) break;                                   // corrupt stream: stop inside the buffers
        const XRaw<NB> xv = x_load<NB>(smem_u32(xs) + st.bpos * (uint32_t)x_col_bytes(NB));
        st.bpos += 1;
        const int rank = read_unary(unS, st.upos, upos_lim);
        const uint32_t k = k0 + (uint32_t)e;
        const uint32_t fword = flC[(k / PER) * 32];
        uint32_t a;
        if constexpr (32 % F == 0) a = __funnelshift_l(fword, fword, (F * (k % PER)) & 31) & MASK;
        else a = packed_field_f32<T>(fword, k % PER);
        x_fma<NB>(xv, a | lut[rank & 255], st.acc);
    }
    return st;
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {         // shared-space byte address
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint32_t lds_u32_off(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF));
    return v;
}

// Dot product of one chunk (32 rows, lane = row) with x.  T = truncated mantissa bits (0 or 4).  Every lane walks
// its row in groups of 8 kept values through 32-bit windows: one bitmap window per group, one unary window per 4
// codewords.  A group whose 8 kept columns span more than 32 columns, or whose 4 codewords take more than 32 bits,
// shows up as a window that ran dry (no bit left to find); that lane then redoes the group with the careful
// walk while the others wait.  The walk addresses shared memory through 32-bit shared-space addresses.
template <int T, int NB>
__device__ __forceinline__ void chunk_dot_fast(const uint32_t* __restrict__ sb, const SbGeom& g, int ch, int lane,
                                               int chunk_elems, const float* __restrict__ xs,
                                               const uint32_t* __restrict__ lut, float (&acc)[NB]) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr bool ROT = 32 % F == 0;                                    // fields tile a word: float-aligned and rotated
    constexpr int NFW = ROT ? kGroupCols / PER : 3;                      // field words a group of 8 can touch
    constexpr uint32_t MASK = 0x80000000u | (((1u << (7 - T)) - 1u) << (16 + T));   // sign + kept mantissa of a binary32
    static_assert(ROT ? (PER == 4 || PER == 8) : (PER >= 4 && PER <= 10), "fast path: 4 to 10 fields per word");
    constexpr uint32_t XS = (uint32_t)x_col_bytes(NB);            // bytes per column of the x slice
    const uint32_t e0 = sb[g.tab + ch * 32 + lane];            // where this row's value ch * chunk_elems sits
    const uint32_t fw = (uint32_t)(ch * chunk_elems) / PER;    // the word of the chunk's first field (fields are numbered through the segment)
    uint32_t upos = e0 & 0xFFFFFu;
    const uint32_t* bmS = sb + g.bm + lane;
    const uint32_t* flS = sb + g.fl + lane;
    const uint32_t* unS = sb + g.un + lane;
    const uint32_t bm_a = smem_u32(bmS), un_a = smem_u32(unS), xs_a = smem_u32(xs), lut_a = smem_u32(lut);
    uint32_t fl_a = smem_u32(flS + fw * 32);
    uint32_t j0 = (uint32_t)(ch * chunk_elems) % PER;           // packed fields: place of the group's first field in its word
    // every row has chunk_elems values in each chunk except its last ones, so the lanes of a warp stay in step
    const int kept = (int)(sb[g.tab + g.n_ch * 32 + lane] >> 20);
    const int m = max(0, min(chunk_elems, kept - ch * chunk_elems));
    const int n_full = __reduce_min_sync(0xffffffffu, m) / kGroupCols;
    const int n_groups = ceil_div(__reduce_max_sync(0xffffffffu, m), kGroupCols);
    uint32_t bpos = e0 >> 20;
    const uint32_t bpos_lim = (uint32_t)(g.bm_words * 32), upos_lim = (uint32_t)(g.w_u * 32);

    // Bit positions are counted from the least significant end (bfind): a window keeps its place and the bit
    // just used is cleared, so a kept column is x[bpos + 31 - p] and a codeword's rank is the distance between two
    // consecutive terminators.  A window that ran dry gives p = -1; once dry it stays dry, so the sign of the last
    // position of each window tells whether the whole group fitted.
    auto group = [&](int grp, auto tail_c) {
        constexpr bool tail = decltype(tail_c)::value;         // two specialisations: full groups carry no per-value tests
        WalkState<NB> st0;
#pragma unroll
        for (int b = 0; b < NB; ++b) st0.acc[b] = acc[b];
        st0.bpos = bpos; st0.upos = upos;
        const uint32_t ba = bm_a + (bpos >> 5) * 128u;
        uint32_t bv = __funnelshift_l(lds_u32_off<128>(ba), lds_u32(ba), bpos);    // 32 columns from bpos on
        const uint32_t xg = xs_a + bpos * XS + 31u * XS;                           // address of x[bpos + 31]
        uint32_t fwd[NFW];
        fwd[0] = lds_u32(fl_a);
        if (NFW > 1) fwd[1] = lds_u32_off<128>(fl_a);
        if (NFW > 2) fwd[2] = lds_u32_off<256>(fl_a);
        const int rem = m - grp * kGroupCols;
        uint32_t dry = 0;                           // sign bit set: a window ran dry under a value that counts
        uint32_t p = 0;
#pragma unroll
        for (int half = 0; half < kGroupCols / kGroupCodes; ++half) {
            const uint32_t ua = un_a + (upos >> 5) * 128u;
            uint32_t uv = __funnelshift_l(lds_u32_off<128>(ua), lds_u32(ua), upos);   // 32 code bits from upos on
            uint32_t la = lut_a + 124u;             // lut + 4 * (position of the previous terminator - 1); none yet: 32
            uint32_t q = 0;
#pragma unroll
            for (int j = 0; j < kGroupCodes; ++j) {
                const int e = half * kGroupCodes + j;
                p = bfind_u32(bv);                                   // next kept column
                const XRaw<NB> xv = x_load<NB>(mad_lo(p, 0u - XS, xg));
                bv &= ~shl_sat(1u, p);
                q = bfind_u32(uv);                                   // next terminator
                const uint32_t eb = lds_u32(mad_lo(q, 0xFFFFFFFCu, la));          // lut[previous - q - 1]
                la = mad_lo(q, 4u, lut_a - 4u);
                uv &= ~shl_sat(1u, q);
                uint32_t wb;
                if constexpr (ROT) {
                    const uint32_t fword = fwd[e / PER];
                    const uint32_t a = __funnelshift_l(fword, fword, (F * (e % PER)) & 31);
                    wb = (a & MASK) | eb;
                } else {
                    const uint32_t jj = j0 + (uint32_t)e;                 // field jj of the group's (up to three) words
                    const uint32_t wsel = jj >= 2u * PER ? 2u : (jj >= (uint32_t)PER ? 1u : 0u);
                    const uint32_t fword = wsel == 2u ? fwd[NFW - 1] : (wsel == 1u ? fwd[1] : fwd[0]);
                    wb = packed_field_f32<T>(fword, jj - wsel * PER) | eb;
                }
                if (!tail) {
                    x_fma<NB>(xv, wb, acc);
                } else if (e < rem) {
                    x_fma<NB>(xv, wb, acc);
                    dry |= p | q;
                }
            }
            upos += 32u - q;                                         // bits up to and including the last terminator
            if (tail) upos = min(upos, upos_lim);                    // rows that ran out of values stay inside the buffers
            else dry |= q;
        }
        bpos += 32u - p;
        if (tail) bpos = min(bpos, bpos_lim);
        else dry |= p;
        if ((int32_t)dry < 0) {
            const WalkState<NB> r = group_slow<T, NB>(bmS, unS, flS, (uint32_t)(ch * chunk_elems + grp * kGroupCols), min(rem, kGroupCols),
                                                      st0, bpos_lim, upos_lim, xs, lut);
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[b] = r.acc[b];
            bpos = r.bpos; upos = r.upos;
        }
        if constexpr (ROT) {
            fl_a += NFW * 128u;
        } else {
            const uint32_t jn = j0 + (uint32_t)kGroupCols;
            const uint32_t adv = jn >= 2u * PER ? 2u : (jn >= (uint32_t)PER ? 1u : 0u);
            fl_a += adv * 128u;
            j0 = jn - adv * PER;
        }
    };

    int grp = 0;
    for (; grp < n_full; ++grp) group(grp, std::false_type{});
    for (; grp < n_groups; ++grp) group(grp, std::true_type{});
}

// ---- Cassandra-2 (MX) chunk: 4-bit fields (sign + 3 magnitude bits, t = 4), one exponent byte per 32 values ------
// Same bitmap walk as above; the unary parse is replaced by a 16-entry table look-up of the signed magnitude, and a
// block's 32 products are summed first and scaled by the block's power of two once (Sec. 5.1, MX decoder: the shared
// exponent is broadcast to the elements of its block).
template <int NB>
__device__ __noinline__ WalkState<NB> group_slow_mx(const uint32_t* bmS, uint32_t fword, int count, WalkState<NB> st,
                                                    uint32_t bpos_lim, const float* xs, const float* nlut) {
    for (int e = 0; e < count; ++e) {
        bool found = false;
        while (st.bpos < bpos_lim) {
            uint32_t w = bmS[(st.bpos >> 5) * 32] << (st.bpos & 31);
            if (w) { st.bpos += __clz(w); found = true; break; }
            st.bpos = (st.bpos | 31u) + 1u;
        }
        if (!found) break;
        const XRaw<NB> xv = x_load<NB>(smem_u32(xs) + st.bpos * (uint32_t)x_col_bytes(NB));
        st.bpos += 1;
        x_fma<NB>(xv, __float_as_uint(nlut[(fword >> (28 - 4 * e)) & 15u]), st.acc);
    }
    return st;
}

template <int NB>
__device__ __forceinline__ void chunk_dot_mx4(const uint32_t* __restrict__ sb, const SbGeom& g, int ch, int lane,
                                              int chunk_elems, const float* __restrict__ xs,
                                              const float* __restrict__ nlut, float (&acc)[NB]) {
    constexpr uint32_t XS = (uint32_t)x_col_bytes(NB);
    const uint32_t e0 = sb[g.tab + ch * 32 + lane];
    const uint32_t* bmS = sb + g.bm + lane;
    const uint32_t bm_a = smem_u32(bmS), xs_a = smem_u32(xs), nl_a = smem_u32(nlut);      // nlut is 64-byte aligned
    uint32_t fl_a = smem_u32(sb + g.fl + lane) + (uint32_t)(ch * chunk_elems / 8) * 128u;
    const uint32_t ex_a = smem_u32(sb + g.un + lane);
    const int kept = (int)(sb[g.tab + g.n_ch * 32 + lane] >> 20);
    const int m = max(0, min(chunk_elems, kept - ch * chunk_elems));
    const int n_full = __reduce_min_sync(0xffffffffu, m) / kGroupCols;
    const int n_groups = ceil_div(__reduce_max_sync(0xffffffffu, m), kGroupCols);
    uint32_t bpos = e0 >> 20;
    const uint32_t blk0 = (e0 & 0xFFFFFu) >> 3;                 // index of the chunk's first exponent byte
    const uint32_t bpos_lim = (uint32_t)(g.bm_words * 32);
    float blk[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) blk[b] = 0.f;

    auto group = [&](int grp, auto tail_c) {
        constexpr bool tail = decltype(tail_c)::value;
        WalkState<NB> st0;
#pragma unroll
        for (int b = 0; b < NB; ++b) st0.acc[b] = blk[b];
        st0.bpos = bpos; st0.upos = 0;
        const uint32_t ba = bm_a + (bpos >> 5) * 128u;
        uint32_t bv = __funnelshift_l(lds_u32_off<128>(ba), lds_u32(ba), bpos);
        const uint32_t xg = xs_a + bpos * XS + 31u * XS;
        const uint32_t fword = lds_u32(fl_a);
        const int rem = m - grp * kGroupCols;
        uint32_t dry = 0, p = 0;
#pragma unroll
        for (int e = 0; e < kGroupCols; ++e) {
            p = bfind_u32(bv);
            const XRaw<NB> xv = x_load<NB>(mad_lo(p, 0u - XS, xg));
            bv &= ~shl_sat(1u, p);
            const uint32_t off = e < 7 ? (fword >> (26 - 4 * e)) : (fword << 2);
            const uint32_t wb = lds_u32((off & 0x3Cu) | nl_a);                         // +-(magnitude << 4) as a float
            if (!tail) {
                x_fma<NB>(xv, wb, blk);
            } else if (e < rem) {
                x_fma<NB>(xv, wb, blk);
                dry |= p;
            }
        }
        bpos += 32u - p;
        if (tail) bpos = min(bpos, bpos_lim);
        else dry |= p;
        if ((int32_t)dry < 0) {
            const WalkState<NB> r = group_slow_mx<NB>(bmS, fword, min(rem, kGroupCols), st0, bpos_lim, xs, nlut);
#pragma unroll
            for (int b = 0; b < NB; ++b) blk[b] = r.acc[b];
            bpos = r.bpos;
        }
        fl_a += 128u;
        if ((grp & 3) == 3 || grp == n_groups - 1) {              // a block of 32 values is complete: apply its scale
            const uint32_t bi = blk0 + (uint32_t)(grp >> 2);
            const uint32_t eb = (lds_u32(ex_a + (bi >> 2) * 128u) >> (24u - 8u * (bi & 3u))) & 0xFFu;
            const float scale = __uint_as_float(eb >= 7u ? (eb - 6u) << 23 : 0u);     // 2^(E - 133)
#pragma unroll
            for (int b = 0; b < NB; ++b) { acc[b] = fmaf(blk[b], scale, acc[b]); blk[b] = 0.f; }
        }
    };
    int grp = 0;
    for (; grp < n_full; ++grp) group(grp, std::false_type{});
    for (; grp < n_groups; ++grp) group(grp, std::true_type{});
}

// T >= 0: fast path for regular chunks, generic path otherwise.  T = -1: generic path only (any t).
// T = 104: Cassandra-2 blob with t = 4 (fast path); T = -2: Cassandra-2 blob, generic path (any t).
// grid = (n_seg, G): CTA (seg, j) handles the superblocks (rb, seg) for rb = j, j + G, ...
// NB vectors x[b] (bf16 [NB][k]) are multiplied in the same pass: every decoded weight is used NB times, and each
// vector's sums are formed in the same order as with NB = 1.
template <int T, int NB>
__global__ void __launch_bounds__(1024) k_draft_gemv(const uint32_t* __restrict__ blob, const uint16_t* __restrict__ x,
                                                     float* __restrict__ partial, int32_t* __restrict__ d_status,
                                                     int stage_bytes, int max_sb, int n, int k, int t, int seg_cols,
                                                     int chunk_cols, int n_seg, int n_rb, unsigned long long blob_bytes) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // The geometry comes from the host's copy of the header (the launch sized shared memory from it); the header
    // itself is fetched now and compared once it has arrived, so that its latency is off the critical path.
    const uint32_t* h = blob;
    const uint32_t h_n = h[H_ROWS], h_k = h[H_COLS], h_t = h[H_T], h_seg = h[H_SEG], h_chunk = h[H_CHUNK], h_nseg = h[H_NSEG],
                   h_nrb = h[H_NRB], h_magic = h[H_MAGIC];
    const int k_pad = ceil_div(k, 32) * 32;
    const int seg = blockIdx.x, rb0 = blockIdx.y, rb_step = gridDim.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;

    float* xs = reinterpret_cast<float*>(smem_raw + (size_t)kGemvStages * stage_bytes);
    uint32_t* lut = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(xs) + (size_t)(seg_cols + kXSlack) * x_col_bytes(NB));
    float* red = reinterpret_cast<float*>(lut + 256);                       // NB = 1: [2][n_warps][32], else [NB][n_warps][32]
    uint64_t* bar = reinterpret_cast<uint64_t*>(red + (NB < 2 ? 2 : NB) * n_warps * 32);    // [kGemvStages]
    __shared__ int s_skip[kGemvStages];

    const int scols = seg_cols_of(k_pad, seg_cols, seg);
    const int n_ch = ceil_div(scols, chunk_cols);
    // The launch sized shared memory from the host's copy of the header; a blob that does not match it is
    // refused instead of overrunning the buffers.
    if (seg >= n_seg || (int)blockDim.x < 32 * n_ch || n_ch > 32 || (T == 104 && (smem_u32(lut) & 63u))) {
        if (tid == 0 && d_status) atomicExch(d_status, CASS_ERR_INVALID_ARG);
        return;
    }
    const int n_tiles = rb0 < n_rb ? (n_rb - rb0 + rb_step - 1) / rb_step : 0;

    if (tid == 0) {
        for (int s = 0; s < kGemvStages; ++s) mbar_init(&bar[s], 1);
        fence_mbar_init();
    }
    __syncthreads();

    // thread 0: start the copy of tile i into stage i % kGemvStages.  Nothing is read beyond blob + blob_bytes (the
    // size the caller's description gives): a directory entry that points outside is skipped and flagged.
    auto issue = [&](int i) {
        const int s = i % kGemvStages;
        const int sb_i = (rb0 + i * rb_step) * n_seg + seg;
        const uint32_t* dir = blob + kBlobDirOffset / 4 + sb_i * 4;
        const bool dir_ok = (unsigned long long)kBlobDirOffset + ((unsigned long long)sb_i + 1ull) * 16ull <= blob_bytes;
        const uint32_t d0 = dir_ok ? dir[0] : 0u, d1 = dir_ok ? dir[1] : 0u, d2 = dir_ok ? dir[2] : 0u, d3 = dir_ok ? dir[3] : 0u;
        const SbGeom g = SbGeom::make(dir_n_ch(d3), scols, (int)d1, (int)d2);
        const uint32_t bytes = (uint32_t)g.total * 4u;
        if (!dir_ok || bytes > (uint32_t)max_sb || dir_n_ch(d3) != n_ch || d1 > 0xFFFFu || d2 > 0xFFFFu ||
            (unsigned long long)d0 * 16ull + bytes > blob_bytes) {                // does not fit: skip the tile, flag it
            s_skip[s] = 1;
            if (d_status) atomicExch(d_status, CASS_ERR_INVALID_ARG);
            mbar_expect_tx(&bar[s], 0);
            return;
        }
        s_skip[s] = 0;
        const uint8_t* src = reinterpret_cast<const uint8_t*>(blob) + (size_t)d0 * 16;
        uint8_t* dst = smem_raw + (size_t)s * stage_bytes;
        mbar_expect_tx(&bar[s], bytes);
        for (uint32_t off = 0; off < bytes; off += 32768u) bulk_g2s(dst + off, src + off, min(32768u, bytes - off), &bar[s]);
    };
    if (tid == 0) {
        for (int i = 0; i < kGemvStages && i < n_tiles; ++i) issue(i);
    }
    // the rank -> exponent table, pre-shifted into place
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(blob) + kBlobHeaderBytes;
    if (T == 104) {
        // signed magnitudes of the 16 field values, as floats: (+-) (m << 4)
        if (tid < 16) reinterpret_cast<float*>(lut)[tid] = (tid & 8 ? -16.f : 16.f) * (float)(tid & 7);
    } else {
        for (int i = tid; i < 256; i += blockDim.x) lut[i] = (uint32_t)cb[i] << 23;
    }
    // Everything above touches only the blob, which no kernel writes.  When the launch allows this grid to start
    // before its predecessor in the stream has finished, wait here: x and the scratch `partial` are the predecessor's.
    pdl_wait();
    // x of this segment (fp32), zero beyond the matrix
    const int c0 = seg * seg_cols;
    if constexpr (NB > 1) {
        // packed bf16 [col][NB]: all vectors' values of one column side by side
        uint16_t* xs16 = reinterpret_cast<uint16_t*>(xs);
        if ((k & 7) == 0 && ((uintptr_t)x & 15) == 0) {
            const int n_oct = (seg_cols + kXSlack) / 8;
            for (int it = tid; it < n_oct * NB; it += blockDim.x) {
                const int i = (it / NB) * 8, b = it % NB;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (i < scols && c0 + i < k) v = *reinterpret_cast<const uint4*>(x + (size_t)b * k + c0 + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    xs16[(size_t)(i + 2 * q) * NB + b] = (uint16_t)(w[q] & 0xFFFFu);
                    xs16[(size_t)(i + 2 * q + 1) * NB + b] = (uint16_t)(w[q] >> 16);
                }
            }
        } else {
            for (int it = tid; it < (seg_cols + kXSlack) * NB; it += blockDim.x) {
                const int i = it / NB, b = it % NB, c = c0 + i;
                xs16[it] = (i < scols && c < k) ? x[(size_t)b * k + c] : (uint16_t)0;
            }
        }
    } else if ((k & 7) == 0 && ((uintptr_t)x & 15) == 0) {
        // eight values per 16-byte load: one round trip to L2 for the whole slice
        for (int i = tid * 8; i < seg_cols + kXSlack; i += blockDim.x * 8) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (i < scols && c0 + i < k) v = *reinterpret_cast<const uint4*>(x + c0 + i);
            float4 lo = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                                    __uint_as_float(v.y & 0xFFFF0000u));
            float4 hi = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u), __uint_as_float(v.w << 16),
                                    __uint_as_float(v.w & 0xFFFF0000u));
            *reinterpret_cast<float4*>(xs + i) = lo;
            *reinterpret_cast<float4*>(xs + i + 4) = hi;
        }
    } else {
        for (int i = tid; i < seg_cols + kXSlack; i += blockDim.x) {
            int c = c0 + i;
            xs[i] = (i < scols && c < k) ? bf16_bits_to_float(x[c]) : 0.f;
        }
    }
    __syncthreads();
    if (h[H_MODE] != ((T == 104 || T == -2) ? kBlobModeMx : kBlobModeUnary) || h_magic != kBlobMagic || (int)h_n != n || (int)h_k != k || (int)h_t != t || (int)h_seg != seg_cols ||
        (int)h_chunk != chunk_cols || (int)h_nseg != n_seg || (int)h_nrb != n_rb) {
        // not the blob the caller described: flag it, let the copies already started land, produce nothing
        if (tid == 0 && d_status) atomicExch(d_status, CASS_ERR_INVALID_ARG);
        for (int j = 0; j < n_tiles && j < kGemvStages; ++j) mbar_wait_bounded(&bar[j % kGemvStages], 0u);
        return;
    }

    for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kGemvStages;
        const int rb = rb0 + i * rb_step;
        if (!mbar_wait_bounded(&bar[s], (uint32_t)(i / kGemvStages) & 1u)) {
            // give up: flag the error, let the copies still in flight into this CTA's buffers land (bounded), leave
            if (d_status) atomicExch(d_status, CASS_ERR_TIMEOUT);
            for (int j = i; j < n_tiles && j < i + kGemvStages; ++j)
                mbar_wait_bounded(&bar[j % kGemvStages], (uint32_t)(j / kGemvStages) & 1u);
            return;
        }
        const uint32_t* sb = reinterpret_cast<const uint32_t*>(smem_raw + (size_t)s * stage_bytes);
        float acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc[b] = 0.f;
        if (warp < n_ch && !s_skip[s]) {
            const uint32_t* dir = blob + kBlobDirOffset / 4 + (rb * n_seg + seg) * 4;
            const SbGeom g = SbGeom::make(n_ch, scols, (int)dir[1], (int)dir[2]);
            if (T == 104) {
                chunk_dot_mx4<NB>(sb, g, warp, lane, dir_chunk_elems(dir[3]), xs, reinterpret_cast<const float*>(lut), acc);
            } else if (T == -2) {
                const uint32_t xs_a = smem_u32(xs);
                decode_chunk_generic_mx(sb, g, dir_chunk_elems(dir[3]), warp, lane, t, [&](int col, uint16_t bits) {
                    x_fma<NB>(x_load<NB>(xs_a + (uint32_t)col * (uint32_t)x_col_bytes(NB)), (uint32_t)bits << 16, acc);
                });
            } else if (T >= 0) {
                chunk_dot_fast<(T >= 0 && T <= 5 ? T : 0), NB>(sb, g, warp, lane, dir_chunk_elems(dir[3]), xs, lut, acc);
            } else {
                const uint32_t xs_a = smem_u32(xs);
                decode_chunk_generic(sb, g, dir_chunk_elems(dir[3]), warp, lane, t, cb, [&](int col, uint16_t bits) {
                    x_fma<NB>(x_load<NB>(xs_a + (uint32_t)col * (uint32_t)x_col_bytes(NB)), (uint32_t)bits << 16, acc);
                });
            }
        }
        const size_t n_pad = (size_t)n_rb * kRowsPerBlock;
        const int row = rb * kRowsPerBlock + lane;
        if constexpr (NB == 1) {
            float* red_i = red + (i & 1) * n_warps * 32;
            red_i[warp * 32 + lane] = acc[0];
            __syncthreads();                              // all reads of stage s are done; partial sums are visible
            if (tid == 0 && i + kGemvStages < n_tiles) {
                fence_proxy_async();
                issue(i + kGemvStages);
            }
            if (warp == 0) {
                float sum = 0.f;
                for (int w = 0; w < n_ch; ++w) sum += red_i[w * 32 + lane];
                if (row < n) partial[(size_t)seg * n_pad + row] = sum;
            }
        } else {
#pragma unroll
            for (int b = 0; b < NB; ++b) red[(b * n_warps + warp) * 32 + lane] = acc[b];
            __syncthreads();
            if (tid == 0 && i + kGemvStages < n_tiles) {
                fence_proxy_async();
                issue(i + kGemvStages);
            }
            for (int b = warp; b < NB; b += n_warps) {    // vector b's chunk sums, added in chunk order as with NB = 1
                float sum = 0.f;
                for (int w = 0; w < n_ch; ++w) sum += red[(b * n_warps + w) * 32 + lane];
                if (row < n) partial[((size_t)b * n_seg + seg) * n_pad + row] = sum;
            }
            __syncthreads();                              // the sums are read before the next tile overwrites them
        }
    }
}

// grid.y = vector b: partial [b][n_seg][n_pad] -> y [b][n]
__global__ void k_gemv_finish(const float* __restrict__ partial, int n, int n_pad, int n_seg,
                              uint16_t* __restrict__ y_bf16, float* __restrict__ y_f32) {
    pdl_wait();
    int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    const int b = blockIdx.y;
    partial += (size_t)b * n_seg * n_pad;
    float acc = 0.f;
    for (int s = 0; s < n_seg; ++s) acc += partial[(size_t)s * n_pad + r];
    if (y_f32) y_f32[(size_t)b * n + r] = acc;
    if (y_bf16) y_bf16[(size_t)b * n + r] = float_to_bf16_bits(acc);
}

static int gemv_sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

int launch_draft_gemv(const void* blob, const cass_blob_info& bi, const void* x_bf16, int nb, float* partial,
                      int32_t* d_status, cudaStream_t stream) {
    const int n_ch = ceil_div(bi.seg_cols, bi.chunk_cols);
    if (n_ch > 32) return CASS_ERR_UNSUPPORTED;
    if (nb != 1 && nb != 2 && nb != 4 && nb != 8) return CASS_ERR_UNSUPPORTED;
    const size_t smem = gemv_smem_bytes(bi, nb);
    if (smem > 227 * 1024) return CASS_ERR_CAPACITY;
    const int threads = 32 * n_ch;
    // One vector: one CTA per superblock -- the hardware hands out CTAs as shared memory frees, which balances the SMs to
    // within one superblock (a grid of as many CTAs as fit at once, each looping over its share, left SMs with 4 x 4
    // superblocks beside SMs with 4 x 3: 56.7 instead of 54.4 us on the 28672 x 4096 matrix).  Several vectors: the x
    // slice a CTA stages is nb times larger, so CTAs keep theirs and loop (one CTA per superblock: 52.3 instead of
    // 48.6 ms per step with 8 sequences).
    int g = bi.n_rowblocks;
    if (nb > 1) {
        int per_sm = (int)((228 * 1024) / (smem + 1024));
        if (per_sm > 2048 / threads) per_sm = 2048 / threads;
        if (per_sm < 1) per_sm = 1;
        g = ceil_div(gemv_sm_count() * per_sm, bi.n_seg);
        if (g > bi.n_rowblocks) g = bi.n_rowblocks;
    }
    if (g < 1) g = 1;
    dim3 grid(bi.n_seg, g), block(threads);
    const uint32_t* b = (const uint32_t*)blob;
    const uint16_t* x = (const uint16_t*)x_bf16;
    const int stage = (int)gemv_stage_bytes(bi);
#define CASS_GEMV_LAUNCH(TT, NN)                                                                               \
    do {                                                                                                       \
        static int attr_smem = 0;      /* largest size already granted to this instantiation */              \
        if ((int)smem > attr_smem) {                                                                           \
            CASS_CUDA_CHECK(cudaFuncSetAttribute(k_draft_gemv<TT, NN>, cudaFuncAttributeMaxDynamicSharedMemorySize,\
                                                 (int)smem));                                                  \
            attr_smem = (int)smem;                                                                             \
        }                                                                                                      \
        cudaLaunchConfig_t cfg = {};                                                                           \
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;            \
        cudaLaunchAttribute at[1];                                                                             \
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   /* prologue may overlap the predecessor */ \
        at[0].val.programmaticStreamSerializationAllowed = pdl_enabled();                                                  \
        cfg.attrs = at; cfg.numAttrs = 1;                                                                      \
        CASS_CUDA_CHECK(cudaLaunchKernelEx(&cfg, k_draft_gemv<TT, NN>, b, x, partial, d_status, stage,         \
                                           (int)bi.max_superblock_bytes, (int)bi.rows, (int)bi.cols,           \
                                           (int)bi.trunc_bits, (int)bi.seg_cols, (int)bi.chunk_cols,           \
                                           (int)bi.n_seg, (int)bi.n_rowblocks,                                 \
                                           (unsigned long long)bi.total_bytes));                               \
    } while (0)
#define CASS_GEMV_LAUNCH_NB(TT)                                                                                \
    do {                                                                                                       \
        if (nb == 1) CASS_GEMV_LAUNCH(TT, 1);                                                                  \
        else if (nb == 2) CASS_GEMV_LAUNCH(TT, 2);                                                             \
        else if (nb == 4) CASS_GEMV_LAUNCH(TT, 4);                                                             \
        else CASS_GEMV_LAUNCH(TT, 8);                                                                          \
    } while (0)
    if (bi.mode == 2 && bi.trunc_bits == 4) CASS_GEMV_LAUNCH_NB(104);
    else if (bi.mode == 2) CASS_GEMV_LAUNCH_NB(-2);
    else if (bi.trunc_bits == 4) CASS_GEMV_LAUNCH_NB(4);
    else if (bi.trunc_bits == 0) CASS_GEMV_LAUNCH_NB(0);
    else if (bi.trunc_bits == 1) CASS_GEMV_LAUNCH_NB(1);          // fields that do not tile a word: the design-space sweep of Sec. 7.2
    else if (bi.trunc_bits == 2) CASS_GEMV_LAUNCH_NB(2);
    else if (bi.trunc_bits == 3) CASS_GEMV_LAUNCH_NB(3);
    else if (bi.trunc_bits == 5) CASS_GEMV_LAUNCH_NB(5);
    else CASS_GEMV_LAUNCH_NB(-1);
#undef CASS_GEMV_LAUNCH_NB
#undef CASS_GEMV_LAUNCH
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

}  // namespace cass

using namespace cass;

extern "C" int cass_draft_gemv(const void* blob, const cass_blob_info* h_info, const void* x_bf16, float* partial,
                               void* y_bf16, float* y_f32, int32_t* d_status, void* stream_) {
    if (!blob || !h_info || !x_bf16 || !partial) return CASS_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    int rc = launch_draft_gemv(blob, *h_info, x_bf16, 1, partial, d_status, stream);
    if (rc) return rc;
    if (!y_bf16 && !y_f32) return CASS_OK;
    int n_pad = h_info->n_rowblocks * kRowsPerBlock;
    k_gemv_finish<<<ceil_div(h_info->rows, 256), 256, 0, stream>>>(partial, h_info->rows, n_pad, h_info->n_seg,
                                                                    (uint16_t*)y_bf16, y_f32);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

extern "C" int cass_draft_gemv_batch(const void* blob, const cass_blob_info* h_info, const void* x_bf16, int n_vec,
                                     float* partial, void* y_bf16, float* y_f32, int32_t* d_status, void* stream_) {
    if (!blob || !h_info || !x_bf16 || !partial) return CASS_ERR_INVALID_ARG;
    if (n_vec != 1 && n_vec != 2 && n_vec != 4 && n_vec != 8) return CASS_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    int rc = launch_draft_gemv(blob, *h_info, x_bf16, n_vec, partial, d_status, stream);
    if (rc) return rc;
    if (!y_bf16 && !y_f32) return CASS_OK;
    int n_pad = h_info->n_rowblocks * kRowsPerBlock;
    k_gemv_finish<<<dim3(ceil_div(h_info->rows, 256), n_vec), 256, 0, stream>>>(partial, h_info->rows, n_pad, h_info->n_seg,
                                                                                 (uint16_t*)y_bf16, y_f32);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

// ---- variant with built-in scratch ------------------------------------------------------------------------
// The split-K partial sums of this variant live in a fixed array inside the library image, so the call needs no
// scratch buffer from its caller.  Every GPU that loads the library holds the array (2 MiB) until the process ends.
static __device__ __align__(256) float g_static_partial[CASS_STATIC_PARTIAL_FLOATS];

extern "C" int cass_draft_gemv_static(const void* blob, const cass_blob_info* h_info, const void* x_bf16, void* y_bf16,
                                      float* y_f32, int32_t* d_status, void* stream_) {
    if (!blob || !h_info || !x_bf16 || (!y_bf16 && !y_f32)) return CASS_ERR_INVALID_ARG;
    if (h_info->n_seg <= 0 || h_info->n_rowblocks <= 0) return CASS_ERR_INVALID_ARG;
    const size_t need = (size_t)h_info->n_seg * h_info->n_rowblocks * kRowsPerBlock;
    if (need > (size_t)CASS_STATIC_PARTIAL_FLOATS) return CASS_ERR_CAPACITY;     // matrix too large for the built-in scratch
    // In host code the array's name is only a handle; its device address is looked up once per device, with that
    // device current, and kept.
    constexpr int kMaxDevices = 64;
    static float* s_scratch[kMaxDevices] = {nullptr};
    int dev = -1;
    CASS_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CASS_ERR_UNSUPPORTED;
    if (!s_scratch[dev]) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_static_partial) != cudaSuccess || !ptr) return CASS_ERR_CUDA;
        s_scratch[dev] = ptr;
    }
    float* partial = s_scratch[dev];
    cudaStream_t stream = (cudaStream_t)stream_;
    int rc = launch_draft_gemv(blob, *h_info, x_bf16, 1, partial, d_status, stream);
    if (rc) return rc;
    const int n_pad = h_info->n_rowblocks * kRowsPerBlock;
    k_gemv_finish<<<ceil_div(h_info->rows, 256), 256, 0, stream>>>(partial, h_info->rows, n_pad, h_info->n_seg,
                                                                    (uint16_t*)y_bf16, y_f32);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
