// Weight-blob format (device side): header indices, superblock geometry, and the generic
// sequential decoder of one (row, chunk).
//
// Blob = header (128 B) | codebook rank->exponent (256 B) | directory (16 B per superblock) | bodies.
// A superblock holds 32 rows x one column segment: chunk table, bitmap, fields and unary sections, each
// interleaved word by word over the 32 rows (word j of row r at index j*32 + r).  A chunk-table entry is
// (index of the chunk's first field word << 20) | bit offset of the chunk's first codeword; the fields of
// every chunk start on a word boundary; the last entry holds the segment totals.  Bit streams are filled
// MSB first.
#pragma once

#include "common.cuh"

namespace cass {

enum BlobHeaderWord {
    H_MAGIC = 0, H_VERSION, H_ROWS, H_COLS, H_P, H_T, H_SEG, H_CHUNK, H_NSEG, H_NRB, H_KEPT,
    H_DIROFF, H_BODYOFF, H_TOTLO, H_TOTHI, H_MAXSB, H_MODE
};
// H_MODE: 0 = Cassandra-1 (unary exponent code, the layout described above), 2 = Cassandra-2 (MX: the kept values of
// a row are cut into blocks of 32 that share one exponent byte; fields hold sign + the high 7-t bits of a 7-bit
// magnitude, packed from the most significant end; the fourth section holds the exponent bytes, four per word from
// the most significant end; a table entry's low 20 bits are 8 x the index of the chunk's first block).
constexpr uint32_t kBlobModeUnary = 0, kBlobModeMx = 2;
constexpr int kMxBlock = 32;
constexpr uint32_t kBlobMagic = 0x57534143u;
constexpr uint32_t kBlobVersion = 3;
constexpr int kBlobHeaderBytes = 128;
constexpr int kBlobCodebookBytes = 256;
constexpr int kBlobDirOffset = kBlobHeaderBytes + kBlobCodebookBytes;

// Word offsets of the sections of one superblock.
struct SbGeom {
    int n_ch;       // chunks in this segment
    int bm_words;   // bitmap words per row
    int w_f, w_u;   // field / unary words per row
    int tab, bm, fl, un, total;   // section starts and total size, in words

    __host__ __device__ static SbGeom make(int n_ch, int seg_cols_here, int w_f, int w_u) {
        SbGeom g;
        g.n_ch = n_ch;
        g.bm_words = seg_cols_here / 32;
        g.w_f = w_f;
        g.w_u = w_u;
        g.tab = 0;
        g.bm = g.tab + (n_ch + 1) * 32;
        g.fl = g.bm + g.bm_words * 32;
        g.un = g.fl + w_f * 32;
        g.total = g.un + w_u * 32;
        return g;
    }
};

__host__ __device__ inline int dir_n_ch(uint32_t w3) { return (int)(w3 & 0xFFu); }
__host__ __device__ inline int dir_chunk_elems(uint32_t w3) { return (int)(w3 >> 8); }
__host__ __device__ inline int chunk_elems_for(int max_kept, int n_ch) {       // smallest multiple of 8 with n_ch * E >= max_kept
    int per_chunk = ceil_div(max_kept, n_ch);
    int e = ceil_div(per_chunk, 8) * 8;
    return e < 8 ? 8 : e;
}

__host__ __device__ inline int mx_chunk_elems_for(int max_kept, int n_ch) {    // smallest multiple of 32 with n_ch * E >= max_kept
    int per_chunk = ceil_div(max_kept, n_ch);
    int e = ceil_div(per_chunk, kMxBlock) * kMxBlock;
    return e < kMxBlock ? kMxBlock : e;
}

// Cassandra-2 element -> bf16 bits: field = sign, magnitude >> t (8-t bits); value = (-1)^s (mag << t) 2^(E-133);
// the leading-zero count of the magnitude gives the shift and the exponent correction; zero magnitude -> +0.
__device__ __forceinline__ uint16_t mx_value_bf16(uint32_t field, uint32_t e_blk, int t) {
    const uint32_t mag = (field & ((1u << (7 - t)) - 1u)) << t;
    if (mag == 0) return 0;
    const int top = 31 - __clz(mag);
    return (uint16_t)(((field >> (7 - t)) << 15) | ((e_blk - 6u + (uint32_t)top) << 7) | ((mag << (7 - top)) & 0x7Fu));
}
__device__ __forceinline__ uint32_t mx_field_of(uint32_t fword, int j, int t) {        // field j of a word
    const int w = 8 - t;
    return (fword >> (32 - w * (j + 1))) & ((1u << w) - 1u);
}

__host__ __device__ inline int seg_cols_of(int k_pad, int seg_cols, int seg) {
    int rest = k_pad - seg * seg_cols;
    return rest < seg_cols ? rest : seg_cols;
}

// Reads one codeword starting at absolute bit `ub` of a row's unary stream (words un[j*32]); returns the
// number of zeros before the terminating one and advances ub past it.  Handles codewords of any length.
// `limit_bits` bounds the scan so that a corrupt stream cannot run away.
__device__ __forceinline__ int read_unary(const uint32_t* un_row, uint32_t& ub, uint32_t limit_bits) {
    int rank = 0;
    while (ub < limit_bits) {
        uint32_t w = un_row[(ub >> 5) * 32] << (ub & 31);
        int avail = 32 - (int)(ub & 31);
        if (w) {
            int s = __clz(w);
            ub += s + 1;
            return rank + s;
        }
        rank += avail;
        ub += avail;
    }
    return rank;
}

// Generic decoder of one (row, chunk): calls emit(col_in_segment, bf16_bits) for every kept value of the chunk, in
// column order.  `sb` points at the superblock's first word (global or shared memory); `row` in [0,32).
template <class Emit>
__device__ inline void decode_chunk_generic(const uint32_t* sb, const SbGeom& g, int chunk_elems, int ch, int row,
                                            int t, const uint8_t* rank_to_exp, Emit&& emit) {
    const int per = 32 / (8 - t);
    const uint32_t e0 = sb[g.tab + ch * 32 + row];
    const int kept = (int)(sb[g.tab + g.n_ch * 32 + row] >> 20);
    const int k0 = ch * chunk_elems;
    const int cnt = min(chunk_elems, kept - k0);
    if (cnt <= 0) return;
    uint32_t col = e0 >> 20, ub = e0 & 0xFFFFFu;
    const uint32_t* fl_row = sb + g.fl + row;
    const uint32_t* un_row = sb + g.un + row;
    const uint32_t limit = (uint32_t)g.w_u * 32u;
    const uint32_t col_lim = (uint32_t)g.bm_words * 32u;
    for (int k = k0; k < k0 + cnt; ++k) {
        bool found = false;
        while (col < col_lim) {
            uint32_t bm = sb[g.bm + (col >> 5) * 32 + row] << (col & 31);
            if (bm) { col += __clz(bm); found = true; break; }
            col = (col | 31u) + 1u;
        }
        if (!found) return;                                   // corrupt stream: stop inside the buffers
        uint32_t fword = fl_row[(k / per) * 32];
        int rank = read_unary(un_row, ub, limit);
        uint32_t e = rank_to_exp[rank & 255];
        emit((int)col, (uint16_t)(field_sign_mant_bf16(fword, k % per, t) | (e << 7)));
        col += 1;
    }
}

// The same with the truncation known at compile time (no run-time divisions in the field arithmetic): what a kernel
// that decodes whole matrices uses.  `lut`: rank -> exponent << 7 (bf16 position), 256 entries.
template <int T, class Emit>
__device__ __forceinline__ void decode_chunk_fixed(const uint32_t* sb, const SbGeom& g, int chunk_elems, int ch, int row,
                                                   const uint16_t* lut, Emit&& emit) {
    constexpr int F = 8 - T, PER = 32 / F;
    constexpr uint32_t KEEP = 0x8000u | (0x7Fu & ~((1u << T) - 1u));    // sign + kept mantissa bits of a bf16
    const uint32_t e0 = sb[g.tab + ch * 32 + row];
    const int kept = (int)(sb[g.tab + g.n_ch * 32 + row] >> 20);
    const int k0 = ch * chunk_elems;
    const int cnt = min(chunk_elems, kept - k0);
    if (cnt <= 0) return;
    uint32_t col = e0 >> 20, ub = e0 & 0xFFFFFu;
    const uint32_t* bm_row = sb + g.bm + row;
    const uint32_t* fl_row = sb + g.fl + row;
    const uint32_t* un_row = sb + g.un + row;
    const uint32_t limit = (uint32_t)g.w_u * 32u, col_lim = (uint32_t)g.bm_words * 32u;
    uint32_t bw = col < col_lim ? bm_row[(col >> 5) * 32] << (col & 31) : 0u;      // bitmap bits from `col` on, left-aligned
    for (uint32_t k = (uint32_t)k0; k < (uint32_t)(k0 + cnt); ++k) {
        while (!bw) {                                                              // nothing kept up to the word's end: next bitmap word
            col = (col + 31u) & ~31u;                                              // the next word boundary (col itself when on one)
            if (col >= col_lim) return;                                            // corrupt stream: stop inside the buffers
            bw = bm_row[(col >> 5) * 32];
            if (!bw) col += 1u;                                                    // an empty word: the next round moves past it
        }
        const uint32_t z = __clz(bw);
        col += z;
        const int rank = read_unary(un_row, ub, limit);
        const uint32_t fword = fl_row[(k / PER) * 32], j = k % PER;
        uint32_t sm;
        if constexpr (32 % F == 0) sm = (__funnelshift_l(fword, fword, (F * j) & 31) >> 16) & KEEP;
        else {
            const uint32_t f = (fword >> (32u - (uint32_t)F * (j + 1u))) & ((1u << F) - 1u);
            sm = ((f >> (F - 1)) << 15) | ((f & ((1u << (F - 1)) - 1u)) << T);
        }
        emit((int)col, (uint16_t)(sm | lut[rank & 255]));
        col += 1;
        bw = z >= 31u ? 0u : (bw << (z + 1u));                                     // bit 31 is column `col` again; 0 once the word is used up
    }
}

// The same for a Cassandra-2 blob (shared exponent per block of 32 kept values instead of a codeword per value).
template <class Emit>
__device__ inline void decode_chunk_generic_mx(const uint32_t* sb, const SbGeom& g, int chunk_elems, int ch, int row,
                                               int t, Emit&& emit) {
    const int per = 32 / (8 - t);
    const uint32_t e0 = sb[g.tab + ch * 32 + row];
    const int kept = (int)(sb[g.tab + g.n_ch * 32 + row] >> 20);
    const int k0 = ch * chunk_elems;
    const int cnt = min(chunk_elems, kept - k0);
    if (cnt <= 0) return;
    uint32_t col = e0 >> 20;
    const uint32_t* fl_row = sb + g.fl + row;
    const uint32_t* ex_row = sb + g.un + row;
    const uint32_t col_lim = (uint32_t)g.bm_words * 32u;
    for (int k = k0; k < k0 + cnt; ++k) {
        bool found = false;
        while (col < col_lim) {
            uint32_t bm = sb[g.bm + (col >> 5) * 32 + row] << (col & 31);
            if (bm) { col += __clz(bm); found = true; break; }
            col = (col | 31u) + 1u;
        }
        if (!found) return;
        const int b = k / kMxBlock;
        if (b / 4 >= g.w_u) return;                           // corrupt geometry: stay inside the buffers
        const uint32_t e_blk = (ex_row[(b / 4) * 32] >> (24 - 8 * (b % 4))) & 0xFFu;
        emit((int)col, mx_value_bf16(mx_field_of(fl_row[(k / per) * 32], k % per, t), e_blk, t));
        col += 1;
    }
}

}  // namespace cass
