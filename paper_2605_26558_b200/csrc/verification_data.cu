// Verification data (Sec. 4.1 target inference, Sec. 5.1 encoder): what the Cassandra-1 speculation data leaves out
// -- the low t mantissa bits of the kept values and the pruned values as they are -- and the exact reconstruction
// of the bf16 matrix from the two parts (k_decode_full).  A session told to verify from the two parts
// (cass_session_verify_from_parts) rebuilds every matrix with it right before the verification GEMM reads it.
//
// Layout: header of 8 words {magic 'CASV', 1, rows, cols, kept per row, t, words per row, 0}; per row
// ceil(kept*t/32) words of t-bit groups (kept values in column order, MSB first), then the pruned values in column
// order as 16-bit halfwords (little endian, padded to a word).  Every row has the same kept count, so rows are
// equally long.  The bitmap is the one in the speculation data.
#include "wblob.cuh"

namespace cass {

constexpr uint32_t kVdataMagic = 0x56534143u;
constexpr int kVdataHeaderWords = 8;

__host__ __device__ inline int vdata_lo_words(int kept, int t) { return (kept * t + 31) / 32; }
__host__ __device__ inline int vdata_row_words(int cols, int kept, int t) { return vdata_lo_words(kept, t) + (cols - kept + 1) / 2; }

// Bitmap word j (32 columns) of `row` inside the blob: superblock (row / 32, segment), bitmap section, interleaved.
__device__ __forceinline__ uint32_t blob_bitmap_word(const uint32_t* __restrict__ blob, int row, int j, int seg_cols, int n_seg,
                                                     int k_pad) {
    const int seg = (j * 32) / seg_cols, jj = j - seg * (seg_cols / 32);
    const uint32_t* dir = blob + kBlobDirOffset / 4 + ((row / kRowsPerBlock) * n_seg + seg) * 4;
    const SbGeom g = SbGeom::make(dir_n_ch(dir[3]), seg_cols_of(k_pad, seg_cols, seg), (int)dir[1], (int)dir[2]);
    return blob[(size_t)dir[0] * 4 + g.bm + jj * 32 + (row % kRowsPerBlock)];
}

// One warp per row.  ENCODE: W -> verification data.  otherwise: W_out (holding the draft reconstruction) |= low bits,
// pruned positions <- raw values.
template <bool ENCODE>
__global__ void __launch_bounds__(256) k_vdata(const uint32_t* __restrict__ blob, const uint16_t* __restrict__ W,
                                               uint32_t* __restrict__ vdata, uint16_t* __restrict__ W_out) {
    const int n = blob[H_ROWS], k = blob[H_COLS], t = blob[H_T], seg_cols = blob[H_SEG], n_seg = blob[H_NSEG];
    const int kept = blob[H_KEPT], k_pad = ceil_div(k, 32) * 32;
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (row >= n) return;
    const int lo_words = vdata_lo_words(kept, t), row_words = vdata_row_words(k, kept, t);
    uint32_t* lo = vdata + kVdataHeaderWords + (size_t)row * row_words;
    uint16_t* raw = reinterpret_cast<uint16_t*>(lo + lo_words);
    if (ENCODE) {
        for (int w = lane; w < row_words; w += 32) lo[w] = 0u;
        __syncwarp();
    }
    uint32_t k_base = 0, p_base = 0;
    for (int j = 0; j < k_pad / 32; ++j) {
        const uint32_t bm = blob_bitmap_word(blob, row, j, seg_cols, n_seg, k_pad);
        const int c = j * 32 + lane;
        const bool in = c < k, is_kept = (bm >> (31 - lane)) & 1u;
        const uint32_t before = lane ? __popc(bm >> (32 - lane)) : 0u;          // kept columns of this word before mine
        if (in && is_kept && t > 0) {
            const uint32_t bit0 = (k_base + before) * (uint32_t)t;               // first bit of my t-bit group
            const uint32_t sh = bit0 & 31u, wi = bit0 >> 5;
            if (ENCODE) {
                const uint64_t v = (uint64_t)(W[(size_t)row * k + c] & ((1u << t) - 1u)) << (64 - t - sh);
                atomicOr(&lo[wi], (uint32_t)(v >> 32));
                if ((uint32_t)v) atomicOr(&lo[wi + 1], (uint32_t)v);
            } else {
                const uint64_t two = ((uint64_t)lo[wi] << 32) | (sh + t > 32 ? lo[wi + 1] : 0u);
                W_out[(size_t)row * k + c] |= (uint16_t)((two >> (64 - t - sh)) & ((1u << t) - 1u));
            }
        } else if (in && !is_kept) {
            const uint32_t i = p_base + ((uint32_t)lane - before);               // pruned columns before mine
            if (ENCODE) raw[i] = W[(size_t)row * k + c];
            else W_out[(size_t)row * k + c] = raw[i];
        }
        const int valid = min(32, k - j * 32);                                   // columns of this word inside the matrix
        const uint32_t kept_here = __popc(valid >= 32 ? bm : (bm & ~(0xFFFFFFFFu >> valid)));
        k_base += kept_here;
        p_base += (uint32_t)valid - kept_here;
    }
    if (ENCODE && row == 0 && lane == 0) {
        vdata[0] = kVdataMagic; vdata[1] = 1; vdata[2] = n; vdata[3] = k; vdata[4] = kept; vdata[5] = t; vdata[6] = row_words;
        vdata[7] = 0;
    }
}

// Exact reconstruction in one pass (Sec. 4.1 target inference: speculation and verification data are loaded and the
// original values rebuilt; Sec. 5.1 mantissa concatenator).  One CTA per superblock, warp = chunk, lane = row: the lane
// walks its chunk's kept values in column order (the blob's streams are interleaved over the 32 rows, so the warp's
// reads are contiguous), appends each value's low t bits from the row's verification data, and fills the columns
// between kept values with the raw pruned values.  Chunk c owns the columns from its first kept value up to the next
// chunk's first kept value (chunk 0 also the columns before its first value).
__global__ void __launch_bounds__(1024) k_decode_full(const uint32_t* __restrict__ blob, const uint32_t* __restrict__ vdata,
                                                      uint16_t* __restrict__ out) {
    const uint32_t* h = blob;
    const int n = h[H_ROWS], k = h[H_COLS], t = h[H_T], seg_cols = h[H_SEG], n_seg = h[H_NSEG], kept = h[H_KEPT];
    const int k_pad = ceil_div(k, 32) * 32;
    const int sb = blockIdx.x, rb = sb / n_seg, seg = sb % n_seg;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const int scols = seg_cols_of(k_pad, seg_cols, seg);
    const SbGeom sg = SbGeom::make(dir_n_ch(dir[3]), scols, (int)dir[1], (int)dir[2]);
    const int chunk_elems = dir_chunk_elems(dir[3]);
    const uint32_t* body = blob + (size_t)dir[0] * 4;
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(blob) + kBlobHeaderBytes;
    const int lo_words = vdata_lo_words(kept, t), row_words = vdata_row_words(k, kept, t);
    const int ch = threadIdx.x >> 5, r = threadIdx.x & 31, row = rb * kRowsPerBlock + r;
    if (ch >= sg.n_ch || row >= n) return;
    // kept values of this row in the segments before this one (their chunk tables end with the segment's kept count)
    uint32_t kept_before = 0;
    for (int s2 = 0; s2 < seg; ++s2) {
        const uint32_t* d2 = blob + kBlobDirOffset / 4 + (rb * n_seg + s2) * 4;
        const SbGeom g2 = SbGeom::make(dir_n_ch(d2[3]), seg_cols_of(k_pad, seg_cols, s2), (int)d2[1], (int)d2[2]);
        kept_before += blob[(size_t)d2[0] * 4 + g2.tab + g2.n_ch * 32 + r] >> 20;
    }
    const uint32_t* lo = vdata + kVdataHeaderWords + (size_t)row * row_words;
    const uint16_t* raw = reinterpret_cast<const uint16_t*>(lo + lo_words);
    uint16_t* orow = out + (size_t)row * k;
    const int c_base = seg * seg_cols;
    const int kept_seg = (int)(body[sg.tab + sg.n_ch * 32 + r] >> 20);
    const int k0 = ch * chunk_elems;                                    // this chunk's first kept value (index inside the segment)
    if (k0 >= kept_seg && ch > 0) return;                               // no values: an earlier chunk owns the rest of the row
    const int col_first = k0 < kept_seg ? (int)(body[sg.tab + ch * 32 + r] >> 20) : scols;
    const int col_end = (ch + 1 < sg.n_ch && (ch + 1) * chunk_elems < kept_seg) ? (int)(body[sg.tab + (ch + 1) * 32 + r] >> 20) : scols;
    int next_col = ch == 0 ? 0 : col_first;                             // first column not yet written
    uint32_t kk = kept_before + (uint32_t)k0;                           // row-wide index of the next kept value
    auto fill_pruned = [&](int from, int to) {                          // columns [from, to) of the segment are pruned
        for (int c = from; c < to; ++c) {
            const int cc = c_base + c;
            if (cc < k) orow[cc] = raw[(uint32_t)cc - kk];              // pruned columns before cc = cc - kept values before cc
        }
    };
    auto emit = [&](int col, uint16_t bits) {
        fill_pruned(next_col, col);
        if (t > 0) {
            const uint32_t bit0 = kk * (uint32_t)t, sh = bit0 & 31u, wi = bit0 >> 5;
            const uint64_t two = ((uint64_t)lo[wi] << 32) | (sh + t > 32 ? lo[wi + 1] : 0u);
            bits |= (uint16_t)((two >> (64 - t - sh)) & ((1u << t) - 1u));
        }
        if (c_base + col < k) orow[c_base + col] = bits;
        ++kk;
        next_col = col + 1;
    };
    if (k0 < kept_seg) decode_chunk_generic(body, sg, chunk_elems, ch, r, t, cb, emit);
    fill_pruned(next_col, col_end);
}

}  // namespace cass

using namespace cass;

extern "C" int cass_verification_data_bytes(const cass_blob_info* bi, size_t* h_bytes) {
    if (!bi || !h_bytes || bi->rows <= 0 || bi->cols <= 0) return CASS_ERR_INVALID_ARG;
    if (bi->mode != 1) return CASS_ERR_UNSUPPORTED;
    *h_bytes = ((size_t)kVdataHeaderWords + (size_t)bi->rows * vdata_row_words(bi->cols, bi->kept_per_row, bi->trunc_bits)) * 4;
    return CASS_OK;
}

extern "C" int cass_encode_verification_data(const void* blob, const cass_blob_info* bi, const void* W_bf16, void* vdata,
                                             size_t vdata_bytes, void* stream_) {
    size_t need = 0;
    int rc = cass_verification_data_bytes(bi, &need);
    if (rc) return rc;
    if (!blob || !W_bf16 || !vdata || ((uintptr_t)vdata & 3)) return CASS_ERR_INVALID_ARG;
    if (vdata_bytes < need) return CASS_ERR_CAPACITY;
    k_vdata<true><<<ceil_div(bi->rows, 8), 256, 0, (cudaStream_t)stream_>>>((const uint32_t*)blob, (const uint16_t*)W_bf16,
                                                                            (uint32_t*)vdata, nullptr);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

extern "C" int cass_decode_full(const void* blob, const cass_blob_info* bi, const void* vdata, void* W_bf16_out, void* stream_) {
    if (!blob || !bi || !vdata || !W_bf16_out) return CASS_ERR_INVALID_ARG;
    if (bi->mode != 1) return CASS_ERR_UNSUPPORTED;
    const int n_ch = ceil_div(bi->seg_cols, bi->chunk_cols);
    if (n_ch > 32) return CASS_ERR_UNSUPPORTED;
    k_decode_full<<<bi->n_rowblocks * bi->n_seg, 32 * n_ch, 0, (cudaStream_t)stream_>>>((const uint32_t*)blob, (const uint32_t*)vdata,
                                                                                         (uint16_t*)W_bf16_out);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
