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

// Exact reconstruction (Sec. 4.1 target inference: speculation and verification data are loaded and the original values
// rebuilt; Sec. 5.1 mantissa concatenator), in two light kernels that keep many warps per SM in flight:
//   k_decode_kept<T>: one CTA per superblock, warp = chunk, lane = row.  The lane walks its chunk's kept values (the
//     blob's streams are interleaved over the 32 rows, so the warp's reads are contiguous) and stores their speculation
//     bits (sign, exponent, high mantissa bits) at their columns of the output.
//   k_merge_vdata: one warp per row, lane = column.  For every 32 columns the kept values get their low t bits from the
//     row's verification data and the pruned columns their raw values; kept and pruned counts before a column are
//     popcounts of the bitmap (prefix sums over the row's bitmap words first, so that the words are then independent
//     and their loads overlap), neighbouring lanes read neighbouring verification data and the row leaves as
//     contiguous stores.
template <int TT>                                                       // truncated bits (0..5), or -1: read from the header
__global__ void __launch_bounds__(1024) k_decode_kept(const uint32_t* __restrict__ blob, uint16_t* __restrict__ out) {
    __shared__ uint16_t lut_s[256];                                     // rank -> exponent at its bf16 position
    const uint32_t* h = blob;
    const int n = h[H_ROWS], k = h[H_COLS], t = TT >= 0 ? TT : (int)h[H_T], seg_cols = h[H_SEG], n_seg = h[H_NSEG];
    const int k_pad = ceil_div(k, 32) * 32;
    const int sb = blockIdx.x, rb = sb / n_seg, seg = sb % n_seg;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const SbGeom sg = SbGeom::make(dir_n_ch(dir[3]), seg_cols_of(k_pad, seg_cols, seg), (int)dir[1], (int)dir[2]);
    const int chunk_elems = dir_chunk_elems(dir[3]);
    const uint32_t* body = blob + (size_t)dir[0] * 4;
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(blob) + kBlobHeaderBytes;
    if ((int)h[H_T] != t) return;                                       // not the blob the launch was told about
    for (int i = threadIdx.x; i < 256; i += blockDim.x) lut_s[i] = (uint16_t)cb[i] << 7;
    __syncthreads();
    const int ch = threadIdx.x >> 5, r = threadIdx.x & 31, row = rb * kRowsPerBlock + r;
    if (ch >= sg.n_ch || row >= n) return;
    uint16_t* orow = out + (size_t)row * k + seg * seg_cols;
    const int cols_here = k - seg * seg_cols;
    auto put = [&](int col, uint16_t bits) { if (col < cols_here) orow[col] = bits; };
    if constexpr (TT >= 0) decode_chunk_fixed<(TT >= 0 ? TT : 0)>(body, sg, chunk_elems, ch, r, lut_s, put);
    else decode_chunk_generic(body, sg, chunk_elems, ch, r, t, cb, put);
}

constexpr int kMergeRowWarps = 8;
__global__ void __launch_bounds__(32 * kMergeRowWarps) k_merge_vdata(const uint32_t* __restrict__ blob, const uint32_t* __restrict__ vdata,
                                                                     uint16_t* __restrict__ out) {
    __shared__ uint32_t kb_s[kMergeRowWarps][64];                       // kept values before each 32-column word of the segment in hand
    const uint32_t* h = blob;
    const int n = h[H_ROWS], k = h[H_COLS], t = h[H_T], seg_cols = h[H_SEG], n_seg = h[H_NSEG], kept = h[H_KEPT];
    const int k_pad = ceil_div(k, 32) * 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kMergeRowWarps + warp;
    if (row >= n) return;
    const int rb = row / kRowsPerBlock, rr = row % kRowsPerBlock;
    const int lo_words = vdata_lo_words(kept, t), row_words = vdata_row_words(k, kept, t);
    const uint32_t* lo = vdata + kVdataHeaderWords + (size_t)row * row_words;
    const uint16_t* raw = reinterpret_cast<const uint16_t*>(lo + lo_words);
    uint32_t k_base = 0;                                                // kept values of the row in the segments already done
    for (int seg = 0; seg < n_seg; ++seg) {
        const uint32_t* dir = blob + kBlobDirOffset / 4 + (rb * n_seg + seg) * 4;
        const int scols = seg_cols_of(k_pad, seg_cols, seg), n_words = scols / 32;       // <= 64 words
        const SbGeom sg = SbGeom::make(dir_n_ch(dir[3]), scols, (int)dir[1], (int)dir[2]);
        const uint32_t* bmw = blob + (size_t)dir[0] * 4 + sg.bm + rr;  // bitmap word j of this row at bmw[j * 32]
        const int c_base = seg * seg_cols;
        uint16_t* orow = out + (size_t)row * k + c_base;
        __syncwarp();
        uint32_t c0 = 0, c1 = 0;
        if (lane < n_words) c0 = __popc(bmw[lane * 32]);
        if (lane + 32 < n_words) c1 = __popc(bmw[(lane + 32) * 32]);
        uint32_t i0 = c0, i1 = c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t a = __shfl_up_sync(0xffffffffu, i0, o), b2 = __shfl_up_sync(0xffffffffu, i1, o);
            if (lane >= o) { i0 += a; i1 += b2; }
        }
        const uint32_t tot0 = __shfl_sync(0xffffffffu, i0, 31), tot1 = __shfl_sync(0xffffffffu, i1, 31);
        kb_s[warp][lane] = k_base + i0 - c0;
        kb_s[warp][lane + 32] = k_base + tot0 + i1 - c1;
        __syncwarp();
#pragma unroll 4
        for (int j = 0; j < n_words; ++j) {
            const uint32_t bm = bmw[j * 32];
            const int c = j * 32 + lane;
            const uint32_t kb = kb_s[warp][j];
            const bool in = c_base + c < k, is_kept = (bm >> (31 - lane)) & 1u;
            const uint32_t before = lane ? __popc(bm >> (32 - lane)) : 0u;          // kept columns of this word before mine
            if (in) {
                uint16_t v;
                if (is_kept) {
                    v = orow[c];                                                    // the speculation bits k_decode_kept left here
                    if (t > 0) {
                        const uint32_t bit0 = (kb + before) * (uint32_t)t, sh = bit0 & 31u, wi = bit0 >> 5;
                        const uint64_t two = ((uint64_t)lo[wi] << 32) | (sh + t > 32 ? lo[wi + 1] : 0u);
                        v |= (uint16_t)((two >> (64 - t - sh)) & ((1u << t) - 1u));
                    }
                } else {
                    v = raw[(uint32_t)(c_base + c) - kb - before];                   // pruned columns before mine = columns - kept before
                }
                orow[c] = v;
            }
        }
        k_base += tot0 + tot1;
    }
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
    const int threads = 32 * n_ch;
    const int grid = bi->n_rowblocks * bi->n_seg;
    cudaStream_t stream = (cudaStream_t)stream_;
    const uint32_t* b32 = (const uint32_t*)blob;
    uint16_t* o16 = (uint16_t*)W_bf16_out;
    switch (bi->trunc_bits) {
        case 0: k_decode_kept<0><<<grid, threads, 0, stream>>>(b32, o16); break;
        case 1: k_decode_kept<1><<<grid, threads, 0, stream>>>(b32, o16); break;
        case 2: k_decode_kept<2><<<grid, threads, 0, stream>>>(b32, o16); break;
        case 3: k_decode_kept<3><<<grid, threads, 0, stream>>>(b32, o16); break;
        case 4: k_decode_kept<4><<<grid, threads, 0, stream>>>(b32, o16); break;
        case 5: k_decode_kept<5><<<grid, threads, 0, stream>>>(b32, o16); break;
        default: k_decode_kept<-1><<<grid, threads, 0, stream>>>(b32, o16); break;
    }
    CASS_LAUNCH_CHECK();
    k_merge_vdata<<<ceil_div(bi->rows, kMergeRowWarps), 32 * kMergeRowWarps, 0, stream>>>(b32, (const uint32_t*)vdata, o16);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
