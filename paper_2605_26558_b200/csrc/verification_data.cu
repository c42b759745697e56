// Verification data (Sec. 4.1 target inference, Sec. 5.1 encoder): what the Cassandra-1 speculation data leaves out
// -- the low t mantissa bits of the kept values and the pruned values as they are -- and the exact reconstruction
// of the bf16 matrix from the two parts.  Not on the decode path of this library (verification reads a bf16 copy);
// it shows that the format is a strict split of the original bits and what the two parts weigh.
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
    int rc = cass_decode_weights(blob, bi, W_bf16_out, stream_);           // kept values without their low bits, zeros elsewhere
    if (rc) return rc;
    k_vdata<false><<<ceil_div(bi->rows, 8), 256, 0, (cudaStream_t)stream_>>>((const uint32_t*)blob, nullptr,
                                                                             (uint32_t*)const_cast<void*>(vdata), (uint16_t*)W_bf16_out);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
