// Offline weight encoder: Wanda-scored per-row pruning, mantissa truncation, unary exponent coding,
// superblock packing (Sec. 4.2, 5.1, 5.3).  Bit-exact counterpart of the CPU oracle's blob.
#include "wblob.cuh"

namespace cass {

// Workspace carve-up (all offsets 256-byte aligned).
struct EncWs {
    uint32_t* keepbm;        // [n_pad][k_pad/32]
    uint32_t* cnt_fw;        // [n_pad][n_seg]  field words of the row in that segment
    uint32_t* ubits;         // [n_pad][n_seg]  code bits of the row in that segment
    unsigned long long* hist;   // [256]
    uint8_t* exp_to_rank;    // [256]
    uint32_t* abort_flag;    // [1]
    size_t bytes;
};

static EncWs carve(void* base, int n_pad, int k_pad, int n_seg) {
    EncWs w;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off = align_up(off + b, 256); return (char*)base + o; };
    w.keepbm = (uint32_t*)take((size_t)n_pad * (k_pad / 32) * 4);
    w.cnt_fw = (uint32_t*)take((size_t)n_pad * n_seg * 4);
    w.ubits = (uint32_t*)take((size_t)n_pad * n_seg * 4);
    w.hist = (unsigned long long*)take(256 * 8);
    w.exp_to_rank = (uint8_t*)take(256);
    w.abort_flag = (uint32_t*)take(256);
    w.bytes = off;
    return w;
}

struct EncGeom {
    int n, k, k_pad, n_pad, n_rb, n_seg, seg_cols, chunk_cols, p, t, n_prune;
    int mx;          // 1: Cassandra-2 (shared exponents), 0: Cassandra-1 (unary code)
};

static int make_geom(const cass_format* fmt, int rows, int cols, EncGeom* g) {
    if (!fmt || rows <= 0 || cols <= 0) return CASS_ERR_INVALID_ARG;
    if (fmt->mode != 1 && fmt->mode != 2) return CASS_ERR_UNSUPPORTED;
    g->mx = fmt->mode == 2;
    int p = fmt->w_prune_permille, t = fmt->w_trunc_bits;
    if (p < 0 || p > 999 || t < 0 || t > 7) return CASS_ERR_INVALID_ARG;
    int chunk = fmt->w_chunk_cols ? fmt->w_chunk_cols : 256;
    int seg = fmt->w_seg_cols ? fmt->w_seg_cols : 2048;
    if (chunk % 32 || chunk <= 0 || seg % chunk || seg > 2048 || seg <= 0) return CASS_ERR_INVALID_ARG;
    if (cols > (1 << 20)) return CASS_ERR_UNSUPPORTED;
    g->n = rows; g->k = cols; g->p = p; g->t = t;
    g->k_pad = ceil_div(cols, 32) * 32;
    g->chunk_cols = chunk;
    int seg_lim = ceil_div(g->k_pad, chunk) * chunk;
    g->seg_cols = seg < seg_lim ? seg : seg_lim;
    g->n_seg = ceil_div(g->k_pad, g->seg_cols);
    g->n_rb = ceil_div(rows, kRowsPerBlock);
    g->n_pad = g->n_rb * kRowsPerBlock;
    g->n_prune = (int)(((long long)cols * p) / 1000);
    return CASS_OK;
}

// ---- E1: per-row selection of the kept set -------------------------------------------------------------
// One block per row.  Score bits (non-negative fp32, so the integer order is the float order) are staged in
// shared memory; the composite key (score << 20 | column) is unique, so "prune the n_prune smallest keys"
// is the rule "lowest score first, lower column first among equals".  The threshold key is found by a
// bitwise binary search on the count of smaller keys.
__global__ void __launch_bounds__(256) k_select(const uint16_t* __restrict__ W, const float* __restrict__ act, EncGeom g,
                                                uint32_t* __restrict__ keepbm, unsigned long long* __restrict__ hist) {
    extern __shared__ uint32_t s_score[];            // [k]
    __shared__ unsigned int s_hist[256];
    __shared__ int s_part[8];
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint16_t* wr = W + (size_t)row * g.k;
    s_hist[tid] = 0;
    for (int c = tid; c < g.k; c += 256) {
        float mag = bf16_bits_to_float(wr[c] & 0x7FFFu);
        float a = act ? act[c] : 1.0f;
        s_score[c] = __float_as_uint(__fmul_rn(mag, a));
    }
    __syncthreads();
    unsigned long long thr = 0;                      // smallest kept key
    if (g.n_prune > 0) {
        for (int bit = 51; bit >= 0; --bit) {
            unsigned long long cand = thr | (1ull << bit);
            int c_lt = 0;
            for (int c = tid; c < g.k; c += 256) {
                unsigned long long key = ((unsigned long long)s_score[c] << 20) | (unsigned)c;
                c_lt += key < cand;
            }
            c_lt = __reduce_add_sync(0xffffffffu, c_lt);
            if (lane == 0) s_part[warp] = c_lt;
            __syncthreads();
            int tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) tot += s_part[i];
            if (tot <= g.n_prune) thr = cand;
            __syncthreads();
        }
    }
    const int words = g.k_pad / 32;
    for (int j = warp; j < words; j += 8) {
        int c = j * 32 + lane;
        bool keep = false;
        if (c < g.k) {
            unsigned long long key = ((unsigned long long)s_score[c] << 20) | (unsigned)c;
            keep = key >= thr;
            if (keep) atomicAdd(&s_hist[(wr[c] >> 7) & 0xFF], 1u);
        }
        uint32_t b = __brev(__ballot_sync(0xffffffffu, keep));     // column c at bit 31 - c%32
        if (lane == 0) keepbm[(size_t)row * words + j] = b;
    }
    __syncthreads();
    if (s_hist[tid]) atomicAdd(&hist[tid], (unsigned long long)s_hist[tid]);
}

// ---- E3: codebook: rank exponents by (count desc, exponent asc) -----------------------------------------
__global__ void k_codebook(const unsigned long long* __restrict__ hist, uint8_t* __restrict__ rank_to_exp,
                           uint8_t* __restrict__ exp_to_rank) {
    __shared__ unsigned long long s[256];
    int e = threadIdx.x;
    s[e] = hist[e];
    __syncthreads();
    unsigned long long mine = s[e];
    int rank = 0;
    for (int o = 0; o < 256; ++o) rank += (s[o] > mine) || (s[o] == mine && o < e);
    rank_to_exp[rank] = (uint8_t)e;
    exp_to_rank[e] = (uint8_t)rank;
}

// ---- E4: per (row, segment) sizes: kept values and code bits ------------------------------------------------
__global__ void k_sizes(const uint16_t* __restrict__ W, EncGeom g, const uint32_t* __restrict__ keepbm,
                        const uint8_t* __restrict__ exp_to_rank, uint32_t* __restrict__ cnt_kept,
                        uint32_t* __restrict__ ubits) {
    int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (gw >= g.n_pad * g.n_seg) return;
    int row = gw / g.n_seg, seg = gw % g.n_seg;
    uint32_t kept_n = 0, ub = 0;
    if (row < g.n) {
        const int words = g.k_pad / 32;
        int scols = seg_cols_of(g.k_pad, g.seg_cols, seg);
        int w0 = seg * (g.seg_cols / 32), nw = scols / 32;
        for (int j = 0; j < nw; ++j) {
            uint32_t bm = keepbm[(size_t)row * words + w0 + j];
            bool kept = (bm >> (31 - lane)) & 1u;
            uint32_t len = 0;
            if (kept) len = exp_to_rank[(W[(size_t)row * g.k + (w0 + j) * 32 + lane] >> 7) & 0xFF] + 1u;
            ub += __reduce_add_sync(0xffffffffu, len);
            kept_n += __popc(bm);
        }
    }
    if (g.mx) ub = 8u * ((kept_n + kMxBlock - 1) / kMxBlock);        // one exponent byte per block of 32 kept values
    if (lane == 0) { cnt_kept[gw] = kept_n; ubits[gw] = ub; }
}

// ---- E5: directory (exclusive scan of superblock sizes) and header -------------------------------------
__global__ void __launch_bounds__(1024) k_directory(EncGeom g, const uint32_t* __restrict__ cnt_fw,
                                                    const uint32_t* __restrict__ ubits, uint32_t* __restrict__ blob,
                                                    unsigned long long blob_cap, uint32_t* abort_flag, int32_t* d_status) {
    __shared__ unsigned long long s_scan[1024];
    __shared__ unsigned long long s_carry;
    __shared__ unsigned int s_maxsb;
    const int tid = threadIdx.x, n_sb = g.n_rb * g.n_seg;
    const unsigned long long body_off = align_up((size_t)kBlobDirOffset + 16ull * n_sb, 128);
    if (tid == 0) { s_carry = body_off; s_maxsb = 0; }
    __syncthreads();
    uint32_t* dir = blob + kBlobDirOffset / 4;
    for (int base = 0; base < n_sb; base += 1024) {
        int sb = base + tid;
        unsigned long long bytes = 0;
        uint32_t wf = 0, wu = 0, max_kept = 0;
        int n_ch = 0;
        if (sb < n_sb) {
            int rb = sb / g.n_seg, seg = sb % g.n_seg;
            const uint32_t per = 32u / (8u - (uint32_t)g.t);
            for (int r = 0; r < kRowsPerBlock; ++r) {
                int row = rb * kRowsPerBlock + r;
                max_kept = max(max_kept, cnt_fw[row * g.n_seg + seg]);
                wu = max(wu, (ubits[row * g.n_seg + seg] + 31u) / 32u);
            }
            wf = (max_kept + per - 1) / per;
            int scols = seg_cols_of(g.k_pad, g.seg_cols, seg);
            n_ch = ceil_div(scols, g.chunk_cols);
            bytes = (unsigned long long)SbGeom::make(n_ch, scols, (int)wf, (int)wu).total * 4ull;
            atomicMax(&s_maxsb, (unsigned int)bytes);
        }
        s_scan[tid] = bytes;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {          // inclusive Hillis-Steele scan
            unsigned long long v = tid >= o ? s_scan[tid - o] : 0;
            __syncthreads();
            s_scan[tid] += v;
            __syncthreads();
        }
        unsigned long long excl = s_scan[tid] - bytes + s_carry;
        if (sb < n_sb) {
            dir[sb * 4 + 0] = (uint32_t)(excl / 16);
            dir[sb * 4 + 1] = wf;
            dir[sb * 4 + 2] = wu;
            const int e_chunk = g.mx ? mx_chunk_elems_for((int)max_kept, n_ch) : chunk_elems_for((int)max_kept, n_ch);
            dir[sb * 4 + 3] = (uint32_t)n_ch | ((uint32_t)e_chunk << 8);
        }
        __syncthreads();
        if (tid == 1023) s_carry += s_scan[1023];
        __syncthreads();
    }
    if (tid == 0) {
        unsigned long long total = s_carry;
        uint32_t* h = blob;
        for (int i = 0; i < kBlobHeaderBytes / 4; ++i) h[i] = 0;
        h[H_MAGIC] = kBlobMagic; h[H_VERSION] = kBlobVersion; h[H_ROWS] = g.n; h[H_COLS] = g.k; h[H_P] = g.p; h[H_T] = g.t;
        h[H_SEG] = g.seg_cols; h[H_CHUNK] = g.chunk_cols; h[H_NSEG] = g.n_seg; h[H_NRB] = g.n_rb;
        h[H_KEPT] = g.k - g.n_prune; h[H_DIROFF] = kBlobDirOffset; h[H_BODYOFF] = (uint32_t)body_off;
        h[H_TOTLO] = (uint32_t)total; h[H_TOTHI] = (uint32_t)(total >> 32); h[H_MAXSB] = s_maxsb;
        h[H_MODE] = g.mx ? kBlobModeMx : kBlobModeUnary;
        // zero the padding between directory and first body
        for (unsigned long long o = kBlobDirOffset + 16ull * n_sb; o < body_off; o += 4) blob[o / 4] = 0;
        if (total > blob_cap) {
            *abort_flag = 1;
            if (d_status) *d_status = CASS_ERR_CAPACITY;
        }
    }
}

// ---- E6: pack one superblock (32 warps = 32 rows) -------------------------------------------------------
__global__ void __launch_bounds__(1024) k_pack(const uint16_t* __restrict__ W, EncGeom g,
                                               const uint32_t* __restrict__ keepbm,
                                               const uint8_t* __restrict__ exp_to_rank, uint32_t* __restrict__ blob,
                                               const uint32_t* __restrict__ abort_flag) {
    if (*abort_flag) return;
    const int sb = blockIdx.x, rb = sb / g.n_seg, seg = sb % g.n_seg;
    const int tid = threadIdx.x, lane = tid & 31, r = tid >> 5;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const int scols = seg_cols_of(g.k_pad, g.seg_cols, seg);
    const int n_ch = dir_n_ch(dir[3]);
    const uint32_t E = (uint32_t)dir_chunk_elems(dir[3]);
    const SbGeom sg = SbGeom::make(n_ch, scols, (int)dir[1], (int)dir[2]);
    uint32_t* body = blob + (size_t)dir[0] * 4;
    for (int i = tid; i < sg.total / 4; i += 1024) reinterpret_cast<uint4*>(body)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    const int row = rb * kRowsPerBlock + r;
    const int t = g.t, F = 8 - t, per = 32 / F;
    const int words = g.k_pad / 32;
    const int w0 = seg * (g.seg_cols / 32);
    uint32_t ub = 0, k_base = 0;
    for (int j = 0; j < sg.bm_words; ++j) {
        uint32_t bm = row < g.n ? keepbm[(size_t)row * words + w0 + j] : 0u;
        if (lane == 0) body[sg.bm + j * 32 + r] = bm;
        bool kept = (bm >> (31 - lane)) & 1u;
        uint32_t len = 0, field = 0;
        if (kept) {
            uint32_t b = W[(size_t)row * g.k + (w0 + j) * 32 + lane];
            len = exp_to_rank[(b >> 7) & 0xFF] + 1u;
            field = ((b >> 15) << (7 - t)) | ((b & 0x7Fu) >> t);
        }
        uint32_t incl = len;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (kept) {
            uint32_t pre = lane ? __popc(bm >> (32 - lane)) : 0u;
            uint32_t k = k_base + pre;
            atomicOr(&body[sg.fl + (k / per) * 32 + r], field_bits_in_word(field, k % per, t));
            uint32_t pos = ub + incl - 1;                                   // the codeword's terminating one
            atomicOr(&body[sg.un + (pos >> 5) * 32 + r], 0x80000000u >> (pos & 31));
            if (k % E == 0 && k / E < (uint32_t)n_ch)                       // first value of a chunk: its column and first code bit
                body[sg.tab + (k / E) * 32 + r] = ((uint32_t)(j * 32 + lane) << 20) | (pos + 1 - len);
        }
        ub += __shfl_sync(0xffffffffu, incl, 31);
        k_base += __popc(bm);
    }
    // chunks the row has no value for, and the totals
    for (int c = lane; c <= n_ch; c += 32) {
        if (c == n_ch) body[sg.tab + c * 32 + r] = (k_base << 20) | ub;
        else if ((uint32_t)c * E >= k_base) body[sg.tab + c * 32 + r] = ((uint32_t)scols << 20) | ub;
    }
}

// ---- E6 for Cassandra-2: the same superblock with shared exponents (Sec. 4.2, MX) --------------------------
// Pass 1 finds the largest exponent of every block of 32 kept values of every row (shared memory), pass 2 writes the
// bitmap, the magnitudes relative to their block's exponent, the exponent bytes and the chunk table.
__global__ void __launch_bounds__(1024) k_pack_mx(const uint16_t* __restrict__ W, EncGeom g,
                                                  const uint32_t* __restrict__ keepbm, uint32_t* __restrict__ blob,
                                                  const uint32_t* __restrict__ abort_flag) {
    __shared__ uint32_t s_exp[kRowsPerBlock][2048 / kMxBlock];
    if (*abort_flag) return;
    const int sb = blockIdx.x, rb = sb / g.n_seg, seg = sb % g.n_seg;
    const int tid = threadIdx.x, lane = tid & 31, r = tid >> 5;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const int scols = seg_cols_of(g.k_pad, g.seg_cols, seg);
    const int n_ch = dir_n_ch(dir[3]);
    const uint32_t E = (uint32_t)dir_chunk_elems(dir[3]);
    const SbGeom sg = SbGeom::make(n_ch, scols, (int)dir[1], (int)dir[2]);
    uint32_t* body = blob + (size_t)dir[0] * 4;
    for (int i = tid; i < sg.total / 4; i += 1024) reinterpret_cast<uint4*>(body)[i] = make_uint4(0, 0, 0, 0);
    for (int i = lane; i < 2048 / kMxBlock; i += 32) s_exp[r][i] = 0;
    __syncthreads();

    const int row = rb * kRowsPerBlock + r;
    const int t = g.t, F = 8 - t, per = 32 / F;
    const int words = g.k_pad / 32;
    const int w0 = seg * (g.seg_cols / 32);
    uint32_t k_base = 0;
    for (int j = 0; j < sg.bm_words; ++j) {                      // pass 1: block maxima
        uint32_t bm = row < g.n ? keepbm[(size_t)row * words + w0 + j] : 0u;
        if ((bm >> (31 - lane)) & 1u) {
            uint32_t k = k_base + (lane ? __popc(bm >> (32 - lane)) : 0u);
            atomicMax(&s_exp[r][k / kMxBlock], ((uint32_t)W[(size_t)row * g.k + (w0 + j) * 32 + lane] >> 7) & 0xFFu);
        }
        k_base += __popc(bm);
    }
    __syncwarp();
    const uint32_t n_blk = (k_base + kMxBlock - 1) / kMxBlock;
    for (uint32_t b = lane; b < n_blk; b += 32) atomicOr(&body[sg.un + (b / 4) * 32 + r], s_exp[r][b] << (24 - 8 * (b % 4)));
    k_base = 0;
    for (int j = 0; j < sg.bm_words; ++j) {                      // pass 2: bitmap, fields, table
        uint32_t bm = row < g.n ? keepbm[(size_t)row * words + w0 + j] : 0u;
        if (lane == 0) body[sg.bm + j * 32 + r] = bm;
        if ((bm >> (31 - lane)) & 1u) {
            const uint32_t b = W[(size_t)row * g.k + (w0 + j) * 32 + lane];
            const uint32_t k = k_base + (lane ? __popc(bm >> (32 - lane)) : 0u);
            const uint32_t e = (b >> 7) & 0xFFu, e_blk = s_exp[r][k / kMxBlock];
            const uint32_t shift = 1u + e_blk - e;
            const uint32_t m7 = (shift < 8u && e > 0u && e_blk >= 7u) ? (0x80u | (b & 0x7Fu)) >> shift : 0u;
            const uint32_t field = ((b >> 15) << (7 - t)) | (m7 >> t);
            atomicOr(&body[sg.fl + (k / per) * 32 + r], field << (32 - F * (k % per + 1)));
            if (k % E == 0 && k / E < (uint32_t)n_ch)
                body[sg.tab + (k / E) * 32 + r] = ((uint32_t)(j * 32 + lane) << 20) | (8u * (k / kMxBlock));
        }
        k_base += __popc(bm);
    }
    for (int c = lane; c <= n_ch; c += 32) {
        if (c == n_ch) body[sg.tab + c * 32 + r] = (k_base << 20) | (8u * n_blk);
        else if ((uint32_t)c * E >= k_base) body[sg.tab + c * 32 + r] = ((uint32_t)scols << 20) | (8u * n_blk);
    }
}

// ---- test hook: zero-padded reconstruction of the whole blob ---------------------------------------------
__global__ void k_decode(const uint32_t* __restrict__ blob, uint16_t* __restrict__ out) {
    const uint32_t* h = blob;
    const int n = h[H_ROWS], k = h[H_COLS], t = h[H_T], seg_cols = h[H_SEG], chunk_cols = h[H_CHUNK], n_seg = h[H_NSEG];
    const int k_pad = ceil_div(k, 32) * 32;
    const int sb = blockIdx.x, rb = sb / n_seg, seg = sb % n_seg;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const SbGeom sg = SbGeom::make(dir_n_ch(dir[3]), seg_cols_of(k_pad, seg_cols, seg), (int)dir[1], (int)dir[2]);
    const int chunk_elems = dir_chunk_elems(dir[3]);
    const uint32_t* body = blob + (size_t)dir[0] * 4;
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(blob) + kBlobHeaderBytes;
    for (int item = threadIdx.x; item < sg.n_ch * 32; item += blockDim.x) {
        int ch = item >> 5, r = item & 31, row = rb * kRowsPerBlock + r;
        if (row >= n) continue;
        auto emit = [&](int col, uint16_t bits) {
            int c = seg * seg_cols + col;
            if (c < k) out[(size_t)row * k + c] = bits;
        };
        if (h[H_MODE] == kBlobModeMx) decode_chunk_generic_mx(body, sg, chunk_elems, ch, r, t, emit);
        else decode_chunk_generic(body, sg, chunk_elems, ch, r, t, cb, emit);
    }
}

// ---- content accounting: sum of the codeword lengths recorded in the chunk tables ------------------------
__global__ void k_code_bits(const uint32_t* __restrict__ blob, unsigned long long* __restrict__ out) {
    const uint32_t* h = blob;
    const int k = h[H_COLS], seg_cols = h[H_SEG], n_seg = h[H_NSEG];
    const int k_pad = ceil_div(k, 32) * 32;
    const int sb = blockIdx.x, seg = sb % n_seg;
    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb * 4;
    const SbGeom sg = SbGeom::make(dir_n_ch(dir[3]), seg_cols_of(k_pad, seg_cols, seg), (int)dir[1], (int)dir[2]);
    const uint32_t* body = blob + (size_t)dir[0] * 4;
    unsigned int bits = body[sg.tab + sg.n_ch * 32 + threadIdx.x] & 0xFFFFFu;       // segment total of row threadIdx.x
    bits = __reduce_add_sync(0xffffffffu, bits);
    if (threadIdx.x == 0) atomicAdd(out, (unsigned long long)bits);
}

}  // namespace cass

using namespace cass;

extern "C" int cass_weight_blob_stats(const void* blob, const cass_blob_info* bi, void* d_scratch, cass_blob_stats* st,
                                      void* stream_) {
    if (!blob || !bi || !d_scratch || !st || ((uintptr_t)d_scratch & 7)) return CASS_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    CASS_CUDA_CHECK(cudaMemsetAsync(d_scratch, 0, 8, stream));
    k_code_bits<<<bi->n_rowblocks * bi->n_seg, 32, 0, stream>>>((const uint32_t*)blob, (unsigned long long*)d_scratch);
    CASS_LAUNCH_CHECK();
    unsigned long long code = 0;
    CASS_CUDA_CHECK(cudaMemcpyAsync(&code, d_scratch, 8, cudaMemcpyDeviceToHost, stream));
    CASS_CUDA_CHECK(cudaStreamSynchronize(stream));
    st->bitmap_bits = (uint64_t)bi->rows * bi->cols;
    st->field_bits = (uint64_t)bi->rows * bi->kept_per_row * (8 - bi->trunc_bits);
    st->code_bits = code;
    st->total_bits = bi->total_bytes * 8;
    return CASS_OK;
}

extern "C" int cass_encoded_weight_bytes(const cass_format* fmt, int rows, int cols, size_t* h_blob_bound,
                                         size_t* h_workspace_bytes) {
    EncGeom g;
    int rc = make_geom(fmt, rows, cols, &g);
    if (rc) return rc;
    const int F = 8 - g.t, per = 32 / F;
    size_t n_sb = (size_t)g.n_rb * g.n_seg;
    int n_ch = ceil_div(g.seg_cols, g.chunk_cols);
    // per superblock: table + bitmap + fields (kept values + one padding word per chunk) + codes at a
    // mean of 8 bits per kept value (+1 word of row padding)
    size_t kept_seg = (size_t)g.seg_cols;
    size_t words_row = (size_t)(n_ch + 1) + g.seg_cols / 32 + (kept_seg + per - 1) / per + n_ch + kept_seg * 8 / 32 + 1;
    size_t sb_bytes = words_row * 32 * 4;
    if (h_blob_bound) *h_blob_bound = align_up((size_t)kBlobDirOffset + 16 * n_sb, 128) + n_sb * sb_bytes;
    if (h_workspace_bytes) *h_workspace_bytes = carve(nullptr, g.n_pad, g.k_pad, g.n_seg).bytes;
    return CASS_OK;
}

extern "C" int cass_encode_weights(const cass_format* fmt, const void* W_bf16, const float* act_norm, int rows,
                                   int cols, void* blob, size_t blob_cap, void* workspace, size_t workspace_bytes,
                                   int32_t* d_status, void* stream_) {
    EncGeom g;
    int rc = make_geom(fmt, rows, cols, &g);
    if (rc) return rc;
    if (!W_bf16 || !blob || !workspace || ((uintptr_t)blob & 127)) return CASS_ERR_INVALID_ARG;
    EncWs ws = carve(workspace, g.n_pad, g.k_pad, g.n_seg);
    if (workspace_bytes < ws.bytes) return CASS_ERR_CAPACITY;
    size_t n_sb = (size_t)g.n_rb * g.n_seg;
    size_t body_off = align_up((size_t)kBlobDirOffset + 16 * n_sb, 128);
    if (blob_cap < body_off) return CASS_ERR_CAPACITY;
    if ((size_t)g.k * 4 > 200 * 1024) return CASS_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)stream_;
    const uint16_t* W = (const uint16_t*)W_bf16;
    uint32_t* b32 = (uint32_t*)blob;

    CASS_CUDA_CHECK(cudaMemsetAsync(workspace, 0, ws.bytes, stream));
    size_t smem = (size_t)g.k * 4;
    CASS_CUDA_CHECK(cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_select<<<g.n, 256, smem, stream>>>(W, act_norm, g, ws.keepbm, ws.hist);
    CASS_LAUNCH_CHECK();
    if (g.mx) {
        CASS_CUDA_CHECK(cudaMemsetAsync((uint8_t*)blob + kBlobHeaderBytes, 0, kBlobCodebookBytes, stream));    // no codebook
    } else {
        k_codebook<<<1, 256, 0, stream>>>(ws.hist, (uint8_t*)blob + kBlobHeaderBytes, ws.exp_to_rank);
        CASS_LAUNCH_CHECK();
    }
    int warps = g.n_pad * g.n_seg;
    k_sizes<<<ceil_div(warps, 8), 256, 0, stream>>>(W, g, ws.keepbm, ws.exp_to_rank, ws.cnt_fw, ws.ubits);
    CASS_LAUNCH_CHECK();
    k_directory<<<1, 1024, 0, stream>>>(g, ws.cnt_fw, ws.ubits, b32, (unsigned long long)blob_cap, ws.abort_flag, d_status);
    CASS_LAUNCH_CHECK();
    if (g.mx) k_pack_mx<<<(unsigned)n_sb, 1024, 0, stream>>>(W, g, ws.keepbm, b32, ws.abort_flag);
    else k_pack<<<(unsigned)n_sb, 1024, 0, stream>>>(W, g, ws.keepbm, ws.exp_to_rank, b32, ws.abort_flag);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

extern "C" int cass_weight_blob_info(const void* blob, cass_blob_info* h_info, void* stream_) {
    if (!blob || !h_info) return CASS_ERR_INVALID_ARG;
    uint32_t h[kBlobHeaderBytes / 4];
    cudaStream_t stream = (cudaStream_t)stream_;
    CASS_CUDA_CHECK(cudaMemcpyAsync(h, blob, sizeof(h), cudaMemcpyDeviceToHost, stream));
    CASS_CUDA_CHECK(cudaStreamSynchronize(stream));
    if (h[H_MAGIC] != kBlobMagic || h[H_VERSION] != kBlobVersion) return CASS_ERR_INVALID_ARG;
    h_info->rows = h[H_ROWS]; h_info->cols = h[H_COLS]; h_info->prune_permille = h[H_P]; h_info->trunc_bits = h[H_T];
    h_info->seg_cols = h[H_SEG]; h_info->chunk_cols = h[H_CHUNK]; h_info->n_seg = h[H_NSEG]; h_info->n_rowblocks = h[H_NRB];
    h_info->kept_per_row = h[H_KEPT]; h_info->max_superblock_bytes = h[H_MAXSB];
    h_info->mode = h[H_MODE] == kBlobModeMx ? 2 : 1; h_info->reserved = 0;
    h_info->total_bytes = (uint64_t)h[H_TOTLO] | ((uint64_t)h[H_TOTHI] << 32);
    return CASS_OK;
}

extern "C" int cass_decode_weights(const void* blob, const cass_blob_info* h_info, void* W_bf16_out, void* stream_) {
    if (!blob || !h_info || !W_bf16_out) return CASS_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    CASS_CUDA_CHECK(cudaMemsetAsync(W_bf16_out, 0, (size_t)h_info->rows * h_info->cols * 2, stream));
    k_decode<<<h_info->n_rowblocks * h_info->n_seg, 256, 0, stream>>>((const uint32_t*)blob, (uint16_t*)W_bf16_out);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
