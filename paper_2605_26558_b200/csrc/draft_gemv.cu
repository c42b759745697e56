// Draft GEMV: y = decode(speculation data) * x with the decode done in registers (Sec. 4.1 draft inference;
// the software form of the decoder dataflow of Sec. 5.1: bitmap de-sparsification, unary exponent decode
// through a rank->exponent table, sign/mantissa concatenation).
//
// One CTA per superblock (32 rows x one column segment).  The whole superblock arrives in shared memory with
// one bulk asynchronous copy (contiguous read, as Sec. 5.3 asks), then warp c decodes chunk c with lane = row:
// every lane walks its own bitmap, field and unary streams, which are interleaved word by word so that all
// shared-memory reads of the streams are conflict free.  Regular chunks (see the irregular mask of the format)
// use 32-bit windows: one bitmap window per 8 kept values, one unary window per 4 codewords.
#include "wblob.cuh"
#include "kernels.cuh"

namespace cass {

size_t gemv_smem_bytes(const cass_blob_info& bi) {
    const int n_ch = ceil_div(bi.seg_cols, bi.chunk_cols);
    return align_up((size_t)bi.max_superblock_bytes + 256, 128) + (size_t)(bi.seg_cols + 64) * 4 + 256 * 4 +
           (size_t)n_ch * 32 * 4 + 64;
}

// Dot product of one regular (row, chunk) with x, lane = row.  T = truncated mantissa bits (0 or 4).
template <int T>
__device__ __forceinline__ float chunk_dot_fast(const uint32_t* __restrict__ sb, const SbGeom& g, int ch, int lane,
                                                int chunk_cols, const float* __restrict__ xs,
                                                const uint32_t* __restrict__ lut) {
    constexpr int F = 8 - T, PER = 32 / F, NFW = kGroupCols / PER;       // field words per group of 8
    constexpr uint32_t MANT = ((1u << (F - 1)) - 1u) << (T + 16);
    static_assert(PER == 4 || PER == 8, "fast path handles 4 or 8 fields per word");
    const uint32_t e0 = sb[g.tab + ch * 32 + lane];
    uint32_t fw = e0 >> 20, upos = e0 & 0xFFFFFu;
    const uint32_t* bmS = sb + g.bm + lane;
    const uint32_t* flS = sb + g.fl + lane;
    const uint32_t* unS = sb + g.un + lane;
    const int wpc = chunk_cols / 32;
    const int w0 = ch * wpc, w1 = min(w0 + wpc, g.bm_words);
    int m = 0;
    for (int w = w0; w < w1; ++w) m += __popc(bmS[w * 32]);
    const int n_full = warp_min_i(m) / kGroupCols;
    const int n_groups = ceil_div(warp_max_i(m), kGroupCols);
    uint32_t bpos = (uint32_t)(w0 * 32);
    const uint32_t bpos_lim = (uint32_t)(g.bm_words * 32), upos_lim = (uint32_t)(g.w_u * 32);
    float acc = 0.f;

    auto group = [&](int grp, bool tail) {
        const uint32_t bw = bpos >> 5;
        uint32_t bv = __funnelshift_l(bmS[(bw + 1) * 32], bmS[bw * 32], bpos);
        const float* xg = xs + bpos;
        uint32_t fwd[NFW];
#pragma unroll
        for (int i = 0; i < NFW; ++i) fwd[i] = flS[(fw + grp * NFW + i) * 32];
        const int rem = m - grp * kGroupCols;
        int s = 0;
#pragma unroll
        for (int half = 0; half < kGroupCols / kGroupCodes; ++half) {
            const uint32_t uw = upos >> 5;
            uint32_t uv = __funnelshift_l(unS[(uw + 1) * 32], unS[uw * 32], upos);
            int tprev = -1;
#pragma unroll
            for (int j = 0; j < kGroupCodes; ++j) {
                const int e = half * kGroupCodes + j;
                s = __clz(bv);
                const float xv = xg[s];
                bv &= ~(0x80000000u >> s);
                const int tt = __clz(uv);
                const uint32_t eb = lut[tt - tprev - 1];
                tprev = tt;
                uv &= ~(0x80000000u >> tt);
                constexpr int dummy = 0; (void)dummy;
                const int sh = (32 - F * (e % PER + 1)) - (T + 16);
                const uint32_t fword = fwd[e / PER];
                const uint32_t a = sh >= 0 ? (fword >> (sh >= 0 ? sh : 0)) : (fword << (sh < 0 ? -sh : 0));
                const uint32_t wb = (a & MANT) | eb | ((a << 8) & 0x80000000u);
                if (!tail || e < rem) acc = fmaf(__uint_as_float(wb), xv, acc);
            }
            upos += (uint32_t)(tprev + 1);
            if (tail) upos = min(upos, upos_lim);
        }
        bpos += (uint32_t)(s + 1);
        if (tail) bpos = min(bpos, bpos_lim);
    };

    int grp = 0;
    for (; grp < n_full; ++grp) group(grp, false);
    for (; grp < n_groups; ++grp) group(grp, true);
    return acc;
}

// T >= 0: fast path for regular chunks, generic path otherwise.  T = -1: generic path only (any t).
template <int T>
__global__ void __launch_bounds__(1024) k_draft_gemv(const uint32_t* __restrict__ blob, const uint16_t* __restrict__ x,
                                                     float* __restrict__ partial, int32_t* __restrict__ d_status,
                                                     int max_sb /* shared-memory room for one superblock */, int seg_cols_host) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const uint32_t* h = blob;
    const int n = h[H_ROWS], k = h[H_COLS], t = h[H_T], seg_cols = h[H_SEG], chunk_cols = h[H_CHUNK];
    const int n_seg = h[H_NSEG], n_rb = h[H_NRB];
    const int k_pad = ceil_div(k, 32) * 32;
    const int sb_i = blockIdx.x, rb = sb_i / n_seg, seg = sb_i % n_seg;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;

    uint32_t* sb = reinterpret_cast<uint32_t*>(smem_raw);
    float* xs = reinterpret_cast<float*>(smem_raw + align_up((size_t)max_sb + 256, 128));
    uint32_t* lut = reinterpret_cast<uint32_t*>(xs + seg_cols + 64);
    float* red = reinterpret_cast<float*>(lut + 256);
    uint64_t* bar = reinterpret_cast<uint64_t*>(red + n_warps * 32);

    const uint32_t* dir = blob + kBlobDirOffset / 4 + sb_i * 4;
    const int scols = seg_cols_of(k_pad, seg_cols, seg);
    const SbGeom g = SbGeom::make((int)dir[3], scols, (int)dir[1], (int)dir[2]);
    const uint32_t bytes = (uint32_t)g.total * 4u;
    // The launch sized shared memory from the host's copy of the header; a blob that does not match it
    // (larger superblock, other segment geometry) is refused instead of overrunning the buffer.
    if (bytes > (uint32_t)max_sb || (int)blockDim.x < 32 * g.n_ch || seg_cols != seg_cols_host || g.n_ch > 32) {
        if (tid == 0 && d_status) atomicExch(d_status, CASS_ERR_INVALID_ARG);
        return;
    }

    if (tid == 0) {
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (tid == 0) {
        const uint8_t* src = reinterpret_cast<const uint8_t*>(blob) + (size_t)dir[0] * 16;
        mbar_expect_tx(bar, bytes);
        for (uint32_t off = 0; off < bytes; off += 32768u) {
            uint32_t nb = min(32768u, bytes - off);
            bulk_g2s(smem_raw + off, src + off, nb, bar);
        }
    }
    // x of this segment (fp32), zero beyond the matrix, and the rank -> exponent table pre-shifted into place
    const int c0 = seg * seg_cols;
    for (int i = tid; i < seg_cols + 64; i += blockDim.x) {
        int c = c0 + i;
        xs[i] = (i < scols && c < k) ? bf16_bits_to_float(x[c]) : 0.f;
    }
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(blob) + kBlobHeaderBytes;
    for (int i = tid; i < 256; i += blockDim.x) lut[i] = (uint32_t)cb[i] << 23;
    // slack words after the superblock may be read (never used) by the window loads
    for (int i = tid; i < 64; i += blockDim.x) sb[g.total + i] = 0;
    __syncthreads();
    if (!mbar_wait_bounded(bar, 0)) {
        if (d_status) atomicExch(d_status, CASS_ERR_TIMEOUT);
        return;
    }

    float acc = 0.f;
    if (warp < g.n_ch) {
        const uint32_t irregular = sb[warp];
        if (T >= 0 && irregular == 0u) {
            acc = chunk_dot_fast<(T >= 0 ? T : 0)>(sb, g, warp, lane, chunk_cols, xs, lut);
        } else {
            decode_chunk_generic(sb, g, chunk_cols, warp, lane, t, cb, [&](int col, uint16_t bits) {
                acc = fmaf(bf16_bits_to_float(bits), xs[col], acc);
            });
        }
    }
    red[warp * 32 + lane] = acc;
    __syncthreads();
    if (warp == 0) {
        float sum = 0.f;
        for (int w = 0; w < n_warps; ++w) sum += red[w * 32 + lane];
        int row = rb * kRowsPerBlock + lane;
        if (row < n) partial[(size_t)seg * (n_rb * kRowsPerBlock) + row] = sum;
    }
}

__global__ void k_gemv_finish(const float* __restrict__ partial, int n, int n_pad, int n_seg,
                              uint16_t* __restrict__ y_bf16, float* __restrict__ y_f32) {
    int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    float acc = 0.f;
    for (int s = 0; s < n_seg; ++s) acc += partial[(size_t)s * n_pad + r];
    if (y_f32) y_f32[r] = acc;
    if (y_bf16) y_bf16[r] = float_to_bf16_bits(acc);
}

int launch_draft_gemv(const void* blob, const cass_blob_info& bi, const void* x_bf16, float* partial,
                      int32_t* d_status, cudaStream_t stream) {
    const int n_ch = ceil_div(bi.seg_cols, bi.chunk_cols);
    if (n_ch > 32) return CASS_ERR_UNSUPPORTED;
    size_t smem = gemv_smem_bytes(bi);
    if (smem > 227 * 1024) return CASS_ERR_CAPACITY;
    dim3 grid(bi.n_rowblocks * bi.n_seg), block(32 * n_ch);
    const uint32_t* b = (const uint32_t*)blob;
    const uint16_t* x = (const uint16_t*)x_bf16;
#define CASS_GEMV_LAUNCH(TT)                                                                                   \
    do {                                                                                                       \
        static int attr_smem = 0;      /* largest size already granted to this instantiation */              \
        if ((int)smem > attr_smem) {                                                                           \
            CASS_CUDA_CHECK(cudaFuncSetAttribute(k_draft_gemv<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize,\
                                                 (int)smem));                                                  \
            attr_smem = (int)smem;                                                                             \
        }                                                                                                      \
        k_draft_gemv<TT><<<grid, block, smem, stream>>>(b, x, partial, d_status, bi.max_superblock_bytes, bi.seg_cols);                              \
    } while (0)
    if (bi.trunc_bits == 4) CASS_GEMV_LAUNCH(4);
    else if (bi.trunc_bits == 0) CASS_GEMV_LAUNCH(0);
    else CASS_GEMV_LAUNCH(-1);
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
    int rc = launch_draft_gemv(blob, *h_info, x_bf16, partial, d_status, stream);
    if (rc) return rc;
    if (!y_bf16 && !y_f32) return CASS_OK;
    int n_pad = h_info->n_rowblocks * kRowsPerBlock;
    k_gemv_finish<<<ceil_div(h_info->rows, 256), 256, 0, stream>>>(partial, h_info->rows, n_pad, h_info->n_seg,
                                                                    (uint16_t*)y_bf16, y_f32);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}
