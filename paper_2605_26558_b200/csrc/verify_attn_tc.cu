// Verification attention on the tensor cores (Sec. 2.2: the gamma+1 rows are verified in one pass; bf16 KV cache).
// One CTA = one (128-token chunk, KV head, sequence).  Both products of the chunk run as tcgen05 MMAs with the
// accumulators in tensor memory:
//   scores^T [128 tokens x NP pairs] = K tile [128 x d] . Q^T          (pairs = (row, query head of the group), padded
//   out^T    [d x NP pairs]          = V tile^T [d x 128 tokens] . P^T   to NP = 32 or 64; P = chunk-local softmax
//                                                                        numerators, bf16)
// K and V tiles arrive by TMA (128-byte swizzle); Q and P are written to shared memory by threads in the same
// swizzled layout.  The V tile is used as it lies in memory (rows = tokens), i.e. as an M-contiguous A operand.
// Chunk results (o, running maximum m, sum l) go to the split-K scratch and k_attn_merge combines the chunks, as for
// the SIMT kernel.  A (row, head) pair is one accumulator column, so its result does not depend on the other rows.
// Needs head_dim = 128 and rows x group <= 64; other shapes use k_verify_attn.
#include "tc.cuh"
#include "kernels.cuh"

namespace cass {

constexpr int kVtTok = 128;            // tokens per CTA: M of the score product, K of the output product
constexpr int kVtMaxPairs = 64;        // largest N of both products (template NP = 32 or 64)
constexpr int kVtD = 128;              // head_dim
constexpr int kVtThreads = 192;        // warp 0: TMA; warp 1: MMA issue and tensor-memory allocation; warps 2-5: softmax, epilogue
constexpr int kVtTileBytes = kVtTok * 64 * 2;          // one TMA box: 128 tokens x 64 dims
constexpr int vt_q_bytes(int np) { return np * 64 * 2; }               // one K-block of the Q or P operand: NP rows x 64 elements
// K tiles (32 KB) | V tiles (32 KB) | Q (2 blocks) | [P (2 blocks) when np = 64] | barriers.  The scores (np x 128
// floats) reuse the K tiles' memory, and with np = 32 so does P: both are written only after the first product has
// finished reading K.
constexpr int vt_smem(int np) { return 4 * kVtTileBytes + (np == 32 ? 2 : 4) * vt_q_bytes(np) + 256 + 1024; }
static_assert(32 * kVtTok * 4 + 2 * vt_q_bytes(32) <= 2 * kVtTileBytes && 64 * kVtTok * 4 <= 2 * kVtTileBytes, "scores (and P) fit the K tiles");
constexpr int vt_tmem_cols(int np) { return 2 * np; }                  // scores^T in columns 0..NP-1, out^T in columns NP..2NP-1

// Byte offset of element (row, col) in a K-major operand block of rows x 64 bf16 with 128-byte swizzle.
__device__ __forceinline__ uint32_t swz_off(int row, int col) {
    return (uint32_t)(row * 128 + ((((col >> 3) ^ (row & 7)) & 7) << 4) + ((col & 7) << 1));
}

__device__ __forceinline__ void named_sync_128() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// 32 consecutive fp32 columns of this warp's 32 tensor-memory lanes: v[i] = column i of the thread's lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int NP>
__global__ void __launch_bounds__(kVtThreads) k_verify_attn_tc(const __grid_constant__ CUtensorMap map_k,
                                                                const __grid_constant__ CUtensorMap map_v,
                                                                const uint16_t* __restrict__ qkv, int rows, int n_q, int n_kv,
                                                                const DevState* __restrict__ st, AttnScratch sc, int n_chunks_alloc,
                                                                int32_t* __restrict__ d_status) {
    extern __shared__ uint8_t smem_dyn[];
    pdl_early<4>();
    pdl_wait();
    const int chunk = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    const int len = st->len[seq];
    const int t0 = chunk * kVtTok;
    if (t0 >= len + rows) return;                              // no row of this call sees the chunk
    constexpr int kVtPairs = NP, kVtQBytes = vt_q_bytes(NP), kVtTmemCols = vt_tmem_cols(NP);
    uint8_t* base = reinterpret_cast<uint8_t*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    uint8_t* sK = base;                                        // 2 boxes [128 tok][64 d]
    uint8_t* sV = sK + 2 * kVtTileBytes;                       // 2 boxes [128 tok][64 d]
    uint8_t* sQ = sV + 2 * kVtTileBytes;                       // 2 blocks [NP pairs][64 d]
    float* sS = reinterpret_cast<float*>(sK);                  // [NP pairs][128 tok] scores: over the K tiles, once consumed
    uint8_t* sP = NP == 32 ? sK + NP * kVtTok * 4 : sQ + 2 * kVtQBytes;      // 2 blocks [NP pairs][64 tok], 1024-aligned
    uint64_t* bar_k = reinterpret_cast<uint64_t*>(sQ + (NP == 32 ? 2 : 4) * kVtQBytes);
    uint64_t* bar_v = bar_k + 1;
    uint64_t* bar_s = bar_k + 2;       // scores complete in tensor memory
    uint64_t* bar_p = bar_k + 3;       // P written to shared memory (128 arrivals)
    uint64_t* bar_o = bar_k + 4;       // output complete in tensor memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_k + 5);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = n_q / n_kv, P = rows * G;
    const int qkv_dim = (n_q + 2 * n_kv) * kVtD;
    if (tid == 0) {
        mbar_init(bar_k, 1); mbar_init(bar_v, 1); mbar_init(bar_s, 1); mbar_init(bar_p, 128); mbar_init(bar_o, 1);
        fence_mbar_init();
        // the chunk's K and V tiles start travelling now, while the other warps stage Q and tensor memory is allocated
        mbar_expect_tx(bar_k, 2 * kVtTileBytes);
        tma_load_3d(sK, &map_k, head * kVtD, t0, seq, bar_k);
        tma_load_3d(sK + kVtTileBytes, &map_k, head * kVtD + 64, t0, seq, bar_k);
        mbar_expect_tx(bar_v, 2 * kVtTileBytes);
        tma_load_3d(sV, &map_v, head * kVtD, t0, seq, bar_v);
        tma_load_3d(sV + kVtTileBytes, &map_v, head * kVtD + 64, t0, seq, bar_v);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kVtTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp >= 2) {
        // Q of this sequence's rows and this group's heads -> sQ (pair p = row * G + head-in-group), zero beyond P
        const int et = tid - 64;
        const uint16_t* q0 = qkv + (size_t)seq * rows * qkv_dim + (size_t)head * G * kVtD;
        for (int i = et; i < kVtPairs * (kVtD / 8); i += 128) {
            const int p = i / (kVtD / 8), c8 = i % (kVtD / 8);           // 8 dims = 16 bytes per item
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (p < P) v = *reinterpret_cast<const uint4*>(q0 + (size_t)(p / G) * qkv_dim + (size_t)(p % G) * kVtD + c8 * 8);
            const int blk = c8 >> 3;                                     // which 64-dim block
            *reinterpret_cast<uint4*>(sQ + blk * kVtQBytes + swz_off(p, (c8 & 7) * 8)) = v;
        }
        fence_proxy_async();                                             // generic-proxy writes -> visible to the MMA
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp == 1 && lane == 0) {
        // ---- scores^T = K . Q^T: A = K tile (K-major over d), B = Q (K-major over d) ----
        if (mbar_wait_bounded(bar_k, 0)) {
            tc_fence_after();
            constexpr uint32_t idesc1 = tc_idesc_mn(kVtTok, kVtPairs, false);
#pragma unroll
            for (int kb = 0; kb < 2; ++kb) {
                const uint64_t ad = tc_smem_desc(sK + kb * kVtTileBytes), bd = tc_smem_desc(sQ + kb * kVtQBytes);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    tc_mma(tmem, ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 2), idesc1, (uint32_t)((kb | kk) != 0));
            }
        } else {
            atomicExch(d_status, CASS_ERR_TIMEOUT); ok = false;
        }
        tc_commit(bar_s);
        // ---- out^T = V^T . P^T: A = V tile as stored (rows = tokens: M-contiguous), B = P (K-major over tokens) ----
        if (ok && mbar_wait_bounded(bar_v, 0) && mbar_wait_bounded(bar_p, 0)) {
            tc_fence_after();
            constexpr uint32_t idesc2 = tc_idesc_mn(kVtD, kVtPairs, true);
#pragma unroll
            for (int kk = 0; kk < kVtTok / 16; ++kk) {                   // 16 tokens per MMA
                // A: 16 token rows of 128 bytes = 2048 bytes further per step; the second 64-dim block is the other box
                const uint64_t ad = tc_smem_desc(sV + kk * 2048, kVtTileBytes);
                // B: block kk / 4 of P (64 tokens each), 32 bytes per 16 tokens inside the swizzled row
                const uint64_t bd = tc_smem_desc(sP + (kk >> 2) * kVtQBytes) + (uint64_t)((kk & 3) * 2);
                tc_mma(tmem + (uint32_t)NP, ad, bd, idesc2, (uint32_t)(kk != 0));
            }
        } else if (ok) {
            atomicExch(d_status, CASS_ERR_TIMEOUT);
        }
        tc_commit(bar_o);
    }
    else if (warp >= 2) {
        const int q = warp & 3;                       // the tensor-memory lane quarter this warp may read
        const int et = q * 32 + lane;                 // this thread's token (scores) and dim (output)
        const float scale = rsqrtf((float)kVtD);
        uint32_t v[32];
        const bool have = mbar_wait_bounded(bar_s, 0);
        if (have) { __syncwarp(); tc_fence_after(); }
        else atomicExch(d_status, CASS_ERR_TIMEOUT);
        // scores^T -> sS[pair][token], scaled, causal: row r of the call sits at position len + r
#pragma unroll
        for (int c0 = 0; c0 < NP; c0 += 32) {
            if (have) tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int p = c0 + i;
                const bool vis = have && p < P && (t0 + et) <= len + p / G;
                sS[p * kVtTok + et] = vis ? __uint_as_float(v[i]) * scale : -INFINITY;
            }
        }
        named_sync_128();
        // chunk softmax of every pair (warp q: pairs q, q + 4, ...), numerators rounded to bf16 into the P operand
        for (int p = q; p < kVtPairs; p += 4) {
            float a[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) a[k] = sS[p * kVtTok + lane + 32 * k];
            const float m = warp_max(fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3])));
            float l = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float e = (m == -INFINITY) ? 0.f : expf(a[k] - m);
                const uint16_t eb = float_to_bf16_bits(e);
                l += bf16_bits_to_float(eb);                  // the sum of what the MMA multiplies
                const int t = lane + 32 * k;
                *reinterpret_cast<uint16_t*>(sP + (t >> 6) * kVtQBytes + swz_off(p, t & 63)) = eb;
            }
            l = warp_sum(l);
            if (lane == 0 && p < P && t0 <= len + p / G) {
                const size_t pair = ((size_t)seq * rows + p / G) * n_q + head * G + p % G;
                sc.m[pair * n_chunks_alloc + chunk] = m;
                sc.l[pair * n_chunks_alloc + chunk] = l;
            }
        }
        fence_proxy_async();
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar_p)) : "memory");
        if (mbar_wait_bounded(bar_o, 0)) {
            __syncwarp();
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < NP; c0 += 32) {
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(NP + c0), v);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int p = c0 + i;
                    if (p < P && t0 <= len + p / G) {
                        const size_t pair = ((size_t)seq * rows + p / G) * n_q + head * G + p % G;
                        sc.o[(pair * n_chunks_alloc + chunk) * kVtD + et] = __uint_as_float(v[i]);
                    }
                }
            }
        } else {
            atomicExch(d_status, CASS_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kVtTmemCols) : "memory");
    }
}

int launch_attn_merge(const AttnScratch& sc, int n_chunks_alloc, int chunk_tokens, int rows, int rps, int n_q, int d,
                      const DevState* st, int draft_mode, int draft_units, uint16_t* out, cudaStream_t s);

bool verify_attn_tc_usable(const KvGeom& g, int rps, int n_q) {
    return g.d == kVtD && rps * (n_q / g.n_kv) <= kVtMaxPairs && (g.seq_stride % 16) == 0;
}

// caches: sequence 0's bf16 K and V of one layer ([max_seq][n_kv][128]); the other sequences lie seq_stride bytes apart.
int launch_verify_attn_tc(const KvGeom& g, const uint16_t* k_cache, const uint16_t* v_cache, const uint16_t* qkv, int n_seq,
                          int rps, int n_q, int np_cols, const DevState* st, const AttnScratch& sc, uint16_t* out,
                          int32_t* d_status, cudaStream_t s) {
    if (!verify_attn_tc_usable(g, rps, n_q) || (np_cols != 32 && np_cols != 64) || rps * (n_q / g.n_kv) > np_cols)
        return CASS_ERR_UNSUPPORTED;
    EncodeTiledFn fn = encode_fn();
    if (!fn) return CASS_ERR_CUDA;
    CUtensorMap mk, mv;
    const cuuint64_t gdim[3] = {(cuuint64_t)g.n_kv * g.d, (cuuint64_t)g.max_seq, (cuuint64_t)n_seq};
    const cuuint64_t gstride[2] = {(cuuint64_t)g.n_kv * g.d * 2, (cuuint64_t)(n_seq > 1 ? g.seq_stride : (size_t)g.max_seq * g.n_kv * g.d * 2)};
    const cuuint32_t box[3] = {64, (cuuint32_t)kVtTok, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    for (int i = 0; i < 2; ++i) {
        CUresult r = fn(i ? &mv : &mk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<uint16_t*>(i ? v_cache : k_cache), gdim, gstride,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return CASS_ERR_INVALID_ARG;
    }
    const int n_chunks = ceil_div(g.max_seq, kVtTok);
    dim3 grid(n_chunks, g.n_kv, n_seq);
    if (np_cols == 32) {
        static bool attr = false;
        if (!attr) {
            CASS_CUDA_CHECK(cudaFuncSetAttribute(k_verify_attn_tc<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, vt_smem(32)));
            attr = true;
        }
        CASS_PDL_LAUNCH(k_verify_attn_tc<32>, grid, dim3(kVtThreads), (size_t)vt_smem(32), s, mk, mv, qkv, rps, n_q, g.n_kv, st, sc,
                        n_chunks, d_status);
    } else {
        static bool attr = false;
        if (!attr) {
            CASS_CUDA_CHECK(cudaFuncSetAttribute(k_verify_attn_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, vt_smem(64)));
            attr = true;
        }
        CASS_PDL_LAUNCH(k_verify_attn_tc<64>, grid, dim3(kVtThreads), (size_t)vt_smem(64), s, mk, mv, qkv, rps, n_q, g.n_kv, st, sc,
                        n_chunks, d_status);
    }
    return launch_attn_merge(sc, n_chunks, kVtTok, n_seq * rps, rps, n_q, g.d, st, 0, 0, out, s);
}

}  // namespace cass
