// Verification projections (Sec. 2.2: the target model processes the gamma+1 drafted rows as one small batch,
// memory-bound on the bf16 weights): Y[r][n] = sum_k W[n][k] X[r][k], bf16 operands, fp32 accumulation.
//
// tcgen05 version, "swap-AB": the weights are the M operand (128 output features per CTA), the token rows the N
// operand (padded to BN = 16, 32 or 64 columns), the accumulator lives in tensor memory.  One CTA = one 128-feature tile x
// one K range (split-K so that small matrices still fill the GPU); warp 0 streams 128x64 weight tiles and the
// BNx64 activation tile through a ring of TMA loads (128-byte swizzle), warp 1 issues the MMAs, warps 2-5 read the
// accumulator back and store fp32 partial sums; a second kernel adds the K ranges in fixed order.
//
// Row-count invariance: an accumulator column belongs to one token row, the tile shape, the K ranges and the order
// of the MMAs depend on (n, k) only, so a row gives the same bits whether it is verified alone or with others.
#include "tc.cuh"
#include "kernels.cuh"

namespace cass {

constexpr int kTcBM = 128, kTcBK = 64;
constexpr int tc_stages(int bn) { return bn <= 16 ? 6 : bn <= 32 ? 5 : 4; }      // two CTAs per SM at every bn
constexpr int kTcABytes = kTcBM * kTcBK * 2;
constexpr int kTcThreads = 192;
constexpr int tc_b_bytes(int bn) { return bn * kTcBK * 2; }
constexpr int tc_smem(int bn) { return tc_stages(bn) * (kTcABytes + tc_b_bytes(bn)) + 256 + 1024; }     // + barriers + alignment slack
constexpr int tc_tmem_cols(int bn) { return bn <= 32 ? 32 : 64; }                                   // a power of two >= 32

// bf16 matrix [rows][cols] row-major -> map with a (box_rows x 64)-element box, 128-byte swizzle, zero fill outside.
static int make_map(CUtensorMap* m, const void* ptr, int rows, int cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return CASS_ERR_CUDA;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTcBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CASS_OK : CASS_ERR_INVALID_ARG;
}

// Instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = bn.
constexpr uint32_t tc_idesc(int bn) { return tc_idesc_mn(kTcBM, bn, false); }

// grid (m tiles, k splits).  partial: fp32 [k splits][BN][n].
template <int BN>
__global__ void __launch_bounds__(kTcThreads) k_verify_gemm_tc(const __grid_constant__ CUtensorMap map_w,
                                                                const __grid_constant__ CUtensorMap map_x,
                                                                float* __restrict__ partial, int rows, int n,
                                                                int kb_total, int kb_per_split, int32_t* __restrict__ d_status,
                                                                int w_static) {
    extern __shared__ uint8_t smem_dyn[];
    uint8_t* base = reinterpret_cast<uint8_t*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);     // swizzled tiles: 1024-byte aligned
    uint8_t* sA = base;
    constexpr int kTcBBytes = tc_b_bytes(BN), kTcTmemCols = tc_tmem_cols(BN), kTcStages = tc_stages(BN);
    constexpr uint32_t kIdesc = tc_idesc(BN);
    uint8_t* sB = base + kTcStages * kTcABytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(sB + kTcStages * kTcBBytes);
    uint64_t* empty = full + kTcStages;
    uint64_t* acc_ready = empty + kTcStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_ready + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kTcBM, ks = blockIdx.y;
    const int kb0 = ks * kb_per_split;
    const int nkb = min(kb_per_split, kb_total - kb0);

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_ready, 1);
        fence_mbar_init();
    }
    if (warp == 1) {                                   // one warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // Barriers and tensor memory are set up.  The weights are nobody's output: the first ring of weight tiles is
    // requested ahead of the wait for the preceding kernels, whose results are the activations and the scratch.
    // (w_static = 0: the weights too come from a preceding kernel, e.g. rebuilt from their two parts: nothing is early)
    const int n_pre = nkb < kTcStages ? nkb : kTcStages;
    if (warp == 0 && lane == 0 && w_static) {
        for (int kb = 0; kb < n_pre; ++kb) {                 // stages are empty at the start: nothing to wait for
            mbar_expect_tx(&full[kb], kTcABytes + kTcBBytes);
            tma_load_2d(sA + kb * kTcABytes, &map_w, (kb0 + kb) * kTcBK, m0, &full[kb]);
        }
    }
    pdl_early<5>();
    pdl_wait();

    if (warp == 0 && lane == 0) {
        // ---- producer: TMA loads into the ring ----
        for (int kb = 0; kb < n_pre; ++kb) {
            if (!w_static) {
                mbar_expect_tx(&full[kb], kTcABytes + kTcBBytes);
                tma_load_2d(sA + kb * kTcABytes, &map_w, (kb0 + kb) * kTcBK, m0, &full[kb]);
            }
            tma_load_2d(sB + kb * kTcBBytes, &map_x, (kb0 + kb) * kTcBK, 0, &full[kb]);
        }
        for (int kb = n_pre; kb < nkb; ++kb) {
            const int s = kb % kTcStages;
            const uint32_t ph = (uint32_t)(kb / kTcStages) & 1u;
            if (!mbar_wait_bounded(&empty[s], ph ^ 1u)) { atomicExch(d_status, CASS_ERR_TIMEOUT); break; }
            mbar_expect_tx(&full[s], kTcABytes + kTcBBytes);
            tma_load_2d(sA + s * kTcABytes, &map_w, (kb0 + kb) * kTcBK, m0, &full[s]);
            tma_load_2d(sB + s * kTcBBytes, &map_x, (kb0 + kb) * kTcBK, 0, &full[s]);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer ----
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % kTcStages;
            const uint32_t ph = (uint32_t)(kb / kTcStages) & 1u;
            if (!mbar_wait_bounded(&full[s], ph)) { atomicExch(d_status, CASS_ERR_TIMEOUT); ok = false; break; }
            tc_fence_after();
            const uint64_t ad = tc_smem_desc(sA + s * kTcABytes), bd = tc_smem_desc(sB + s * kTcBBytes);
#pragma unroll
            for (int kk = 0; kk < kTcBK / 16; ++kk)      // 16 bf16 = 32 bytes along K inside the swizzle row: +2 in the address field
                tc_mma(tmem, ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 2), kIdesc, (uint32_t)((kb | kk) != 0));
            tc_commit(&empty[s]);                        // frees the stage once these MMAs have read it
        }
        tc_commit(acc_ready);                            // accumulator complete (or abandoned after a time-out)
    } else if (warp >= 2) {
        // ---- epilogue: warp w may read the 32 accumulator lanes of quarter w % 4 ----
        if (mbar_wait_bounded(acc_ready, 0)) {
            __syncwarp();
            tc_fence_after();
            const int q = warp & 3;
            const int feat = m0 + q * 32 + lane;
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 16) {          // 16 accumulator columns (token rows) at a time
                uint32_t v[16];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                      "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                    : "r"(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (feat < n && nkb > 0) {
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if (c0 + r < rows) partial[((size_t)ks * BN + c0 + r) * n + feat] = __uint_as_float(v[r]);
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
    }
}

__global__ void k_verify_gemm_finish(const float* __restrict__ partial, int rows, int bn, int n, int n_split,
                                     uint16_t* __restrict__ y_bf16, float* __restrict__ y_f32) {
    pdl_early<5>();
    pdl_wait();
    const int j = blockIdx.x * blockDim.x + threadIdx.x, r = blockIdx.y;
    if (j >= n || r >= rows) return;
    float acc = 0.f;
    for (int s = 0; s < n_split; ++s) acc += partial[((size_t)s * bn + r) * n + j];
    if (y_f32) y_f32[(size_t)r * n + j] = acc;
    if (y_bf16) y_bf16[(size_t)r * n + j] = float_to_bf16_bits(acc);
}

// K ranges: a function of (n, k) only.  Enough CTAs for about two per SM, at least 4 k-blocks per range.  A plan that
// needs a few CTAs more than the 296 that run at once pays a second, nearly empty wave for them (320 CTAs for the
// 4096 x 4096 matrix: 12.5 us; 256: see the microbenchmark summary), so such a plan gives up ranges until it fits.
static void split_plan(int n, int k, int* kb_total, int* kb_per_split, int* n_split) {
    constexpr int kSlots = 296;
    const int tiles = ceil_div(n, kTcBM);
    *kb_total = ceil_div(k, kTcBK);
    int want = ceil_div(kSlots, tiles);
    int max_split = *kb_total / 4 > 0 ? *kb_total / 4 : 1;
    if (want > max_split) want = max_split;
    if (want < 1) want = 1;
    auto plan = [&](int w, int* per, int* ns) { *per = ceil_div(*kb_total, w); *ns = ceil_div(*kb_total, *per); return tiles * *ns; };
    int ctas = plan(want, kb_per_split, n_split);
    while (ctas > kSlots && 2 * ctas <= 3 * kSlots && want > 1) {             // a little over one wave
        int per, ns;
        const int fewer = plan(want - 1, &per, &ns);
        if (fewer <= kSlots && 5 * fewer < 4 * kSlots) break;                 // would leave the single wave too empty: keep the plan
        --want;
        *kb_per_split = per; *n_split = ns; ctas = fewer;
    }
}

Partials verify_gemm_partials(const float* partial, int n, int k, int bn) {
    int kbt, kbs, ns;
    split_plan(n, k, &kbt, &kbs, &ns);
    return Partials{partial, ns, (size_t)bn * n, (size_t)n};
}

size_t verify_gemm_partial_floats(int n, int k, int bn) {
    int kbt, kbs, ns;
    split_plan(n, k, &kbt, &kbs, &ns);
    return (size_t)ns * bn * n;
}

template <int BN>
static int launch_tc(const CUtensorMap& mw, const CUtensorMap& mx, float* partial, int rows, int n, int kbt, int kbs, int ns,
                     int32_t* d_status, int w_static, cudaStream_t s) {
    static bool attr = false;
    if (!attr) {
        CASS_CUDA_CHECK(cudaFuncSetAttribute(k_verify_gemm_tc<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc_smem(BN)));
        attr = true;
    }
    dim3 grid(ceil_div(n, kTcBM), ns);
    CASS_PDL_LAUNCH(k_verify_gemm_tc<BN>, grid, dim3(kTcThreads), (size_t)tc_smem(BN), s, mw, mx, partial, rows, n, kbt, kbs, d_status, w_static);
    return CASS_OK;
}

int launch_verify_gemm(const uint16_t* W, const uint16_t* X, int rows, int bn, int n, int k, float* partial, uint16_t* y_bf16,
                       float* y_f32, int32_t* d_status, cudaStream_t s, int w_static) {
    if (rows < 1 || rows > bn || (bn != 16 && bn != 32 && bn != 64) || (k % 8) || n < 1 || !partial || !d_status)
        return CASS_ERR_INVALID_ARG;
    if (((uintptr_t)W & 15) || ((uintptr_t)X & 15)) return CASS_ERR_INVALID_ARG;
    CUtensorMap mw, mx;
    int rc = make_map(&mw, W, n, k, kTcBM);
    if (rc) return rc;
    rc = make_map(&mx, X, bn, k, bn);      // the activation buffer always has bn rows
    if (rc) return rc;
    int kbt, kbs, ns;
    split_plan(n, k, &kbt, &kbs, &ns);
    if (bn == 16) rc = launch_tc<16>(mw, mx, partial, rows, n, kbt, kbs, ns, d_status, w_static, s);
    else if (bn == 32) rc = launch_tc<32>(mw, mx, partial, rows, n, kbt, kbs, ns, d_status, w_static, s);
    else rc = launch_tc<64>(mw, mx, partial, rows, n, kbt, kbs, ns, d_status, w_static, s);
    if (rc) return rc;
    if (!y_bf16 && !y_f32) return CASS_OK;          // the caller's next kernel adds the parts itself
    dim3 g2(ceil_div(n, 256), rows);
    CASS_PDL_LAUNCH(k_verify_gemm_finish, g2, dim3(256), 0, s, (const float*)partial, rows, bn, n, ns, y_bf16, y_f32);
    return CASS_OK;
}

}  // namespace cass

using namespace cass;

extern "C" size_t cass_verify_gemm_scratch_bytes(int n, int k) {
    if (n < 1 || k < 1) return 0;
    return verify_gemm_partial_floats(n, k, kMaxRows) * sizeof(float);
}

extern "C" int cass_verify_gemm(const void* W_bf16, const void* X_bf16, int rows, int n, int k, void* scratch,
                                size_t scratch_bytes, void* y_bf16, float* y_f32, int32_t* d_status, void* stream) {
    if (!W_bf16 || !X_bf16 || !scratch || (!y_bf16 && !y_f32)) return CASS_ERR_INVALID_ARG;
    if (n < 1 || k < 1 || scratch_bytes < cass_verify_gemm_scratch_bytes(n, k)) return CASS_ERR_CAPACITY;
    if (rows < 1 || rows > kMaxRows) return CASS_ERR_INVALID_ARG;
    return launch_verify_gemm((const uint16_t*)W_bf16, (const uint16_t*)X_bf16, rows, verify_gemm_bn(rows), n, k, (float*)scratch,
                              (uint16_t*)y_bf16, y_f32, d_status, (cudaStream_t)stream);
}
