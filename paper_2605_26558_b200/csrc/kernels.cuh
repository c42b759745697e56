// Internal launchers shared between the translation units of the library.
#pragma once

#include "common.cuh"

namespace cass {

size_t gemv_smem_bytes(const cass_blob_info& bi);
// partial: fp32 [n_seg][n_rowblocks*32]; the caller sums the segments (fixed order) afterwards.
int launch_draft_gemv(const void* blob, const cass_blob_info& bi, const void* x_bf16, float* partial,
                      int32_t* d_status, cudaStream_t stream);

}  // namespace cass
