// Interface of the tensor-core quantisation path (tq_quantize_tc.cu) towards the API layer.
#pragma once

#include <cuda.h>

#include "tq_internal.h"

namespace tq {
namespace tc {

int pick_bn(int d);            // N extent of one MMA tile for this dimension
bool supported(int d);         // d large enough for the tensor path and the driver offers tensor maps

cudaError_t build_matrix_limbs(const float* dM, int rows, int d, int dpad, int bn, MatrixLimbs* out);
void free_matrix_limbs(MatrixLimbs* m);

size_t scratch_bytes_per_row(const tq_plan* plan);

int sm_count();                // SMs of the current device
// TMA descriptor of a byte matrix [rows, row_bytes] (row pitch `pitch` bytes), box = box_bytes x box_rows
// bytes, zero fill outside the matrix; swizzle = 0 (plain rows in shared memory) or 32 / 64 / 128.
// False when the driver offers no tensor maps.
bool make_byte_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint64_t pitch,
                   uint32_t box_bytes, uint32_t box_rows, int swizzle = 0);

// Quant_mse / Quant_prod of n rows through the tcgen05 GEMMs (qjl, gamma unused for TQ_MSE).
int quantize(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx, uint8_t* idx, uint8_t* qjl,
             float* gamma, float* norms, void* scratch, size_t scratch_bytes, cudaStream_t st, const char* who);

}  // namespace tc
}  // namespace tq
