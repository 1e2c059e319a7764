// Internal interface of the projection GEMMs (gemm.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "dash.h"

namespace dash {

enum GemmEpilogueKind { GEMM_PLAIN = 0, GEMM_ROPE = 1, GEMM_RESID = 2, GEMM_SWIGLU = 3 };

struct GemmEpilogue {
    // ROPE: heads of D columns; columns below n_rot_cols (a multiple of 256) belong to Q and K heads and are rotated with
    // rope_table [n, D/2] = (cos, sin) of every row
    int D = 0, n_rot_cols = 0;
    const float2* rope_table = nullptr;
    // rope_pos null: the table holds one entry per row; else one per position and row t uses entry min(rope_pos[t], rope_len - 1)
    const int32_t* rope_pos = nullptr; int64_t rope_len = 0;
    // ROPE, SWIGLU: row_scale (null: none) multiplies the accumulators of a row first -- 1 / rms(row) when the RMSNorm in front of the
    // projection is folded into it (its weight into W, its row factor here)
    const float* row_scale = nullptr;
    // RESID: x_full[tok_index[row]] (tok_index null: row) = H[row] + (A W)[row]; sums [n, N/256] = (sum u^2, sum h^2, sum (h+u)^2, 0)
    // per column tile
    const void* H = nullptr; int64_t ldh = 0;
    const int32_t* tok_index = nullptr;
    void* x_full = nullptr; int64_t ldx = 0;
    float4* sums = nullptr;
    // SWIGLU: W = [K, 2m] (gate | up); C [n, m] = silu(A Wg) * (A Wu)
    int m = 0;
};

// true if the kernel takes this problem with this epilogue.  PLAIN: any N % 4 == 0, K % 8 == 0 (rows on 16-byte boundaries); the
// fused epilogues: whole 256-column tiles (SWIGLU: m % 128 == 0) and K in steps of 64 -- otherwise the caller runs the projection
// PLAIN and the element-wise work as passes of their own.
bool gemm_shape_ok(GemmEpilogueKind kind, int64_t n, int64_t N, int64_t K, int64_t lda, int64_t ldw, const GemmEpilogue& e);
// C (or the epilogue's outputs) = A[n, K] W[K, N], A and W bf16; ld* in elements; n_dev: device true row count or null;
// out_f32 (PLAIN only): C is fp32 instead of bf16
int gemm_bf16(GemmEpilogueKind kind, const void* A, int64_t lda, const void* W, int64_t ldw, void* C, int64_t ldc, int64_t n, int64_t N,
              int64_t K, const GemmEpilogue& e, const int32_t* n_dev, cudaStream_t st, bool out_f32 = false);
// dst (bf16, row stride ld_dst) = src (fp32, row stride ld_src) rounded to nearest even; cols % 4 == 0
int launch_f32_to_bf16(const float* src, int64_t ld_src, void* dst, int64_t ld_dst, int64_t rows, int64_t cols, cudaStream_t st);
// per row: (cos, sin) of pos * base^(-2i/D) into table [n, D/2] (table null: not formed; pos null: the row number is the position);
// with inv_rms non-null also 1 / sqrt(mean(H_row^2) + eps) (bf16 H, row stride ldh)
int launch_row_prep(const int32_t* pos, int64_t n, int D, double rope_base, float2* table, const void* H, int64_t ldh, int d, float rms_eps,
                    float* inv_rms, const int32_t* n_dev, cudaStream_t st, bool beside_front = false);

}  // namespace dash
