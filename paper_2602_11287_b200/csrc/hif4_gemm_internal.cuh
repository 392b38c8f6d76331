// Internal launchers behind hif4_gemm / hif4_grouped_gemm (arguments already validated).
#pragma once
#include "hif4_common.cuh"

namespace hif4 {

// CUDA-core path: any M, N, K % 64 == 0, 4-byte aligned operands.
hif4_status launch_gemm_simt(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                             int64_t ldc, cudaStream_t st);
hif4_status launch_grouped_gemm_simt(const void* A, const void* B, float* C, const int64_t* offsets,
                                     int num_groups, int64_t total_rows, int64_t N, int64_t K, int64_t ldc,
                                     cudaStream_t st);

// Tensor-core path (tcgen05 + TMA): needs K % 256 == 0 and 16-byte aligned operands.
bool gemm_tc_supported(const void* A, const void* B, int64_t a_rows, int64_t b_rows, int64_t N, int64_t K);
hif4_status launch_gemm_tc(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                           cudaStream_t st);
// Tensor-core path on CTA pairs (256 x 256 tiles, tcgen05 cta_group::2): same requirements.
bool gemm_tc2_supported(const void* A, const void* B, int64_t M, int64_t N, int64_t K);
// Workspace: completion words of the tiles that two or more pairs share along K (0 when the schedule splits none).
size_t gemm_tc2_workspace_bytes(int64_t M, int64_t N, int64_t K);
hif4_status launch_gemm_tc2(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                            void* workspace, size_t workspace_bytes, cudaStream_t st);
// The same kernel with the activation conversion inside: X is [M, K] BF16 (row stride ld_x elements, rows 16-byte
// aligned), converted with Algorithm 1 (round-half-to-even) by the A-side decode threads, once per column tile.
hif4_status launch_gemm_tc2_fused_bf16(const void* X, int64_t ld_x, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                                       int64_t ldc, void* workspace, size_t workspace_bytes, cudaStream_t st);
// Weight-streaming path for M <= kGemvMaxM tokens (mma.sync on register-decoded weights): needs
// K % 256 == 0, 16-byte aligned B and a workspace of gemv_workspace_bytes (the decoded tokens).
constexpr int64_t kGemvMaxM = 32;
bool gemv_supported(const void* A, const void* B, int64_t M, int64_t N, int64_t K);
size_t gemv_workspace_bytes(int64_t M, int64_t K);
hif4_status launch_gemv(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                        void* workspace, cudaStream_t st);
// The same with the activations not yet quantized ([M, K] of `dt`, row stride ld_x elements, 16-byte aligned rows):
// the token preparation quantizes (Algorithm 1) and decodes in one kernel, the packed units are never written.
bool gemv_linear_supported(const void* X, hif4_dtype dt, int64_t ld_x, const void* B, int64_t M, int64_t N, int64_t K);
hif4_status launch_gemv_linear(const void* X, hif4_dtype dt, int64_t ld_x, int rha, const void* B, float* C, int64_t M,
                               int64_t N, int64_t K, int64_t ldc, void* workspace, cudaStream_t st);
// The weight-streaming path on Eq. 3's factorisation: E4M3 operands that hold the elements with their micro-exponents,
// the two level-1 scales applied to the FP32 sum of each unit pair.  Same requirements as the path above; workspace
// of gemv8_workspace_bytes (the tokens as E4M3 operand bytes and per-unit scales).  Slower than the BF16 form on
// sm_100a (the legacy FP8 mma.sync has no native path there); reachable through the test hook only.
size_t gemv8_workspace_bytes(int64_t M, int64_t K);
hif4_status launch_gemv8(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int64_t ldc,
                         void* workspace, cudaStream_t st);
size_t grouped_tc_workspace_bytes(int num_groups, int64_t total_rows);
hif4_status launch_grouped_gemm_tc(const void* A, const void* B, float* C, const int64_t* offsets, int num_groups,
                                   int64_t total_rows, int64_t N, int64_t K, int64_t ldc, void* workspace,
                                   cudaStream_t st);

// Grouped GEMM on CTA pairs with swapped operands (weights on the MMA M side, token tiles of 32..256
// rows on the N side); same requirements as the tensor-core path, workspace = its tile table.
size_t grouped_tc2_workspace_bytes(int num_groups, int64_t total_rows, int64_t N);
// (dense problems with fewer weight tiles than CTA pairs are cut along K; their workspace holds the slices' completion words)
size_t gemm_tc2_swapped_workspace_bytes(int64_t M, int64_t N, int64_t K);
hif4_status launch_gemm_tc2_swapped(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                                    int64_t ldc, void* workspace, size_t workspace_bytes, cudaStream_t st);
hif4_status launch_grouped_gemm_tc2(const void* A, const void* B, float* C, const int64_t* offsets, int num_groups,
                                    int64_t total_rows, int64_t N, int64_t K, int64_t ldc, void* workspace,
                                    cudaStream_t st);

}  // namespace hif4
