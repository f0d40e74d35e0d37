// Global-memory layout of the B operand ("covariance image") of the tensor-core log-score kernel, per
// (unit, KV head, head subset): what sigma_image_kernel (or, fused, the statistics kernel) writes and the
// log-score kernel loads with plain bulk copies.
//
//   [ main: KCH chunks of 64 channels | linear-term operand | diagonal blocks (head_dim <= 128) ]
//   main, chunk kc: IMG_ROWS rows of 128 bytes (64 bf16, K-major), 128-byte swizzled: the 16-byte unit u of
//     row r sits at r * 128 + ((u ^ (r & 7)) << 4); row col(j, c) belongs to channel c of head j of the subset
//   linear term: per row 32 bytes of a K = 16 step as unswizzled core matrices: row r at
//     (r / 8) * 256 + (r % 8) * 16 (K columns 0..7) and 128 bytes further (K columns 8..15)
//   diagonal blocks: D / 16 blocks of 16 * HPC rows x 16 K-columns, the same core-matrix layout
#pragma once

template <int D>
struct EaImage {
    static constexpr int HPC = 256 / D;                  // query heads per pass (1, 2 or 4)
    static constexpr int KCH = D / 64;                   // 64-channel (128-byte) chunks per row
    static constexpr int IMG_ROWS = HPC * D;             // rows of a whole image (accumulator columns)
    static constexpr int CHUNK_B_FULL = IMG_ROWS * 128;  // bytes of one chunk of a whole image
    static constexpr int IMG_MAIN = KCH * CHUNK_B_FULL;  // bytes of the covariance part
    static constexpr int LIN_FULL = IMG_ROWS * 32;       // bytes of the linear-term operand
    // At d <= 128 the diagonal goes to the tensor cores as well: its bf16 part sits on the image's diagonal,
    // the bf16 rounding of what that leaves in 16 x 16 diagonal blocks.  At d = 256 the diagonal stays in
    // fp32 in the epilogue.
    static constexpr bool DIAG_MMA = D <= 128;
    static constexpr int DIAG_BLOCK = 16 * HPC * 32;                         // bytes: 16 HPC rows x 16 bf16
    static constexpr int DIAG_FULL = DIAG_MMA ? (D / 16) * DIAG_BLOCK : 0;
    static constexpr int IMG_FULL = IMG_MAIN + LIN_FULL + DIAG_FULL;
    // Accumulator column (= image row) of channel c of head j.  With the diagonal blocks the heads are
    // interleaved in runs of 16 channels, so that the 16 channels of one MMA step are 16 HPC adjacent
    // columns and every head's share of the diagonal is added by one instruction per step.
    __host__ __device__ static constexpr int col(int j, int c) {
        return DIAG_MMA ? (c / 16) * (16 * HPC) + j * 16 + c % 16 : j * D + c;
    }
};
