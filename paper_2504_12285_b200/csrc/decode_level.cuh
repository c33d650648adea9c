// Parameters of the one-level decode launch (decode_level.cu): everything the kernel needs travels in its arguments.
#pragma once

#include "quant_row.cuh"

namespace bitlinear {

constexpr int kLevelMaxProblems = 4;

struct LevelProblem {
    const uint8_t* packed;
    const float* s_w;
    void* y;
    int32_t* acc_out;  // nullable
    int N, y_dtype;
};

struct LevelParams {
    LevelProblem prob[kLevelMaxProblems];
    int count;
    const void* x;  // the input row's first operand (see RowOp)
    RowOp op;
    const __nv_bfloat16* gain;
    float eps;
    int K, x_row0;
    int8_t* xq_out;  // nullable, all three or none: [K] codes in the layout of the quantiser launch (LAYOUT 1), scale, code sum
    float* d_out;
    int32_t* xsum_out;
    int total_rb, rb_per_cta;
    int* status_word;
};

// Can this call run as one level launch?  (At most kLevelMaxProblems problems of one token in the 2-bit layout that
// share their input row, a CTA's share of the weights small enough for two such launches to sit side by side on an SM.)
bool decode_level_fits(int count, int total_rb, int K, int sm_count);
// Fills in the split and launches; P.total_rb = sum of N / 16 over the problems.  dependent: the packed weights, their
// scales and the gain are not written by the launch before this one on the stream, so the kernel may start beside it.
int decode_level_forward(LevelParams& P, int sm_count, cudaStream_t st, bool dependent);

}  // namespace bitlinear
