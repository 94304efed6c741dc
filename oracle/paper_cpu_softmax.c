/*
 * The CPU Softmax method of Section VI-A, restated: C, 32-bit floats, one core,
 * one row at a time, separate input and output buffers.
 *
 * TEST / BASELINE INFRASTRUCTURE, not product code (same rule as oracle.c).
 * It exists so that the CPU columns of Table I have a like-for-like neighbour
 * measured on the host this library is benchmarked on.  It is NOT the parity
 * oracle (that one is double precision, oracle.c).
 *
 * Per row (Section VI-A): search the maximum and subtract it from every
 * element, exponentiate and sum, divide by the sum.
 *   "caching"     - the exponentials are stored at the summing step and reused;
 *   "recomputing" - they are computed again at the final step.
 * Both give the same values up to float rounding.
 */
#include <math.h>
#include <stddef.h>

void paper_cpu_softmax_caching_f32(const float *Z, float *out, long rows, long cols)
{
    for (long i = 0; i < rows; ++i) {
        const float *z = Z + (size_t)i * (size_t)cols;
        float *o = out + (size_t)i * (size_t)cols;
        float m = z[0];
        for (long j = 1; j < cols; ++j)
            if (z[j] > m)
                m = z[j];
        for (long j = 0; j < cols; ++j)
            o[j] = z[j] - m;
        float sum = 0.0f;
        for (long j = 0; j < cols; ++j) {
            o[j] = expf(o[j]);
            sum += o[j];
        }
        for (long j = 0; j < cols; ++j)
            o[j] = o[j] / sum;
    }
}

void paper_cpu_softmax_recomputing_f32(const float *Z, float *out, long rows, long cols)
{
    for (long i = 0; i < rows; ++i) {
        const float *z = Z + (size_t)i * (size_t)cols;
        float *o = out + (size_t)i * (size_t)cols;
        float m = z[0];
        for (long j = 1; j < cols; ++j)
            if (z[j] > m)
                m = z[j];
        for (long j = 0; j < cols; ++j)
            o[j] = z[j] - m;
        float sum = 0.0f;
        for (long j = 0; j < cols; ++j)
            sum += expf(o[j]);
        for (long j = 0; j < cols; ++j)
            o[j] = expf(o[j]) / sum;
    }
}
