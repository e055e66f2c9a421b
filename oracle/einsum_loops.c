/*
 * TEST INFRASTRUCTURE - the CPU oracle's only native part.  Not part of the product library and
 * shares nothing with it.
 *
 * Named-dimension Einstein summation by its plain definition (Section 6, "Einstein Summation"):
 * every input is broadcast to the union of all dimensions, the inputs are multiplied component-wise,
 * and every dimension that is not in the output is summed out.  Written as one loop nest in fp64:
 *
 *     out[o] = sum over all index tuples r of the reduced dimensions of  prod_q in_q[(o, r) restricted to in_q]
 *
 * The iteration space is given as `n_out` output dimensions followed by `n_red` reduced dimensions.
 * A dimension an input does not carry has stride 0 for that input (that is the broadcast).  There is
 * no blocking, no reordering and no use of a BLAS; OpenMP only spreads independent output elements
 * over the host cores (each output element is still summed by one thread in index order).
 */
#include <stdint.h>
#include <stddef.h>

#define ORACLE_MAX_DIMS 16
#define ORACLE_MAX_INPUTS 8

int oracle_einsum_f64(int n_in, int n_out, int n_red,
                      const int64_t* sizes,       /* [n_out + n_red] */
                      const int64_t* in_strides,  /* [n_in][n_out + n_red], in elements, 0 = broadcast */
                      const int64_t* out_strides, /* [n_out], in elements */
                      const double* const* in, double* out)
{
    const int nd = n_out + n_red;
    if (n_in < 1 || n_in > ORACLE_MAX_INPUTS || nd > ORACLE_MAX_DIMS || n_out < 0 || n_red < 0) return 1;

    int64_t n_out_elems = 1, n_red_elems = 1;
    for (int d = 0; d < n_out; ++d) n_out_elems *= sizes[d];
    for (int d = n_out; d < nd; ++d) n_red_elems *= sizes[d];

#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < n_out_elems; ++o) {
        /* decode the output multi-index (last output dimension fastest) */
        int64_t base[ORACLE_MAX_INPUTS];
        for (int q = 0; q < n_in; ++q) base[q] = 0;
        int64_t out_off = 0, rem = o;
        for (int d = n_out - 1; d >= 0; --d) {
            const int64_t i = rem % sizes[d];
            rem /= sizes[d];
            out_off += i * out_strides[d];
            for (int q = 0; q < n_in; ++q) base[q] += i * in_strides[(size_t)q * nd + d];
        }
        /* sum over the reduced index tuples (last reduced dimension fastest) */
        double acc = 0.0;
        int64_t idx[ORACLE_MAX_DIMS];
        for (int d = 0; d < n_red; ++d) idx[d] = 0;
        for (int64_t r = 0; r < n_red_elems; ++r) {
            double prod = 1.0;
            for (int q = 0; q < n_in; ++q) {
                int64_t off = base[q];
                for (int d = 0; d < n_red; ++d) off += idx[d] * in_strides[(size_t)q * nd + n_out + d];
                prod *= in[q][off];
            }
            acc += prod;
            for (int d = n_red - 1; d >= 0; --d) { /* odometer step */
                if (++idx[d] < sizes[n_out + d]) break;
                idx[d] = 0;
            }
        }
        out[out_off] = acc;
    }
    return 0;
}
