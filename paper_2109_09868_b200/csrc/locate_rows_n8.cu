// Thread-per-class locator (locate_rows_impl.cuh), kernels for groups of at most 8 workers.
#define APPROXIFER_ROWS_NMAX 8
#include "locate_rows_impl.cuh"
