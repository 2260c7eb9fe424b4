// Thread-per-class locator (locate_rows_impl.cuh), kernels for groups of at most 24 workers.
#define APPROXIFER_ROWS_NMAX 24
#include "locate_rows_impl.cuh"
