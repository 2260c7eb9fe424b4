// Thread-per-class locator (locate_rows_impl.cuh), kernels for groups of at most 32 workers.
#define APPROXIFER_ROWS_NMAX 32
#include "locate_rows_impl.cuh"
