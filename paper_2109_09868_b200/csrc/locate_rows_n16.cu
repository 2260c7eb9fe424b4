// Thread-per-class locator (locate_rows_impl.cuh), kernels for groups of at most 16 workers.
#define APPROXIFER_ROWS_NMAX 16
#include "locate_rows_impl.cuh"
