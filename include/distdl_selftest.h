/* Self-test entry points of libdistdl.so.  They are not part of the operator interface
 * (include/distdl.h): they exist so that the library's failure paths can be exercised on a GPU
 * without a fault, a trap or an endless wait. */
#ifndef DISTDL_SELFTEST_H
#define DISTDL_SELFTEST_H

#include "distdl.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Launches one block in which one thread waits, with the same bounded wait the tensor-core
 * kernels use between their TMA, MMA and epilogue roles, on a shared-memory barrier that nothing
 * ever signals.  After `limit_cycles` SM clock cycles (1 .. 2e8, i.e. at most about 0.1 s; a real
 * kernel uses about 2 s) the wait gives up, the kernel records DISTDL_ERR_TIMEOUT in the device
 * status word and returns by itself; the CUDA context stays usable.  The next
 * distdl_device_status() reports DISTDL_ERR_TIMEOUT once and clears the word.
 * Returns DISTDL_ERR_INVALID_ARG for a limit outside the range, DISTDL_ERR_CUDA if the launch
 * fails.  `stream`: a cudaStream_t. */
distdl_status_t distdl_selftest_wait_timeout(int64_t limit_cycles, void *stream);

/* Copies the row plan of a partition (see distdl_partition_uses_row_plan; adjoint != 0: the plan of the row
 * ends of H*) to host arrays of 32-bit words: the header (rank, workers, workers per dimension, first record
 * and worker stride of every dimension, record and line counts, and for the two kinds of block -- ghost rows,
 * row ends -- the rows per block, blocks per worker or line and blocks per group, then the number of groups)
 * and one 16-word record per (dimension, worker coordinate): padded extent, low ghost width, bulk extent,
 * coordinates of the low / high neighbour (-1: none), index shifts into them, the neighbours' reach into the
 * bulk at both ends, five division constants, their shift counts, one unused word.  Lets a host-side test
 * replay the index arithmetic of the kernels without a GPU.  DISTDL_ERR_UNSUPPORTED if the partition has no
 * such plan, DISTDL_ERR_INVALID_ARG if an array is too small (the message gives the sizes needed). */
distdl_status_t distdl_selftest_row_plan(const distdl_partition_t *p, int32_t adjoint, int32_t *header, int32_t header_words,
                                         int32_t *records, int32_t record_words, int32_t *num_records);

#ifdef __cplusplus
}
#endif
#endif
