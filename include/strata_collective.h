/*
 * Full-mesh collectives over R emulated ranks (C ABI, sm_100a).
 *
 * Paper Sec. 6.1 ("Full-Mesh Programming Abstraction"): an operator is a set of remote-slice
 * transfers that complete in one logical step.  Data-movement operators run in pull mode (a rank
 * reads the peers' slices and writes them into its own output, no producer-consumer handshake);
 * reduction-bearing operators load the peers' operands on chip and accumulate them into the local
 * destination.  The paper measures them at 32 ranks with 1 MiB .. 1 GiB per rank (Sec. 8.1).
 *
 * Here all R ranks are partitions of ONE GPU's memory, as for the MoE path: rank r's input is the
 * r-th equal part of `in`, its output the r-th equal part of `out`.  Nothing crosses a link, so what
 * is measured is the memory system serving the operator's slice map, not a fabric.  One kernel
 * launch per call; every operand of an output vector is seen by one thread, so the reductions need
 * neither atomics nor locks.
 *
 * Arithmetic of the reductions (this build's reading; the paper names none): bf16 operands, one
 * binary32 addition per peer in rank order 0..R-1 starting from +0, one rounding to bf16 (nearest,
 * ties to even) at the end.  The result is bit-for-bit reproducible.
 *
 * All pointers are DEVICE pointers owned by the caller, 16-byte aligned; `in` and `out` must not
 * overlap.  The calls enqueue on `stream` (a cudaStream_t passed as void*) and return; they take
 * the device, the workspace and the trace buffer from the context, and R from the argument (it
 * need not equal the context's MoE shape).  Errors found on the host are returned before any launch:
 * STRATA_ERR_INVALID_ARG (NULL, R outside [1, 1024], root out of range), STRATA_ERR_SHAPE (a size
 * that is not a multiple of 16 bytes / 8 elements, or more than 2^32-1 work units),
 * STRATA_ERR_ALIGNMENT, STRATA_ERR_WORKSPACE, STRATA_ERR_CUDA (host-only context, launch failure).
 * A size of 0 is legal and launches nothing.  A bounded device wait that runs out reports
 * STRATA_ERR_TIMEOUT through strata_device_status().  Like the MoE calls they belong to the
 * context's single stream at a time.
 */
#ifndef STRATA_COLLECTIVE_H
#define STRATA_COLLECTIVE_H

#include "strata_moe.h"

#ifdef __cplusplus
extern "C" {
#endif

/* all-gather.  in: [R][bytes_per_rank], out: [R][R][bytes_per_rank];
 * out[r][p][j] = in[p][j].  bytes_per_rank % 16 == 0. */
strata_status strata_allgather(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t bytes_per_rank,
                               void* stream);

/* all-to-all.  in: [R][R][bytes_per_slice], out: [R][R][bytes_per_slice];
 * out[r][p][j] = in[p][r][j] (rank r's p-th output slice is what rank p addressed to r).
 * bytes_per_slice % 16 == 0. */
strata_status strata_alltoall(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t bytes_per_slice,
                              void* stream);

/* broadcast.  in: [R][bytes] (only rank `root`'s part is read), out: [R][bytes];
 * out[r][j] = in[root][j].  bytes % 16 == 0. */
strata_status strata_broadcast(strata_ctx* ctx, int32_t R, int32_t root, const void* in, void* out, size_t bytes,
                               void* stream);

/* reduce-scatter.  in: bf16 [R][R][elems_per_slice], out: bf16 [R][elems_per_slice];
 * out[r][j] = bf16( sum over p = 0..R-1, in that order, of in[p][r][j] ).  elems_per_slice % 8 == 0. */
strata_status strata_reducescatter(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t elems_per_slice,
                                   void* stream);

/* all-reduce.  in: bf16 [R][elems], out: bf16 [R][elems];
 * out[r][j] = bf16( sum over p = 0..R-1, in that order, of in[p][j] ) for every r.  elems % 8 == 0. */
strata_status strata_allreduce(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t elems, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* STRATA_COLLECTIVE_H */
