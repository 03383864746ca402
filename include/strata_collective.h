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
 * launch per call (two for all-to-all-v); every operand of an output vector is seen by one thread, so the reductions need
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
 * The collectives do not consult the registration pool: any device buffers are accepted (only the MoE
 * receive buffer has a readiness check).  A size of 0 is legal and launches nothing.  A bounded device wait that runs out reports
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

/* point-to-point.  in: [R][bytes], out: [R][bytes]; out[dst_rank][j] = in[src_rank][j]; the other parts of
 * out are not touched.  bytes % 16 == 0. */
strata_status strata_p2p(strata_ctx* ctx, int32_t R, int32_t src_rank, int32_t dst_rank, const void* in, void* out,
                         size_t bytes, void* stream);

/* all-to-all-v: pairs exchange different volumes (the operator the paper names, with MoE dispatch/combine,
 * as the source of uneven traffic, Sec. 6.2).  in: [R][in_stride_bytes], out: [R][out_stride_bytes].
 * send_bytes, send_offset, recv_offset: DEVICE arrays int64 [R][R], read by the kernel (they may be written
 * by an earlier kernel on the same stream; nothing is copied to the host):
 *   rank p sends send_bytes[p][r] bytes, found at in[p] + send_offset[p][r], to rank r, where they land at
 *   out[r] + recv_offset[r][p].  Bytes of out that no pair addresses are not touched; pairs must not
 *   overlap in out (not checked).
 * Counts and offsets must be multiples of 16 and every pair must fit its two buffers: a pair that does
 * not is skipped and STRATA_ERR_ALIGNMENT / STRATA_ERR_CAPACITY is raised in the device status word.
 * R <= 32 (STRATA_ERR_SHAPE beyond: the pair table lives in shared memory); strides are non-zero multiples
 * of 16.  The work is cut into 16 KB units claimed in order by a persistent grid, so a heavy pair is
 * spread over all CTAs instead of being owned by one. */
strata_status strata_alltoallv(strata_ctx* ctx, int32_t R, const void* in, size_t in_stride_bytes, void* out,
                               size_t out_stride_bytes, const int64_t* send_bytes, const int64_t* send_offset,
                               const int64_t* recv_offset, void* stream);

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
