/*
 * gpuvm_workloads.h -- C ABI of the workload kernels written against the device
 * accessors (gpuvm_device.cuh), and of their twins on plain device-accessible
 * pointers (for the same kernels over cudaMallocManaged memory).
 *
 * Common rules
 *   - `h` is a handle from gpuvm_create; *_off arguments are BYTE offsets of an
 *     array inside its backing store, multiples of 16.
 *   - d_* arguments are device pointers owned by the caller (results live in
 *     ordinary device memory, only the large inputs are paged); `stream` is a
 *     cudaStream_t passed as void* (NULL = default stream).
 *   - calls enqueue work and return without synchronising unless stated; device
 *     errors (a wait that ran out, an offset out of range) are sticky in the handle
 *     and show up in gpuvm_stats().  Return value: 0 or a negative gpuvm_status.
 *   - device scratch (queues of the graph workloads, request tables of the gather, row
 *     staging of the embedding bag) belongs to the handle: it is allocated the first
 *     time a workload needs it, grown when a later call needs more, and freed by
 *     gpuvm_destroy; calls that do not outgrow it allocate nothing (a per-call
 *     cudaMalloc / cudaFree pair was measured to stall for 0.1-0.5 s now and then).
 *     All workload calls on one handle share that scratch: do not let two of them
 *     overlap on the GPU.  The gpuvm_raw_* twins allocate and free per call.
 */
#ifndef GPUVM_WORKLOADS_H
#define GPUVM_WORKLOADS_H

#include "gpuvm.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Streaming read-reduce: *d_sum = sum of the n int32 values at a_off, as int64.
 * One warp per page: the page is pinned once, read with 16-byte loads and released
 * (the access pattern of the paper's transfer benchmark, Section 5.1: each warp is
 * assigned a page, consecutive addresses).  d_sum: device int64, overwritten.
 */
int gpuvm_stream_sum_i32(gpuvm_t h, size_t a_off, size_t n, int64_t *d_sum, void *stream);

/*
 * Random gather: for each block b of `block` consecutive indices,
 *   d_fsum[b] = float( sum of x[idx[k]] accumulated in double )
 *   d_bsum[b] = sum of the 32-bit patterns of the gathered values (int64, exact).
 * x: fp32 array at x_off; d_idx: n_idx int64 element indices in device memory.
 * d_fsum, d_bsum: ceil(n_idx / block) elements.  block <= 2^20.
 *
 * gpuvm_gather_f32: a requester warp keeps 2048 to 16384 requests registered in the page
 * table at once (gpuvm_batch.cuh), so that one migrated page serves many waiting requests
 * (Section 3.3: inter-warp coalescing); the faults go through a ring of page ids in shared
 * memory to the thread block's migrator warps, which move pages with bulk copies.  With up to
 * 16384 * 28 * (number of SMs) indices every request is in flight at once and each page is
 * fetched once.  Two forms of the request table:
 *   - block >= 256 and no scratch bound set: the index list itself is the table (read in
 *     place) and every gathered value is added to the double / int64 sums of its index
 *     block at once, in shared memory.  No device scratch.  The double sum is taken in the
 *     order of arrival, so d_fsum can differ from a fixed-order sum in the last bit when the
 *     sum lies within about 1e-13 (relative) of a float rounding boundary.
 *   - otherwise: 32-bit element indices staged in device scratch owned by the handle, 4
 *     bytes per request in flight (the array must then have fewer than 2^32 - 1 elements:
 *     GPUVM_E_RANGE otherwise), replaced by the values as they arrive and summed in index
 *     order; the warps take the deepest power of two that covers their share of the index
 *     list and fits gpuvm_set_scratch_limit.
 * gpuvm_gather_f32_unbatched: one thread per index through gpuvm_read<float>, one
 * thread block per index block; at most 32 requests per warp are in flight.
 */
int gpuvm_gather_f32(gpuvm_t h, size_t x_off, const int64_t *d_idx, size_t n_idx, size_t block,
                     float *d_fsum, int64_t *d_bsum, void *stream);
int gpuvm_gather_f32_unbatched(gpuvm_t h, size_t x_off, const int64_t *d_idx, size_t n_idx, size_t block,
                               float *d_fsum, int64_t *d_bsum, void *stream);

/*
 * BFS over a CSR graph whose int64 row offsets (nv + 1 of them, at off_off) and int32
 * column indices (at col_off) are paged (Section 5.2 runs BFS on CSR through the paged
 * arrays).  d_level: nv int32 in device memory, receives the hop distance from `source`,
 * -1 where unreachable (nv < 2^30).
 *
 * The sweeps go over the vertices in address order (warps draw chunks of 32 consecutive
 * vertices from a ticket counter, so the grid moves through the arrays as a narrow window;
 * per chunk the column pages its edges span are pinned one at a time), alternating
 * direction.  They are label-correcting rather than level-synchronous: a vertex is
 * expanded whenever its level has been lowered since it was last expanded (the level
 * array holds level << 1 | dirty while the sweeps run; lowering is an atomicMin that sets
 * the bit), so one sweep carries as many hops as the vertex order allows, and a vertex
 * that is lowered behind the sweep position is queued and re-expanded in the same sweep by
 * whichever warp is free.  No page is fetched for such a vertex: its two row offsets and its
 * edges are read from their frames where the pages are still in the pool
 * (gpuvm_ptr_if_resident) and in place from the backing store where they are not (the CSR
 * arrays are never written, so the backing store is current; gpuvm_stats counts these bytes as
 * bytes_direct).  A sweep that follows one with few updates works the same way throughout: it
 * reads the few scattered lists it needs in place instead of fetching a page for each.  The
 * fixed point is the BFS level.  With a pool of half the graph every page is fetched once per
 * run, where one sweep per level fetched most of the graph once per level.
 * Very long neighbour lists are cut at page boundaries into pieces that go to a queue which
 * all warps of the same launch serve between their chunks (the imbalance Section 5.2
 * describes).  The first sweep expands the source alone.  One launch per sweep; the stream is
 * synchronised between sweeps.  *n_levels (host pointer, may be NULL) receives the largest
 * level + 1.  Uses 2 MiB + max(nv, 2^18) bytes of the handle's device scratch (the two
 * queues and the counters).  The row offsets and column indices must not be written through
 * the runtime while the call runs.
 */
int gpuvm_bfs_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, size_t source,
                  int32_t *d_level, int *n_levels, void *stream);

/*
 * BFS over Balanced CSR (Section 5.2, Fig. 8): besides the row offsets and the column
 * indices, a third paged array at chunk_off holds, for every chunk of `chunk_edges`
 * consecutive edges, the number of the vertex whose neighbour list contains the chunk's
 * first edge (int32, ceil(n_edges / chunk_edges) + 1 entries, the last one = the vertex
 * of the last edge; built by gpuvm_bcsr_build).  Workers take chunks instead of
 * vertices, so each gets the same number of edges and exactly one column page however
 * skewed the degrees are, and a long list is expanded by as many warps as it has chunks.
 * A chunk must lie inside one page: col_off is a multiple of the page size and the page
 * size a multiple of 4 * chunk_edges.  Same result as gpuvm_bfs_csr.  Uses 16 bytes of
 * the handle's device scratch.  One launch and one synchronisation per level.
 */
int gpuvm_bfs_bcsr(gpuvm_t h, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges,
                   size_t chunk_edges, size_t source, int32_t *d_level, int *n_levels, void *stream);

/*
 * Connected components over Balanced CSR (Section 5.2, Fig. 8 runs CC on it): the union-find pass of
 * gpuvm_cc_csr, with workers that take chunks of edges instead of vertices.  Arguments as for
 * gpuvm_bfs_bcsr; d_label as for gpuvm_cc_csr.  One launch; synchronises the stream.
 */
int gpuvm_cc_bcsr(gpuvm_t h, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges,
                  size_t chunk_edges, int32_t *d_label, void *stream);

/*
 * Build the chunk table of Balanced CSR (Section 5.2, Fig. 8) from a graph's row offsets, on
 * the host: a format conversion done once, before the graph is handed to gpuvm_create.
 *   row_off       host pointer, nv + 1 int64 row offsets, row_off[0] = 0.
 *   chunk_vertex  host pointer, receives ceil(n_edges / chunk_edges) + 1 int32 entries: entry c
 *                 is the vertex whose neighbour list holds edge c * chunk_edges, the last entry
 *                 the vertex of the last edge (0 for a graph without edges).  NULL: only the
 *                 number of chunks is computed.
 *   capacity      entries that chunk_vertex can hold (GPUVM_E_RANGE when too few).
 *   n_chunks_out  host pointer (may be NULL), receives the number of chunks.
 * Runs on the CPU in one pass over the row offsets; needs no device.
 */
int gpuvm_bcsr_build(const int64_t *row_off, size_t nv, size_t chunk_edges, int32_t *chunk_vertex, size_t capacity,
                     size_t *n_chunks_out);

/*
 * Connected components of the same kind of graph (Section 5.2 evaluates CC next to BFS):
 * d_label[v] receives the smallest vertex number of the weakly connected component of v
 * (edges count in both directions).  Concurrent union-find in ONE sweep over the edges:
 * d_label starts as the identity and serves as the parent array; for every edge the roots
 * of both ends are found (with path halving) and the larger root is hooked under the
 * smaller with a compare-and-swap that succeeds only while it still is a root; a finishing
 * kernel replaces every parent by its root.  Every page of the graph is fetched once.
 * *n_sweeps (host pointer, may be NULL) receives the number of sweeps over the edges (1).
 * Uses 2 MiB of the handle's device scratch.  Synchronises the stream.
 */
int gpuvm_cc_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, int32_t *d_label, int *n_sweeps,
                 void *stream);

/*
 * Single-source shortest paths with int32 edge weights >= 0 stored in a third paged
 * array parallel to the column indices (Section 5.2; the weights are a separate
 * array as in the paper's Table 2).  w_off must differ from col_off by a multiple of
 * the page size, so that the weights of an edge range sit at the same place in their
 * page as the columns do in theirs; both pages are held together while the range is
 * relaxed, hence the pool needs at least two frames per warp of the grid
 * (GPUVM_E_FRAMES otherwise).  The same label-correcting sweeps as gpuvm_bfs_csr with
 * the edge weight in place of 1; d_dist[v] receives the distance from `source`,
 * 0x7FFFFFFF where unreachable (path lengths must stay below 2^30).  *n_rounds (host
 * pointer, may be NULL) receives the number of sweeps.  Uses 2 MiB + max(2 nv, 2^18) bytes of
 * the handle's device scratch.  Synchronises per sweep.
 */
int gpuvm_sssp_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t w_off, size_t nv, size_t source,
                   int32_t *d_dist, int *n_rounds, void *stream);

/*
 * gpuvm_bfs_csr for callers that must not allocate.  (The paper has no counterpart:
 * this entry point exists for the sake of such callers only.)
 *
 * Some callers cannot afford a cudaMalloc / cudaFree pair in the middle of their
 * work: code that runs between the phases of a latency-sensitive pipeline (device
 * allocation synchronises the whole device and may take a driver lock), plug-ins
 * whose host forbids allocation after start-up, and processes that have handed
 * all free device memory to their own pool, where cudaMalloc would simply fail.
 * For them this variant computes what gpuvm_bfs_csr computes, same arguments, same
 * results, with one sweep per level (the queue that gpuvm_bfs_csr keeps for vertices
 * lowered behind the sweep grows with the graph and has no place in a fixed array),
 * and takes its scratch (the queue of neighbour-list pieces and the sweep counters,
 * 2 MiB + 1 KiB) from an array that is part of the library's device image.  It calls no cudaMalloc, cudaFree or other
 * allocating routine.
 *
 *   - Limit: nv <= GPUVM_BFS_NOALLOC_MAX_VERTICES, the graph size the fixed queue
 *     is sized for; anything larger returns GPUVM_E_RANGE and runs nothing.
 *   - Cost: every device that loads the library holds the 2 MiB array until the
 *     process exits, whether or not this function is ever called.
 *   - The first call on a device looks up the array's device address (once per
 *     device, with that device current).  Make that first call during set-up,
 *     before any stream capture is started.
 *   - All calls on one device share the array.  Two calls whose kernels overlap
 *     on the GPU (different streams, different threads) race on it and give wrong
 *     levels; issue them one after the other.  Nothing needs clearing between
 *     calls: each call zeroes the queue's ready words on its stream before its
 *     first level, each level re-zeroes the counters.
 *   - The looked-up address is kept for the life of the process; it does not
 *     survive a cudaDeviceReset of that device (do not reset a device this
 *     library is still to be used on).
 * d_level, n_levels, stream, return value: as for gpuvm_bfs_csr.
 */
#define GPUVM_BFS_NOALLOC_MAX_VERTICES ((size_t)1 << 26)
int gpuvm_bfs_csr_noalloc(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, size_t source,
                          int32_t *d_level, int *n_levels, void *stream);

/*
 * Vector add c[i] = a[i] + b[i] over three paged fp32 arrays of n elements
 * (Listing 1).  c is written through the runtime: its pages become dirty and reach
 * the host by eviction write-back or gpuvm_flush.  One IEEE binary32 addition per
 * element, no fused operations.  A warp processes one page of the element range at a
 * time.  When the pool has at least two frames for every warp of the grid and c starts
 * on a page boundary, the page of c is kept pinned while its chunks are produced and,
 * being overwritten entirely, is not fetched from the host first (GPUVM_WRITE_ALL);
 * otherwise every chunk pins a, b and c one after the other and c is fetched like any
 * page that is written to.  c may be the same array as a or b (c_off == a_off or c_off ==
 * b_off: in place, taken one page at a time); any other overlap of c with an input is refused
 * with GPUVM_E_ARG.
 */
int gpuvm_vadd_f32(gpuvm_t h, size_t a_off, size_t b_off, size_t c_off, size_t n, void *stream);

/*
 * Embedding-bag gather: d_out[g][d] = sum over the `bag` rows of bag g of
 * table[row][d], added in list order in fp32.  table: fp32 [rows][dims] at t_off,
 * dims a multiple of 4 with dims/4 <= 32 lanes (a lane owns 4 consecutive dims);
 * d_rows: n_bags * bag int64 row ids; d_out: n_bags * dims fp32 (device memory, or pinned mapped host memory:
 * the sums are then written straight to the host; measured, that saves the copy afterwards and costs the kernel
 * as much).
 *
 * gpuvm_embag_f32: a requester warp registers the rows of 32 to 256 bags (up to 32 lookups
 * each) at once (gpuvm_batch.cuh); rows that arrive are staged in device scratch and added
 * per bag in list order once the batch is complete, so the result has the bits of a
 * sequential fp32 sum.  Scratch owned by the handle (allocated at the first call, freed by
 * gpuvm_destroy): 8 + 4 * dims bytes per request in flight.  The warps take as many groups
 * of 32 bags (1, 2, 4 or 8) as it takes to have every bag in flight at once, within
 * gpuvm_set_scratch_limit: 2.1 GiB for one group, dims = 128, on a full grid of 148 SMs.
 * The batched kernel reads a whole row from the frame of the row's first byte, so it needs rows
 * that never straddle a page: the page size a multiple of the row size (4 * dims bytes) and
 * t_off a multiple of the row size.  Any other layout (dims = 20 or 100, pages smaller than a
 * row) is served by the unbatched kernel, with the same result.  A row id whose row does not lie
 * inside the backing store entirely sets the sticky GPUVM_E_RANGE.
 * Which pages are fetched (gpuvm_set_inplace_divisor, gpuvm_set_inplace_counted in gpuvm.h): by default a short
 * kernel first counts the lookups per page (4 bytes of scratch per page); the rows of pages with fewer lookups than
 * the page holds rows are read in place from the backing store, page by page (counted as bytes_direct, no fault,
 * the page table untouched), every other page is fetched once, and when those pages fit the pool twice over the
 * rows are added up straight from their frames: the scratch is then 4 * dims + 4 bytes per row read in place and
 * 4 bytes per lookup instead of the tables and staged rows described above.  With the divisor 0 every first touch fetches
 * its page, as in the paper.  The result is the same bit for bit; the table must not be written through the
 * runtime while the call runs.
 * gpuvm_embag_f32_unbatched: one warp per bag, one row request at a time through
 * gpuvm_read; no scratch.
 */
int gpuvm_embag_f32(gpuvm_t h, size_t t_off, size_t dims, const int64_t *d_rows, size_t n_bags,
                    size_t bag, float *d_out, void *stream);
int gpuvm_embag_f32_unbatched(gpuvm_t h, size_t t_off, size_t dims, const int64_t *d_rows, size_t n_bags,
                              size_t bag, float *d_out, void *stream);

/*
 * Read-modify-write through the element accessors: for every k < n,
 * a[idx[k]] = a[idx[k]] * 3 + 1 on uint32 elements at a_off (wrapping).  Indices
 * must be distinct.  Exercises gpuvm_read + gpuvm_write with scattered dirty pages.
 */
int gpuvm_scatter_update_u32(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream);

/* The same update through gpuvm_batch_access in write mode, 1024 requests per warp staged in
 * shared memory, without migrator warps: each warp migrates the pages of its own faults. */
int gpuvm_scatter_update_u32_batched(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream);

/* The same update in write mode with the thread block's fault ring and two migrator warps per
 * block of six requester warps (512 requests per requester warp staged in shared memory):
 * migrators write dirty victims back with 16-byte stores and bring pages in with bulk copies;
 * with pages of 256 KiB or more the grid-wide ring is used as well (256 KiB of the handle's
 * device scratch). */
int gpuvm_scatter_update_u32_queued(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream);

/*
 * Transfer micro-benchmark (Section 5.1, Fig. 7): touch n_pages consecutive pages
 * starting at page first_page, one warp per page, `warps_per_sm` warps on every SM;
 * each warp pins its page (faulting it in) and releases it.  No payload is read.
 */
int gpuvm_touch_pages(gpuvm_t h, size_t first_page, size_t n_pages, int warps_per_sm, void *stream);

/* The same with a given total number of warps (rounded up to whole thread blocks of at most 8
 * warps, spread over the SMs): how many migrating warps the link needs (Section 3.2, Little's
 * law; Section 5.2, sensitivity to the number of queues). */
int gpuvm_touch_pages_warps(gpuvm_t h, size_t first_page, size_t n_pages, int total_warps, void *stream);

/* ---- the same kernels on plain pointers (cudaMallocManaged or device memory) */
int gpuvm_raw_stream_sum_i32(const int32_t *a, size_t n, int64_t *d_sum, void *stream);
int gpuvm_raw_gather_f32(const float *x, const int64_t *d_idx, size_t n_idx, size_t block,
                         float *d_fsum, int64_t *d_bsum, void *stream);
int gpuvm_raw_bfs_csr(const int64_t *row_off, const int32_t *col, size_t nv, size_t source,
                      int32_t *d_level, int *n_levels, void *stream);
int gpuvm_raw_cc_csr(const int64_t *row_off, const int32_t *col, size_t nv, int32_t *d_label, int *n_sweeps,
                     void *stream);
int gpuvm_raw_sssp_csr(const int64_t *row_off, const int32_t *col, const int32_t *weight, size_t nv,
                       size_t source, int32_t *d_dist, int *n_rounds, void *stream);
int gpuvm_raw_vadd_f32(const float *a, const float *b, float *c, size_t n, void *stream);
int gpuvm_raw_embag_f32(const float *table, size_t dims, const int64_t *d_rows, size_t n_bags,
                        size_t bag, float *d_out, void *stream);

/*
 * Host-link peaks measured with SM-issued 16-byte loads / stores on `bytes` of
 * pinned mapped host memory (host_ptr: host pointer, pinned) and a device buffer
 * d_buf of the same size: out[0] = host->device GB/s, out[1] = device->host GB/s,
 * out[2] = both directions at once (sum), each the best of `reps` (CUDA events).
 * out: host pointer to 3 doubles.  Synchronises.
 */
int gpuvm_link_peak(void *host_ptr, void *d_buf, size_t bytes, int reps, double *out);

/*
 * The same link read as scattered rows: n_rows rows of row_bytes (a multiple of 16, at most 512) at hashed
 * positions of the pinned region [host_ptr, host_ptr + host_bytes) are loaded by warps, four rows in flight
 * each, and stored to the device buffer d_buf of d_bytes (reused round-robin).  out[0] = GB/s, best of `reps`.
 * run = 1: every row at a position of its own: the ceiling of rows read in place as their lookups come up; it
 * falls with the size of the region (measured on one host: 51.4 GB/s over 1 GiB, 33.4 over 8 GiB, 24.5 over
 * 64 GiB, whatever the number of reads in flight).  run > 1: `run` consecutive rows fall into the same 2 MiB
 * of the region (a hashed 2 MiB block, hashed rows inside it): the pattern of rows bucketed by page, which the
 * same host serves at the sequential rate from a few dozen rows per block on.
 * out: host pointer to 1 double.  Synchronises.
 */
int gpuvm_link_peak_scattered(void *host_ptr, size_t host_bytes, size_t row_bytes, size_t n_rows, size_t run,
                              void *d_buf, size_t d_bytes, int reps, double *out);

/* Number of kernels this library has launched in the calling process. */
unsigned long long gpuvm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GPUVM_WORKLOADS_H */
