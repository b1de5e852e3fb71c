/*
 * bcs.h -- C ABI of the B200 (sm_100a) library that constructs the round-optimal
 * n-block broadcast schedules on circulant graphs of J. L. Traff, "(Poly)Logarithmic
 * Time Construction of Round-optimal n-Block Broadcast Schedules for Broadcast and
 * irregular Allgather in MPI" (arXiv 2205.10072), Section 2.
 *
 * Notation (Section 2): p processors ranked 0..p-1, q = ceil(log2 p), skips[0..q]
 * the jumps of the circulant graph (Algorithm 1), root = rank 0.  A schedule of
 * rank r is two arrays of q block numbers in [-q, q-1]: recvsched[k] and
 * sendsched[k] for round k of a phase; a non-negative entry is a block of the
 * current phase, a negative entry b-q is block b of the previous phase.
 *
 * Conventions of every entry point
 *   - "device" pointers are CUDA device addresses valid on the current device;
 *     "host" pointers are ordinary host addresses.  The caller owns every buffer.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work on that stream; they do not synchronise, and the
 *     library holds no device memory of its own unless an entry point says so
 *     (scratch memory is passed in by the caller as a `workspace`).
 *   - Schedule tables are int8, rank-major and unpadded: the row of rank r of a
 *     call for ranks r_begin..r_end-1 starts at byte (r - r_begin) * q.
 *   - Errors are return codes.  Arguments are checked before the first CUDA call: when
 *     BCS_ERR_ARG, BCS_ERR_RANGE, BCS_ERR_ALIGN or BCS_ERR_UNSUPPORTED is returned nothing
 *     was enqueued and no output byte was written.  BCS_ERR_CUDA means that the runtime
 *     refused a launch or a copy in the middle of a call: kernels enqueued before that point
 *     still run, and the outputs of that call are to be discarded.
 *   - Supported: 1 <= p <= 2^31 - 1 (block sets are 32-bit masks).  p == 1 has
 *     q == 0: every call succeeds and writes nothing.
 *   - An entry that the construction could not determine (Algorithm 4 finding no
 *     new block in either window; never observed) is written as BCS_BAD_ENTRY.
 */
#ifndef BCS_H_
#define BCS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BCS_OK = 0,
    BCS_ERR_ARG = 1,          /* NULL where a buffer is required, n == 0, bad combination */
    BCS_ERR_RANGE = 2,        /* p == 0, r_begin > r_end, r_end > p, offsets not monotone */
    BCS_ERR_ALIGN = 3,        /* an output pointer is not 16-byte aligned */
    BCS_ERR_UNSUPPORTED = 4,  /* p > 2^31 - 1, or a size beyond a stated maximum */
    BCS_ERR_CUDA = 5          /* the CUDA runtime refused a launch or a copy */
} bcs_status;

#define BCS_BAD_ENTRY 127
#define BCS_MAX_Q 31
#define BCS_SKIPS_STRIDE 32   /* words per row of a skips table */
#define BCS_STATIC_WORKSPACE_BYTES (8u << 20)   /* scratch built into the library, see bcs_build_static */

/* Human-readable name of a status code (static string, never NULL). */
const char *bcs_status_str(bcs_status st);

/* q = ceil(log2 p) (Section 2, first paragraph); 0 for p == 1, -1 for p == 0. */
int bcs_q(uint32_t p);

/* Algorithm 1: skips[q] = p, skips[k] = ceil(skips[k+1] / 2), skips[0] = 1.
 * skips_host: host array of at least q+1 words.  Errors: p == 0 -> BCS_ERR_RANGE,
 * p > 2^31-1 -> BCS_ERR_UNSUPPORTED, NULL -> BCS_ERR_ARG. */
bcs_status bcs_skips(uint32_t p, uint32_t *skips_host);

/* Receive and send schedules (Algorithm 4; Algorithm 5 resp. the table lookup of
 * Algorithm 9, sendsched[r][k] = recvsched[(r+skips[k]) mod p][k]) of the ranks
 * r_begin..r_end-1 of one p.
 *   recv_out, send_out: device, int8, (r_end-r_begin)*q bytes each, 16-byte
 *   aligned; either may be NULL (not wanted), not both unless the range is empty.
 *   workspace: device scratch owned by the caller, 16-byte aligned, or NULL.  With at
 *   least bcs_build_workspace_bytes(p, r_begin, r_end) bytes the call runs its fast
 *   construction: one pass writes a 32-bit "skip code" per rank of p (which skips add
 *   up to the rank, the sums Algorithm 2 walks down), a second finds each round's
 *   block from the codes of the two ranks bounding the window of Algorithm 4 and also
 *   keeps a round-major copy of the receive rows, a third reads the send rows from
 *   that copy.  With NULL (or too few bytes) a self-contained, several times slower
 *   construction runs (homerange descent per window; send entries whose to-processor
 *   lies outside the range are recomputed with Algorithm 4).  Both give identical
 *   tables, and any sub-range is self-contained either way.  The workspace holds
 *   nothing of value after the call; calls that share one must not overlap.
 * Errors: see the status codes. */
size_t bcs_build_workspace_bytes(uint32_t p, uint64_t r_begin, uint64_t r_end);
bcs_status bcs_build(uint32_t p, uint64_t r_begin, uint64_t r_end,
                     int8_t *recv_out, int8_t *send_out,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The same tables in two steps, for building one p in several rank chunks (or both
 * tables of the same ranks at different times) without repeating the construction:
 *   bcs_prepare runs the construction once for ALL ranks of p and leaves, in the caller's
 *   workspace of at least bcs_prepare_workspace_bytes(p) bytes (4 bytes of skip code plus q
 *   bytes per rank: 36.5 GB for p = 2^30-1), the receive schedule in round-major order;
 *   bcs_build_prepared then writes the rank-major receive rows of any range (a
 *   transposition of that copy) and its send rows (the same transposition with row k
 *   rotated by skips[k]: sendsched[r][k] = recvsched[(r+skips[k]) mod p][k], Algorithm 9).
 * The workspace must stay untouched between the two calls; any number of
 * bcs_build_prepared calls may follow one bcs_prepare.  Outputs, alignment and error codes
 * as for bcs_build; a workspace that is NULL or too small is BCS_ERR_ARG. */
size_t bcs_prepare_workspace_bytes(uint32_t p);
bcs_status bcs_prepare(uint32_t p, void *workspace, size_t workspace_bytes, void *cuda_stream);
/* bcs_prepare in two steps, for callers that want the rank-major receive rows of a chunk straight
 * from the construction instead of from a transposition afterwards:
 *   bcs_prepare_codes writes the skip codes of ALL ranks of p into the workspace;
 *   bcs_prepare_rows then runs Algorithm 4 for the ranks r_begin..r_end-1: their entries go into
 *   the round-major copy in the workspace and, if recv_out is not NULL, their rank-major rows to
 *   recv_out (device, (r_end-r_begin)*q bytes, 16-byte aligned).  r_begin must be a multiple of
 *   16 (BCS_ERR_ALIGN).  Chunks may be prepared in any order; once every rank of p has been
 *   through bcs_prepare_rows the workspace is what bcs_prepare leaves, and bcs_build_prepared
 *   gives the send rows of any range (sendsched[r][k] = recvsched[(r+skips[k]) mod p][k] reaches
 *   into other chunks, hence only then).
 * bcs_prepare(p, ...) is bcs_prepare_codes followed by bcs_prepare_rows(p, 0, p, NULL, ...). */
bcs_status bcs_prepare_codes(uint32_t p, void *workspace, size_t workspace_bytes, void *cuda_stream);
bcs_status bcs_prepare_rows(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);
bcs_status bcs_build_prepared(uint32_t p, uint64_t r_begin, uint64_t r_end,
                              int8_t *recv_out, int8_t *send_out,
                              const void *workspace, size_t workspace_bytes, void *cuda_stream);

/* bcs_build for callers that have no device memory to offer as a workspace and may not
 * allocate any (the paper has no counterpart; this is a convenience of the library).  Think of
 * code that runs after a framework has claimed the whole GPU for its own memory pool, or of a
 * latency-critical loop in which a cudaMalloc -- which can stall the whole device -- is not
 * acceptable.  The fast construction of bcs_build runs with its scratch taken from an array of
 * BCS_STATIC_WORKSPACE_BYTES (8 MiB) that is part of the library's device image: every GPU on
 * which the library is loaded gives up that much memory until the process exits, whether or
 * not this function is ever called.  The call itself allocates and frees nothing.
 *   Limit: bcs_build_workspace_bytes(p, r_begin, r_end) must not exceed
 *   BCS_STATIC_WORKSPACE_BYTES (all ranks of p up to about 300 000; of a larger p a
 *   correspondingly shorter range, and none once 4*p alone exceeds the array);
 *   otherwise BCS_ERR_UNSUPPORTED is returned and nothing is written.  Use bcs_build with
 *   your own workspace, or with NULL, beyond that.
 *   First use: the first call on each device asks the CUDA runtime for the array's device
 *   address (with that device current) and remembers it for the life of the process, so do
 *   not use this entry point across a cudaDeviceReset.  Where the runtime loads the library's
 *   device code lazily, that first call is also what sets the 8 MiB aside: make it early --
 *   before other code has claimed the rest of the device memory -- and outside any stream
 *   capture.  Later calls touch no allocator at all.
 *   Sharing: all calls on a device use the same array.  Two calls whose kernels can overlap
 *   on the GPU (different streams, or several host threads) race on it and produce garbage;
 *   order them on one stream or with events.  The array keeps whatever the last call left
 *   in it; this function needs none of it to be zero and reads only what it has written.
 * Outputs, range and error codes otherwise as for bcs_build. */
bcs_status bcs_build_static(uint32_t p, uint64_t r_begin, uint64_t r_end,
                            int8_t *recv_out, int8_t *send_out, void *cuda_stream);

/* Schedules of a broadcast rooted at processor `root` (Section 2: the processors are renumbered
 * by subtracting the root, so processor r uses the rank-0-rooted rows of virtual rank
 * (r - root) mod p; the skips, and with them the neighbours (r +- skips[k]) mod p, do not depend
 * on the root).  A thin remap over bcs_build:
 *   out[(r - r_begin)*q + k] = entry k of virtual rank (r - root) mod p,  r in [r_begin, r_end).
 * The virtual ranks of the range are one run, or two when they pass p - 1; each run is built
 * by bcs_build.  The second run starts (p - v0)*q bytes into the outputs (v0 the first virtual
 * rank); where that is not a multiple of 16 it is built in the workspace and copied into place
 * on the stream (cudaMemcpyAsync, device to device).
 *   root < p, else BCS_ERR_RANGE.  Outputs as for bcs_build.
 *   workspace, workspace_bytes: at least bcs_build_rooted_workspace_bytes(...) bytes (16-byte
 *   aligned) select the fast construction; NULL or less: the self-contained construction, which
 *   is then refused with BCS_ERR_ARG if the range needs the copy described above. */
size_t bcs_build_rooted_workspace_bytes(uint32_t p, uint32_t root, uint64_t r_begin, uint64_t r_end);
bcs_status bcs_build_rooted(uint32_t p, uint32_t root, uint64_t r_begin, uint64_t r_end,
                            int8_t *recv_out, int8_t *send_out, void *workspace,
                            size_t workspace_bytes, void *cuda_stream);

/* As bcs_build, then copies the tables to HOST memory on the same stream
 * (cudaMemcpyAsync; pinned host memory makes the copies asynchronous).
 *   recv_host, send_host: host, (r_end-r_begin)*q bytes each, either may be NULL.
 *   stage_dev: device staging buffer supplied by the caller, 16-byte aligned, of
 *   at least 2 * align256((r_end-r_begin)*q) bytes (align256 = round up to 256);
 *   what exceeds that is handed to bcs_build as its workspace, so adding
 *   bcs_build_workspace_bytes(...) bytes selects the fast construction.
 * The host buffers are complete once the stream has been synchronised. */
bcs_status bcs_build_to_host(uint32_t p, uint64_t r_begin, uint64_t r_end,
                             int8_t *recv_host, int8_t *send_host,
                             void *stage_dev, size_t stage_bytes, void *cuda_stream);

/* Host helper for bcs_build_batch: for a list of num_p values of p fills
 *   rank_off_host[num_p+1]  prefix sums of p_j            (flattened rank index),
 *   entry_off_host[num_p+1] prefix sums of p_j * q_j      (byte offset of p_j's table),
 *   tile_off_host[num_p+1]  prefix sums of ceil(p_j / 512) over the p_j above 1024, 0 for the
 *                           others (the fast construction works on a larger p in tiles of 512
 *                           ranks that start anew with every p, and builds both tables of a
 *                           p_j <= 1024 in one thread block that keeps everything on chip),
 *   copy_off_host[num_p+1]  prefix sums of q_j * align16(p_j) over the p_j above 1024 (where
 *                           p_j's round-major scratch copy starts in the workspace; align16 =
 *                           round up to 16),
 *   skips_tab_host[num_p * BCS_SKIPS_STRIDE] row j = skips[0..q_j] of p_j (Algorithm 1),
 *                           the rest of the row 0,
 *   full_tab_host[num_p * BCS_SKIPS_STRIDE]  row j, word d = skip code of rank
 *                           skips[d]-1 of p_j, d = 0..q_j.
 * The caller copies the six arrays and p_list to the device. */
bcs_status bcs_batch_plan(const uint32_t *p_list_host, uint32_t num_p,
                          uint64_t *rank_off_host, uint64_t *entry_off_host,
                          uint64_t *tile_off_host, uint64_t *copy_off_host,
                          uint32_t *skips_tab_host, uint32_t *full_tab_host);

/* All ranks of many p at once (the "full schedule" of Algorithm 9 for each p_j),
 * one launch sequence over the list of (p_j, r) pairs.  Device inputs as laid out by
 * bcs_batch_plan; total_ranks = rank_off[num_p], total_entries = entry_off[num_p],
 * total_tiles = tile_off[num_p], total_copy = copy_off[num_p] (the host knows all four).
 * Outputs: device int8, total_entries bytes each, 16-byte aligned; the table of p_j starts at
 * byte entry_off[j] and is rank-major with q_j bytes per rank, unpadded.  send_out may be NULL;
 * recv_out is required.  workspace as for bcs_build, of
 * bcs_build_batch_workspace_bytes(total_ranks, total_copy) bytes for the fast construction
 * (which also needs tile_off_dev and copy_off_dev; 256 bytes, never touched, when no p of the
 * list is above 1024: the pointer then only selects the construction), or NULL: then
 * tile_off_dev and copy_off_dev may be NULL too and the self-contained construction runs. */
size_t bcs_build_batch_workspace_bytes(uint64_t total_ranks, uint64_t total_copy);
bcs_status bcs_build_batch(const uint32_t *p_list_dev, const uint64_t *rank_off_dev,
                           const uint64_t *entry_off_dev, const uint64_t *tile_off_dev,
                           const uint64_t *copy_off_dev, const uint32_t *skips_tab_dev,
                           const uint32_t *full_tab_dev,
                           uint32_t num_p, uint64_t total_ranks, uint64_t total_entries,
                           uint64_t total_tiles, uint64_t total_copy,
                           int8_t *recv_out, int8_t *send_out,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Round tables of the n-block broadcast (Algorithm 6 without the Send||Recv): for
 * each rank r of r_begin..r_end-1 and each round j of 0..n-2+q one record of four
 * int32 {send block, receive block, to-processor, from-processor} with
 *   x = (q - (n-1+q) mod q) mod q, i = j + x, k = i mod q,
 *   block = sched[k] - x + q * floor(i / q); below 0 -> -1 (nothing is sent or
 *   received), above n-1 -> n-1; to = (r+skips[k]) mod p, from = (r-skips[k]+p) mod p.
 *   recv, send: device int8 rows of exactly these ranks as bcs_build writes them (the rows
 *   of the range, not the full [p][q] tables, so that a chunk can be built and expanded
 *   without the rest), or both NULL: the kernel then computes the rows of its ranks itself,
 *   as Algorithm 6 does by calling recvsched and sendsched -- each entry by the paper's
 *   per-rank construction (Algorithm 4 up to that round; the send entry as the receive entry
 *   of the to-processor, Algorithm 5), O(log^3 p) per rank, without scratch memory.  Meant
 *   for a few ranks or many rounds; for whole tables build the schedules once with bcs_build.
 *   One of the two NULL and the other not: BCS_ERR_ARG.
 *   table_out: device, (r_end-r_begin) * (n-1+q) records of 16 bytes, 16-byte
 *   aligned; record of (r, j) at index (r-r_begin)*(n-1+q) + j. */
bcs_status bcs_expand(uint32_t p, uint32_t n, uint64_t r_begin, uint64_t r_end,
                      const int8_t *recv, const int8_t *send, int32_t *table_out,
                      void *cuda_stream);

/* Round tables of the two other algorithms on the same circulant graph (Section 2.3), whose
 * edges run opposite to the broadcast's: q records of four int32 per rank, record of (r, k) at
 * index (r - r_begin) * q + k.
 *   census == 0, regular allgather (Algorithm 7): {to = (r - skips[k] + p) mod p,
 *     from = (r + skips[k]) mod p, number of blocks exchanged = skips[k+1] - skips[k] (blocks
 *     0..count-1 of the buffer are sent), offset skips[k] at which the received ones are stored};
 *   census != 0, census / allreduce (Algorithm 8): {to, from, 1 if x_r (+) S is sent and 0 if S
 *     alone, 0}; when skips[k] + skips[k] > skips[k+1] the edges are (r - skips[k] + 1) and
 *     (r + skips[k] - 1) and S alone is sent (the listing writes skips[i]; k is meant).
 * table_out: device, (r_end - r_begin) * q records, 16-byte aligned. */
bcs_status bcs_circulant_rounds(uint32_t p, uint64_t r_begin, uint64_t r_end, int census,
                                int32_t *table_out, void *cuda_stream);

/* Index tables of the irregular allgather (Algorithm 9 without the pack / Send||Recv / unpack
 * data movement) for ONE processor r: in round jr (0..n-2+q) processor r packs block
 * pack_out[jr * p + j] of buffer[j] for its to-processor and unpacks what it receives into
 * block unpack_out[jr * p + j] of buffer[j], j = 0..p-1; -1 = nothing for that buffer in that
 * round, blocks above n-1 are n-1.  Processor r handles buffer j as virtual processor
 * (r-j) mod p of the broadcast rooted at j, so the entries are the send / receive blocks of
 * that virtual processor's round, with the schedule adjustment of Algorithm 6 (-x, first use
 * of the first x entries in the second phase) applied to every row -- Algorithm 9 as printed
 * omits it and would then start with block x instead of block 0.  The to- and from-processors
 * of the round are those of bcs_expand.
 *   recv, send: device int8, the FULL [p][q] tables, 16-byte aligned; pack_out, unpack_out:
 *   device int32, (n-1+q) * p entries each, 4-byte aligned, either may be NULL. */
bcs_status bcs_allgather_tables(uint32_t p, uint32_t n, uint32_t r,
                                const int8_t *recv, const int8_t *send,
                                int32_t *pack_out, int32_t *unpack_out, void *cuda_stream);

/* Counts the ranks of r_begin..r_end-1 whose rows break a property that every schedule of the
 * construction has (text after Theorem 1; Algorithms 4, 5 and 9) -- a check that scales to
 * tables far too large to compare entry by entry:
 *   violations_dev[0]  receive row: the home round (skips[h] <= r < skips[h+1]) must hold the
 *                      baseblock of r (Algorithm 2), every other round a negative entry b-q,
 *                      the q-1 blocks b different from each other and from the baseblock; for
 *                      the root q different negative entries;
 *   violations_dev[1]  send row: the root sends block k in round k; any other rank sends a
 *                      previous-phase block that it received in an earlier round of the row,
 *                      or its own baseblock of the previous phase, or -- in the rounds after
 *                      its home round -- its baseblock (without recv only "some previous-phase
 *                      block" can be checked for the first two);
 *   violations_dev[2]  pairing: send[r][k] == recv[(r+skips[k]) mod p][k] wherever the
 *                      to-processor lies inside the range (needs both tables).
 * recv, send: device int8 rows of the ranks of the range as bcs_build writes them, 16-byte
 * aligned, either may be NULL (its checks are skipped).  violations_dev: device, three uint64,
 * overwritten.  Baseblocks are recomputed with Algorithm 2, independently of bcs_build. */
bcs_status bcs_validate(uint32_t p, uint64_t r_begin, uint64_t r_end,
                        const int8_t *recv, const int8_t *send,
                        uint64_t *violations_dev, void *cuda_stream);

/* Brute-force run of the n-block broadcast (Algorithm 6 without the data) over the complete
 * tables of one p, all ranks at once, n-1+q rounds, for p far beyond what a host can simulate.
 * Rank 0 starts with all n blocks.  Counted over all rounds and ranks:
 *   counts_dev[0]  a rank sends a block it does not hold at that time (condition a) of Section 2),
 *   counts_dev[1]  what a rank sends differs from what its to-processor receives in that round,
 *   counts_dev[2]  a non-root rank receives a block it already has (condition b)),
 *   counts_dev[3]  ranks that do not hold all n blocks after the last round,
 *   counts_dev[4]  ranks that already held all n blocks before the last round (the root always
 *                  does; n-1+q rounds being necessary, at least one rank must not).
 * A correct round-optimal schedule gives 0, 0, 0, 0 and counts_dev[4] < p.
 *   recv, send: device int8, the FULL [p][q] tables; n <= 64 (BCS_ERR_UNSUPPORTED beyond);
 *   state_dev: device scratch of 2 * p uint64, 8-byte aligned; counts_dev: five uint64,
 *   overwritten.  n + q + 1 kernels are enqueued on the stream. */
bcs_status bcs_simulate(uint32_t p, uint32_t n, const int8_t *recv, const int8_t *send,
                        uint64_t *state_dev, uint64_t *counts_dev, void *cuda_stream);

/* Bounded waits (no counterpart in the paper).  The transposition kernels of bcs_build,
 * bcs_build_prepared and bcs_build_batch wait for their bulk copies on a shared-memory barrier
 * with a poll limit; a CTA whose copies did not arrive within the limit gives up, leaves its
 * ranks of the output unwritten and counts itself in a device-wide counter that is never
 * reset.  The build call that enqueued the kernel has long returned BCS_OK by then, so this
 * poll is the only report.  The call waits for all work of the current device
 * (cudaDeviceSynchronize, whatever streams it was enqueued on) and then stores the counter in
 * *count_host (host).  0: every table written so far is complete.  Any increase since the last
 * reading: discard EVERY table built in between, not only the counted tiles -- a copy that
 * arrives after its CTA has gone may land in the shared memory of another CTA. */
bcs_status bcs_wait_expired(uint64_t *count_host);

/* Position-weighted 64-bit checksum of a stretch of schedule entries, additive
 * over disjoint stretches (no counterpart in the paper; used to compare outputs
 * that are too large to copy back).  The bytes are read as little-endian 32-bit
 * words of the whole entry stream: word g covers entries 4g..4g+3.
 *   sum = sum over words g of  word_g * weight(g)   mod 2^64,
 *   weight(g) = fmix32(low32(g) ^ (0x9E3779B9 * high32(g))) | 1,
 * fmix32 = the 32-bit finaliser of MurmurHash3.  buf_dev: device, 4-byte aligned;
 * first_entry_index must be a multiple of 4; a last partial word is zero-padded.
 * sum_dev: device uint64, overwritten with the sum (set to 0 first, then
 * accumulated atomically). */
bcs_status bcs_checksum(const int8_t *buf_dev, uint64_t n_entries,
                        uint64_t first_entry_index, uint64_t *sum_dev, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BCS_H_ */
