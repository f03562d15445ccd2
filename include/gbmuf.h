/* gbmuf.h -- C ABI of libgbmuf: the random-gossip BMUF synchronisation round on one GPU.
 *
 * The operation is the body of `if t mod H_i == 0` in Algorithm 1 ("gossip-MA (gossip-BMUF) for
 * node k") of "A Random Gossip BMUF Process for Neural Language Modeling": every worker k, for
 * every model component i that is due, picks q random neighbours on a p-symmetric ring
 * (Definition 1), averages its copy of the component with theirs, and passes the average through
 * the block-momentum filter (block delta G, momentum Delta <- eta Delta + zeta G, global model
 * omega <- omega + Delta, restart point theta <- omega + eta Delta).  The K workers are K
 * parameter replicas that live side by side in one GPU's memory.
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the context's GPU, owned by the CALLER (the
 *     library never frees or reallocates them); "host" pointers are ordinary host memory read or
 *     written before the call returns -- also when that memory is page-locked: small host tables
 *     (masks, offsets) are copied into the library's own staging memory before their upload is
 *     enqueued, so the caller may overwrite or free them as soon as the call is back.
 *   - theta, omega, delta are row-major [K][ld]: worker k's element e is at k*ld + e.  ld >= N,
 *     ld a multiple of 32, base pointers 128-byte aligned.  Columns N..ld-1 are padding: never
 *     written, contents irrelevant.  theta is fp32 or bf16 (theta_dtype); omega and delta are
 *     always fp32.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls that
 *     take a stream only enqueue work; they do not wait for it.
 *   - Every function returns a gbmuf_status; nothing throws or aborts across this boundary.
 *     Argument, state and size errors are found before any device work is enqueued, and
 *     out-parameters are untouched on error.  Only if a kernel launch itself is refused by the
 *     CUDA runtime (GBMUF_ERR_CUDA) may earlier steps of the same call (a table upload, the
 *     set-up kernel) already be in the stream; no round kernel has run in that case.
 *     gbmuf_last_error() gives a sentence about the most recent failure on that context.
 *   - Device-side waits are bounded (see gbmuf_selftest_wait_timeout).  A kernel whose wait
 *     expired leaves early and records GBMUF_ERR_TIMEOUT in the context's status word; nothing
 *     else reports it.  The buffers a round has written are therefore known to be good once
 *     gbmuf_device_status has returned GBMUF_OK for the stream the round ran in; one check after
 *     a sequence of rounds covers all of them (the word keeps the error until it is read).
 *   - Stream capture: calls that only launch kernels (gbmuf_init, gbmuf_local_perturb,
 *     gbmuf_local_adagrad without a new clip scratch, gbmuf_sync_round with comp_mask == NULL,
 *     gbmuf_final_average) may be recorded into a capture.  Calls that upload host tables
 *     (a comp_mask, gbmuf_sync_round_noalloc, gbmuf_set_partition) or wait for the device
 *     (gbmuf_device_status, gbmuf_get_neighbors, the host-memory calls) may not; the first two
 *     kinds return GBMUF_ERR_BAD_STATE inside a capture.
 *   - All arithmetic is fp32 with round-to-nearest-even on every single operation of Algorithm 1
 *     (no contraction into fused multiply-adds, no flush-to-zero), in the order Algorithm 1 writes
 *     it; the division by q+1 yields the correctly rounded quotient (see gbmuf_selftest_divide);
 *     a bf16 theta is widened exactly on load and rounded to nearest-even on store.
 *   - There is no CPU path and no other back-end: without a CUDA device every compute call
 *     returns GBMUF_ERR_CUDA.
 */
#ifndef GBMUF_H_
#define GBMUF_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gbmuf_ctx gbmuf_ctx; /* opaque, owned by the library, freed by gbmuf_destroy */

typedef enum {
  GBMUF_OK = 0,
  GBMUF_ERR_INVALID_ARG = 1, /* a size, pointer, alignment or hyper-parameter is out of range   */
  GBMUF_ERR_BAD_STATE = 2,   /* call order: e.g. sync_round before set_partition               */
  GBMUF_ERR_ALLOC = 3,       /* a small device table could not be allocated                     */
  GBMUF_ERR_CUDA = 4,        /* a CUDA runtime call failed (text in gbmuf_last_error)           */
  GBMUF_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (see gbmuf_device_status)    */
  GBMUF_ERR_UNSUPPORTED = 6  /* valid request outside what the kernels cover (e.g. K too large) */
} gbmuf_status;

typedef enum { GBMUF_F32 = 0, GBMUF_BF16 = 1 } gbmuf_dtype;

/* Algorithm 1 has two branches after the averaging line: gossip-BMUF (the filter) and gossip-MA
 * (theta <- average; omega and Delta are then neither read nor written). */
typedef enum { GBMUF_MODE_BMUF = 0, GBMUF_MODE_MA = 1 } gbmuf_mode;

typedef struct {
  int32_t K;           /* number of workers n (Definition 1), 1 <= K <= 256                       */
  int64_t N;           /* parameters per replica, >= 1                                            */
  int64_t ld;          /* row stride in elements: >= N, multiple of 32                            */
  int32_t p;           /* symmetric degree of the ring (Definition 1), >= 0; the candidate set of
                          worker k is (k-1)%K..(k-p)%K,(k+1)%K..(k+p)%K without k itself and
                          without repeats, so it has c = min(2p, K-1) members; c <= 64            */
  int32_t q;           /* gossip neighbours per draw, 0 <= q <= c (Algorithm 1: q <= 2p)          */
  float eta;           /* block momentum                                                          */
  float zeta;          /* block learning rate                                                     */
  int32_t mode;        /* gbmuf_mode                                                              */
  int32_t theta_dtype; /* gbmuf_dtype                                                             */
  uint64_t seed;       /* keys the neighbour draws and the synthetic local steps                  */
  int32_t device;      /* CUDA device ordinal                                                     */
  int32_t comp_base;   /* global index of this context's component 0 (>= 0).  Non-zero when the
                          buffers hold a column range of a larger model: draws are keyed by the
                          global component index, so a range reproduces the full model's choices */
  int64_t elem_base;   /* global index of column 0 (>= 0); keys the synthetic local-step noise     */
} gbmuf_config;

/* Bind a context to three caller-owned device buffers (theta, omega, delta: [K][ld], see the
 * conventions above).  Allocates only small tables (a few KB plus 4*K*m*q bytes later on).
 * The buffers must stay valid until gbmuf_destroy.  Errors: INVALID_ARG (any range, alignment or
 * NULL violation; q > c), UNSUPPORTED (K > 256, ld >= 2^31, c > 64),
 * CUDA, ALLOC. */
gbmuf_status gbmuf_create(const gbmuf_config* cfg, void* theta_device, float* omega_device,
                          float* delta_device, gbmuf_ctx** out);

/* Split theta = [theta_1^T .. theta_m^T]^T (Algorithm 1, second REQUIRE line): component i covers
 * elements offsets[i] .. offsets[i+1]-1.  offsets: host, m+1 entries, offsets[0] = 0, strictly
 * increasing, offsets[m] = N; no alignment is required of interior offsets.  periods: host, m
 * entries >= 1 (the synchronous period H_i of each component), or NULL for all 1.  May be called
 * again to re-partition; it then waits for the work THIS context has enqueued (in whatever
 * streams), not for the rest of the device.  1 <= m <= 65536.
 * Errors: INVALID_ARG, ALLOC, CUDA. */
gbmuf_status gbmuf_set_partition(gbmuf_ctx* ctx, int32_t m, const int64_t* offsets_host,
                                 const int32_t* periods_host);

/* Initialisation line of Algorithm 1: theta^k <- theta_0, omega^k <- theta_0, Delta^k <- 0 for
 * all k.  theta0: device, [N], theta's dtype, 16-byte aligned; may not alias theta. */
gbmuf_status gbmuf_init(gbmuf_ctx* ctx, const void* theta0_device, void* stream);

/* Synthetic stand-in for the local SGD line theta <- theta - alpha g of Algorithm 1 (there is no
 * model or data here): nsteps times, theta^k[e] <- store(theta^k[e] - lr * (sigma * z)), with
 * z(seed, step + s, k, elem_base + e) a counter-based, approximately standard normal value
 * (Philox4x32-10; sum of four 16-bit uniforms, centred and scaled to unit variance).  In place;
 * omega and Delta are not touched.  nsteps >= 0, step + nsteps <= 2^32 - 1. */
gbmuf_status gbmuf_local_perturb(gbmuf_ctx* ctx, uint64_t step, float lr, float sigma,
                                 int32_t nsteps, void* stream);

/* The local step with the optimiser of the paper's experiments (Section 3.2: Adagrad; the norm of
 * the LSTM gradients clipped to 10.0) in place of the plain SGD line of Algorithm 1, on gradients
 * the caller supplies.  grad: device fp32 [K][ld] (read only); accum: device fp32 [K][ld], the
 * Adagrad accumulator, caller-owned and caller-initialised (the usual start is 0.1), updated in
 * place; both 128-byte aligned.  Per worker k: norm_k = sqrt(sum of g^2 over the components whose
 * clip_mask byte is non-zero) (double accumulation, fixed order); inside those components
 * g' = g * (clip_norm / max(norm_k, clip_norm)), elsewhere g' = g; a <- a + g'g';
 * theta <- store(theta - (lr * g') / (sqrt(a) + eps)).  clip_mask: host, m bytes, or NULL (no
 * clipping; clip_norm <= 0 also switches it off); at most 16 separate runs of adjacent masked
 * components.  lr is the caller's alpha_t (the paper decays 0.1 by 0.9 per epoch).
 * Errors: INVALID_ARG, BAD_STATE (mask without set_partition), UNSUPPORTED, ALLOC, CUDA. */
gbmuf_status gbmuf_local_adagrad(gbmuf_ctx* ctx, const float* grad_device, float* accum_device,
                                 float lr, float eps, float clip_norm,
                                 const uint8_t* clip_mask_host, void* stream);

/* One synchronisation round `round` (the t of Algorithm 1).  Components taking part:
 * comp_mask != NULL: host, m bytes, component i takes part iff comp_mask[i] != 0;
 * comp_mask == NULL: component i takes part iff round % periods[i] == 0.
 * For each worker k and participating component i: the q neighbours are drawn for
 * (seed, round, k, comp_base + i); theta_bar = (theta^k + sum_j theta^{k_j}) / (q+1), own value
 * first, then the neighbours in draw order, all read as they were before this round;
 * G = theta_bar - R, with R the component as the worker's previous sync left it (theta_0 before
 * any); Delta <- eta Delta + zeta G; omega <- omega + Delta; theta <- omega + eta Delta.
 * R is not stored: it is recomputed as store(omega + eta Delta) from the values before the round,
 * which is bit-for-bit the expression that produced it (so a caller that fills omega and Delta
 * itself, rather than through gbmuf_init and earlier rounds, thereby defines R).  In MA mode
 * theta <- theta_bar only.
 * Everything happens in place in one pass; components not taking part are not touched.
 * Requires set_partition.  With a comp_mask the call may not be recorded into a stream capture
 * (BAD_STATE).  Errors: BAD_STATE, INVALID_ARG, CUDA. */
gbmuf_status gbmuf_sync_round(gbmuf_ctx* ctx, uint64_t round, const uint8_t* comp_mask_host,
                              void* stream);

/* The neighbour choices of round `round`: out is host, [K][m][q] int32 (worker ids).  Runs the
 * sampler kernel on a private stream and waits for it; does not disturb rounds in flight. */
gbmuf_status gbmuf_get_neighbors(gbmuf_ctx* ctx, uint64_t round, int32_t* out_host);

/* Return line of Algorithm 1: out[e] = (1/K) sum_k theta^k[e], summed for k = 0..K-1 in that
 * order.  out: device, [N], theta's dtype, 16-byte aligned. */
gbmuf_status gbmuf_final_average(gbmuf_ctx* ctx, void* out_device, void* stream);

/* Reads and clears the device-side status word (waits for `stream` first).  *out is GBMUF_OK, or
 * GBMUF_ERR_TIMEOUT if a kernel's bounded wait on a staged tile expired; the kernel then stopped
 * early and the buffers' contents are unspecified. */
gbmuf_status gbmuf_device_status(gbmuf_ctx* ctx, void* stream, int32_t* out);

/* Self-test of the failure reporting.  Every device-side wait in this library is bounded (two
 * seconds of the GPU's wall clock); when one expires the kernel records GBMUF_ERR_TIMEOUT in the
 * status word and leaves instead of hanging.  This call launches a one-warp kernel that waits on a
 * barrier nothing ever signals, waits for it, and returns GBMUF_OK iff the wait expired and the
 * kernel returned; *seconds_out (host, may be NULL) receives the kernel's duration.  Afterwards
 * gbmuf_device_status reports GBMUF_ERR_TIMEOUT once (reading clears it) and the context remains
 * fully usable.  No fault, trap or unbounded loop is involved. */
gbmuf_status gbmuf_selftest_wait_timeout(gbmuf_ctx* ctx, void* stream, double* seconds_out);

/* Self-test of the averaging division.  Algorithm 1's averaging line divides a sum by q+1; the
 * kernels compute that quotient for a small integer divisor that is not a power of two as
 * q0 = RN(s * RN(1/b)), r = fma(-b, q0, s), RN(q0 + r * RN(1/b)) when the exponent of s is in the
 * middle range, and with the division instruction sequence otherwise.  The result must equal the
 * IEEE-754 quotient rounded to nearest even in every bit.  This call evaluates both over ALL 2^32
 * bit patterns of s for the given divisor (2..256) and writes the number of patterns whose
 * results differ to *mismatches_out (host) and the smallest such pattern to *first_bad_out (host,
 * may be NULL; 0xFFFFFFFF if none).  Synchronises the stream.  Errors: INVALID_ARG, CUDA. */
gbmuf_status gbmuf_selftest_divide(gbmuf_ctx* ctx, int32_t divisor, void* stream,
                                   uint64_t* mismatches_out, uint32_t* first_bad_out);

/* Launch shape of the fused kernel (one persistent CTA per SM).  Any argument may be 0 to keep
 * the built-in choice.  Two variants exist.  (a) theta tile in tensor memory, outputs through bulk
 * stores: chosen automatically in gossip-BMUF mode when the resident rows of a tile fit the 512
 * columns of tensor memory.  Resident rows r: all K workers' rows, or -- because worker k only ever
 * averages with workers within ring distance p (Definition 1) -- a window of 2p + i rows that
 * slides along the ring plus the first p rows kept for the last workers, r = 3p + i (i = 2 for
 * fp32 theta, 4 for bf16; the last p rows of a tile are then read twice), or r = 4p + i with the
 * last p rows kept as well (every row read once; taken when it costs no tile width); the window
 * is possible when 2p + i < K and is taken when it allows a wider tile than K rows would (in
 * practice from about 20 workers on).  tile_elems must be a
 * multiple of 512 with r * tile_elems / 128 <= 512 for fp32 theta, <= 1024 for bf16; ring_slots
 * (2..8, at most three tiles' worth of rows) is the number of shared-memory slots every row
 * streams through.  (b) theta tile in shared memory: everything else, and whenever
 * consumer_threads or theta_stages is given or flags bit 3 is set; consumer_threads: multiple of
 * 32 in 32..992 (one more warp issues the copies); tile_elems: a multiple of 8 and, above 256, of
 * 256; theta_stages: 1..4; ring_slots: 2..8 rows of omega/Delta in flight.  (c) On request
 * (flags bit 4; by itself only for fp32 theta with 192 or more workers) and with K >= 2p + 2,
 * gossip-MA streams a window of rows along the ring
 * through shared memory instead of holding all K rows of a tile: rows 0 .. p-1 are kept (two sets,
 * for alternate tiles), the other rows pass through a ring of 2p + 6 .. 64 row slots, the last p
 * rows are read twice; tile_elems (a row slot) must be a multiple of 128 for fp32 theta, 256 for
 * bf16, at most 512 16-byte vectors.  flags: bit 0 = 256-byte L2 promotion for the theta loads of
 * (b); bit 1 = force (a), bit 2 (with bit 1) = with bulk stores (without: stores from registers);
 * bit 3 = force (b); bit 4 = force the ring window of (a) / of gossip-MA, bit 5 = never use it,
 * bit 6 = window of (a) with every row read once.  All choices give the same bits.
 * Errors: INVALID_ARG, UNSUPPORTED (does not fit, or (a) forced where it does not apply). */
gbmuf_status gbmuf_set_tuning(gbmuf_ctx* ctx, int32_t consumer_threads, int32_t tile_elems,
                              int32_t theta_stages, int32_t ring_slots, int32_t flags);

/* What the next full round would launch: tiles (work items), grid and block size, dynamic shared
 * memory in bytes, elements per tile, theta stages in shared memory (0 = the theta tile is kept in
 * tensor memory, all K rows; -r = in tensor memory as a ring window, r resident rows; 1000 + r =
 * gossip-MA ring window in shared memory with r ring slots).  Any out
 * pointer may be NULL.  Requires set_partition. */
gbmuf_status gbmuf_get_launch_info(gbmuf_ctx* ctx, int64_t* tiles, int32_t* grid, int32_t* block,
                                   int32_t* smem_bytes, int32_t* tile_elems, int32_t* stages);

/* Synchronisation rounds (as gbmuf_sync_round, same arithmetic and the same neighbour draws --
 * Algorithm 1, the body of `if t mod H_i == 0`) over replicas that live in HOST memory: theta,
 * omega, delta are host arrays [K][ld] (ld >= N, no alignment rule; page-locked memory lets the
 * copies overlap, pageable memory works but serialises them).  Given the neighbour table every
 * element of the round is independent, so the columns are cut into chunks of chunk_cols (a
 * multiple of 32; 0 = 2,097,152) that rotate through three sets of device buffers: copy in,
 * set-up + fused kernel, copy out, each set on its own stream.  Chunks in which no component
 * takes part are not copied at all.
 *   gbmuf_host_create allocates the device buffers (3 * K * chunk_cols * (element size + 8)
 *   bytes; gossip-MA: 3 * K * chunk_cols * element size), the three streams and the chunk tables
 *   once; cfg as for gbmuf_create (ld is the row stride of the HOST arrays), offsets host [m+1].
 *   flags: bit 0 = move each array of a chunk by K row copies instead of one 2-D copy.
 *   gbmuf_host_sync_round runs one round over the given host arrays (omega, delta may be NULL in
 *   gossip-MA mode) and returns when they hold the result; it allocates nothing.  comp_mask: host
 *   [m] or NULL (= all components take part).  Calls on one handle must not overlap.
 *   gbmuf_host_destroy frees everything (NULL is accepted).
 *   gbmuf_sync_round_host is create + one round + destroy in one call, for a single round.
 * Errors: INVALID_ARG, ALLOC, CUDA, TIMEOUT, UNSUPPORTED; text via gbmuf_last_error(NULL). */
typedef struct gbmuf_host gbmuf_host;
gbmuf_status gbmuf_host_create(const gbmuf_config* cfg, int32_t m, const int64_t* offsets_host,
                               int64_t chunk_cols, int32_t flags, gbmuf_host** out);
gbmuf_status gbmuf_host_sync_round(gbmuf_host* h, void* theta_host, float* omega_host,
                                   float* delta_host, const uint8_t* comp_mask_host, uint64_t round);
gbmuf_status gbmuf_host_destroy(gbmuf_host* h);
gbmuf_status gbmuf_sync_round_host(const gbmuf_config* cfg, void* theta_host, float* omega_host,
                                   float* delta_host, int32_t m, const int64_t* offsets_host,
                                   const uint8_t* comp_mask_host, uint64_t round, int64_t chunk_cols);

/* (No counterpart in the paper: this entry point exists for the library's callers, not for the
 * method.)  One synchronisation round that allocates nothing, for callers that must not or cannot
 * allocate device memory at the point where they synchronise: a training process whose memory pool
 * has already claimed the whole GPU, code running under an allocator that forbids foreign
 * cudaMalloc calls, or a plug-in that is handed buffers and a stream and nothing else.  It does
 * what gbmuf_create + gbmuf_set_partition + gbmuf_sync_round do for one round -- same kernels,
 * same results bit for bit -- but the library-side tables (component offsets, participation
 * flags, tile work-list, neighbour table, status word) live in one fixed array inside the loaded
 * library image instead of in cudaMalloc'ed memory.  The call itself uses no cudaMalloc/cudaFree
 * and no allocating library routine; theta, omega and delta are still the caller's.
 *   Limits: m <= 1024 components and K * m * q <= 65536 neighbour draws per round; larger
 *   requests are refused with GBMUF_ERR_UNSUPPORTED (use a context for them).  The array is
 *   276,224 bytes and every GPU on which the library is loaded keeps it until the process ends.
 *   Arguments: cfg as for gbmuf_create (device selects the GPU); theta/omega/delta device [K][ld];
 *   offsets host [m+1]; comp_mask host [m] or NULL (= every component takes part); round as in
 *   gbmuf_sync_round; stream a cudaStream_t.  device_status_out: NULL, or a host int32 -- then the
 *   call waits for the stream and stores the device status word (GBMUF_OK or GBMUF_ERR_TIMEOUT).
 *   First use on a device: the first call on each GPU looks up the device address of the array
 *   (cudaGetSymbolAddress, with that GPU current) and raises the kernels' shared-memory limit.
 *   Stream capture: every call uploads two small host tables (offsets, participation flags), so
 *   this entry point is not meant to be recorded into a stream capture at all, first call or
 *   later: inside a capture it returns GBMUF_ERR_BAD_STATE and enqueues nothing.  The tables
 *   are copied into static staging memory of the library before the upload, so offsets and
 *   comp_mask may be page-locked and may be overwritten as soon as the call returns.
 *   Sharing: all calls on a GPU use the same array.  It keeps the previous call's contents; this
 *   function clears the status word and rewrites every table it reads, so calls one after another
 *   on one stream are independent.  Calls that overlap on the GPU (different streams, or several
 *   host threads) race on the array and give undefined results: serialise them.
 * Errors: INVALID_ARG, UNSUPPORTED, BAD_STATE, CUDA; text via gbmuf_last_error(NULL) on the
 * calling thread. */
gbmuf_status gbmuf_sync_round_noalloc(const gbmuf_config* cfg, void* theta_device,
                                      float* omega_device, float* delta_device, int32_t m,
                                      const int64_t* offsets_host, const uint8_t* comp_mask_host,
                                      uint64_t round, void* stream, int32_t* device_status_out);

/* ---- one worker per GPU ("peer" form) ------------------------------------------------------------
 * The deployment the paper describes: every worker owns a GPU and, at a synchronisation step,
 * obtains the chosen neighbours' copies of each component (Algorithm 1, neighbour choice and
 * averaging lines; Section 3, experimental platform).  Here worker `rank` holds its own theta in
 * TWO buffers (a round reads one and writes the other), its omega and Delta ([ld] each), and
 * pointers to every other worker's two theta buffers, mapped into this process (CUDA IPC / peer
 * access; setting that up is the caller's business).  A round draws this worker's neighbours
 * exactly as gbmuf_sync_round does for worker `rank` (same seed, round, global component index),
 * and ONE kernel pulls their slices from peer memory (single-destination bulk copies), averages
 * (own value first, then draw order), filters, writes omega and Delta in place and the new theta
 * into the worker's other buffer.  Components that do not take part are copied to the other
 * buffer unchanged, so after the round the other buffer is the worker's complete theta.
 * Protocol: all workers call gbmuf_peer_sync_round(round, read_buffer = b), then synchronise
 * with one another (every worker's kernel finished), then use b' = 1 - b for the next round.
 * Within a round nobody writes a buffer that anybody reads, so no other ordering is needed.
 * theta_bufs: host array of 2*K device pointers, theta_bufs[b*K + j] = buffer b of worker j
 * (entry `rank` is this worker's own memory); all [ld] elements of theta's dtype, 128-byte
 * aligned, valid until gbmuf_peer_destroy.  cfg: K = number of workers, N, ld, p, q <= 15, eta,
 * zeta, mode, theta_dtype, seed, device, comp_base as for gbmuf_create.
 * Errors as for the context calls; text via gbmuf_last_error(NULL) on the calling thread. */
typedef struct gbmuf_peer gbmuf_peer;
gbmuf_status gbmuf_peer_create(const gbmuf_config* cfg, int32_t rank, void* const* theta_bufs_host,
                               float* omega_device, float* delta_device, gbmuf_peer** out);
gbmuf_status gbmuf_peer_set_partition(gbmuf_peer* h, int32_t m, const int64_t* offsets_host,
                                      const int32_t* periods_host);
gbmuf_status gbmuf_peer_sync_round(gbmuf_peer* h, uint64_t round, const uint8_t* comp_mask_host,
                                   int32_t read_buffer, void* stream);
gbmuf_status gbmuf_peer_device_status(gbmuf_peer* h, void* stream, int32_t* out);
gbmuf_status gbmuf_peer_destroy(gbmuf_peer* h);

/* Sentence about the last error on this context ("" if none); valid until the next call on it.
 * With ctx == NULL: the last error of a failed gbmuf_create on this thread. */
const char* gbmuf_last_error(const gbmuf_ctx* ctx);

/* Waits for the work this context has enqueued (not for the whole device), frees the library's
 * tables.  NULL is accepted. */
gbmuf_status gbmuf_destroy(gbmuf_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* GBMUF_H_ */
