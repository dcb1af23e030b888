/*
 * kvh.h — C ABI of the per-chunk KV-cache codec (CUDA, sm_100a).
 *
 * The codec is the executor's data path in the paper's design (Design
 * section: estimator, policy optimizer, executor): it stores a context's KV
 * tensors at the quality the policy chose ("evict, store in full quality or
 * compress", last paragraph of the Design section) and, on a cache hit,
 * decompresses a stored chunk into the serving engine's paged bf16 KV (the
 * "decompression overhead" the estimator profiles).  A KV tensor is l layers
 * x {K,V} x N tokens x c channels of bf16 (the paper's N, c, l); a quality
 * level k is one rung of the ladder below.
 *
 * Levels (the paper prints only "2 bits" and "full quality"; the ladder, the
 * group geometry and the byte format are this library's definition):
 *   0  raw bf16, lossless                      16 bits/element
 *   1  8-bit asymmetric group quantisation      9 bits/element
 *   2  4-bit                                    5 bits/element
 *   3  2-bit                                    3 bits/element
 * K groups: one channel over 32 consecutive tokens of a chunk.  V groups: 32
 * consecutive channels of one token.  Per group a u32 = bf16(min) |
 * bf16(max) << 16.  A chunk is at most 256 tokens; its stream is, per layer,
 * Kmeta | Kcodes | Vmeta | Vcodes, each zero-padded to 128 bytes, with
 * Kmeta[ceil(n/32)][c], Vmeta[n][c/32], and the code of element (t, ch) in
 * bits [b*(t*c+ch), +b) of its section read as a little-endian bit string.
 * Level 0 has no metadata; its code sections are the bf16 rows themselves.
 * Arithmetic, binary32 round-to-nearest-even: r = max - min; when
 * 2^-100 <= r <= FLT_MAX, inv = qmax / r and scale = r / qmax, otherwise both
 * are 0 (every code 0, decodes to min); q = clamp(rint((x - min) * inv), 0,
 * qmax); xhat = bf16_rne(fma(q, scale, min)).  Inputs must be finite.
 *
 * Conventions.  Pointers marked [device] are CUDA device pointers, [host]
 * host pointers.  The caller owns every buffer; the library allocates no
 * device memory and keeps no state between calls (the one exception is
 * described with kvh_load_host_static).  Device work is enqueued on
 * `stream` (a cudaStream_t passed as void*, NULL = the default stream) and
 * the call returns without waiting.  Argument errors are reported by the
 * return value with nothing enqueued.  Errors only the GPU can see (a page id
 * outside the pool, a descriptor that does not fit its buffer) make the
 * kernel skip the offending chunk or page and atomicMax the status code into
 * *dev_status [device, may be NULL]; nothing traps.  No CPU fallback exists.
 *
 * Waits inside the kernels.  The persistent kernels feed themselves with
 * asynchronous copies and wait for them on shared-memory barriers.  No such
 * wait lasts longer than 2 seconds: a CTA whose wait runs out reports
 * KVH_ERR_TIMEOUT through *dev_status, stops taking work, lets its copies in
 * flight land and returns, so the launch ends and the context stays usable.
 * The work that CTA had not finished is then missing from the output; treat
 * the whole call as failed.  In a healthy process this never happens (a wait
 * is over within microseconds).
 */
#ifndef KVH_H
#define KVH_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVH_FORMAT_VERSION 1
#define KVH_CHUNK_TOKENS 256   /* most tokens in one chunk */
#define KVH_GROUP 32           /* tokens per K group, channels per V group */
#define KVH_SECTION_ALIGN 128  /* every section and chunk starts on this boundary */

typedef int kvh_status;
enum {
    KVH_OK = 0,
    KVH_ERR_INVALID_ARG = 1,      /* NULL pointer, negative count */
    KVH_ERR_BAD_LEVEL = 2,        /* level outside 0..3 */
    KVH_ERR_BAD_SHAPE = 3,        /* c not a multiple of 32, n_tok outside 1..256, ... */
    KVH_ERR_MISALIGNED = 4,       /* base not 128-byte (streams) / 16-byte (KV, pool) aligned */
    KVH_ERR_BUFFER_TOO_SMALL = 5, /* stream or page table shorter than a descriptor needs */
    KVH_ERR_PAGE_OOB = 6,         /* page id outside [0, num_pages): device-reported */
    KVH_ERR_CUDA = 7,             /* a CUDA runtime call failed (launch error) */
    KVH_ERR_TIMEOUT = 8           /* a bounded wait inside a kernel ran out: device-reported */
};

/* The serving engine's paged KV pool: element (layer, kv, page, slot, ch) is at
 * base + layer*layer_stride + kv*kv_stride + page*page_stride + slot*n_channels
 * + ch, in bf16 elements.  Strides must be multiples of 8 elements. */
typedef struct {
    void *base;            /* [device] bf16 */
    int64_t layer_stride;
    int64_t kv_stride;     /* kv = 0 for K, 1 for V */
    int64_t page_stride;
    int32_t num_pages;
    int32_t page_tokens;   /* tokens per page; must divide 256 (16 in the benchmark) */
    int32_t n_layers;
    int32_t n_channels;
} kvh_pool;

/* One stored chunk.  stream_off: byte offset of the chunk in the stream buffer
 * (multiple of 128).  pt_off: index in the page table of the chunk's first
 * page id (decode only); the chunk uses ceil(n_tok / page_tokens) entries. */
typedef struct {
    uint64_t stream_off;
    int32_t level;
    int32_t n_tok;
    int32_t pt_off;
    int32_t reserved;      /* must be 0 */
} kvh_chunk_desc;

int kvh_format_version(void);
int kvh_num_levels(void);
/* "default" for the library proper; the test builds of the same sources that select other
 * kernels or another tile schedule at compile time answer with their own name. */
const char *kvh_build_variant(void);
const char *kvh_status_string(kvh_status s);

/* Properties of a level: code bits per element, group size, 1 if lossless.
 * Any out pointer may be NULL.  [host] */
kvh_status kvh_level_info(int level, int *bits, int *group, int *lossless);

/* size(i, M, R) of the paper's utility definition for one chunk: bytes the
 * stored form of n_tokens (1..256) tokens takes at `level`.  Pure host
 * arithmetic.  *out [host]. */
kvh_status kvh_level_bytes(int level, int n_layers, int n_channels, int n_tokens,
                           uint64_t *out);

/* Lay out a context of n_tokens as ceil(n_tokens/256) chunks.  chunk_levels
 * [host, one entry per chunk] or NULL to use `level` for all.  Chunk i gets
 * stream_off = stream_base + sum of the sizes before it, pt_off = pt_base +
 * i * (256 / page_tokens).  descs_out [host, n chunks] may be NULL to ask only
 * for *total_bytes [host] (bytes from stream_base to the end of the last chunk).
 * Pure host arithmetic. */
kvh_status kvh_plan_chunks(int n_layers, int n_channels, int64_t n_tokens,
                           const int32_t *chunk_levels, int level,
                           uint64_t stream_base, int32_t pt_base, int32_t page_tokens,
                           kvh_chunk_desc *descs_out, uint64_t *total_bytes);

/* Encode a whole context at one level (the per-entry decision (M_i, R_i) of
 * the utility definition).  kv [device]: bf16 [n_layers][2][n_tokens][n_channels],
 * contiguous, 16-byte aligned.  out [device]: 128-byte aligned, out_capacity
 * bytes; chunk i lands at i * kvh_level_bytes(level, ..., 256).  Returns
 * KVH_ERR_BUFFER_TOO_SMALL if the context does not fit. */
kvh_status kvh_encode(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                      int level, void *out, uint64_t out_capacity,
                      int32_t *dev_status, void *stream);

/* Encode a context with a level per chunk.  descs [device, n_chunks =
 * ceil(n_tokens/256)]: desc i describes tokens [256 i, 256 i + n_tok) and where
 * its stream goes (as laid out by kvh_plan_chunks).  A descriptor with a bad
 * level, an n_tok that does not match the context, a misaligned offset or an
 * extent beyond out_capacity is skipped and reported through *dev_status.
 * descs_host [host, may be NULL]: the same n_chunks descriptors in host memory.
 * With them the call sorts the chunks by level and runs, per level, the kernel
 * that holds only that level's code (about 1.7 times faster on mixed contexts
 * than the one kernel that holds them all, which runs when descs_host is NULL);
 * a chunk whose two descriptors disagree on the level is skipped and reported. */
kvh_status kvh_encode_chunks(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                             const kvh_chunk_desc *descs, const kvh_chunk_desc *descs_host, int n_chunks,
                             void *out, uint64_t out_capacity,
                             int32_t *dev_status, void *stream);

/* Token dropping, the paper's second compression method (Introduction: contexts that matter "at
 * the beginning and the end"; the method cited keeps the first tokens, the attention sinks, and a
 * window of the most recent ones).  A kept run is a range of consecutive source tokens; the kept
 * tokens of all runs, in order, form the sequence that is stored, at any level, exactly as
 * kvh_encode_chunks would store a context of n_kept tokens.  On a hit the chunks decode into
 * consecutive page slots like any other context, so the engine sees the compacted cache. */
#define KVH_MAX_KEPT_RUNS 8
typedef struct {
    int64_t first;         /* first source token of the run */
    int64_t count;         /* tokens in the run, > 0 */
} kvh_token_run;

/* Runs kept when the first n_sink and the last n_recent tokens of an n_tokens context survive:
 * one or two runs, or the single run [0, n_tokens) when the windows meet.  runs_out [host, room
 * for 2]; *n_runs, *n_kept [host].  Pure host arithmetic. */
kvh_status kvh_keep_sinks_and_recent(int64_t n_tokens, int64_t n_sink, int64_t n_recent,
                                     kvh_token_run *runs_out, int *n_runs, int64_t *n_kept);

/* Encode the kept tokens of a context.  kv [device] as for kvh_encode ([n_layers][2][n_tokens]
 * [n_channels]).  runs [host, n_runs <= KVH_MAX_KEPT_RUNS]: ascending, disjoint, inside the
 * context.  descs [device, n_chunks = ceil(n_kept / 256)] describe the chunks of the compacted
 * sequence (lay them out with kvh_plan_chunks for n_kept tokens).  level >= 0 says that every
 * chunk is stored at this one level: descs may then be NULL (chunk i lands at i *
 * kvh_level_bytes(level, ..., 256), as with kvh_encode), a kernel holding only that level's code
 * runs, and a descriptor of another level is skipped and reported; level = -1 takes a level per
 * chunk from descs.  Everything else as for kvh_encode_chunks.  Rows wider than 1024 channels must
 * be divisible into equal blocks of at most 1024 channels that are multiples of 128
 * (KVH_ERR_BAD_SHAPE otherwise). */
kvh_status kvh_encode_kept(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                           const kvh_token_run *runs, int n_runs,
                           const kvh_chunk_desc *descs, int n_chunks, int level,
                           void *out, uint64_t out_capacity,
                           int32_t *dev_status, void *stream);

/* Decode one stored chunk (cache hit) into the pool.  chunk [device, 128-byte
 * aligned]: the chunk's stream.  page_ids [device]: ceil(n_tok/page_tokens)
 * page ids; token t goes to page page_ids[t / page_tokens], slot
 * t % page_tokens, in every layer and for K and V alike.  Slots past n_tok in
 * the last page are not written.  pool [host struct, device memory]. */
kvh_status kvh_decode_to_pages(const void *chunk, int level, int n_tok,
                               const int32_t *page_ids, const kvh_pool *pool,
                               int32_t *dev_status, void *stream);

/* Decode many stored chunks of mixed levels in one launch.  streams_base
 * [device, 128-byte aligned, streams_bytes long]; descs [device, n_chunks];
 * page_table [device, page_table_len entries].  Chunk i reads its stream at
 * streams_base + descs[i].stream_off and its page ids at page_table +
 * descs[i].pt_off.  Bad descriptors are skipped and reported. */
kvh_status kvh_decode_batch(const void *streams_base, uint64_t streams_bytes,
                            const kvh_chunk_desc *descs, int n_chunks,
                            const int32_t *page_table, int64_t page_table_len,
                            const kvh_pool *pool, int32_t *dev_status, void *stream);

/* Transcode stored chunks to a coarser level on the device ("compress furthermore" in the
 * paper's marginal-utility step, applied to an entry that is already stored).  Chunk i is read at
 * in_streams + in_descs[i].stream_off at level in_descs[i].level and written at out_streams +
 * out_descs[i].stream_off at level out_descs[i].level; the result is, bit for bit, the encoding at
 * the new level of the bf16 values the old chunk decodes to.  Both descriptor arrays [device,
 * n_chunks] must agree on n_tok, and the new level must be coarser (greater) than the old one;
 * chunks that break a rule are skipped and reported through *dev_status (pt_off is not used).
 * level_in / level_out: when every chunk goes from one level to one other level, pass them and a
 * kernel specialised for the pair runs (chunks with other levels are skipped and reported);
 * pass -1 / -1 for any mix.  in_descs_host / out_descs_host [host, n_chunks each, may both be
 * NULL]: host copies of the two arrays; with them a mix is sorted by pair of levels on the host
 * and every pair runs through its specialised kernel (as kvh_encode_chunks does per level).  The
 * two stream buffers must not overlap.  Rows wider than 1024 channels: as for kvh_encode_kept. */
kvh_status kvh_transcode(const void *in_streams, uint64_t in_bytes, const kvh_chunk_desc *in_descs,
                         void *out_streams, uint64_t out_capacity, const kvh_chunk_desc *out_descs,
                         const kvh_chunk_desc *in_descs_host, const kvh_chunk_desc *out_descs_host,
                         int n_chunks, int n_layers, int n_channels, int level_in, int level_out,
                         int32_t *dev_status, void *stream);

/* ---- host-tier entry points: the stored form lives in (pinned) host memory ------------------
 *
 * The paper keeps compressed entries in DRAM and SSD and loads them on a hit; its loading delay
 * is size / bandwidth (utility definition).  These two calls move a context between pinned host
 * memory and the GPU in slices of about slice_bytes, overlapping the PCIe copy of one slice (on
 * copy_stream) with the kernel of the previous one (on stream).  descs_host [host] and descs_dev
 * [device] hold the same n_chunks descriptors, laid out by kvh_plan_chunks with ascending,
 * contiguous stream offsets; offsets index both the host buffer and dev_staging [device,
 * 128-byte aligned, staging_bytes long].  If host_status [host, pinned] is not NULL, *dev_status
 * is copied to it on `stream` after the last kernel.  copy_stream must be a non-NULL stream
 * other than `stream`, created non-blocking if `stream` is the default stream; the calls return
 * without waiting and create no device memory. */

/* Cache hit on the host tier: copy the stored chunks host -> device and decode them into the
 * pool.  The load path of the paper's hierarchy. */
kvh_status kvh_load_host(const void *host_streams, void *dev_staging, uint64_t staging_bytes,
                         const kvh_chunk_desc *descs_host, const kvh_chunk_desc *descs_dev,
                         int n_chunks, const int32_t *page_table, int64_t page_table_len,
                         const kvh_pool *pool, int32_t *dev_status, int32_t *host_status,
                         uint64_t slice_bytes, void *copy_stream, void *stream);

/* Store to the host tier: encode the context kv [device] chunk by chunk and copy the streams
 * device -> host.  descs describe the whole context (chunk i = tokens [256 i, ...)). */
kvh_status kvh_store_host(const void *kv, int n_layers, int64_t n_tokens, int n_channels,
                          const kvh_chunk_desc *descs_host, const kvh_chunk_desc *descs_dev,
                          int n_chunks, void *dev_staging, uint64_t staging_bytes, void *host_out,
                          int32_t *dev_status, int32_t *host_status, uint64_t slice_bytes,
                          void *copy_stream, void *stream);

/* ---- the policy: which stored form every entry gets ---------------------------------------------
 *
 * Host arithmetic only.  The paper's Design section: Utility(i) = Freq(i) * (alpha * Quality(i, M_i,
 * R_i) - size(i, M_i, R_i) / Bandwidth); the choice of (M_i, R_i) under a tier's capacity is a
 * multiple-choice knapsack, solved greedily by the smallest marginal utility drop (utility lost
 * per byte saved) over each entry's LP-undominated options, eviction included.  An option is one
 * stored form of an entry: its size in bytes (kvh_level_bytes / kvh_plan_chunks for the level and
 * the kept tokens) and the estimated quality of answers generated from it.  The options of all
 * entries are concatenated; option_begin [n_entries + 1] delimits each entry's. */
typedef struct {
    uint64_t size;         /* stored bytes */
    double quality;        /* estimated quality, any scale (alpha converts it to seconds) */
} kvh_option;

typedef struct {
    double alpha;          /* weight of quality against loading delay */
    double bandwidth;      /* bytes per second from this tier to the GPU, > 0 */
    uint64_t capacity;     /* bytes */
} kvh_tier;

/* One tier.  choice_out [n_entries]: index of the chosen option within the entry's own options,
 * or -1 = evicted.  used_bytes, total_utility [host] may be NULL.  Slopes are compared in extended
 * precision; ties go to the lower entry index. */
kvh_status kvh_policy_assign(const double *freq, const kvh_option *options, const int32_t *option_begin,
                             int n_entries, const kvh_tier *tier, int32_t *choice_out,
                             uint64_t *used_bytes, double *total_utility);

/* Several tiers, fastest first (DRAM, then SSD in the paper): what a tier evicts is offered to
 * the next; what the last one evicts is recomputed on a hit.  tier_out [n_entries]: tier index or
 * -1; choice_out as above. */
kvh_status kvh_policy_assign_tiers(const double *freq, const kvh_option *options, const int32_t *option_begin,
                                   int n_entries, const kvh_tier *tiers, int n_tiers,
                                   int32_t *tier_out, int32_t *choice_out);

/* A check callers can run on their page table before a load [host arithmetic].  KVH_ERR_PAGE_OOB
 * if an id lies outside [0, num_pages), KVH_ERR_INVALID_ARG if an id occurs twice (two chunks
 * decoded into the same page would race); *first_bad [host, may be NULL] receives the index of the
 * first offending entry (for a duplicate: the later of the two). */
kvh_status kvh_check_page_table(const int32_t *page_table, int64_t len, int32_t num_pages,
                                int64_t *first_bad);

/* ---- a load entry point that allocates nothing -------------------------------------------------
 *
 * The paper has no counterpart to this call; it exists for how the library gets deployed.  Some
 * callers of kvh_load_host have no device allocator at hand when a cache hit arrives: a plug-in
 * running inside a serving engine that has already handed all free HBM to its paged KV pool, a
 * thread that must not take the allocator's lock, or code running while a stream capture is open
 * elsewhere in the process, where cudaMalloc is not permitted.  For them the staging area that
 * kvh_load_host takes as an argument is a fixed array inside the library's device image,
 * KVH_STATIC_STAGING_BYTES long.  Every GPU on which the library is loaded gives up that much
 * memory until the process exits, whether or not this call is ever made.
 *
 * Arguments and behaviour are those of kvh_load_host without dev_staging / staging_bytes.  The
 * descriptors' stream offsets index the host buffer and the fixed array alike, so the end of the
 * last chunk (its stream_off plus its size) must not exceed KVH_STATIC_STAGING_BYTES; a larger
 * request returns KVH_ERR_BUFFER_TOO_SMALL with nothing enqueued.  Split such a request into
 * several calls whose descriptors start again at offset 0.  Splitting stops at one chunk: a single
 * 256-token chunk that is larger than the array cannot be served by this call at all.  A full
 * chunk takes 1024, 576, 320 or 192 bytes per layer and channel at levels 0..3, so one chunk fits
 * while n_layers * n_channels is at most 65,536 / 116,508 / 209,715 / 349,525; at 80 layers of
 * 1024 channels a level-0 chunk (80 MiB) does not fit, the quantised levels (45, 25, 15 MiB) do.
 *
 * What the call does create: no device memory and no host buffers, but one short-lived CUDA event
 * per slice and direction of hand-over (created, recorded, waited on and destroyed inside the
 * call, exactly as in kvh_load_host), and, like every launch, it makes the runtime load the code of
 * the decode kernel instance it uses the first time that instance runs.
 *
 * Set-up.  The first call on each device looks up the array's device address (with that device
 * current) and remembers it for the life of the process: the one piece of state this library
 * keeps.  Make that first call, and one call for every pool geometry that will be used (channel
 * count and page size select the kernel instance), outside any stream capture and before the
 * engine claims the rest of the device's memory: the array is part of the library's device image,
 * which is loaded as a whole, so if the image does not fit, every kvh call on that device fails
 * with KVH_ERR_CUDA, not only this one.
 *
 * Sharing.  All calls on a device share the one array and it keeps whatever the last call left
 * there: nothing in it needs to start at zero, because every byte a decode reads is copied in by
 * the same call first.  Two calls whose GPU work can overlap (different `stream`s, or several
 * host threads) overwrite each other's staged chunks; order them on one stream or with events. */
#define KVH_STATIC_STAGING_BYTES (64u << 20)

kvh_status kvh_load_host_static(const void *host_streams,
                                const kvh_chunk_desc *descs_host, const kvh_chunk_desc *descs_dev,
                                int n_chunks, const int32_t *page_table, int64_t page_table_len,
                                const kvh_pool *pool, int32_t *dev_status, int32_t *host_status,
                                uint64_t slice_bytes, void *copy_stream, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* KVH_H */
