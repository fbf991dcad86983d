/*
 * mkv.h -- C ABI of libmkv: mixed-format (FP8 + TQ3) paged KV cache and decode attention for
 * NVIDIA B200 (sm_100a), after the Minima-KV paper.
 *
 * One pool holds the KV pages of ONE attention layer in two physical stores (Section 4.1,
 * "Physical stores and decode dispatch"): an FP8 arena for Recent and Anchor pages and a TQ3
 * arena for Stale pages.  A request's logical cache is a row of a block table; every entry
 * carries a tier tag that selects the arena and a physical page id inside it (Section 3.1:
 * z_p in {R, A, S}).  Decode attention walks that single table in one pass and merges the FP8
 * and TQ3 tokens under one softmax (Section 3.3, Eq. softmax-merge); no dequantised copy of the
 * cache is ever built.
 *
 * Conventions
 *   - page = 16 tokens by default, or 16 M tokens, M <= 256 (Section 4.1 stores blocks of 1,792 and of
 *     832 tokens); head_dim d in {128, 256}; query head h reads KV head h / (n_q/n_kv); at most 8
 *     query heads per KV head.
 *   - "device" pointers are CUDA device memory owned by the caller, 16-byte aligned (arenas and
 *     workspace 256-byte aligned); "host" pointers are ordinary host memory.  The library
 *     allocates no device memory: the caller hands it arenas and workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).  Calls that take
 *     a stream only enqueue work and never synchronise with the host unless stated.
 *   - every function returns 0 (MKV_OK) or a negative mkv_status; no exceptions cross the ABI.
 *     Host-detectable misuse (bad sizes, null pointers, unaligned pointers, unsupported shapes)
 *     returns MKV_E_INVALID without launching anything.  Out-of-range page ids or tags met ON
 *     THE DEVICE never fault: the kernel skips the access and records the event in the pool's
 *     status word, read with mkv_pool_status().
 *   - bf16 / fp16 / e4m3 data are passed as raw 16- / 8-bit words.
 *
 * Record formats (per page and KV head), little endian:
 *   FP8 record, 32*d bytes:   K e4m3 [16 tokens][d], then V e4m3 [d channels][16 tokens].
 *     stored = e4m3(x / scale) rounded to nearest even, saturating at +-448.
 *   TQ3 record, 16*d + 32 bytes (Section 4.1: three-bit rotated key codes, FP16 key-norm
 *     correction, three-bit value codes, FP16 scale/zero):
 *       [0, 6d)   key codes,   [6d, 12d) value codes,   [12d, 12d+32) norm correction g[16],
 *       [12d+32, 16d+32) value scale/zero.  Bit positions are those of the tensor-core
 *     fragment that consumes them; mkv_page_read_raw() returns the bytes as stored.
 *   TQ3 record format 2 (mkv_pool_config.tq3_format = 2; Section 3.1 fixes neither codebook nor layout):
 *     the four key magnitudes are the e4m3 numbers nearest to the Lloyd-Max levels (0.25, 0.75, 1.375,
 *     2.25; thresholds 0.5, 1.0625, 1.8125; about 1 % more Gaussian distortion), and the key section is
 *     cut so that four consecutive dims of a token are the nibbles of one half-word.  All levels are
 *     eighths of small integers (2, 6, 11, 18), so the decode scan turns four codes into four signed bytes
 *     with one byte-table lookup and multiplies them in integer tensor-core instructions against the rotated
 *     query carried as three base-128 digits per head (exact integer sums).  Value codes, norm corrections,
 *     scale/zero, sizes and every other encoder step are those of format 1.  A pool has one format; pages
 *     written under one format must not be read under the other.  MKV_DECODE_TMEM serves format 1 only.
 *   Pages of 16 M tokens (page_size = 16 M) are M tiles of 16 tokens:
 *     FP8 page, M * 32*d bytes: tile m is the FP8 record of tokens [16 m, 16 m + 16) at m * 32*d.
 *     TQ3 page, M * (12*d + 32) + 4*d bytes: tile m at m * (12*d + 32) holds [key codes | value codes |
 *       g[16]] of its 16 tokens as in the 16-token record; the value scale/zero of the PAGE (one pair per
 *       channel over all 16 M tokens) follow the tiles.  M = 1 is the 16-token record.  At M = 112,
 *       d = 256 this is 348,672 bytes per page and head: the 3.04 bit/scalar of Section 5.4.
 *     Block-table rows have one entry per page; slot_mapping = page * page_size + position.  With M > 1
 *     mkv_decode_attention() and mkv_decode_attention_scored() run the tensor-core kernel or, if
 *     selected, the CUDA-core kernel (MKV_DECODE_TMEM is refused with MKV_E_INVALID); the page mass is per page of 16 M
 *     tokens; mkv_demote() takes two launches (page scale/zero, then the tiles) and mkv_promote() one when the call
 *     converts at most 48 pages -- the table entries are then published from inside the tile kernel by the last
 *     group of blocks to finish a page, counted in 48 ticket words of the pool's status tail -- and one more
 *     launch (publication) for larger calls.  Two publishing calls on ONE pool must not overlap on the GPU
 *     (issue them on one stream or order them with events): they would share the ticket words.
 */
#ifndef MKV_H_
#define MKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mkv_pool mkv_pool;
typedef struct mkv_seq mkv_seq;

typedef enum {
    MKV_OK = 0,
    MKV_E_INVALID = -1,  /* bad argument (null, size, alignment, unsupported geometry)          */
    MKV_E_OOM_FP8 = -2,  /* FP8 arena has no free page                                          */
    MKV_E_OOM_TQ3 = -3,  /* TQ3 arena has no free page                                          */
    MKV_E_STATE = -4,    /* transition not allowed from the page's current tier / double free   */
    MKV_E_BOUNDS = -5,   /* page id, slot or logical page out of range                          */
    MKV_E_CUDA = -6,     /* a CUDA runtime call failed (see mkv_last_cuda_error)                */
    MKV_E_TIMEOUT = -7   /* a bounded device-side wait gave up                                  */
} mkv_status;

enum { MKV_TAG_RECENT = 0, MKV_TAG_ANCHOR = 1, MKV_TAG_STALE = 2 };
enum { MKV_FMT_FP8 = 0, MKV_FMT_TQ3 = 1 };
/* decode kernels: the tensor-core kernel (mma.sync, accumulators in registers) is the product; the
 * CUDA-core kernel computes the same thing with scalar FMAs and exists so that the choice of tensor
 * cores can be measured; MKV_DECODE_TMEM runs the products as tcgen05.mma with operands and
 * accumulators in tensor memory and the stages of a page in specialised warps (head_dim 256; other
 * sizes and the scored call use the tensor-core kernel) -- same results, at present slower */
enum { MKV_DECODE_TENSOR = 0, MKV_DECODE_SCALAR = 1, MKV_DECODE_TMEM = 2 };

typedef struct {
    int32_t page_size;          /* tokens per page: 16, or a multiple of 16 up to 4096          */
    int32_t head_dim;           /* 128 or 256                                                   */
    int32_t n_kv_heads;
    int32_t n_q_heads;          /* multiple of n_kv_heads, at most 8 per KV head                */
    int32_t fp8_pages;          /* capacity of the FP8 arena (Recent + Anchor), in pages        */
    int32_t tq3_pages;          /* capacity of the TQ3 arena (Stale), in pages                  */
    float k_scale;              /* FP8 key scale   (dequantised = stored * scale); 1.0 typical  */
    float v_scale;              /* FP8 value scale                                              */
    const int8_t* k_rot_signs;  /* host, head_dim entries of +1/-1: diagonal of the randomised  */
                                /* Hadamard rotation applied to keys before 3-bit quantisation  */
    int32_t tq3_format;         /* TQ3 record format: 1 (0 means 1), or 2 (see "Record formats") */
} mkv_pool_config;

typedef struct {
    int64_t fp8_pages_total, fp8_pages_used, tq3_pages_total, tq3_pages_used;
    int64_t fp8_bytes_used, tq3_bytes_used;   /* physical bytes of used pages (all KV heads)     */
    int64_t bf16_bytes_equivalent;            /* the same pages held as BF16                     */
} mkv_stats;

/* ---- pool -------------------------------------------------------------------------------- */

/* Bytes the caller must allocate for the two arenas (Section 4.1: FP8 store and TQ3 side store).
 * fp8_bytes includes a 256-byte tail that holds the pool's device status word. */
int32_t mkv_pool_query(const mkv_pool_config* cfg, size_t* fp8_arena_bytes, size_t* tq3_arena_bytes);

/* Workspace for mkv_decode_attention with up to max_batch requests: the split partials (m, l, O)
 * of Section 3.3.  Independent of sequence lengths. */
int32_t mkv_decode_workspace_bytes(const mkv_pool_config* cfg, int32_t max_batch, size_t* bytes);

/* Clear a workspace buffer.  Call it once on every newly allocated workspace before the first
 * mkv_decode_attention that uses it: the row tickets at its start (by which the last block of a
 * split row knows that it has to merge, Eq. softmax-merge) must start at zero.  Every decode call
 * leaves them at zero again, so one call per allocation is enough. */
int32_t mkv_workspace_init(void* workspace_dev, size_t bytes, void* stream);

/* Create a pool over caller-owned arenas.  Zero-fills both arenas (so that never-written slots
 * decode to zeros, not NaN) and synchronises `stream` before returning.  The pool owns host
 * bookkeeping only; the arenas stay the caller's and must outlive the pool. */
int32_t mkv_pool_create(const mkv_pool_config* cfg, void* fp8_arena_dev, void* tq3_arena_dev,
                        void* stream, mkv_pool** out);
/* Bookkeeping-only pool (no arenas, no device): free lists, sequence rows and statistics work;
 * every call that would touch the device returns MKV_E_INVALID.  For schedulers that plan page
 * transitions in a process without a GPU. */
int32_t mkv_pool_create_host_only(const mkv_pool_config* cfg, mkv_pool** out);
int32_t mkv_pool_destroy(mkv_pool* pool);

/* Per-format free lists (Section 4.4: "per-kind free list").  ids is a host array of n entries.
 * alloc: all-or-nothing; MKV_E_OOM_* leaves the lists untouched.  A fresh list hands out
 * 0, 1, 2, ...; a freed id is reused first.  free: MKV_E_BOUNDS for a bad id, MKV_E_STATE for a
 * page that is not allocated or is the retiring source of a planned conversion (mkv_seq_release);
 * nothing is freed in either case. */
int32_t mkv_page_alloc(mkv_pool* pool, int32_t fmt, int32_t* ids_host, int32_t n);
int32_t mkv_page_free(mkv_pool* pool, int32_t fmt, const int32_t* ids_host, int32_t n);

/* Physical-byte counter of the pool (Section 6.3 "active-cache counter"). */
int32_t mkv_pool_stats(const mkv_pool* pool, mkv_stats* out);

/* Read and clear the device status word; synchronises `stream`.  Returns MKV_OK, or
 * MKV_E_BOUNDS / MKV_E_STATE / MKV_E_TIMEOUT if a kernel since the last call met an out-of-range
 * id or tag, a forbidden tier transition, or a wait that ran out. */
int32_t mkv_pool_status(mkv_pool* pool, void* stream);

/* Select the decode kernel (MKV_DECODE_TENSOR by default). */
int32_t mkv_pool_set_decode_variant(mkv_pool* pool, int32_t variant);

/* Wall-time limit, in nanoseconds, of the decode scan's waits for a page copy (Section 4.1: the direct
 * path "fails closed").  Default 20,000,000 (20 ms).  A wait that runs out makes the block stop scanning,
 * wait (with the default limit) for the copies it still has in flight, and finish; the call's output is
 * then not valid and mkv_pool_status() returns MKV_E_TIMEOUT.  0 makes every wait that is not satisfied
 * at once give up: a diagnostic setting that exercises this path. */
int32_t mkv_pool_set_wait_limit_ns(mkv_pool* pool, uint64_t ns);

/* Test hooks: copy one page (all KV heads; n_kv_heads * record bytes) between the arena and a
 * host buffer, synchronously.  Lets a test compare packed bytes with a reference encoder, or
 * install pages encoded elsewhere. */
int32_t mkv_page_read_raw(mkv_pool* pool, int32_t fmt, int32_t id, void* host_buf, void* stream);
int32_t mkv_page_write_raw(mkv_pool* pool, int32_t fmt, int32_t id, const void* host_buf, void* stream);

const char* mkv_last_cuda_error(void);

/* ---- hot path ---------------------------------------------------------------------------- */

/* Append (Algorithm 1 step 1, Section 3.1 "Recent"): write the K and V of n_tokens new tokens
 * into FP8 pages as e4m3.
 *   k, v          device, bf16 [n_tokens][n_kv_heads][d]
 *   slot_mapping  device, int32 [n_tokens]: page_id * page_size + position in the FP8 arena;
 *                 negative = skip the token.  An id beyond the arena is skipped and flagged (MKV_E_BOUNDS).
 * The caller publishes the page in the block table (tag MKV_TAG_RECENT) when it opens it. */
int32_t mkv_append(mkv_pool* pool, const void* k_dev, const void* v_dev, const int32_t* slot_mapping_dev,
                   int32_t n_tokens, void* stream);

/* Demote / Retier(p, TQ3) (Algorithm 1 step 2; Section 4, "normalize-rotate-pack"): encode
 * n_pages full FP8 pages (all KV heads) into TQ3 pages, then publish.
 *   src_fp8_ids, dst_tq3_ids   device, int32 [n_pages]
 *   block_table, tier_tag      device tables to publish into, or NULL
 *   entry_index                device, int64 [n_pages]: flat index of each page's entry in the two
 *                              tables (negative = do not publish), or NULL
 *   table_entries              number of entries of block_table / tier_tag (ignored when entry_index is
 *                              NULL); an index at or beyond it is not written and flags MKV_E_BOUNDS
 * For every page the TQ3 record is complete and fenced before its id and MKV_TAG_STALE are
 * written (copy-before-publish).  The FP8 source is not modified; return it to its free list with
 * mkv_page_free() once every reader enqueued before this call has been ordered before the next
 * writer (same-stream order suffices).  Key encoder: sign flip, Walsh-Hadamard, 3-bit Lloyd-Max
 * codes of the normalised coordinates, fp16 norm correction |x|/|c|.  Value encoder: per channel
 * over the page's 16 tokens, asymmetric 3-bit codes with fp16 scale and zero. */
int32_t mkv_demote(mkv_pool* pool, const int32_t* src_fp8_ids_dev, const int32_t* dst_tq3_ids_dev,
                   int32_t n_pages, int32_t* block_table_dev, uint8_t* tier_tag_dev,
                   const int64_t* entry_index_dev, int64_t table_entries, void* stream);

/* Promote (Algorithm 1 step 3; Section 3.1, Anchor tier: a Stale page that becomes protected again
 * is rebuilt at FP8): reconstruct n_pages TQ3 pages (all KV heads) into newly allocated FP8 pages, then publish id and MKV_TAG_ANCHOR; arguments as for mkv_demote with the
 * arenas swapped.  Keys: inverse Walsh-Hadamard of the signed levels times the norm correction and
 * d^-1/2, rotation signs undone; values: scale * code + zero; both rounded to e4m3 like Append.  The
 * TQ3 source is not modified; free it once earlier readers are ordered before its next writer. */
int32_t mkv_promote(mkv_pool* pool, const int32_t* src_tq3_ids_dev, const int32_t* dst_fp8_ids_dev,
                    int32_t n_pages, int32_t* block_table_dev, uint8_t* tier_tag_dev,
                    const int64_t* entry_index_dev, int64_t table_entries, void* stream);

/* Protect / unprotect (Fig. lifecycle: Recent -> Anchor): set the tag of one table entry to
 * MKV_TAG_ANCHOR (flag != 0) or MKV_TAG_RECENT (flag == 0).  No data moves.  If the entry is
 * Stale the tag is left alone and MKV_E_STATE is recorded in the status word (a Stale page is
 * promoted into a new FP8 page with mkv_promote instead).  entry_index >= table_entries (the number of
 * entries of tier_tag) returns MKV_E_BOUNDS without launching.
 * Publication writes the id, then the tag, as two stores: a reader on ANOTHER stream must be ordered after
 * the publishing call (an event), readers on the same stream are by stream order. */
int32_t mkv_set_anchor(mkv_pool* pool, uint8_t* tier_tag_dev, int64_t table_entries, int64_t entry_index, int32_t flag,
                       void* stream);

/* Decode attention (Section 3.3; Section 4.1 "fused decode path"): for every request b and query
 * head h, softmax(scale * q K^T) V over the seq_lens[b] tokens of row b, where each page is read
 * in its own physical format and all tokens share one softmax normalisation.
 *   q            device, bf16 [B][n_q_heads][d]
 *   block_table  device, int32 [B][max_pages]; unused entries are ignored; max_pages <= 65535
 *                (tensor-core variant; MKV_E_INVALID beyond)
 *   tier_tag     device, uint8 [B][max_pages]; 0/1 = FP8 arena, 2 = TQ3 arena
 *   seq_lens     device, int32 [B]; pages beyond ceil(len/16) are not read; the last page may be
 *                partial (FP8 only); len == 0 gives out = 0 and lse = -inf
 *   out          device, fp32 [B][n_q_heads][d]
 *   lse          device, fp32 [B][n_q_heads] natural-log-sum-exp of the scaled scores, or NULL
 *   workspace    device, at least mkv_decode_workspace_bytes(cfg, B) bytes, cleared once with
 *                mkv_workspace_init; two decode calls that overlap on the GPU need two buffers
 * One launch (tensor-core variant): a persistent split-KV scan; the block that finishes a split
 * row last merges its partials with Eq. (softmax-merge).  No host synchronisation. */
int32_t mkv_decode_attention(mkv_pool* pool, const void* q_dev, const int32_t* block_table_dev,
                             const uint8_t* tier_tag_dev, const int32_t* seq_lens_dev, int32_t B,
                             int32_t max_pages, float scale, float* out_dev, float* lse_dev,
                             void* workspace_dev, size_t workspace_bytes, void* stream);

/* The decode step of several layers in one launch (Section 4.1 runs the direct FP8/TQ3 path of all
 * full-attention layers of a decode step from one CUDA graph; Section 5, evaluated profiles).  Layer i
 * has its own pool, query, table, tags, outputs and workspace; the requests (seq_lens, B, max_pages,
 * scale) are common to all layers, and all pools have the same geometry (head_dim, heads, page_size,
 * record format).  Every block of the persistent scan walks its share of layer 0, then of layer 1, ... without
 * waiting for the other blocks, so the table walk and query rotation of one layer and the merge of the
 * layer before overlap the page scans of their neighbours; results are those of n_layers calls of
 * mkv_decode_attention (the same kernel code per layer).
 *   layers_host  host array of n_layers entries (copied into the launch; free to reuse on return);
 *                lse_dev may be NULL; every workspace_dev as for mkv_decode_attention, distinct per layer
 *   n_layers     1 .. MKV_MAX_LAYERS_PER_CALL; MKV_E_INVALID beyond, for pools of different geometry,
 *                page size or record format, or for a pool set to another decode variant */
#define MKV_MAX_LAYERS_PER_CALL 32
typedef struct {
    mkv_pool* pool;
    const void* q_dev;                  /* bf16 [B][n_q_heads][d]                   */
    const int32_t* block_table_dev;     /* int32 [B][max_pages]                     */
    const uint8_t* tier_tag_dev;        /* uint8 [B][max_pages]                     */
    float* out_dev;                     /* fp32 [B][n_q_heads][d]                   */
    float* lse_dev;                     /* fp32 [B][n_q_heads] or NULL              */
    void* workspace_dev;                /* this layer's workspace                   */
} mkv_layer_call;
int32_t mkv_decode_attention_layers(const mkv_layer_call* layers_host, int32_t n_layers, const int32_t* seq_lens_dev,
                                    int32_t B, int32_t max_pages, float scale, size_t workspace_bytes, void* stream);

/* Append (Algorithm 1 step 1) of the same n_tokens positions into the pools of several layers in one
 * launch: layer i converts k_dev[i], v_dev[i] (bf16 [n_tokens][n_kv_heads][d]) into its own FP8 arena at
 * slot_mapping (common to the layers: every layer's table names the same page ids).  Decode-sized
 * calls only (n_tokens <= 64); same bytes as n_layers calls of mkv_append. */
typedef struct {
    mkv_pool* pool;
    const void* k_dev;
    const void* v_dev;
} mkv_layer_append;
int32_t mkv_append_layers(const mkv_layer_append* layers_host, int32_t n_layers, const int32_t* slot_mapping_dev,
                          int32_t n_tokens, void* stream);

/* The same decode attention for callers that cannot give the library a workspace because they are
 * not allowed to allocate device memory once they are running (a server that handed its whole
 * memory budget to the KV pool at start-up, code living inside another component's memory manager,
 * a process whose allocator is frozen while it serves).  (The paper has no counterpart: this is a
 * property of the library, not of the method.)  The split partials go to a fixed array inside the
 * library image, MKV_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the process
 * exits.  Arguments, results and kernel are those of mkv_decode_attention with the tensor-core variant;
 * a pool that was switched to another variant is refused with MKV_E_INVALID.
 *   - allocates nothing: no cudaMalloc / cudaFree, no allocating library call, on any call.
 *   - limits: B <= MKV_STATIC_MAX_BATCH, and the scan must not launch more than MKV_STATIC_MAX_BLOCKS
 *     blocks on this GPU (it launches one per SM on B200); beyond either the call launches nothing and
 *     returns MKV_E_INVALID, with the reason in mkv_last_cuda_error().
 *   - the pool's device must be the current device.  The first call on a device looks up the array's
 *     device address; make that first call before any stream capture begins.
 *   - all calls on a device share the one array, which keeps whatever the previous call left in it
 *     (partials are rewritten before they are read; the ticket words start at zero when the library is
 *     loaded and every call returns them to zero, so nothing needs clearing).  Two calls that overlap
 *     on the GPU, e.g. on different streams, race on it: serialise them or use mkv_decode_attention
 *     with separate workspaces. */
#define MKV_STATIC_MAX_BLOCKS 160
#define MKV_STATIC_MAX_BATCH 1024
#define MKV_STATIC_SCRATCH_BYTES (2u * MKV_STATIC_MAX_BLOCKS * (8u * 256u + 16u) * 4u + 1024u) /* 2,642,944 bytes */
int32_t mkv_decode_attention_static(mkv_pool* pool, const void* q_dev, const int32_t* block_table_dev,
                                    const uint8_t* tier_tag_dev, const int32_t* seq_lens_dev, int32_t B,
                                    int32_t max_pages, float scale, float* out_dev, float* lse_dev, void* stream);

/* Section 3.1 (Eq. score-partial, Eq. score-global-weight): mkv_decode_attention that also reports
 * the globally normalised attention mass of every page, taken from the same scores, the same softmax
 * and the same one pass over the mixed-format pages as the output (no dense view of the cache).
 *   page_mass    device, fp32 [B][n_q_heads][max_pages]: q~_{h,p} = sum over the tokens of page p of
 *                softmax weight of head h, divided by the sum over all pages (1 up to rounding, since
 *                every page is addressable); pages beyond ceil(len/16) are set to 0
 *   lse          required here (the second launch needs it)
 * Other arguments, workspace and errors as mkv_decode_attention; always the tensor-core kernel.
 * Two launches: the scan (which stores log2 of every page's exponential sum) and a small kernel
 * that refers them to the row's log-sum-exp and normalises. */
int32_t mkv_decode_attention_scored(mkv_pool* pool, const void* q_dev, const int32_t* block_table_dev,
                                    const uint8_t* tier_tag_dev, const int32_t* seq_lens_dev, int32_t B,
                                    int32_t max_pages, float scale, float* out_dev, float* lse_dev,
                                    float* page_mass_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Eq. (attention-score): r_p = mean over the sampled head set of q~_{h,p}, a_p <- beta a_p + (1-beta) r_p
 * for every page below each request's length (others untouched).
 *   page_mass    device, fp32 [B][n_q_heads][max_pages] from mkv_decode_attention_scored
 *   head_mask    bit h selects query head h (n_q_heads <= 64); no selected head: MKV_E_INVALID
 *   beta         in [0, 1]
 *   score        device, fp32 [B][max_pages], updated in place */
int32_t mkv_page_score_update(const float* page_mass_dev, const int32_t* seq_lens_dev, int32_t B,
                              int32_t n_q_heads, int32_t max_pages, uint64_t head_mask, float beta,
                              float* score_dev, void* stream);

/* The same for pools whose pages hold page_size tokens (a multiple of 16): a request of len tokens has
 * ceil(len / page_size) pages.  mkv_page_score_update() is this call with page_size = 16. */
int32_t mkv_page_score_update_paged(const float* page_mass_dev, const int32_t* seq_lens_dev, int32_t B,
                                    int32_t n_q_heads, int32_t max_pages, int32_t page_size, uint64_t head_mask,
                                    float beta, float* score_dev, void* stream);

/* ---- host-side sequence bookkeeping (Algorithm 1; no device work) ------------------------- */

/* A sequence owns a row of logical pages -> (tag, physical id).  These calls only plan: they
 * move ids between the free lists and the row and tell the caller which device call to issue. */
int32_t mkv_seq_create(mkv_pool* pool, mkv_seq** out);
/* Finish(q): release every page of the sequence to its free list and destroy the handle. */
int32_t mkv_seq_finish(mkv_seq* seq);
/* Append: slot for the next token; opens a Recent page every 16 tokens (MKV_E_OOM_FP8 if none). */
int32_t mkv_seq_append(mkv_seq* seq, int32_t* page_id, int32_t* slot, int32_t* opened_page);
/* Recent <-> Anchor tag of a logical page (MKV_E_STATE if it is Stale). */
int32_t mkv_seq_protect(mkv_seq* seq, int32_t logical_page, int32_t flag);
/* Retier to TQ3 (Algorithm 1 step 2): allocates the destination and updates the row.  Only full, non-Stale
 * pages qualify (MKV_E_STATE otherwise).  The caller then enqueues mkv_demote().  The source FP8 id leaves
 * the row but is RETIRING: it is on no free list and is handed to nobody until mkv_seq_release(), which the
 * caller issues once every reader enqueued before the conversion, and the conversion itself, are ordered
 * before any later writer of that page (on one stream: as soon as mkv_demote() has been enqueued; across
 * streams: after the event that marks it).  mkv_pool_stats() counts retiring pages as used. */
int32_t mkv_seq_demote(mkv_seq* seq, int32_t logical_page, int32_t* src_fp8_id, int32_t* dst_tq3_id);
/* Promote (Algorithm 1 step 3): Stale -> Anchor through a newly allocated FP8 page (MKV_E_STATE if the page
 * is not Stale, MKV_E_OOM_FP8 if none is free).  The caller then enqueues mkv_promote(); the TQ3 source is
 * retiring until mkv_seq_release(), as for mkv_seq_demote(). */
int32_t mkv_seq_promote(mkv_seq* seq, int32_t logical_page, int32_t* src_tq3_id, int32_t* dst_fp8_id);
/* Release a retiring source (Algorithm 1: "after readers and the conversion event clear") to its free list.
 * MKV_E_STATE if (fmt, id) is not a retiring source of this sequence, MKV_E_BOUNDS for a bad id.
 * mkv_seq_finish() releases what is still retiring. */
int32_t mkv_seq_release(mkv_seq* seq, int32_t fmt, int32_t id);
/* Age: plan the demotion of every full Recent page wholly before the last `recent_tokens`
 * tokens (their sources become retiring, as with mkv_seq_demote).  Writes up to `cap` triples and returns their number in *n (MKV_E_INVALID if more
 * would be needed; nothing changes then). */
int32_t mkv_seq_age(mkv_seq* seq, int32_t recent_tokens, int32_t* logical_pages, int32_t* src_fp8_ids,
                    int32_t* dst_tq3_ids, int32_t cap, int32_t* n);
int32_t mkv_seq_len(const mkv_seq* seq, int32_t* len, int32_t* n_pages);
/* Copy the row (n_pages entries) to host arrays. */
int32_t mkv_seq_row(const mkv_seq* seq, int32_t* ids_host, uint8_t* tags_host, int32_t cap);

#ifdef __cplusplus
}
#endif
#endif /* MKV_H_ */
