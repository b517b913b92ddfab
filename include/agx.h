/*
 * agx - prefix-cached block attention and greedy speculative acceptance for NVIDIA B200 (sm_100a).
 *
 * One GPU hot path, shared by the two halves of the Agent-X method:
 *   prefill with prefix caching  : attention of the q uncached suffix tokens of a prompt over a
 *                                  KV cache that already holds the cached prefix (Sec. 2.3,
 *                                  "Prefix caching"; Sec. 4.2 makes the prefix long and the suffix short);
 *   speculative-decoding verify  : attention of the most recent token followed by N draft tokens
 *                                  (q = N + 1) over the whole cached context, then acceptance
 *                                  (Sec. 2.3, "Speculative decoding"; Sec. 4.3 supplies the drafts
 *                                  from an n-gram table and falls back to q = 1 on a table miss).
 *
 * Conventions shared by every call
 *   - All functions are extern "C", return an agx_status (0 = AGX_OK, negative = error) unless
 *     stated otherwise, never throw and never abort.  Work is enqueued on the caller's stream and
 *     the call returns without synchronising (except agx_get_status and the *_host call).
 *   - "device" pointers are device memory owned by the caller; "host" pointers are ordinary host
 *     memory read during the call only (the caller may reuse it as soon as the call returns).
 *     The library never frees or retains caller memory.
 *   - A handle must be used from one stream at a time: calls on the same handle that overlap on
 *     the GPU share that state and race.  Host threads: a handle is not thread-safe (it caches the last
 *     launch plan, the pools' tensor maps and the last error text); use it from one host thread at a
 *     time, or one handle per thread.  Different handles may be used concurrently: the only
 *     process-wide state is a per-device note that a kernel's launch attributes have been set, which
 *     every thread writes with the same value.
 *   - The handle owns 512 KB of device memory (a status word, the accept step's ticket counter and one
 *     64-bit key per logits row it can take, 65535).
 *   - Ragged batches: B sequences; sequence s has a cached prefix of prefix_len[s] tokens and a
 *     block of q_len[s] >= 1 new tokens; cu_q[B+1] is the exclusive prefix sum of q_len and
 *     total_q = cu_q[B].  Rows of q_block, k_new, v_new, out and logits are sequence-major,
 *     position-minor: row cu_q[s] + i is block position i of sequence s.
 *   - Element type: AGX_BF16 (bfloat16) or AGX_F32 (float), fixed per handle.  Accumulation and
 *     softmax are always fp32; outputs are rounded to the element type (nearest-even).
 *   - KV pool layout (library-defined): k_pool and v_pool are [num_pages][num_kv_heads][16][head_dim],
 *     256-byte aligned.  Token t of sequence s lives in page page_table[s*page_table_stride + t/16],
 *     slot t%16.  prefix_len need not be a multiple of 16 (a reused prefix may be cut anywhere).
 *     Pages may be shared between sequences for reading; pages that a call appends into must be
 *     private to that sequence.
 *   - Query head h reads KV head h / (num_q_heads / num_kv_heads).
 */
#ifndef AGX_H_
#define AGX_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define AGX_API __attribute__((visibility("default")))
#else
#define AGX_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct agx_handle agx_handle;
typedef int32_t agx_status;

enum {
    AGX_OK = 0,
    AGX_E_INVAL = -1,       /* null / misaligned pointer, bad shape, q_len < 1, workspace too small */
    AGX_E_RANGE = -2,       /* lengths exceed the page table, or too many sequences/rows */
    AGX_E_UNSUPPORTED = -3, /* head_dim, page size or dtype combination not built */
    AGX_E_CUDA = -4,        /* a CUDA runtime call or launch failed; see agx_last_error */
    AGX_E_DEVICE = -5,      /* the device status word is non-zero (see agx_get_status) */
    AGX_E_NOMEM = -6
};

enum { AGX_BF16 = 0, AGX_F32 = 1 };

/* Bits of the device status word (sticky until agx_get_status clears them). */
enum {
    AGX_DEV_BAD_PAGE = 1,    /* a page id outside [0, num_pages) was met; the access was skipped */
    AGX_DEV_WAIT_TIMEOUT = 2, /* a bounded in-kernel wait gave up; results of that launch are invalid */
    AGX_DEV_BAD_TOKEN = 4     /* agx_ngram_build met a token id outside [0, 2^21); its windows were skipped */
};

typedef struct agx_config {
    int32_t num_q_heads;  /* Hq */
    int32_t num_kv_heads; /* Hkv, divides Hq */
    int32_t head_dim;     /* d: 64 or 128 (AGX_BF16 with 64 and AGX_F32 run a scalar fp32 kernel: a correctness path) */
    int32_t page_size;    /* must be 16 */
    int32_t dtype;        /* AGX_BF16 or AGX_F32 */
    float scale;          /* softmax scale; 0 selects 1/sqrt(head_dim) */
} agx_config;

/* Create / destroy a handle on the current CUDA device.  No paper counterpart (plumbing). */
AGX_API agx_status agx_create(const agx_config* config, agx_handle** out_handle);
AGX_API agx_status agx_destroy(agx_handle* handle);

/* Text for a status code; and the detail message of the last failing call on this handle
 * (valid until the next call on the handle).  Never NULL. */
AGX_API const char* agx_status_string(agx_status status);
AGX_API const char* agx_last_error(const agx_handle* handle);

/*
 * agx_kv_append - write the block's K and V rows into the sequences' pages.
 * Sec. 2.3: prefill fills the KV cache; with prefix caching only the uncached suffix is
 * written, after the cached prefix.  In a verify step the rows are speculative: acceptance later
 * commits a length and moves no data; dead slots are overwritten by the next append.
 *   k_pool, v_pool : device, pools as laid out above (written)
 *   k_new, v_new   : device, [total_q][num_kv_heads][head_dim], 16-byte aligned
 *   page_table     : device int32, [B][page_table_stride]
 *   prefix_len     : device int32 [B]; row i of sequence s goes to token slot prefix_len[s] + i
 *   cu_q           : device int32 [B+1]
 * Errors: AGX_E_INVAL on null/misaligned pointers or B/total_q < 0; a page id outside
 * [0, num_pages) sets AGX_DEV_BAD_PAGE and that row is not written.  B == 0 or total_q == 0 is a no-op.
 */
AGX_API agx_status agx_kv_append(agx_handle* handle, void* k_pool, void* v_pool, int64_t num_pages,
                         const void* k_new, const void* v_new, const int32_t* page_table,
                         int32_t page_table_stride, const int32_t* prefix_len, const int32_t* cu_q,
                         int32_t B, int32_t total_q, void* stream);

/*
 * agx_attn_workspace_bytes - scratch bytes agx_attn_prefixed needs for this batch (host lengths).
 * Returns a negative agx_status on bad arguments.  The figure depends only on the config, the
 * lengths and the device's SM count.
 */
AGX_API int64_t agx_attn_workspace_bytes(agx_handle* handle, int32_t B, const int32_t* h_prefix_len,
                                 const int32_t* h_q_len);

/*
 * agx_attn_prefixed - attention of each sequence's block over its cached prefix plus the block.
 * Sec. 2.3 (prefix caching): a token looks only at the tokens up to itself, so row i of the block
 * (absolute position P + i) attends to tokens 0 .. P + i of the sequence: all of the cached prefix, and the
 * block rows up to and including itself.  The same call serves the verify block of speculative
 * decoding (q = N + 1) and plain decode (q = 1).  agx_kv_append for the same block must have
 * been enqueued before, so the pages already hold tokens P .. P + q - 1.
 *   out[r][h][:] = sum_j softmax_j(scale * <q_block[r][h], K[j][h/G]>) V[j][h/G],  j in [0, P + i]
 *   q_block      : device, [total_q][num_q_heads][head_dim], 16-byte aligned
 *   k_pool,v_pool: device pools (read only); page_table: device int32 [B][page_table_stride]
 *   h_prefix_len, h_q_len : HOST int32 [B].  They size the launch and are copied into kernel
 *                  arguments, so the values in force are the ones passed here.
 *   out          : device, [total_q][num_q_heads][head_dim], element type of the handle
 *   lse          : device float [total_q][num_q_heads] or NULL; natural-log sum of exp of the
 *                  scaled scores
 *   workspace    : device, >= agx_attn_workspace_bytes(...) bytes, 256-byte aligned (may be NULL
 *                  when that figure is 0)
 * Dispatch (G = num_q_heads / num_kv_heads; bf16 handles with head_dim 128 - other handles run the scalar kernel): up to 32 query rows per KV head (q_len * G) over a context
 * shorter than about 7k tokens (10k for q_len * G <= 8) run the split-KV warp-MMA kernel (latency-bound); up to 32 rows over a
 * longer context, or 33..128 rows over any context, run the tensor-core kernel with one padded Q tile
 * whose KV tiles alternate between two softmax warpgroups (HBM-bound); longer blocks run the
 * tensor-core kernel with 256-row tiles (tensor-bound).  Sequences of all kinds may share a batch; two or
 * more blocks of at most 32 rows whose contexts add up to 24576 tokens or more (at 8 KV heads) all take the
 * padded-tile kernel, whatever their single lengths.
 * Errors: AGX_E_INVAL (null/misaligned, q_len < 1, prefix_len < 0, workspace too small),
 * AGX_E_RANGE ((P + q) exceeds 16 * page_table_stride), AGX_E_CUDA.  Page ids outside
 * [0, num_pages) set AGX_DEV_BAD_PAGE and read as zeros.
 */
AGX_API agx_status agx_attn_prefixed(agx_handle* handle, const void* q_block, const void* k_pool,
                             const void* v_pool, int64_t num_pages, const int32_t* page_table,
                             int32_t page_table_stride, const int32_t* h_prefix_len,
                             const int32_t* h_q_len, int32_t B, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * agx_attn_prefixed_append - agx_kv_append and agx_attn_prefixed of the same block as one call.
 * Sec. 2.3: the block's K/V rows join the cache (after the cached prefix) and the block then attends to
 * prefix plus block.  Results, in the pools and in `out`, are those of the two calls made one after the
 * other.  Where every sequence of a launch has at most 256 query rows per KV head (q_len * G; bf16 handles), the
 * rows are written inside the attention kernel: each CTA stores the rows of its own KV head that fall into
 * its own KV split before it reads them, which saves the append launch of a decode or verify step.
 * Longer blocks and fp32 handles get an append launch in front of the attention launch.
 *   k_new, v_new : device, [total_q][num_kv_heads][head_dim], 16-byte aligned (rows in the order of q_block)
 *   k_pool, v_pool : device pools (written, then read); the other arguments as for agx_attn_prefixed
 * Errors: those of agx_attn_prefixed; a page id outside [0, num_pages) sets AGX_DEV_BAD_PAGE, the row is
 * not written and reads as zeros.
 */
AGX_API agx_status agx_attn_prefixed_append(agx_handle* handle, const void* q_block, const void* k_new,
                                            const void* v_new, void* k_pool, void* v_pool, int64_t num_pages,
                                            const int32_t* page_table, int32_t page_table_stride,
                                            const int32_t* h_prefix_len, const int32_t* h_q_len, int32_t B,
                                            void* out, float* lse, void* workspace, size_t workspace_bytes,
                                            void* stream);

/* Scratch bytes agx_accept_greedy needs for total_q logits rows (the rows' winners; a few KB). */
AGX_API int64_t agx_accept_workspace_bytes(agx_handle* handle, int32_t total_q, int32_t vocab);

/*
 * agx_accept_greedy - per-row vocabulary argmax, longest matching draft prefix, commit.
 * Sec. 2.3 (speculative decoding, steps 2-3): drafts are kept up to the first one the target
 * disagrees with; that draft and every later one are dropped, and the kept drafts plus the
 * target's own next token start the next round.  With
 * an n-gram draft source (Sec. 4.3) there are no draft logits, so a draft is accepted iff it
 * equals the target's greedy token.
 * For sequence s with k = q_len[s] - 1 drafts d_1..d_k, logits row 0 belongs to the most recent
 * token and row i to draft d_i:
 *   t_r        = lowest index attaining max_v logits[r][v]   (NaN never beats a number; a row of
 *                only NaN gives 0; -0 and +0 tie)
 *   accept_len = number of leading i in 1..k with d_i == t_{i-1}
 *   next_token = t_{accept_len};   seq_lens[s] <- seq_lens[s] + accept_len + 1
 *   logits     : device, [total_q][row_stride] of logits_dtype (AGX_BF16 / AGX_F32); only the
 *                first vocab entries of a row are read; rows 16-byte aligned
 *   drafts     : device int32 [total_q - B]; sequence s owns entries cu_q[s]-s .. (any int32 is
 *                legal; values outside [0, vocab) never match)
 *   cu_q       : device int32 [B+1]
 *   accept_len, next_token : device int32 [B] (written)
 *   argmax     : device int32 [total_q] or NULL (written)
 *   seq_lens   : device int32 [B] or NULL; in: committed length before the block (the prefix
 *                length), out: prefix + accept_len + 1
 * Prefill uses the same call with no drafts (q_len = 1 per sequence, the last row's logits).
 * Errors: AGX_E_INVAL, AGX_E_RANGE (vocab < 1, row_stride < vocab), AGX_E_CUDA.
 */
AGX_API agx_status agx_accept_greedy(agx_handle* handle, const void* logits, int32_t logits_dtype,
                             int64_t row_stride, int32_t vocab, const int32_t* drafts,
                             const int32_t* cu_q, int32_t B, int32_t total_q, int32_t* accept_len,
                             int32_t* next_token, int32_t* argmax, int32_t* seq_lens,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * agx_accept_greedy_static - agx_accept_greedy for callers that cannot allocate device memory.
 * The paper has no counterpart: this is a packaging variant of the accept step above, with the
 * same inputs, outputs and results.
 *
 * Who needs it: code that verifies drafts from inside a memory arena sized once at start-up (an
 * embedded or serving runtime with a fixed device-memory budget), or next to an allocator it does
 * not own, where a cudaMalloc may synchronise the whole device, fragment the pool or simply be
 * forbidden.  This call takes no handle and no workspace and performs no allocation of any kind;
 * it uses a fixed scratch array inside the library (about 16 KB of device memory on every GPU that
 * loads the library, held until the process exits).
 *
 * Limit: total_q <= 2048 logits rows per call; more rows return AGX_E_RANGE and should use
 * agx_accept_greedy with a workspace.  (The array holds one 64-bit key per row and a counter.)
 *
 * The first call on each device looks up the device address of the scratch array (that device
 * must be current); make that first call outside any stream capture.  The look-up is guarded, so
 * several host threads may make their first calls at the same time.  Every call uses the same
 * array: the call clears the part that has to start at zero, but two calls that overlap on the GPU
 * (different streams, no ordering between them) race on it and give undefined results.  Calls on
 * one stream, or ordered by events, are safe.
 *
 * Arguments and error codes are those of agx_accept_greedy; every pointer is a device pointer.
 * There is no handle, so no error text is kept: the status code is all a failing call reports.
 */
AGX_API agx_status agx_accept_greedy_static(const void* logits, int32_t logits_dtype,
                                            int64_t row_stride, int32_t vocab,
                                            const int32_t* drafts, const int32_t* cu_q, int32_t B,
                                            int32_t total_q, int32_t* accept_len,
                                            int32_t* next_token, int32_t* argmax,
                                            int32_t* seq_lens, void* stream);

/*
 * agx_get_status - synchronise the stream, read and clear the device status word.
 * *device_status receives the AGX_DEV_* bits (0 = clean).  Returns AGX_E_DEVICE when non-zero.
 */
AGX_API agx_status agx_get_status(agx_handle* handle, void* stream, int32_t* device_status);

/*
 * agx_verify_step_host - one whole step (append, attention, acceptance) for callers whose
 * activations live in HOST memory.  Same operations as the three calls above (Sec. 2.3), plus the
 * host<->device copies: q_block, k_new, v_new, logits, drafts and the lengths go to the device,
 * out, accept_len, next_token and seq_lens come back, and the stream is synchronised before the
 * call returns.  The KV pools and the page table stay on the device: they are the cache.
 *   k_pool, v_pool, page_table : device (as in agx_kv_append)
 *   h_prefix_len, h_q_len      : host int32 [B]
 *   h_q_block, h_k_new, h_v_new: host, element type of the handle (pinned memory makes the
 *                                copies asynchronous; pageable memory works but serialises).
 *                                When the three are pinned, mapped into the device's address space
 *                                (cudaHostAlloc / cudaHostRegister) and together at most 1 MiB, one
 *                                kernel reads them across the bus instead of three transfers; a
 *                                pinned, mapped h_out of at most 1 MiB is written by the attention
 *                                kernels directly.  Results are the same either way.
 *   h_logits                   : host, [total_q][row_stride] of logits_dtype; a megabyte or more of them is
 *                                uploaded on a stream the handle owns, beside the attention kernels (it starts
 *                                behind the work already on `stream`, and `stream` waits for it before the
 *                                accept step)
 *   h_drafts                   : host int32 [total_q - B] (may be NULL when total_q == B)
 *   h_out                      : host, [total_q][num_q_heads][head_dim]
 *   h_accept_len, h_next_token, h_seq_lens : host int32 [B]; h_seq_lens receives
 *                                prefix_len + accept_len + 1
 *   vocab == 0                 : attention only (a middle layer of a model): the logits, drafts
 *                                and accept outputs are ignored and may be NULL.  Such a step that moves
 *                                4 MiB or more is cut into several attention calls: runs of whole blocks of
 *                                about a thousand rows, or, where that gives fewer than three calls, chunks of
 *                                384 rows of a block (environment variable AGX_HOST_PIPELINE_ROWS, 0 = never
 *                                cut), rows [r0, r1) of a block being a block of their own behind a prefix longer
 *                                by r0 (chunked prefill); the uploads of a chunk, the attention calls of the chunks
 *                                before it and the downloads of their rows overlap on two streams the handle owns,
 *                                which start
 *                                behind the work already on `stream` and which `stream` waits for at the end
 *                                of the call.  Results are those of the single call; on an error in the middle
 *                                the chunks already enqueued still run.
 *   workspace                  : device, >= agx_verify_step_host_workspace_bytes(...) bytes,
 *                                256-byte aligned; holds the staged copies and both scratch areas
 * Errors: as the three calls; nothing is launched when a check fails.
 */
AGX_API int64_t agx_verify_step_host_workspace_bytes(agx_handle* handle, int32_t B,
                                                     const int32_t* h_prefix_len,
                                                     const int32_t* h_q_len, int32_t logits_dtype,
                                                     int64_t row_stride, int32_t vocab);
AGX_API agx_status agx_verify_step_host(agx_handle* handle, void* k_pool, void* v_pool,
                                        int64_t num_pages, const int32_t* page_table,
                                        int32_t page_table_stride, const int32_t* h_prefix_len,
                                        const int32_t* h_q_len, int32_t B, const void* h_q_block,
                                        const void* h_k_new, const void* h_v_new,
                                        const void* h_logits, int32_t logits_dtype,
                                        int64_t row_stride, int32_t vocab, const int32_t* h_drafts,
                                        void* h_out, int32_t* h_accept_len, int32_t* h_next_token,
                                        int32_t* h_seq_lens, void* workspace,
                                        size_t workspace_bytes, void* stream);

/*
 * agx_verify_step_host_enqueue - the same step (Sec. 2.3: append, attention, acceptance) and the same
 * arguments as agx_verify_step_host, but the call returns as soon as the copies and kernels are enqueued.
 * A model calls it once per layer and synchronises the stream once per step, so the copies of one layer
 * overlap the kernels of another.  Until the caller has synchronised the stream, the host input buffers
 * must stay unchanged when they are pinned memory (pageable buffers are staged before the call returns),
 * the host outputs are not valid, and the workspace belongs to the calls in flight (calls on one stream
 * may share it: they run in order).
 */
AGX_API agx_status agx_verify_step_host_enqueue(agx_handle* handle, void* k_pool, void* v_pool,
                                                int64_t num_pages, const int32_t* page_table,
                                                int32_t page_table_stride, const int32_t* h_prefix_len,
                                                const int32_t* h_q_len, int32_t B, const void* h_q_block,
                                                const void* h_k_new, const void* h_v_new,
                                                const void* h_logits, int32_t logits_dtype,
                                                int64_t row_stride, int32_t vocab, const int32_t* h_drafts,
                                                void* h_out, int32_t* h_accept_len, int32_t* h_next_token,
                                                int32_t* h_seq_lens, void* workspace,
                                                size_t workspace_bytes, void* stream);

/*
 * agx_ngram_build - the draft table of example-based speculative decoding, built on the device.
 * Sec. 4.3: a window of n consecutive tokens slides over one token stream (the prompt's examples and
 * the query); the first n-1 tokens of a window are a key, and the key's value is the token that follows
 * it most often in the stream.  The paper does not say which successor wins when counts are equal:
 * here the lowest token id does.
 *   stream_tokens : device int32 [num_tokens], ids in [0, 2^21); a window holding any other id is
 *                   skipped and sets AGX_DEV_BAD_TOKEN
 *   n             : 2 or 3 (3, the trigram table, is the paper's choice)
 *   lut           : device, >= agx_ngram_lut_bytes(num_tokens) bytes, 16-byte aligned; opaque, valid
 *                   until overwritten; read by agx_ngram_draft
 *   workspace     : device, >= agx_ngram_workspace_bytes(num_tokens) bytes, 16-byte aligned
 * num_tokens < n builds an empty table.  Errors: AGX_E_INVAL, AGX_E_UNSUPPORTED (n), AGX_E_RANGE
 * (num_tokens > 2^24), AGX_E_CUDA.
 */
AGX_API int64_t agx_ngram_lut_bytes(int32_t max_stream_tokens);
AGX_API int64_t agx_ngram_workspace_bytes(int32_t stream_tokens);
AGX_API agx_status agx_ngram_build(agx_handle* handle, const int32_t* stream_tokens, int32_t num_tokens,
                                   int32_t n, void* lut, size_t lut_bytes, void* workspace,
                                   size_t workspace_bytes, void* stream);

/*
 * agx_ngram_draft - k draft tokens per sequence by chained table lookups (Sec. 4.3).
 * Draft 1 is the table's value for the sequence's last n-1 tokens, draft 2 the value for the last n-2
 * tokens followed by draft 1, and so on.  Selective decoding: has_draft[s] = 0 when the FIRST lookup
 * misses - the caller then runs a plain one-token step (q_len = 1) instead of paying for a verify block
 * that cannot be accepted; after a first hit, a later miss takes the caller's guess fill[s][i] (the
 * paper's "random token", drawn by the caller) and the chain goes on from it.
 *   lut        : device, built by agx_ngram_build
 *   context    : device int32 [B][n-1], the most recent n-1 tokens of each sequence, oldest first
 *   fill       : device int32 [B][k]
 *   drafts     : device int32 [B][k] (written in any case); has_draft : device int32 [B] (written)
 * Errors: AGX_E_INVAL (null pointers, B < 0, k < 0), AGX_E_CUDA.
 */
AGX_API agx_status agx_ngram_draft(agx_handle* handle, const void* lut, const int32_t* context,
                                   const int32_t* fill, int32_t B, int32_t k, int32_t* drafts,
                                   int32_t* has_draft, void* stream);

/*
 * agx_pw_select_combinations - which cluster combinations to precompute (Algorithm 1, Sec. 4.2).  HOST code.
 * A sample is the ordered sequence of clusters a training query activates.  The coverage of a cached set
 * is, summed over samples, the length of the longest prefix of the sample that is cached.  Starting from
 * the empty set, `budget` times the candidate that raises the coverage most is added; candidates are the
 * samples' prefixes that are a single cluster or a cached sequence extended by one cluster.  Equal gains
 * (the paper is silent): the shorter candidate, then the lexicographically smaller one.  The selection
 * ends early when no candidate is left.
 *   samples      : host int32 [num_samples][max_len], cluster ids >= 0, rows padded with -1
 *   selected     : host int32 [budget][max_len] (written, padded with -1), in the order of selection
 *   selected_len : host int32 [budget]; gains : host int32 [budget] or NULL (coverage gained by each step)
 *   num_selected : host int32 (written)
 * Errors: AGX_E_INVAL.
 */
AGX_API agx_status agx_pw_select_combinations(const int32_t* samples, int32_t num_samples, int32_t max_len,
                                              int32_t budget, int32_t* selected, int32_t* selected_len,
                                              int32_t* gains, int32_t* num_selected);

/*
 * agx_pw_longest_prefix - online lookup with tail cut (Sec. 4.2).  HOST code.
 * Among the stored combinations, the one that shares the longest run of leading clusters with the query;
 * the stored combination may go on after the run (its tail is cut off: only the KV of the run is reused).
 * Equal runs: the first stored combination.  *index = -1, *length = 0 when nothing matches.
 *   stored : host int32 [num_stored][max_len]; stored_len : host int32 [num_stored]; query : host int32 [query_len]
 */
AGX_API agx_status agx_pw_longest_prefix(const int32_t* stored, const int32_t* stored_len, int32_t num_stored,
                                         int32_t max_len, const int32_t* query, int32_t query_len,
                                         int32_t* index, int32_t* length);

/*
 * agx_kv_copy_pages - private copies of KV pages.  Sec. 4.2: a reused prefix may be cut anywhere (the
 * mismatched tail of a stored combination is dropped), so its last page can be partly valid and still
 * shared with other sequences; a sequence that appends behind the cut needs that page for itself.  The
 * caller points the first prefix_len / 16 entries of the new page-table row at the stored pages, copies
 * page prefix_len / 16 with this call when prefix_len % 16 != 0, and uses fresh pages after it.
 *   k_pool, v_pool : device pools (pages dst[i] are overwritten with pages src[i], K and V, all heads)
 *   src, dst       : device int32 [count]; ids outside [0, num_pages) set AGX_DEV_BAD_PAGE and are skipped
 * Errors: AGX_E_INVAL, AGX_E_CUDA.
 */
AGX_API agx_status agx_kv_copy_pages(agx_handle* handle, void* k_pool, void* v_pool, int64_t num_pages,
                                     const int32_t* src, const int32_t* dst, int32_t count, void* stream);

/*
 * agx_kv_import_pages - bring precomputed KV pages from host memory into the pool.
 * Sec. 4.2 / Sec. 5.1: the KV caches of the static prefix and of the selected cluster combinations are computed
 * once, kept in storage and loaded when a request reuses them (the paper loads from SSD into unified
 * memory; here the stored pages sit in host memory and cross to the GPU).  When h_k and h_v are pinned and
 * mapped into the device's address space (cudaHostAlloc / cudaHostRegister), the scatter kernel reads the pages
 * across the bus itself, one pass at bus speed; otherwise two host-to-device copies fill the staging area first.
 * Everything runs on `stream`: issued on a stream of its own, an import overlaps attention that runs on other
 * streams over pages already resident.
 *   h_k_pages, h_v_pages : HOST, [count][num_kv_heads][16][head_dim] of the handle's element type (pinned
 *                          memory makes the copies asynchronous)
 *   dst_pages            : device int32 [count]: pool page that receives imported page i; ids outside
 *                          [0, num_pages) set AGX_DEV_BAD_PAGE and are skipped
 *   staging              : device, >= agx_kv_import_staging_bytes(count) bytes, 16-byte aligned; busy until the
 *                          scatter kernel has run
 * Errors: AGX_E_INVAL, AGX_E_CUDA.
 */
AGX_API int64_t agx_kv_import_staging_bytes(const agx_handle* handle, int32_t count);
AGX_API agx_status agx_kv_import_pages(agx_handle* handle, void* k_pool, void* v_pool, int64_t num_pages,
                                       const void* h_k_pages, const void* h_v_pages, const int32_t* dst_pages,
                                       int32_t count, void* staging, size_t staging_bytes, void* stream);

/*
 * agx_set_option - per-handle switches.  No paper counterpart (plumbing).
 *   AGX_OPT_EARLY_PREFIX_LOADS (value 0 / 1, default 0; environment AGX_EARLY_PREFIX sets the default)
 *       The attention kernels are chained to the launch in front of them by programmatic dependent launch: their CTAs
 *       take their seats while that launch drains and wait for it before touching memory it may have written.  With
 *       this option on, the CTAs fetch page-table entries and K/V pages that lie wholly below the cached-prefix length
 *       (tokens < 16 * floor(prefix_len / 16)) BEFORE that wait, so the first loads of one attention call overlap the
 *       tail of the previous kernel.  The caller thereby vouches that no work still in flight on the stream when the
 *       call is enqueued writes the page table or those pages: true for a cache written by earlier steps or by other
 *       layers' calls on other pools; NOT true directly behind agx_kv_import_pages, agx_kv_copy_pages or a
 *       chunked prefill's previous chunk on the same pool (leave the option off there, or put an event or any launch
 *       that is not part of this library in between).  The block's own rows and Q are always read after the wait.
 *   AGX_OPT_WAIT_LIMIT_CYCLES (value >= 1000, default 4e9 ~ 2 s)
 *       Clock ticks after which an in-kernel wait gives up, sets AGX_DEV_WAIT_TIMEOUT and winds the CTA down.
 *   AGX_OPT_ZERO_COPY (value = bits 0..3, default 3; environment AGX_ZERO_COPY sets the default)
 *       Bit 0: kernels read small pinned, device-mapped host inputs (agx_verify_step_host*) and stored pages
 *       (agx_kv_import_pages) across the bus themselves; cleared, every host buffer goes through copy-engine
 *       transfers into device staging first.  Bit 1: the attention kernels write `out` straight into a pinned, mapped
 *       host buffer.  Reading across the bus is the faster way for a call on an idle GPU; the copy engine is the
 *       better one for an import that should run beside attention on another stream, since it needs no SM.
 *   AGX_OPT_TEST_DROP_STAGE (value = stage index, -1 = off, default -1)
 *       Test hook for the give-up path: the copy-issuing warp of every attention CTA leaves that K/V pipeline stage out
 *       (nothing is armed, nothing is copied), so the waits for it run out after the wait limit and the launch ends
 *       with AGX_DEV_WAIT_TIMEOUT.  Meant to be used with a short wait limit; results of such a launch are invalid.
 * Errors: AGX_E_INVAL (unknown option), AGX_E_RANGE.
 */
enum { AGX_OPT_EARLY_PREFIX_LOADS = 1, AGX_OPT_WAIT_LIMIT_CYCLES = 2, AGX_OPT_TEST_DROP_STAGE = 3, AGX_OPT_ZERO_COPY = 4 };
AGX_API agx_status agx_set_option(agx_handle* handle, int32_t option, int64_t value);

/* Number of kernels the last agx_attn_prefixed / agx_accept_greedy / agx_kv_append call on this
 * handle launched (for launch accounting in benchmarks). */
AGX_API int32_t agx_last_launch_count(const agx_handle* handle);

#ifdef __cplusplus
}
#endif
#endif /* AGX_H_ */
