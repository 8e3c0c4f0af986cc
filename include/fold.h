/*
 * fold.h -- C ABI of the declared-reference ("fold") softmax-attention decode library
 * for NVIDIA B200 (sm_100a).
 *
 * The library computes single-token decode attention over a BF16 key/value cache.  A
 * finite per-row reference Z_i is fixed before the cache is scanned (Section 3, Eq. 2),
 * so every weight 2^(s_ij - Z_i) is final when computed and the per-range pairs
 * (A, L) = (sum_j 2^(s_ij - Z_i) v_j, sum_j 2^(s_ij - Z_i)) add across key ranges with no
 * maximum compared and nothing rescaled (Prop. 1).  A per-call depth T cuts keys whose
 * weight is below 2^-T: they keep their weight in L, add nothing to A, and their value
 * rows are not read (Section 4, "Depth as a dial", Algorithm 1).
 *
 * Units.  Scores are base 2: s_ij = log2(e) * softmax_scale * <q_i, k_j> (Section 2).
 * z, lse and depth_T are all in binades; natural-log lse = ln(2) * lse.
 *
 * Pointers.  Unless a comment says HOST, every pointer is a DEVICE pointer owned by the
 * caller.  The library allocates and frees nothing and keeps no device resource (no stream,
 * no event, no buffer beyond the static scratch array of fold_decode_static); the only state it
 * holds is, per device, "this kernel has been allowed its shared memory" flags and the address of
 * that array, both set at a first call and safe against host threads racing on it.  Every call
 * enqueues work on `stream` and returns without synchronising the host; every call can be captured
 * in a CUDA graph.  Calls that share a workspace must be ordered by the caller (same stream, or events).
 *
 * Values.  Key and value rows of tokens below seqlens[] must be finite.  The depth gate never reads the value row
 * of a key no row keeps, but a row that IS read under a weight of zero (a cut key inside a group of keys fetched
 * whole) is multiplied, not skipped: a NaN or infinity stored there would reach the outputs of that (sequence, kv
 * head).  Rows at or beyond seqlens[] may hold anything.
 *
 * Errors.  Functions return a fold_status.  Only host-detectable conditions are
 * returned (bad arguments, unsupported shapes, workspace too small, a CUDA launch
 * error).  Conditions found on the device are reported in `row_status` bits and in the
 * workspace header (see fold_ws_header); no kernel traps, asserts or waits unboundedly.
 */
#ifndef FOLD_H_
#define FOLD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *fold_stream;            /* a cudaStream_t; NULL is the legacy default stream */

typedef enum fold_status {
  FOLD_OK = 0,
  FOLD_EINVAL = 1,        /* null / misaligned pointer, inconsistent sizes, T < 0 or NaN */
  FOLD_EUNSUPPORTED = 2,  /* head_dim not in {64,128}, page_size not a power of two >= 16, batch > 65535, ... */
  FOLD_EWORKSPACE = 3,    /* workspace_bytes < fold_workspace_bytes(args) */
  FOLD_ECUDA = 4,         /* a CUDA runtime / driver call failed (launch error, no sm_100 device) */
  FOLD_ETOOLARGE = 5      /* fold_decode_static only: the call needs more scratch than the built-in array holds */
} fold_status;

/* How the per-row reference Z_i (Section 3, "Choosing the reference") is obtained. */
typedef enum fold_zmode {
  FOLD_Z_ESTIMATE = 0,  /* the 192-key estimate: sink + 63 most recent keys exactly, plus a
                           trimmed stratified estimate from 128 stratum centres; written to z[] */
  FOLD_Z_GIVEN = 1,     /* caller supplies z[] (e.g. the lse of a previous step, or a cascade's
                           flat estimate shared by all its levels) */
  FOLD_Z_EXACT_MAX = 2, /* test mode: an extra full pass sets z = max_j s_ij; written to z[] */
  FOLD_Z_ZERO = 3       /* z = 0 for every row; written to z[] */
} fold_zmode;

/* Bits of fold_args.flags. */
enum {
  FOLD_INPUTS_SETTLED = 1, /* q, the cache rows, seqlens, page_table and draft_mask were complete before the kernel that
                              precedes this call on `stream` STARTED (they were not written by it).  The call's first
                              kernel may then begin, and read them, while that kernel is still draining (programmatic
                              dependent launch); everything it writes still waits.  Without the flag the first kernel is
                              launched in plain stream order, which is what a decode loop that appends to the cache or
                              projects q just before the call needs. */
  FOLD_SEPARATE_LAUNCHES = 2, /* fold_decode: always run reference, scan and partial add as separate kernels */
  FOLD_ONE_LAUNCH = 4      /* fold_decode: run them inside ONE cooperative kernel launch wherever the decode is one wave:
                              head_dim 128, up to 8 rows per (sequence, kv head), stack 1, FOLD_Z_ESTIMATE or
                              FOLD_Z_GIVEN, no split hint below the chunk count, and at most two canonical chunks per
                              SM in all (each (sequence, kv head)'s count rounded up to even).  Section 3's three steps
                              then follow one another on chip; Algorithm 1 is unchanged, and out, lse, z, row_status and
                              the header are bit for bit those of the separate launches.  With neither flag the library
                              takes the one launch where it measured faster on a B200 -- FOLD_Z_GIVEN -- and separate
                              launches for FOLD_Z_ESTIMATE (three short kernels that overlap by programmatic dependent
                              launch beat one kernel that forms the estimate in every CTA).  Where the one launch does
                              not apply the flag is ignored. */
};

/* Bits of row_status[b * num_q_heads + h]. */
enum {
  FOLD_ROW_RANGE = 1,     /* L outside [2^-1, 2^100]: the range certificate of Section 3 failed;
                             decode the row again with z = the returned lse */
  FOLD_ROW_NONFINITE = 2, /* an output element or L is not finite */
  FOLD_ROW_EMPTY = 4      /* the row has no keys: out = 0, lse = -inf */
};

/* A key/value cache view.  Elements are BF16; the head_dim elements of one (token, head)
 * row are contiguous and every row starts on a 16-byte boundary (all strides, in
 * elements, are multiples of 8).
 *
 * Contiguous (page_table == NULL): row (seq, tok, head) is at
 *     k + seq*stride_seq + tok*stride_tok + head*stride_head,   tok < capacity.
 * Paged (page_table != NULL): logical token j of sequence `seq` is row
 *     (page = page_table[seq*max_pages_per_seq + j / page_size], j % page_size, head) at
 *     k + page*stride_seq + (j % page_size)*stride_tok + head*stride_head.
 * Rows at or beyond seqlens[seq] (and unused page tails) are never used, whatever they hold.
 *
 * Block tail (Section 4, "Depth as a dial": the block model, its mean only -- the fitted rank-16 map is
 * not part of this library).  v_block_mean, when not NULL, holds for every LOGICAL block of 64
 * consecutive keys [64 b, 64 b + 64) of every sequence the mean of that block's value rows as BF16
 * (a short last block: the mean of the keys it has), row (seq, b, head) at
 *     v_block_mean + seq*mean_stride_seq + b*mean_stride_block + head*mean_stride_head
 * (elements; multiples of 8; rows 16-byte aligned; blocks are logical for paged caches too).  A decode
 * at finite depth then adds, for every row, the summed weight of the keys that row cuts in a block
 * times that block's mean to A, instead of nothing (Algorithm 1: the step that gives the cut keys' weights to the
 * tile's virtual row).  fold_block_means() fills the table from the cache; keeping it current when
 * tokens are appended is the caller's business (only the last block changes).  Every row-block and
 * stacked-row shape takes it (a stacked level with a table runs on the mma.sync kernel, not on tcgen05).
 * Ignored at depth_T = INFINITY (nothing is cut).
 *
 * Two-plane INT8 keys (Section 4, "Cache format"; Algorithm 1).  When k_plane_a is not NULL the decode
 * reads keys from two INT8 planes and a BF16 scale per (token, kv head) instead of from k:
 *     H k_j ~ e_j (a_j + b_j / 256),   H the orthonormal Hadamard matrix of order head_dim,
 * written by fold_quantize_keys() (below, which states the arithmetic).  Plane rows are head_dim bytes,
 * contiguous, 16-byte aligned: row (seq-or-page, tok, head) of plane X at
 *     k_plane_X + seq*plane_stride_seq + tok*plane_stride_tok + head*plane_stride_head   (bytes; multiples of 16),
 * both planes with the same strides, paged exactly as k is (same page_table).  The scales lie token-fastest,
 *     k_scale + seq*scale_stride_seq + head*scale_stride_head + tok                       (BF16 elements; multiples of 8),
 * and every (sequence-or-page, head) scale row must be readable up to the next multiple of 8 tokens past
 * capacity (page_size).  With planes, k may be NULL for the decode calls; v stays BF16.  Each scan scores every
 * key against plane A alone (head_dim + 2 bytes per key), ORs the verdicts over the rows that share the kv head,
 * and only then requests plane B rows (refined keys) and value rows (live keys).  Up to 16 rows per
 * (sequence, kv head) (stack * group, draft rows included) form one block whose verdicts are ORed over all of them;
 * more stacked rows (a cascade's shared level) are cut into blocks of 16 rows in row order, each block scanned as
 * Algorithm 1 over its own rows with its own verdicts.  With or without the block tail; no FOLD_Z_EXACT_MAX, and
 * draft rows only within one block (FOLD_EUNSUPPORTED otherwise).  A cascade may run on two-plane keys when every
 * level has them (see fold_decode_cascade); a level's automatic refine gate follows that level's own length.
 *
 * Two E4M3 value planes (Section 4, "Cache format": two FP8 planes that share one power-of-two scale per layer; only
 * together with the two-plane keys).  When v_plane_1 is not NULL the scan reads values from
 *     v_j ~ 2^v_scale_log2 * (v1_j + v2_j),   v1, v2 E4M3 codes (1-4-3 bits, bias 7, largest value 448),
 * written by fold_quantize_values(): rows of head_dim bytes laid out exactly like the key planes (the same
 * plane_stride_* and paging).  A live key's plane-1 row is always read; its plane-2 row only when some row of
 * the group gives the key a coarse weight >= 2^-refine_tau_v ("refine V"): head_dim + head_dim * r_V bytes per live
 * key instead of 2 * head_dim.  The codes widen to BF16 exactly; v1 + v2 is rounded to BF16 once.  v may then be
 * NULL for the decode calls.  Draft masks apply as on BF16 values.  The cut model of this format is not the block
 * model but the sequence's mean value row (Section 4, "Depth as a dial": a mean kept per request): with value
 * planes, v_block_mean (when not NULL) is read as ONE row per (sequence, kv head) -- block index 0 of the layout
 * above, mean_stride_block unused -- holding the mean of all the sequence's value rows as BF16
 * (fold_running_means() fills it), and a decode at finite depth adds, for every row, the summed weight of the keys
 * that row cuts times that mean row to A. */
typedef struct fold_kv {
  const void *k, *v;
  int64_t stride_seq, stride_tok, stride_head;   /* elements */
  const int32_t *page_table;                     /* [num_seqs, max_pages_per_seq] or NULL */
  int32_t page_size;                             /* tokens per page, power of two >= 16; 0 if contiguous */
  int32_t max_pages_per_seq;
  int32_t num_pages;                             /* pages in the pool (paged) */
  int32_t capacity;                              /* tokens allocated per sequence (contiguous) */
  int32_t num_seqs;                              /* KV sequences */
  const int32_t *seqlens;                        /* [num_seqs] keys per sequence */
  int32_t max_seqlen;                            /* HOST upper bound on seqlens[]; sizes grids and slots */
  const void *v_block_mean;                      /* BF16 block means, or NULL: no block tail */
  int64_t mean_stride_seq, mean_stride_block, mean_stride_head;   /* elements */
  const int8_t *k_plane_a, *k_plane_b;           /* INT8 key planes, or NULL: BF16 keys from k */
  int64_t plane_stride_seq, plane_stride_tok, plane_stride_head;  /* bytes */
  const void *k_scale;                           /* BF16 scale per (token, kv head), token-fastest */
  int64_t scale_stride_seq, scale_stride_head;   /* elements */
  const uint8_t *v_plane_1, *v_plane_2;          /* E4M3 value planes (strides: plane_stride_*), or NULL: BF16 values from v */
  int32_t v_scale_log2;                          /* the value planes' power-of-two scale */
} fold_kv;

/* One decode call.  `batch` requests with one query token each; request b reads KV
 * sequence b / stack (stack consecutive requests share a sequence: stack = 1 for plain
 * decode; a cascade's shared-prefix level stacks the query rows of all requests that hold
 * the prefix, Section 4 "Value product" last sentence).  batch == kv.num_seqs * stack.
 * Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *
 * Drafts and verification trees (Section 4 "Value product": extra query rows masked to their ancestors).
 * With draft_len = m in 1..32 the last m keys of every sequence are draft tokens already appended to the
 * cache: key n - m + t (n the sequence's length) is used by request b only if bit t of draft_mask[b] is
 * set; earlier keys are used by every request; all heads of a request share its mask.  The requests that
 * verify one sequence are the `stack` consecutive requests that read it (a chain of m drafts: stack = m,
 * draft_mask[r] = 2^(r+1) - 1).  A key a row does not use has weight exactly 0 everywhere: in the
 * reference estimate, in L and in A.  A row must use at least one key.  In a cascade only the level that
 * holds the drafts (the last) carries them.  draft_len = 0: no masking. */
typedef struct fold_args {
  int32_t batch, num_q_heads, num_kv_heads, head_dim;  /* head_dim in {64, 128} */
  int32_t stack;
  const void *q;                       /* BF16 [batch, num_q_heads, head_dim], head_dim contiguous */
  int64_t q_stride_b, q_stride_h;      /* elements, multiples of 8 */
  fold_kv kv;
  float softmax_scale;                 /* c; > 0, finite */
  int32_t z_mode;                      /* fold_zmode */
  float *z;                            /* [batch, num_q_heads] fp32, binades; read (GIVEN) or written */
  float depth_T;                       /* binades, >= 0; INFINITY = dense decode */
  int32_t num_splits;                  /* CTAs per (sequence, kv head); 0 = choose.  A scheduling
                                          hint only: it never changes a bit of the result */
  void *workspace;                     /* 256-byte aligned */
  size_t workspace_bytes;              /* >= fold_workspace_bytes(args) */
  void *out;                           /* BF16 [batch, num_q_heads, head_dim], contiguous */
  float *lse;                          /* [batch, num_q_heads] base-2 log-sum-exp, or NULL */
  int32_t *row_status;                 /* [batch, num_q_heads] bit flags, or NULL */
  const uint32_t *draft_mask;          /* [batch] or NULL (draft_len = 0) */
  int32_t draft_len;                   /* 0..32 */
  float refine_tau;                    /* two-plane keys only: the refine gate tau_K of Algorithm 1, binades.  A live key
                                          reads plane B iff some row of its group has coarse weight >= 2^-refine_tau.
                                          0 = choose: max(log2(n) - 2, 4) for a sequence of n keys (its own length only:
                                          a key is refined when some row gives it >= 4/n of the row's mass);
                                          INFINITY = every live key; negative = none (plane A scores only) */
  float refine_tau_v;                  /* E4M3 value planes only: the refine-V gate, binades, like refine_tau.
                                          0 = choose: max(log2(n) + 1, 4); INFINITY = every live key; negative = none */
  int32_t flags;                       /* FOLD_INPUTS_SETTLED, FOLD_SEPARATE_LAUNCHES, FOLD_ONE_LAUNCH: ORed, or 0 */
  fold_stream side_stream;             /* fold_decode_cascade, levels[0] only: a second stream of the caller's and two */
  void *side_fork_event;               /* cudaEvent_t of the caller's (created with timing disabled, say) on which the */
  void *side_join_event;               /* first level is scanned; all three NULL: every level on `stream` */
  float live_hint;                     /* finite depth_T: the fraction of value rows the caller expects to be kept (what
                                          v_rows_fetched / v_rows_total of the step before was, say), in (0, 1]; 0 = no
                                          expectation.  Scheduling only -- how the row-block scan splits its on-chip ring
                                          between key and value tiles (Section 4, "Weight-gated reads": the byte mix
                                          2D + 2D lambda varies with lambda) -- never a bit of any result.  NaN or
                                          negative values count as 0. */
} fold_args;

/* First 64 bytes of every workspace, zeroed at the start of each scan. */
typedef struct fold_ws_header {
  uint32_t wait_timeouts;      /* != 0: a bounded on-chip wait gave up; the results are invalid */
  uint32_t reserved;
  uint64_t v_rows_fetched;     /* value rows actually requested from memory, all (seq, kv head) */
  uint64_t v_rows_total;       /* value rows a dense decode would read (= keys scanned) */
  uint64_t v_slices_skipped;   /* warp slices (16 keys at head_dim 128, 32 at 64) whose value work was skipped entirely */
  uint64_t k_rows_refined;     /* two-plane keys: plane B rows requested from memory */
  uint64_t v2_rows_refined;    /* E4M3 value planes: plane-2 rows requested from memory */
  uint64_t pad[2];
} fold_ws_header;

/* The (A, L) partial pairs one scan leaves in its workspace (Algorithm 1, last line).
 * The key axis of every sequence is cut into canonical chunks of fold_chunk_keys(n) keys,
 * aligned to absolute key index; chunk c of (seq, kv head) owns slot c:
 *     slot = slots + ((seq*num_kv_heads + kvh)*max_slots + c) * slot_stride   (floats)
 *     A[r][d] = slot[r*head_dim + d],  L[r] = slot[rows*head_dim + r],
 *     r = (request % stack) * group + (q head % group),  rows = stack * group.
 * Slots 0 .. fold_num_chunks(seqlens[seq])-1 are valid; the rest are never read.  A slot's
 * content depends only on (q rows, that chunk's keys/values, z, T): not on num_splits,
 * batch composition or cache layout.  Partial sets can be added only if they were
 * scanned under the same z. */
typedef struct fold_partials {
  float *slots;
  const int32_t *seqlens;      /* [num_seqs], the scanned sequence lengths */
  const float *z;              /* [batch, num_q_heads] the reference the partials were formed under */
  int32_t batch, num_q_heads, num_kv_heads, head_dim, stack;
  int32_t num_seqs, max_slots, rows;
  int32_t max_seqlen;          /* the HOST bound the slots were sized for */
  int64_t slot_stride;         /* floats */
} fold_partials;

/* Keys per canonical chunk for a sequence of n keys, and the number of chunks.  Pure
 * host functions of n (and of nothing else), so results cannot depend on the batch. */
int32_t fold_chunk_keys(int32_t n);
int32_t fold_num_chunks(int32_t n);

/* Bytes of workspace fold_decode / fold_decode_split need for `args` (header + slots; with two-plane keys
 * also the split query rows).  Depends only on shapes, kv.max_seqlen and whether kv.k_plane_a is set.
 * Returns 0 if args is invalid. */
size_t fold_workspace_bytes(const fold_args *args);

/* Reference estimate (Section 3): writes levels[0]->z for every (request, q head).
 * The logical key sequence of request b is the concatenation of its sequences in
 * levels[0], levels[1], ... (a cascade's prefix then suffix; Appendix "Cascades and
 * drafts": the cascade takes its references from the flat estimate).  q, z and the head
 * counts are taken from levels[0]; each level contributes its kv and stack.  n_levels
 * in 1..4.  `levels` is a HOST array of HOST pointers.  The levels keep to one key format; with two-plane keys the
 * sampled keys are scored with both planes, and every level's workspace (required, as for fold_decode_split)
 * receives the split query rows. */
int fold_estimate_z(const fold_args *const *levels, int n_levels, fold_stream stream);

/* Scan only (Algorithm 1 with a BF16 cache): obtains z per args->z_mode, scores every key
 * against it, accumulates FP32 (A, L) per canonical chunk into args->workspace and fills
 * *dst (HOST struct) describing them.  out / lse / row_status are not touched. */
int fold_decode_split(const fold_args *args, fold_partials *dst, fold_stream stream);

/* Order-free partial add (Prop. 1(i); summation on a declared integer grid, Eq. 3 /
 * Prop. 2, so that the result is a function of the SET of partials): for every
 * (request, q head) adds all valid slots of all levels, writes out = A / L (BF16, round
 * to nearest even), lse = z + log2 L and row_status.  Used for the split-KV merge
 * (n_levels = 1) and the shared-prefix cascade (prefix level + suffix level).  All levels
 * must describe the same batch / heads / head_dim and the same z.  `levels` is a HOST
 * array of HOST pointers to HOST structs; n_levels in 1..4. */
int fold_cascade_merge(const fold_partials *const *levels, int n_levels, void *out, float *lse,
                       int32_t *row_status, fold_stream stream);

/* Whole decode: reference (per z_mode) -> scan -> partial add.  Equivalent to
 * fold_decode_split followed by fold_cascade_merge over its one level. */
int fold_decode(const fold_args *args, fold_stream stream);

/* How many kernels fold_decode(args) launches: 1 when the decode is one wave and runs in a single launch (see
 * FOLD_ONE_LAUNCH), else the reference kernel (if the mode has one), the scan and the partial add; 0 for
 * arguments fold_decode would refuse.  A host-side query: nothing is enqueued.  (No counterpart in the paper.) */
int32_t fold_decode_launches(const fold_args *args);

/* Shared-prefix cascade in one call (Section 4, "Value product"; Appendix "Cascades and drafts"):
 * one reference estimate over each request's concatenated levels, one scan per level under
 * that reference, one order-free add over all levels' partials.  levels[l] (HOST array of HOST
 * pointers, n_levels in 1..4) describe the same requests: the same q, z, batch, head counts,
 * head_dim, softmax_scale and depth_T; each level has its own kv, stack and workspace.
 * levels[0]->z_mode is FOLD_Z_ESTIMATE (estimate over all levels, written to z) or FOLD_Z_GIVEN;
 * out, lse and row_status are taken from levels[0].  The levels' keys are all BF16 or all two-plane
 * (FOLD_EUNSUPPORTED otherwise); with two-plane keys one front kernel splits the query rows for every level.
 * With two or more levels and levels[0]->side_stream / side_fork_event / side_join_event set (a stream and two events the
 * CALLER owns, the stream different from `stream`), the first level is scanned on the side stream, forked from and
 * joined back into `stream` with the events, so to the caller the call is still one ordered piece of work on `stream`;
 * the events are recorded by every such call, so calls that share them must not overlap.  Without them every level
 * is scanned on `stream`. */
int fold_decode_cascade(const fold_args *const *levels, int n_levels, fold_stream stream);

/* Fill kv->v_block_mean (DEVICE memory of the caller, laid out as the fold_kv comment says, at least
 * ceil(kv->max_seqlen / 64) blocks per sequence) from kv->v: for every sequence, block b < ceil(n / 64)
 * and kv head, the mean of the block's value rows, summed in float64 in key order, divided by the key
 * count, rounded to FP32 and then to BF16 (both to nearest even) -- Section 4, "Depth as a dial".  Blocks
 * at or beyond ceil(n / 64) are left untouched.  Asynchronous on `stream`; reads seqlens on the device.
 * num_kv_heads / head_dim as in fold_args.  FOLD_EINVAL for a NULL or misaligned table. */
int fold_block_means(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, fold_stream stream);

/* The same for the 8-bit value format's cut model (Section 4, "Depth as a dial"): writes, for every sequence and kv
 * head, the mean of ALL its value rows j < seqlens[s] (float64 sums, one rounding to FP32 and one to BF16) into block
 * 0 of kv->v_block_mean; a sequence of length 0 gets zeros.  Reads kv->v (BF16 values; FOLD_EINVAL if NULL). */
int fold_running_means(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, fold_stream stream);

/* Cache write for two-plane INT8 keys (Section 4, "Cache format"): for every sequence s, kv head and token
 * first_token[s] <= j < seqlens[s] (first_token == NULL: from 0; a DEVICE array otherwise -- pass the old lengths
 * to quantize only appended tokens) read the BF16 key row from kv->k, rotate it and write its two planes and
 * scale into kv->k_plane_a / k_plane_b / k_scale (DEVICE memory of the caller; written although the struct
 * says const).  A row's code depends on that row alone.  The arithmetic is FP32, one rounding per step, so the
 * codes are reproducible bit for bit:
 *   y = H x:   log2(head_dim) butterfly stages with strides 1, 2, 4, ..., each (lo, hi) -> (lo + hi, lo - hi),
 *              then one multiply by fp32(1 / sqrt(head_dim));
 *   e = the smallest BF16 value >= max|y| / 127 (1 if the row is all zero), so plane A never saturates;
 *   t = y / e;   a = rint(t) within +-127;   b = rint((t - a) * 256) within [-128, 127]   (ties to even).
 * The decode splits each query row the same way at every step (into its workspace) and carries
 * eta = e_q * fp32(log2(e) * softmax_scale).  Asynchronous on `stream`. */
int fold_quantize_keys(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, const int32_t *first_token,
                       fold_stream stream);

/* Cache write for the E4M3 value planes: for every sequence, kv head and token first_token[s] <= j < seqlens[s]
 * (first_token as in fold_quantize_keys) read the BF16 value row from kv->v and write
 *     p1 = e4m3(v / 2^v_scale_log2),   p2 = e4m3(v / 2^v_scale_log2 - p1)
 * (round to nearest, ties to even, magnitudes beyond 448 saturate; both subtractions and the scaling are exact)
 * into kv->v_plane_1 / v_plane_2 (DEVICE memory of the caller, written although the struct says const).  The scale
 * is the caller's: 2^v_scale_log2 >= max|v| / 448 keeps plane 1 from saturating.  Asynchronous on `stream`. */
int fold_quantize_values(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, const int32_t *first_token,
                         fold_stream stream);

/* The same decode for callers whose tensors live in HOST memory (pinned for the copies to
 * be asynchronous): q, kv.k, kv.v, kv.page_table, kv.seqlens, z (if GIVEN), out, lse and
 * row_status of *host_args are HOST pointers laid out as described above (the cache is
 * copied as the single span its strides cover).  `staging` is DEVICE memory of at least
 * fold_host_staging_bytes(host_args) bytes, 256-byte aligned, which receives the copies,
 * the workspace and the results before they are copied back.  Everything is enqueued on
 * `stream`; the host buffers are valid after the caller synchronises the stream.  With two-plane keys (and
 * E4M3 value planes) kv.k_plane_a / k_plane_b / k_scale (v_plane_1 / v_plane_2) are HOST pointers too and are copied
 * as the spans their strides cover (a scale row up to the next multiple of 8 tokens); kv.k (kv.v) may then be NULL.
 * The block tail is not offered here: kv.v_block_mean must be NULL (FOLD_EUNSUPPORTED otherwise); nor are draft
 * masks (draft_len must be 0). */
size_t fold_host_staging_bytes(const fold_args *host_args);
int fold_decode_host(const fold_args *host_args, void *staging, size_t staging_bytes, fold_stream stream);

/* Decode without a caller workspace.  (The paper has no counterpart: this entry point exists for
 * integration, not for the method.)
 *
 * Who needs it: callers that cannot hand the library device memory at call time because they are
 * not allowed to allocate any -- a plugin inside a host program that owns the whole device heap and
 * forbids cudaMalloc, a decode loop that must never reach the allocator because cudaMalloc /
 * cudaFree synchronise the device and stall every stream, or code that is only given its input and
 * output tensors and has nowhere to keep a buffer between calls.
 *
 * What it does: exactly fold_decode(args, stream), except that args->workspace and
 * args->workspace_bytes are ignored and the scratch the scan and the partial add need (the
 * fold_ws_header and the (A, L) slots) lives in an array built into the library:
 * FOLD_STATIC_SCRATCH_BYTES bytes of device memory, 256-byte aligned, that every GPU which loads
 * the library holds from load to exit.  The call allocates and frees nothing, on the host side of
 * the CUDA API or through any other library.
 *
 * Limits and rules:
 *  - A call whose fold_workspace_bytes(args) exceeds FOLD_STATIC_SCRATCH_BYTES is refused with
 *    FOLD_ETOOLARGE before anything is enqueued (16 requests x 8 kv heads x 32768 keys at group 4,
 *    head_dim 128, need 8.1 MiB).
 *  - The first call on each device looks up the array's device address (with that device current);
 *    make that first call outside any stream capture.  Later calls on the device reuse the address.
 *    Host threads that race on that first call look up the same address and store the same value.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left.  The
 *    library re-zeroes the part that must start at zero (the header) at the start of every call and
 *    never reads a slot the same call has not written, so stale contents are harmless -- but two
 *    calls that can overlap on the GPU (different streams, or a call racing a graph replay that
 *    contains one) would write the same slots: order them yourself.
 *  - The partials are not exposed: there is no split / cascade form of this entry point. */
#define FOLD_STATIC_SCRATCH_BYTES (16u << 20)
int fold_decode_static(const fold_args *args, fold_stream stream);

/* Measurement aid (the paper has no counterpart): reads `bytes` bytes (16-byte aligned; a multiple of 16 is read) of
 * DEVICE memory once with streaming loads on every SM and XORs a digest of them into *sink (DEVICE, may be NULL).
 * Timed with events around it, buffer bytes / time is the read-only bandwidth a kernel can get from this memory
 * system: the third denominator beside the nominal and the measured-copy figures.  Asynchronous on `stream`. */
int fold_probe_read(const void *buffer, size_t bytes, uint64_t *sink, fold_stream stream);

const char *fold_status_string(int status);
/* Library version as major*10000 + minor*100 + patch. */
int fold_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FOLD_H_ */
