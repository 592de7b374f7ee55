/*
 * libsepllm — separator-masked causal attention for one B200 (sm_100a).
 *
 * The operations follow "SepLLM" (arXiv 2412.12094): a query at position i
 * attends to the first n_init tokens, to every earlier separator token and to
 * its n_neighbor closest tokens, itself included (Section 3.1; Eq. 1 and
 * Eq. 2), in forward and backward; generation keeps a four-block KV cache
 * (Section 3.3).
 *
 * Conventions for every call
 *  - C ABI, plain pointers and sizes.  "dev" = device pointer, "host" = host
 *    pointer.  Descriptors are host structs read during the call.
 *  - The caller owns every buffer.  Unless a call says otherwise the library
 *    allocates nothing and keeps no state between calls.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *    only enqueue work; they do not synchronise unless stated.
 *  - Errors are return codes.  Shape, alignment and capacity errors are found
 *    on the host before anything is launched.  Conditions only the device can
 *    see (more side entries than side_cap, a wait that ran out) are written to
 *    a status word at the start of the workspace / state buffer and read with
 *    sepllm_last_device_status(); kernels clamp instead of writing out of
 *    bounds.
 *  - Tensors are bf16 (two bytes, upper half of an IEEE fp32), row-major,
 *    contiguous, base pointers 16-byte aligned:
 *        Q, O, dO, dQ : [B][Hq][L][d]        K, V, dK, dV : [B][Hkv][L][d]
 *        LSE          : [B][Hq][L] fp32, natural logarithm
 *    Query head h reads KV head h / (Hq/Hkv).
 *  - Sequences shorter than L are padded at the end (any token ids, any finite
 *    K, V, Q values): the mask is causal, so no valid row sees a padded key,
 *    and with dO = 0 on the padded rows the padded queries add nothing to dK
 *    and dV.  Outputs of padded rows are to be ignored.  An index built with
 *    sepllm_build_index_varlen also tells the attention calls where each
 *    sequence ends: query tiles that hold only padding are then skipped (their
 *    rows of O, LSE and dQ are not written; their rows of dK and dV are
 *    written as 0), and padded positions are never initial tokens or
 *    separators.
 *  - Supported: d in {64, 80, 96, 112, 128} for the attention calls (rows of
 *    exactly d elements, no padding in memory; sizes above 64 run in the
 *    128-wide kernels and cost what d = 128 costs), d in {64, 128} for the
 *    cache calls; Hq a multiple of Hkv; n_neighbor >= 1; n_init >= 0; index
 *    tiles BM = BN = 128 for the attention calls.
 */
#ifndef SEPLLM_H_
#define SEPLLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int sepllm_status;
enum {
  SEPLLM_OK = 0,
  SEPLLM_INVALID_ARG = 1,       /* null pointer, non-positive size, misaligned buffer */
  SEPLLM_UNSUPPORTED = 2,       /* valid request outside the supported set above */
  SEPLLM_BUFFER_TOO_SMALL = 3,
  SEPLLM_CUDA_ERROR = 4,        /* a CUDA runtime / driver call failed */
  SEPLLM_CAPACITY_EXCEEDED = 5, /* device status: more side entries than side_cap */
  SEPLLM_TIMEOUT = 6,           /* device status: a bounded wait in a kernel ran out */
  SEPLLM_NOT_BUILT = 7
};

#define SEPLLM_MAX_SEP_IDS 64

/* Index description.  side_cap = capacity (entries per sequence) of the side
 * list, i.e. initial tokens plus separators; L is always enough. */
typedef struct {
  int32_t B, L, n_init, n_neighbor, n_sep, BM, BN, side_cap;
} sepllm_index_desc;

/* scale = 0 means 1/sqrt(d) (Eq. 1).  grad_dtype: 0 = bf16, 1 = fp32 outputs
 * for dQ, dK, dV.
 * flags: SEPLLM_ATTN_SIDE_READY = the workspace already holds the side K/V rows
 *   gathered from these K, V by an earlier attention call on the same workspace
 *   (a backward given the forward's workspace); the call then skips its gather
 *   and leaves the workspace's status word as the earlier call left it.
 * events / n_events: a measurement aid, not part of the operation: optional host
 *   array of cudaEvent_t handles (NULL / 0 = off, the normal use).
 *   The call records events[0] on `stream` before its first launch and
 *   events[i] after its i-th launch, for as many as the array holds, so a
 *   caller can time each kernel.  Forward launches: 1 side gather, 2 attention.
 *   Backward launches: 1 side gather, 2 Delta, 3 dQ, 4 dK/dV of side tiles,
 *   5 dK/dV of window tiles.  A skipped gather still records its event. */
#define SEPLLM_ATTN_SIDE_READY 1
typedef struct {
  int32_t B, Hq, Hkv, d, L;
  float scale;
  int32_t grad_dtype;
  int32_t flags;
  void* const* events;
  int32_t n_events;
} sepllm_attn_desc;

/* Streaming cache capacities in the paper's names (Section 3.3): a initial,
 * s separator, w local window, c total; a + s + w < c, w >= 1.  The cache
 * calls take up to 16 query heads per kv head (Hq / Hkv <= 16).
 * flags = 0: the four-block cache of Section 3.3 (the neighbour run grows until
 *   Size_run reaches c, then its Past Window part is compacted).
 * flags = SEPLLM_CACHE_FIXED_WINDOW: generation in the fundamental design
 *   (Section 3.2 "Generation"; Section 4.2 keeps all separator KV there): the
 *   neighbour run is exactly the w most recent tokens (w plays n's role); a
 *   token that leaves it moves to the Separator Cache if it is a separator and
 *   is dropped otherwise; the Separator Cache never evicts.  s is then its
 *   capacity, chosen by the caller for the longest text (c only sizes the
 *   buffers: slots = c + s as before, a + s + w < c).  After token t the
 *   retained set is row t of Eq. 2's mask with n_init = a, n_neighbor = w.  A
 *   sequence with more than s separators outside the window reports
 *   SEPLLM_CAPACITY_EXCEEDED in the state's status word and keeps the newest s. */
#define SEPLLM_CACHE_FIXED_WINDOW 1
typedef struct {
  int32_t B, Hkv, Hq, d, a, s, w, c;
  int32_t flags;
} sepllm_cache_desc;

/* ---- index blob -----------------------------------------------------------
 * The index is one device buffer: this header, then five int32 arrays at the
 * byte offsets it gives (each 256-byte aligned):
 *   cnt       [B][L+1]      cnt[j] = side members (j < n_init or separator) at positions < j
 *   lim       [B][L]        lim[i] = cnt[max(0, i-n_neighbor+1)]: side entries row i keeps
 *                           outside its neighbour window
 *   side_pos  [B][side_cap] ascending positions of side members (-1 beyond n_side)
 *   n_side    [B]           number of side members (may exceed side_cap: then the status
 *                           word reads SEPLLM_CAPACITY_EXCEEDED and side_pos is truncated)
 *   seq_len   [B]           tokens in each sequence (L unless built by sepllm_build_index_varlen)
 *   tile_meta [B][ceil(L/BM)][8] per query tile of BM rows (all 0 for a tile of padding; the last
 *       valid tile ends at the sequence's last token):
 *       0 side_full   floor(lim[first row]/BN)   side tiles all rows see in full
 *       1 side_last   ceil(lim[last row]/BN)     side tiles any row sees
 *       2 win_lo      max(0, first row - n_neighbor + 1)
 *       3 win_hi      last row + 1
 *       4 win_tile_lo win_lo / BN
 *       5 win_tile_hi ceil(win_hi / BN)
 *       6 pairs       kept (query,key) pairs in the tile
 *       7 side_first  first side tile any row sees (0 unless the index holds documents)
 *   doc_start [B][L], doc_end [B][L]   bounds of the document each position belongs to; written
 *       by sepllm_build_index_packed only (the header's `packed` word is then 1)
 * The mask these arrays encode is Eq. 2 with M[i][j] = 1 iff j <= i and
 * (j < n_init or token j is a separator or i - j < n_neighbor).
 */
#define SEPLLM_INDEX_MAGIC 0x58444953u /* "SIDX" */
typedef struct {
  int32_t status;      /* device status word of sepllm_build_index (first word) */
  uint32_t magic, version;
  sepllm_index_desc desc;
  int32_t n_tiles;     /* ceil(L/BM) */
  int64_t off_cnt, off_lim, off_side_pos, off_n_side, off_tile_meta, total_bytes;
  int64_t off_seq_len;
  int64_t off_doc_start, off_doc_end;
  int64_t packed;      /* 1: built by sepllm_build_index_packed, the document arrays are valid */
  int64_t reserved[16];
} sepllm_index_header; /* 256 bytes */

/* Sizes of the index blob and of the scratch buffer sepllm_build_index needs. */
sepllm_status sepllm_index_bytes(const sepllm_index_desc* desc, size_t* index_bytes,
                                 size_t* scratch_bytes);

/* Builds the index of Eq. 2's mask from token ids (Section 3.1: initial,
 * separator and neighbouring tokens; Section 4.1 for the separator set).
 *   token_ids dev  int32 [B][L]
 *   sep_ids   host int32 [n_sep], n_sep <= SEPLLM_MAX_SEP_IDS (0 = no separators)
 *   index     dev  sepllm_index_bytes() bytes, 256-byte aligned; written in full
 *   scratch   dev  scratch_bytes, 256-byte aligned; contents undefined afterwards
 * Integer output, deterministic. */
sepllm_status sepllm_build_index(const sepllm_index_desc* desc, const int32_t* token_ids,
                                 const int32_t* sep_ids, void* index, void* scratch,
                                 void* stream);

/* Index of a batch of sequences of unequal lengths padded to L (the paper
 * trains and pre-fills on full rows and does not treat padding; the reading
 * taken is that a padded position is no token at all): seq_len dev int32 [B],
 * 0 <= seq_len[b] <= L (values outside are clamped).  Positions from
 * seq_len[b] on are neither initial tokens nor separators, query tiles that
 * start at or behind seq_len[b] carry no work, and the tile that holds the
 * last token ends there.  With every seq_len[b] = L the result equals
 * sepllm_build_index's.  Other arguments as there. */
sepllm_status sepllm_build_index_varlen(const sepllm_index_desc* desc, const int32_t* token_ids,
                                        const int32_t* seq_len, const int32_t* sep_ids,
                                        void* index, void* scratch, void* stream);

/* Index of rows that pack several documents one after the other.  The paper
 * trains on full rows and does not treat packing; the reading taken: Eq. 2
 * holds inside each document and nothing is seen across a boundary, so the
 * initial tokens are the first n_init tokens of every document and a row's
 * neighbour window stops at its document's first token.
 *   doc_first dev int32 [B][L]: non-zero where a document begins (position 0
 *             begins one whatever it holds)
 *   seq_len   dev int32 [B] or NULL (every row full), as for _varlen
 * Row i then keeps the side entries [cnt[doc_start[i]], lim[i]) and the keys
 * from max(i-n_neighbor+1, doc_start[i]) to i, with lim[i] = cnt of that first
 * window key; a key j is kept by queries before doc_end[j] only.  The
 * attention calls read the header's `packed` word on the device and follow
 * the document bounds; sepllm_cache_from_prompt takes no such index.
 * scratch is not used (may be NULL).  Integer output, deterministic; a plain
 * multi-pass build (one block per row scans it in 8192-token steps), not
 * tuned like sepllm_build_index. */
sepllm_status sepllm_build_index_packed(const sepllm_index_desc* desc, const int32_t* token_ids,
                                        const int32_t* doc_first, const int32_t* seq_len,
                                        const int32_t* sep_ids, void* index, void* scratch,
                                        void* stream);

/* Same result as sepllm_build_index, for callers that cannot hand over a scratch
 * buffer because they cannot allocate device memory at the point of the call: a
 * serving process whose memory pool is already fully handed out, a plugin or
 * callback that runs where cudaMalloc is forbidden, or a latency-critical loop
 * that must not take cudaMalloc's device-wide synchronisation.  (The paper has
 * no counterpart; this is a packaging variant of the index build.)
 * The scratch lives in a fixed 256 KB array (65536 words) inside the library
 * image, present on every device that loads the library until the process
 * exits.  A call needs two words per 4096-token chunk plus one per sequence,
 * so the limit is B * (2 * ceil(L / 4096) + 1) <= 65536 (for example 31
 * sequences of 2^22 ids, or 21845 sequences of 4096); beyond it the call
 * returns SEPLLM_BUFFER_TOO_SMALL and launches nothing.  The call itself
 * allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 * Every call looks up the array's device address on the current device (a
 * host-side lookup); the first call on a device also makes the runtime load
 * the library's kernels there, so make that first call outside any stream
 * capture.  All calls on a device share the one
 * array: two calls whose kernels may overlap on the GPU (different streams
 * without ordering, or different host threads) race on it and must be
 * serialised by the caller.  The array keeps the last call's contents; each
 * call clears the words it is going to use (a memset on `stream`, before its
 * kernel), so back-to-back calls are independent.  Other arguments and the
 * written index are exactly those of sepllm_build_index. */
sepllm_status sepllm_build_index_static(const sepllm_index_desc* desc, const int32_t* token_ids,
                                        const int32_t* sep_ids, void* index, void* stream);

/* Index of the fixed-interval variant (Section 4.7 and the appendix, both
 * under "Fixed-Interval Variant": instead of the separators, one token every
 * `interval` positions is attended to between the initial and the
 * neighbouring tokens).  The side
 * members are the first n_init positions and every position j with
 * j % interval == 0 (the paper does not say where the intervals start; they
 * start at position 0 here).  No token ids are read; desc->n_sep must be 0,
 * interval >= 1.  The written index has the layout of sepllm_build_index and
 * serves the same attention and hand-off calls.  Other arguments as there. */
sepllm_status sepllm_build_index_fixed_interval(const sepllm_index_desc* desc, int32_t interval,
                                                void* index, void* scratch, void* stream);

/* Workspace sizes for the attention calls (bytes; either pointer may be NULL). */
sepllm_status sepllm_attn_workspace_bytes(const sepllm_attn_desc* desc,
                                          const sepllm_index_desc* idesc, size_t* fwd_bytes,
                                          size_t* bwd_bytes);

/* Forward of Eq. 1 under the mask of Eq. 2: O = softmax(Q K^T * scale | M) V and
 * the row log-sum-exp.  Q, K, V dev bf16; index dev (built with the same B, L and
 * BM = BN = 128); O dev bf16; LSE dev fp32; workspace dev fwd_bytes, 256-byte
 * aligned (its first word is the device status). */
sepllm_status sepllm_attn_fwd(const sepllm_attn_desc* desc, const sepllm_index_desc* idesc,
                              const void* Q, const void* K, const void* V, const void* index,
                              void* O, float* LSE, void* workspace, void* stream);

/* Backward of the same operation (the gradient of softmax attention, training
 * with the mask: Section 3.1 "Separator Tokens", Section 4.3): given dO, the
 * inputs and the forward's O and LSE, writes dQ [B][Hq][L][d] and dK, dV
 * [B][Hkv][L][d] (summed over the query heads sharing a KV head) in
 * desc->grad_dtype.  Deterministic: no floating-point atomics.  workspace dev
 * bwd_bytes, 256-byte aligned. */
sepllm_status sepllm_attn_bwd(const sepllm_attn_desc* desc, const sepllm_index_desc* idesc,
                              const void* dO, const void* Q, const void* K, const void* V,
                              const void* O, const float* LSE, const void* index, void* dQ,
                              void* dK, void* dV, void* workspace, void* stream);

/* ---- streaming cache (Section 3.3, Tailored Streaming Design) --------------
 * Kc and Vc are bf16 [B][Hkv][slots][d] with slots = c + s: slots [0,a) are the
 * Initial Cache, [a, a+s) a ring holding the Separator Cache, [a+s, c+s) a ring
 * holding the neighbour run whose newest w entries are the Local Window Cache
 * and whose older entries are the Past Window Cache.  `state` holds the sizes,
 * ring starts, per-slot token position (int64) and separator flag of every
 * sequence; its first word is the device status.  Saving and restoring a cache
 * is a copy of state, Kc and Vc.
 */
#define SEPLLM_CACHE_MAGIC 0x48434353u /* "SCCH" */
typedef struct {
  int32_t status;                /* device status word (first word) */
  uint32_t magic, version;
  int32_t slots;                 /* c + s */
  sepllm_cache_desc desc;
  int64_t off_seq, off_slot_pos, off_slot_is_sep, total_bytes;
  int64_t reserved[21];
} sepllm_cache_header; /* 256 bytes */

/* Per-sequence record inside the state, 16 int32.  reserved[0] is a scratch
 * counter of sepllm_cache_update (zero between calls); the rest is zero. */
typedef struct {
  int32_t size_init, sep_start, size_sep, win_start, size_win, compactions;
  int64_t next_pos;              /* tokens seen so far */
  int32_t reserved[8];
} sepllm_cache_seq;

/* state_bytes: the state buffer; kv_bytes: ONE of Kc / Vc. */
sepllm_status sepllm_cache_bytes(const sepllm_cache_desc* desc, size_t* state_bytes,
                                 size_t* kv_bytes);

/* Empties the cache (writes the whole state buffer). */
sepllm_status sepllm_cache_init(const sepllm_cache_desc* desc, void* state, void* stream);

/* Takes in one token per sequence: fills the Initial Cache first, then appends
 * to the neighbour run; when Size_run reaches c the separators of the Past
 * Window Cache move, in position order, to the Separator Cache, which drops its
 * oldest entries beyond s, and the other Past Window entries are dropped.
 *   new_token_ids dev int32 [B]; sep_ids host int32 [n_sep];
 *   k_new, v_new dev bf16 [B][Hkv][d]. */
sepllm_status sepllm_cache_update(const sepllm_cache_desc* desc, void* state, void* Kc, void* Vc,
                                  const int32_t* new_token_ids, const int32_t* sep_ids,
                                  int32_t n_sep, const void* k_new, const void* v_new,
                                  void* stream);

/* Hand-off from pre-filling to generation (Section 3.2: after the prompt only
 * the K/V of initial, separator and neighbouring tokens are kept; Section 3.3
 * for the four blocks).  Fills the cache with what the first prompt_len[b]
 * tokens of sequence b leave behind: the same sizes, retained positions (in the
 * same order), separator flags, compaction count and K/V rows as giving those
 * tokens one by one to sepllm_cache_update on an empty cache, with both rings
 * starting at their first slot.  The separator flag of an Initial Cache slot,
 * which no call reads, is written as 0.  sepllm_cache_update and the decode
 * calls continue from the result.
 *   idesc, index   the index built from the prompts' token ids with
 *                  n_init = desc->a and B = desc->B (its n_neighbor and tiles
 *                  play no part; the prefix counts and the side list are read,
 *                  and a side list cut short by side_cap is made up for from
 *                  the counts)
 *   prompt_len     dev int32 [B], 0 <= prompt_len[b] <= L; NULL = L for all
 *   K, V           dev bf16 [B][Hkv][L][d], the prompt's keys and values
 *   state, Kc, Vc  as for sepllm_cache_update; written in full / in every
 *                  retained slot (no sepllm_cache_init needed before)
 *   Kr, rope_table NULL, or the rotated key buffer and the table of
 *                  sepllm_cache_update_rope below: Kr is then filled as well
 * A prompt_len outside [0, L], or an index that was not built for idesc, leaves
 * that sequence's cache empty and SEPLLM_INVALID_ARG in the device status. */
sepllm_status sepllm_cache_from_prompt(const sepllm_cache_desc* desc,
                                       const sepllm_index_desc* idesc, const void* index,
                                       const int32_t* prompt_len, const void* K, const void* V,
                                       void* state, void* Kc, void* Vc, void* Kr,
                                       const void* rope_table, void* stream);

/* The decode workspace holds the per-split partial results; its status word is
 * always written as 0 (the decode kernels contain no bounded wait and clamp
 * nothing). */
sepllm_status sepllm_decode_workspace_bytes(const sepllm_cache_desc* desc, size_t* bytes);

/* One query per sequence over every retained entry (Section 3.2 "Generation",
 * Section 3.3): o = softmax(q Kc^T * scale) Vc.  q dev bf16 [B][Hq][d]; o dev bf16
 * [B][Hq][d]; lse dev fp32 [B][Hq] (may be NULL); scale 0 = 1/sqrt(d). */
sepllm_status sepllm_decode(const sepllm_cache_desc* desc, float scale, const void* q,
                            const void* state, const void* Kc, const void* Vc, void* o,
                            float* lse, void* workspace, void* stream);

/* Generation with positions taken inside the cache (Section 3.3, "Positional
 * Encoding": as in StreamingLLM, the streaming setting uses an entry's place in
 * the cache, not its place in the text; Table 8 shows the effect of leaving
 * this out).  Keys and queries are handed over un-rotated.  The retained
 * entries, walked as initial, separator (oldest first), neighbour (oldest
 * first), have positions 0 .. Size_run-1 and the query has Size_run-1.  The
 * paper fixes no rotary formula; this library uses the rotate-half form:
 * with theta_i = base^(-2i/d), i < d/2, a vector x at position p becomes
 *   y[i]       = x[i] cos(p theta_i) - x[i + d/2] sin(p theta_i)
 *   y[i + d/2] = x[i + d/2] cos(p theta_i) + x[i] sin(p theta_i).
 * rope_table holds (cos, sin) as fp32 pairs [c][d/2]: size it with
 * sepllm_rope_table_bytes and fill it once per (desc, base) with
 * sepllm_rope_table_build (dev, 16-byte aligned).
 *
 * Kr is a second key buffer of Kc's size and layout (dev bf16, 16-byte
 * aligned, caller-owned) in which every retained key stands rotated to its
 * current position, computed in fp32 from the un-rotated key in Kc and rounded
 * to bf16 once, however many compactions the key has been through.
 * sepllm_cache_update_rope does what sepllm_cache_update does and keeps Kr
 * current: an update without compaction moves no entry, so it rotates the new
 * key only; a compaction shifts every entry behind the Initial Cache, and the
 * call rewrites those rows of Kr from Kc.  Use it for every update of a cache
 * that is decoded with sepllm_decode_rope (sepllm_cache_from_prompt fills Kr
 * when given it).  sepllm_decode_rope rotates q to position Size_run-1, rounds
 * it to bf16 and attends over Kr and Vc; other arguments as sepllm_decode. */
sepllm_status sepllm_rope_table_bytes(const sepllm_cache_desc* desc, size_t* bytes);
sepllm_status sepllm_rope_table_build(const sepllm_cache_desc* desc, float rope_base, void* table,
                                      void* stream);
sepllm_status sepllm_cache_update_rope(const sepllm_cache_desc* desc, void* state, void* Kc,
                                       void* Vc, void* Kr, const void* rope_table,
                                       const int32_t* new_token_ids, const int32_t* sep_ids,
                                       int32_t n_sep, const void* k_new, const void* v_new,
                                       void* stream);
sepllm_status sepllm_decode_rope(const sepllm_cache_desc* desc, float scale, const void* q,
                                 const void* state, const void* Kr, const void* Vc,
                                 const void* rope_table, void* o, float* lse, void* workspace,
                                 void* stream);

/* Copies the device status word at the start of an index, workspace or state
 * buffer to *out (host) after synchronising `stream`. */
sepllm_status sepllm_last_device_status(const void* buffer, int32_t* out, void* stream);

const char* sepllm_status_string(sepllm_status);

#ifdef __cplusplus
}
#endif
#endif /* SEPLLM_H_ */
