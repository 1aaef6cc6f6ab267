/*
 * wmtp.h -- C ABI of the Windowed-MTP draft-attention library (single GPU, sm_100a).
 *
 * The library implements the draft head's GQA decode attention over its KV cache in the two
 * forms the paper compares: windowed (attention sink + the last W tokens, kept in a compact
 * ring buffer; Section 4 "Mechanism" and "Memory", Appendix A pseudocode) and full context
 * (the native-MTP draft that re-reads all S keys at every draft step; Section 3).
 *
 * Conventions for every call
 *  - Pointers marked "device" are CUDA device memory owned by the caller; the library
 *    allocates nothing on the device and keeps no reference after the call's work has run.
 *    Process-wide state: a launch counter, per-device caches of device attributes, and the three
 *    test knobs at the end of this file (wmtp_set_max_ctas, wmtp_set_work_stealing,
 *    wmtp_set_wait_limit); nothing else outlives a call.
 *    Descriptors (wmtp_ring, wmtp_kv) are plain host structs, read during the call only.
 *  - bf16 tensors are row-major with head_dim D contiguous; base pointers 16-byte aligned.
 *  - `stream` is a cudaStream_t passed as void*. Calls only enqueue work on it; nothing
 *    synchronises except wmtp_device_status and the *_host loop variants.
 *  - Sequence lengths live in device memory (`len`), are advanced by the append kernels and
 *    read by the attention kernels, so a chain of calls needs no host round trip.
 *  - Return value: WMTP_OK or an error; nothing is launched when an argument is rejected.
 *    wmtp_last_error() gives a thread-local detail string. Problems only visible on the
 *    device (a page id out of range, an append past capacity, a bounded wait that expired)
 *    set a sticky word in the workspace, the kernel skips the offending access, and
 *    wmtp_device_status reports it.
 *  - Query head h reads KV head h / (Hq / Hkv). Supported: D in {128, 256}, Hq / Hkv in [1, 8].
 *  - sm_scale <= 0 selects 1 / sqrt(D).
 */
#ifndef WMTP_H_
#define WMTP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WMTP_OK = 0,
    WMTP_ERR_INVALID_ARG = 1,    /* NULL / misaligned pointer, non-positive size, Hq % Hkv != 0, cap < W ... */
    WMTP_ERR_UNSUPPORTED = 2,    /* head_dim or group size the kernels are not built for */
    WMTP_ERR_CAPACITY = 3,       /* a length would exceed the ring / KV capacity */
    WMTP_ERR_WORKSPACE = 4,      /* workspace missing, misaligned or too small */
    WMTP_ERR_CUDA = 5,           /* a CUDA runtime / driver call failed (no device, launch error) */
    WMTP_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait expired; outputs of that call are invalid and the workspace
                                    must be initialised again (wmtp_workspace_init) before it is reused */
    WMTP_ERR_DEVICE_BOUNDS = 7   /* a device-side index check failed (page id, append past capacity) */
} wmtp_status;

/*
 * Entry type of a KV store (ring or full-context). WMTP_KV_BF16: bf16 values. WMTP_KV_FP8_E4M3: the fp8-KV variant
 * (Section 6, "Robustness to KV-cache quantization": the KV dtype only sets the bytes per entry, the key set and the
 * attention are unchanged): every entry is one e4m3 code (1 sign, 4 exponent, 3 mantissa bits; no infinities, largest
 * finite value 448) and stands for code_value * k_scale[g] (resp. v_scale[g]) with g its KV head. Layouts, shapes and
 * alignment rules are the same with 1-byte entries. q, k_new, v_new and out stay bf16: the append calls (and the
 * appends fused into the draft loops) quantise a new row as code = e4m3(x / scale[g]) -- fp32 division, round to
 * nearest even, magnitudes beyond 448 saturate -- and the attention kernels widen the codes exactly and apply the
 * scales to the scores and to the read-out. NaN codes are not valid store contents.
 */
typedef enum { WMTP_KV_BF16 = 0, WMTP_KV_FP8_E4M3 = 1 } wmtp_kv_dtype;

/* Bytes per entry of a store of that type (2 or 1); 0 for an unknown type. */
size_t wmtp_kv_elem_bytes(int kv_dtype);

/*
 * Ring-buffer draft KV store (Section 4 "Memory": the draft KV is kept in a compact
 * n_sink + W + d ring; Appendix A: slot = ring_base(r) + logical position under a modulus).
 * Per sequence r the store has n_sink fixed sink slots followed by `cap` window slots used
 * circularly: position p lives in slot p if p < n_sink, else n_sink + ((p - n_sink) mod cap).
 * cap == W is the plain window; cap = W + d reserves the paper's d slots of slack. The draft
 * attends over the sink slots and the slots holding the last W positions.
 */
typedef struct wmtp_ring {
    void*    k;         /* device bf16 [batch][Hkv][n_sink + cap][D] */
    void*    v;         /* device bf16 [batch][Hkv][n_sink + cap][D] */
    int32_t* slot_pos;  /* device [batch][n_sink + cap]: logical position held by each slot, -1 = never written
                           (32 bits: the bookkeeping is exact for logical lengths up to 2^31 - 1 tokens) */
    int64_t* len;       /* device [batch]: logical sequence length S (tokens appended so far) */
    int32_t  batch, Hkv, D, n_sink, W, cap;
    int32_t  kv_dtype;        /* wmtp_kv_dtype; 0 (bf16) keeps the fields below unused */
    const float* k_scale;     /* device fp32 [Hkv], WMTP_KV_FP8_E4M3 only: positive, finite */
    const float* v_scale;     /* device fp32 [Hkv] */
} wmtp_ring;

/*
 * Full-context draft KV (the native draft's cache, Section 3).
 * Contiguous layout (page_table == NULL): bf16 [batch][Hkv][S_cap][D].
 * Paged layout: pool bf16 [num_pages][Hkv][page_size][D]; token p of sequence r lives in page
 * page_table[r][p / page_size] at row p % page_size. page_size must be 64.
 */
typedef struct wmtp_kv {
    void*          k;
    void*          v;
    const int32_t* page_table; /* device [batch][max_pages], or NULL */
    int64_t*       len;        /* device [batch] */
    int64_t        S_cap;      /* host-known capacity in tokens per sequence (contiguous: row count; paged: max_pages * page_size) */
    int32_t        batch, Hkv, D, page_size, max_pages, num_pages;
    int32_t        kv_dtype;   /* wmtp_kv_dtype */
    const float*   k_scale;    /* device fp32 [Hkv], WMTP_KV_FP8_E4M3 only */
    const float*   v_scale;
} wmtp_kv;

const char* wmtp_status_string(wmtp_status s); /* static storage */
const char* wmtp_last_error(void);             /* thread-local, valid until the thread's next failing call */

/* Bytes of the ring's K (== V) tensor (bf16 entries; an fp8 ring needs half) and of slot_pos, for the caller's
 * allocation. Returns k_bytes. */
size_t wmtp_ring_bytes(int batch, int Hkv, int D, int n_sink, int cap, size_t* pos_bytes);

/*
 * Workspace for the attention calls: split-KV partial results, their completion counters and
 * the sticky device status word. Size depends only on (batch, Hq, Hkv, D). The workspace must be
 * 256-byte aligned and initialised once with wmtp_workspace_init before its first use; after that
 * the kernels leave it ready for the next call, whatever its shape: one workspace sized for the
 * largest (batch, Hq, Hkv, D) serves decode steps and draft-extend launches in any order. Calls
 * sharing one workspace must be ordered on one stream.
 */
size_t      wmtp_workspace_bytes(int batch, int Hq, int Hkv, int D);
wmtp_status wmtp_workspace_init(void* workspace, size_t ws_bytes, void* stream);

/* Synchronises `stream`, then returns (and clears) the sticky device status of the workspace. */
wmtp_status wmtp_device_status(void* workspace, void* stream);

/* ---- ring store -------------------------------------------------------------------------- */

/* len = 0, every slot_pos = -1 (K/V bytes are left as they are). */
wmtp_status wmtp_ring_reset(const wmtp_ring* ring, void* stream);

/*
 * Snapshot and restore of a ring. The paper defines no checkpoint format: this is the store of Appendix A (RING) copied
 * as it stands -- K rows, V rows, slot_pos, len, in that order, each starting on a 256-byte boundary of the blob.
 * wmtp_ring_state_bytes: size of the snapshot (0 for an invalid descriptor). wmtp_ring_export copies the four arrays
 * into `blob`, wmtp_ring_import copies them back into a ring of the same geometry (batch, Hkv, D, n_sink, cap,
 * kv_dtype are the caller's to keep; only the size is checked; the scales of an fp8 ring are not part of the state).
 * `blob` is device memory or page-locked host memory, 16-byte aligned, blob_bytes >= wmtp_ring_state_bytes(ring);
 * the copies are asynchronous on `stream`. A ring restored from a snapshot taken between two draft steps continues
 * bit-identically.
 */
size_t      wmtp_ring_state_bytes(const wmtp_ring* ring);
wmtp_status wmtp_ring_export(const wmtp_ring* ring, void* blob, size_t blob_bytes, void* stream);
wmtp_status wmtp_ring_import(const wmtp_ring* ring, const void* blob, size_t blob_bytes, void* stream);

/*
 * Seeds the ring from a context KV holding S = kv->len[r] tokens per sequence: copies positions
 * [0, min(S, n_sink)) and [max(n_sink, S - cap), S) into their slots, sets slot_pos and len = S.
 * The result is bit-identical to S sequential wmtp_ring_append calls (Section 6, "Prefill
 * sparsification": only O(W + n_sink) of the context is needed by the windowed draft).
 * Rows are copied as stored: ring and kv must have the same kv_dtype and, for fp8, equal scales.
 * The call has no workspace to flag device-side findings in: a position whose page id lies outside [0, num_pages)
 * is not copied and its slot is marked empty (slot_pos = -1) while len is still set to S; callers that cannot vouch for
 * their page table check it first (wmtp_reduced_block_table and wmtp_kv_append flag bad ids in a workspace).
 */
wmtp_status wmtp_ring_init_from_kv(const wmtp_ring* ring, const wmtp_kv* kv, void* stream);

/*
 * Appends one token per sequence (Appendix A, RING): p = len[r]; the K/V rows k_new, v_new
 * (device bf16 [batch][Hkv][D]) go to the slot of position p, slot_pos[slot] = p, len[r] = p + 1.
 */
wmtp_status wmtp_ring_append(const wmtp_ring* ring, const void* k_new, const void* v_new, void* stream);

/* Same for the full-context KV: writes position p = len[r] (through the page table if paged), len[r] = p + 1.
 * A position beyond S_cap, or a page id outside [0, num_pages), is skipped and flagged in `workspace` (may be NULL). */
wmtp_status wmtp_kv_append(const wmtp_kv* kv, const void* k_new, const void* v_new, void* workspace, void* stream);

/* ---- draft attention --------------------------------------------------------------------- */

/*
 * Windowed draft attention (Section 4 "Mechanism"; Appendix A): for each sequence, one query
 * per head attends over the first n_sink tokens and the last W tokens, read from the ring
 * (all of it when S <= n_sink + W). q: device bf16 [batch][Hq][D]; out: device bf16
 * [batch][Hq][D]; lse: device fp32 [batch][Hq] (natural-log sum of exp of the scaled logits)
 * or NULL. Softmax in fp32; split-KV partials are merged by log-sum-exp.
 * A sequence of length 0 yields out = 0, lse = -inf.
 */
wmtp_status wmtp_draft_attn_windowed(const void* q, int Hq, const wmtp_ring* ring, float sm_scale,
                                     void* out, float* lse, void* workspace, size_t ws_bytes, void* stream);

/* Full-context draft attention (Section 3: the native draft re-reads all S keys): same, over positions [0, len[r]). */
wmtp_status wmtp_draft_attn_full(const void* q, int Hq, const wmtp_kv* kv, float sm_scale,
                                 void* out, float* lse, void* workspace, size_t ws_bytes, void* stream);

/*
 * gamma sequential draft steps on one stream (Section 3, Eq. 1: gamma draft forwards per decode
 * step): for i in [0, gamma): append(k_new[i], v_new[i]) then attention(q[i]) -> out[i].
 * q: device bf16 [gamma][batch][Hq][D]; k_new, v_new: device bf16 [gamma][batch][Hkv][D];
 * out: device bf16 [gamma][batch][Hq][D]; lse: device fp32 [gamma][batch][Hq] or NULL.
 */
wmtp_status wmtp_draft_loop_windowed(const wmtp_ring* ring, int gamma, const void* q, int Hq,
                                     const void* k_new, const void* v_new, float sm_scale,
                                     void* out, float* lse, void* workspace, size_t ws_bytes, void* stream);
wmtp_status wmtp_draft_loop_full(const wmtp_kv* kv, int gamma, const void* q, int Hq,
                                 const void* k_new, const void* v_new, float sm_scale,
                                 void* out, float* lse, void* workspace, size_t ws_bytes, void* stream);

/*
 * The same loops for a caller whose step inputs and outputs live in HOST memory (pinned memory
 * makes the copies asynchronous): q, k_new, v_new are copied to the device staging buffer
 * `stage` (device, at least wmtp_stage_bytes, 256-byte aligned), the loop runs, `out` (and `lse`
 * if not NULL) are copied back to the host pointers, and the stream is synchronised before
 * returning. The KV cache / ring stay device-resident: they are state, not step inputs.
 */
size_t      wmtp_stage_bytes(int gamma, int batch, int Hq, int Hkv, int D);
wmtp_status wmtp_draft_loop_windowed_host(const wmtp_ring* ring, int gamma, const void* q_host, int Hq,
                                          const void* k_new_host, const void* v_new_host, float sm_scale,
                                          void* out_host, float* lse_host, void* stage,
                                          void* workspace, size_t ws_bytes, void* stream);
wmtp_status wmtp_draft_loop_full_host(const wmtp_kv* kv, int gamma, const void* q_host, int Hq,
                                      const void* k_new_host, const void* v_new_host, float sm_scale,
                                      void* out_host, float* lse_host, void* stage,
                                      void* workspace, size_t ws_bytes, void* stream);

/* ---- windowed attention straight from the KV store (no ring) ----------------------------------- */

/*
 * The paper's own realisation of the window (Section 4 "Mechanism"; Appendix A pseudocode): the draft keeps its
 * full-length KV, and each draft step attends over a reduced key set taken from it -- the first n_sink positions and
 * the last W positions, [0, S) when S <= n_sink + W -- which in a paged store is the per-request block table reduced
 * to [sink blocks] || [recent-W blocks]. Here the reduced table is never materialised: the kernel walks the sink
 * tiles and the tiles of the last W tokens through the page table (or the contiguous rows) arithmetically, O(W) per
 * step, and masks the ragged ends row by row, so the window is token-granular whatever the page size. Same result as
 * wmtp_draft_attn_windowed on a ring that holds the same tokens; arguments as wmtp_draft_attn_full plus n_sink >= 0,
 * W >= 1.
 */
wmtp_status wmtp_draft_attn_windowed_kv(const void* q, int Hq, const wmtp_kv* kv, int n_sink, int W, float sm_scale,
                                        void* out, float* lse, void* workspace, size_t ws_bytes, void* stream);

/* gamma draft steps on the KV store: append (k_new[i], v_new[i]) at position len, then attend over sink + last W. */
wmtp_status wmtp_draft_loop_windowed_kv(const wmtp_kv* kv, int n_sink, int W, int gamma, const void* q, int Hq,
                                        const void* k_new, const void* v_new, float sm_scale, void* out, float* lse,
                                        void* workspace, size_t ws_bytes, void* stream);

/*
 * The reduced block table itself, for callers that run another paged attention backend through it (the paper's
 * deployment, Section 4 "Mechanism": table = [sink blocks] || [recent-W blocks]). Paged stores only. Per sequence r with
 * S = len[r]: table[r][0 .. n_s) = pages of the sink positions [0, min(S, n_sink)), table[r][n_s .. n_s + n_w) = pages of
 * the window positions [max(min(S, n_sink), S - W), S), remaining entries -1; a page holding both kinds appears in both
 * parts. meta[r][0..5) = { n_s, n_w, rows used in the last sink page, first row used in the first window page, rows
 * used in the last window page }: the ends stay token-granular. table: device int32 [batch][table_stride],
 * table_stride >= wmtp_reduced_block_table_width(n_sink, W, page_size) = ceil(n_sink/ps) + ceil(W/ps) + 1;
 * meta: device int32 [batch][5]. O((n_sink + W) / page_size) work per sequence, no host arithmetic on S (the O(S)
 * per-step index construction the paper removes has no counterpart in this library: the attention kernels index the
 * stores arithmetically). A page id outside [0, num_pages) is written as -1 and flagged in `workspace` (may be NULL).
 */
int         wmtp_reduced_block_table_width(int n_sink, int W, int page_size);
wmtp_status wmtp_reduced_block_table(const wmtp_kv* kv, int n_sink, int W, int32_t* table, int table_stride, int32_t* meta,
                                     void* workspace, void* stream);

/*
 * The O(S) counterpart, for comparison: the pool row of every token of a paged store, which a full-context (native)
 * draft rebuilds before every attention call (Section 3, t_ctx; Appendix B, per-kernel table: the draft's KV index
 * build). index[r][s] = page_table[r][s / page_size] * page_size + s mod page_size for s < len[r], -1 for
 * len[r] <= s < index_stride; `index` is device int32 [batch][index_stride]. A length beyond index_stride or a page id
 * outside the pool is flagged WMTP_ERR_DEVICE_BOUNDS in `workspace` (may be NULL) and the entry is -1. The attention
 * entry points of this library never need it (they walk the page table arithmetically); it exists so that the O(S)
 * and the O(W) structure can be timed side by side.
 */
wmtp_status wmtp_full_token_index(const wmtp_kv* kv, int32_t* index, int64_t index_stride, void* workspace, void* stream);

/* ---- after verification: rollback and draft-extend -------------------------------------------- */

/*
 * A decode step ends with the target accepting some of the proposed tokens. The draft then (a) discards the K/V of the
 * rejected ones -- the ring reserves d slots of slack for exactly this (Section 4 "Memory"; Section 6 "Compatibility
 * with tree speculation": n_sink + W + d) -- and (b) re-processes the accepted tokens in one "draft-extend" pass,
 * several new tokens per sequence at once, each attending causally up to itself (Section 5 "The backend is not the
 * confound"; Appendix B, per-kernel table).
 *
 * wmtp_ring_rewind: drops the last n_drop[r] tokens of every sequence (device int32 [batch]): len shrinks and the
 *   slots of the dropped positions get slot_pos = -1. Requires 0 <= n_drop[r] <= min(len[r], cap - W): the rows those
 *   tokens overwrote are then outside every later window. A violation is flagged in `workspace` (may be NULL) and the
 *   sequence is left unchanged. The bound is on the distance below the longest length the sequence has reached:
 *   the kernel checks each call by itself, so a caller that rewinds twice without appending in between keeps the
 *   sum within cap - W.
 * wmtp_ring_append_many / wmtp_kv_append_many: n_tok tokens per sequence in one launch; k_new, v_new are device bf16
 *   [batch][n_tok][Hkv][D]; token j goes to position len + j; len += n_tok (all or nothing for the KV store).
 * wmtp_ring_replace_tail: both in one launch, the draft's state update after a verify step: drops the last n_drop[r]
 *   tokens (n_drop may be NULL: none), then appends n_tok tokens at the positions that follow; slots of dropped
 *   positions that are not rewritten get slot_pos = -1. Same conditions and error behaviour as wmtp_ring_rewind.
 * wmtp_draft_extend_windowed / _full: q is device bf16 [batch][q_len][Hq][D]; the q_len tokens must already be in the
 *   store. Query i of a sequence attends as a decode step would have at length len - (q_len - 1 - i): over sink + last W
 *   of that length (windowed; needs cap >= W + q_len - 1) or over all positions below it (full). out: device bf16
 *   [batch][q_len][Hq][D]; lse: device fp32 [batch][q_len][Hq] or NULL. The workspace must be sized for
 *   batch * q_len sequences: wmtp_workspace_bytes(batch * q_len, Hq, Hkv, D). The windowed form is one launch (the
 *   ring is L2-resident; each query reads it). The full-context form reads every K/V tile from HBM once for up to four
 *   queries of a sequence (one attention launch and one small merge launch; bf16 and fp8 stores); only a batch whose
 *   per-sequence tables do not fit the kernel's shared memory is served query by query in a single launch.
 */
wmtp_status wmtp_ring_rewind(const wmtp_ring* ring, const int32_t* n_drop, void* workspace, void* stream);
wmtp_status wmtp_ring_append_many(const wmtp_ring* ring, int n_tok, const void* k_new, const void* v_new, void* stream);
wmtp_status wmtp_ring_replace_tail(const wmtp_ring* ring, const int32_t* n_drop, int n_tok, const void* k_new, const void* v_new,
                                   void* workspace, void* stream);
wmtp_status wmtp_kv_append_many(const wmtp_kv* kv, int n_tok, const void* k_new, const void* v_new, void* workspace,
                                void* stream);
wmtp_status wmtp_draft_extend_windowed(const void* q, int q_len, int Hq, const wmtp_ring* ring, float sm_scale, void* out,
                                       float* lse, void* workspace, size_t ws_bytes, void* stream);
wmtp_status wmtp_draft_extend_full(const void* q, int q_len, int Hq, const wmtp_kv* kv, float sm_scale, void* out,
                                   float* lse, void* workspace, size_t ws_bytes, void* stream);

/* ---- diagnostics ------------------------------------------------------------------------------ */

/*
 * Attention-mass diagnostics of a windowed against a full-context read-out of the same queries (Appendix D, the
 * attention-mass table), from the outputs of wmtp_draft_attn_windowed and wmtp_draft_attn_full. Per row
 * (sequence, query head), rows = batch * Hq:
 *   mass[r]    = exp(lse_win - lse_full)                 share of the softmax mass inside sink + window
 *   perturb[r] = ||o_full - o_win|| / ||o_full||           relative L2 change of the read-out when the far keys are dropped
 *   tail[r]    = ||o_full - mass * o_win|| / ||o_full||    share of the read-out norm contributed by the far keys
 *                (o_full = mass * o_win + (1 - mass) * o_far)
 * out_*: device bf16 [rows][D]; lse_*: device fp32 [rows]; mass / perturb / tail: device fp32 [rows], any may be NULL.
 */
wmtp_status wmtp_attn_mass_diagnostics(const void* out_win, const float* lse_win, const void* out_full, const float* lse_full,
                                       int rows, int D, float* mass, float* perturb, float* tail, void* stream);

/* ---- tuning and accounting ---------------------------------------------------------------- */

/* Upper bound on the CTAs (KV splits) of the attention kernels; 0 restores the default (up to one CTA per SM).
 * Windowed launches, which run one thread-block cluster per (sequence, KV head), take the largest cluster size that
 * keeps the launch within the bound (never less than one CTA per pair). Process-wide; meant for tests that exercise
 * the split/merge paths. */
void    wmtp_set_max_ctas(int max_ctas);
/* Tile-level work stealing between CTAs (default on): SMs that stream faster take tiles from slower ones, which
 * shortens long launches by several percent but makes the low bits of the result depend on timing. 0 selects a
 * fixed partition: bit-reproducible results. Process-wide. */
void    wmtp_set_work_stealing(int enabled);
/* Polls a CTA of the attention kernels spends waiting for a word another CTA of the same launch writes (a segment's
 * arrival count, the end-of-launch count) before it gives up, flags WMTP_ERR_DEVICE_TIMEOUT in the workspace and
 * carries on to the end of the kernel; 0 restores the default (2^22 polls, seconds). Waits on the kernel's own
 * shared-memory barriers are not affected. Process-wide; meant for tests of the give-up path: with a limit of one
 * poll a multi-CTA launch reports the timeout, its outputs are invalid and the workspace needs wmtp_workspace_init. */
void    wmtp_set_wait_limit(int polls);
/* Number of kernels this library has launched in this process (all threads). */
int64_t wmtp_launch_count(void);

/* ---- for callers that cannot allocate device memory --------------------------------------------- */

/*
 * (The paper has no counterpart to this entry point; it exists for integration.)
 * Windowed draft attention, same result as wmtp_draft_attn_windowed, for callers that cannot give the
 * library a workspace because they cannot allocate device memory themselves: plug-ins inside a runtime
 * that owns the allocator, processes whose device-memory budget is frozen at start-up, loops that must
 * not allocate once they are running. The split-KV scratch is a fixed array inside the library
 * (about 4 MiB, held by every GPU that loads the library until the process exits); the call, and the
 * library on its behalf, performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   - Limits: batch * Hkv <= 32, Hq / Hkv <= 8, D in {128, 256}; more is rejected with
 *     WMTP_ERR_CAPACITY / WMTP_ERR_UNSUPPORTED and nothing is launched. At most 160 CTAs are used.
 *   - The first call on each device looks up the array's device address (a one-time set-up, with that
 *     device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the call
 *     clears the words that must start at zero. Two calls whose GPU work can overlap (different
 *     streams without ordering) race on it: order them on one stream or with events.
 *   - The sticky device status lives in the array too and is cleared at the start of each call; it is
 *     not reported. The windowed path has no page table whose ids could be out of range; a bounded
 *     device-side wait that expired goes unnoticed here, so callers that need that report use the
 *     workspace form and wmtp_device_status.
 * Arguments as wmtp_draft_attn_windowed, without workspace.
 */
wmtp_status wmtp_draft_attn_windowed_noalloc(const void* q, int Hq, const wmtp_ring* ring, float sm_scale,
                                             void* out, float* lse, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* WMTP_H_ */
