/*
 * libmala -- C ABI of the B200 (sm_100a) MassAlloc Attention (MALA) hot path.
 *
 * The operator is the one the paper's Methodology section states for a query head and its
 * key/value head: QK^T scores are formed for every legal causal tile; a forward tile is skipped
 * when, for every relevant row, rowmax(S) - m - log(l) < log(tau / L_q) (Eq. 3, Algorithm 1);
 * a backward tile is skipped when S - lse < log(tau / L_q) on all its valid entries (Eq. 4,
 * Algorithm 2); split-KV decode applies the forward rule per split against the split's partial
 * normalizer with L = N_k and merges the partials ("Fused decoding execution").  tau = 0 selects
 * the dense FullAttn kernels (Section 2.3: tau -> 0 recovers FullAttn).
 *
 * Conventions common to all calls
 *   - Every pointer is a DEVICE pointer owned by the caller unless stated otherwise; the library
 *     never frees or retains one.  Tensors are bf16 views [B, N, H, d] given as a base pointer and
 *     element strides (sb, sn, sh); the last dimension is contiguous.  Base pointers must be
 *     16-byte aligned and all strides multiples of 8 elements (16 bytes).
 *   - d is a multiple of 8 between 8 and 256 for the forward calls (mala_fwd*) and the decode calls on a bf16 cache
 *     (mala_decode, _multi, _paged, _static), between 8 and 128 for the backward calls and a multiple of 16 up to
 *     128 for the calls on an e4m3 cache (the paper's symbols put no limit on d_h, Section 2.1; its models use 128).
 *     The kernels exist for 64, 128 and 256 columns; another head size runs on the next of them at that size's cost
 *     (the missing columns are read as zeros and never stored).
 *     Hq must be a multiple of Hkv; query head h uses key/value head h / (Hq / Hkv).  N may be any positive length (the last tile may be ragged).
 *   - scale (> 0, finite) multiplies the fp32 scores; lse is in nats, of the scaled scores, over
 *     the retained set.  tau >= 0, finite.
 *   - Tile partition: mala_tile_shape() reports it; forward and backward use the same partition.
 *   - Two environment variables, read once per process, change what a call does around its launches (both off by
 *     default): MALA_NVTX=1 makes every launching call an NVTX range of its own name; MALA_DEBUG=1 makes error
 *     reporting synchronous -- the call waits for its stream and returns MALA_ERR_CUDA or MALA_ERR_DEVICE_TIMEOUT
 *     itself (with a line on stderr) instead of leaving the error to a later call.  A debug call therefore
 *     synchronises, which a call otherwise never does.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t, may be NULL for the default
 *     stream), allocate nothing and never synchronise.  `ws` is caller-provided scratch of at
 *     least mala_workspace_bytes() bytes, 256-byte aligned; its contents are undefined afterwards.
 *   - Return value: MALA_OK or a negative MALA_ERR_* code; nothing is launched on error.
 *     A bounded device-side wait that expires does not hang: the kernels finish, later launches
 *     become no-ops, and mala_device_status() reports MALA_ERR_DEVICE_TIMEOUT until cleared.
 */
#ifndef MALA_H_
#define MALA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MALA_OK 0
#define MALA_ERR_INVALID_ARG (-1)        /* NULL pointer, non-positive size, bad tau / scale */
#define MALA_ERR_UNSUPPORTED (-2)        /* d not a multiple of 8 in the call's range, Hq % Hkv != 0, too many splits ... */
#define MALA_ERR_MISALIGNED (-3)         /* pointer / stride alignment rules above violated */
#define MALA_ERR_WORKSPACE_TOO_SMALL (-4)
#define MALA_ERR_WRONG_ARCH (-5)         /* current device is not compute capability 10.x */
#define MALA_ERR_CUDA (-6)               /* a CUDA runtime call or launch failed */
#define MALA_ERR_TENSOR_MAP (-7)         /* the driver rejected a TMA tensor map */
#define MALA_ERR_DEVICE_TIMEOUT (-8)     /* a bounded device-side wait expired (status word) */
#define MALA_ERR_STATIC_SCRATCH_EXCEEDED (-9) /* mala_decode_static: problem exceeds the built-in scratch */

/* Size of the scratch array compiled into the library for mala_decode_static (24 MiB per device). */
#define MALA_STATIC_SCRATCH_BYTES (24u << 20)

#define MALA_OP_FWD 0
#define MALA_OP_BWD 1
#define MALA_OP_DECODE 2

typedef struct { const void* p; int64_t sb, sn, sh; } mala_tin;   /* read-only bf16 [B,N,H,d] view */
typedef struct { void* p; int64_t sb, sn, sh; } mala_tout;        /* written bf16 [B,N,H,d] view */

/* Optional telemetry (any member may be NULL; the struct pointer itself may be NULL).
 *   retained_per_block : u32, overwritten.  fwd [B,Hq,Tr] (per query block), bwd [B,Hq,Tc] (per key
 *                        block and query head), decode [B,Hkv,num_splits].
 *   tile_bitmask       : u32 words, overwritten.  fwd [B,Hq,Tr,ceil(Tc/32)], bit j of row i set iff
 *                        tile (i,j) was retained; bwd [B,Hq,Tc,ceil(Tr/32)], bit i of row j;
 *                        decode [B,Hkv,num_splits,ceil(tiles_per_split/32)].  Meant for parity checks.
 *   totals             : u64[2], ACCUMULATED: += retained tiles, += legal (visited) tiles. */
typedef struct {
  uint32_t* retained_per_block;
  uint32_t* tile_bitmask;
  uint64_t* totals;
} mala_stats;

/* Algorithm 1 (forward / prefill).  q [B,N,Hq,d]; k, v [B,N,Hkv,d]; o [B,N,Hq,d]; lse fp32 [B,Hq,N].
 * causal != 0: equal-length causal attention, L_q = q + 1, tiles visited from the diagonal toward
 * earlier keys.  causal == 0: every key legal, L_q = N, tiles visited from the last to the first. */
int mala_fwd(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B, int Hq,
             int Hkv, int N, int d, int causal, float scale, float tau, void* ws, size_t ws_bytes,
             void* cuda_stream);

/* Algorithm 2 (backward).  o, dout [B,N,Hq,d]; lse as written by mala_fwd; dq [B,N,Hq,d];
 * dk, dv [B,N,Hkv,d] (summed over the query heads of the group).  D = rowsum(O o dO) is computed
 * from the given o.  dQ is accumulated in fp32 in the workspace and converted at the end. */
int mala_bwd(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
             mala_tout dk, mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int N, int d, int causal,
             float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream);

/* Algorithms 1 and 2 with fewer queries than keys (chunked prefill; cross attention when causal == 0).
 * q, o, dout, dq [B,Nq,Hq,d]; k, v, dk, dv [B,Nk,Hkv,d]; lse fp32 [B,Hq,Nq].
 * causal != 0: the queries are the LAST Nq of the Nk positions (Nk >= Nq): query row q attends to the keys
 * 0 .. q + Nk - Nq and L_q = q + 1 + Nk - Nq, the number of keys it sees (Section 2.1); a query block visits its
 * tiles from its diagonal toward earlier keys.  The query blocks follow the key positions -- block i holds the rows q
 * with 128 i <= q + (Nk - Nq) % 128 < 128 (i + 1), so the first block of a chunk that starts inside a tile is a short
 * one -- and the result therefore equals rows Nk - Nq .. Nk - 1 of the equal-length call on the whole sequence wherever
 * the chunk holds a whole block of that call (for the backward: with dout zero on the earlier rows).
 * Both calls take any Nk >= Nq.
 * causal == 0: every key legal for every query, L_q = Nk, any Nq and Nk.
 * Telemetry: fwd retained_per_block [B,Hq,Tq], tile_bitmask [B,Hq,Tq,ceil(ceil(Nk/128)/32)] with
 * Tq = ceil((Nq + (Nk - Nq) % 128) / 128) (causal) or ceil(Nq/128);
 * bwd retained_per_block [B,Hq,ceil(Nk/128)], tile_bitmask [B,Hq,ceil(Nk/128),ceil(Tq/32)].
 * Workspace of the backward: mala_workspace_bytes(MALA_OP_BWD, B, Hq, Hkv, Nq + (Nk - Nq) % 128, d, 0) when causal
 * (the accumulator holds whole query blocks), mala_workspace_bytes(MALA_OP_BWD, B, Hq, Hkv, Nq, d, 0) otherwise.  Everything else as
 * mala_fwd / mala_bwd, which are these calls with Nq = Nk = N. */
int mala_fwd_chunk(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B, int Hq,
                   int Hkv, int Nq, int Nk, int d, int causal, float scale, float tau, void* ws, size_t ws_bytes,
                   void* cuda_stream);
int mala_bwd_chunk(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
                   mala_tout dk, mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int Nq, int Nk, int d,
                   int causal, float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream);

/* mala_fwd_chunk with the keys cut into num_splits ranges that run on different SMs: for a short chunk of queries
 * against a long context (where mala_fwd_chunk has fewer query blocks than the GPU has SMs).  The key blocks
 * 0 .. ceil(Nk/128)-1 are cut into num_splits contiguous ranges of ceil(ceil(Nk/128)/num_splits) blocks; every range
 * runs Algorithm 1 on its blocks with its own running state, i.e. its skip test sees the range's PARTIAL normalizer
 * (the split-local rule of "Fused decoding execution"; more conservative than the unsplit test), and the ranges are
 * merged by lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s.  num_splits = 1 is mala_fwd_chunk; tau = 0
 * gives FullAttn for any num_splits.  Telemetry as for mala_fwd_chunk.  ws: device scratch of
 * mala_workspace_bytes(MALA_OP_FWD, B, Hq, Hkv, Nq, d, num_splits) bytes, 256-byte aligned.  B * num_splits <= 65535. */
int mala_fwd_chunk_split(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B,
                         int Hq, int Hkv, int Nq, int Nk, int d, int causal, float scale, float tau, int num_splits,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Algorithms 1 and 2 on B packed sequences of different lengths (self attention, equal query and key lengths per
 * sequence).  q, o, dout, dq are [1,total,Hq,d] tensors, k, v, dk, dv [1,total,Hkv,d] (sb is ignored); sequence b
 * holds the rows cu_seqlens[b] .. cu_seqlens[b+1]-1; cu_seqlens: device int32 [B+1], non-decreasing, cu_seqlens[0] = 0,
 * cu_seqlens[B] = total; max_seqlen >= every length (it sizes the grid and the telemetry).  Every sequence is treated
 * exactly as a mala_fwd / mala_bwd call on its own rows (its own tile partition, starting at its first row; its own
 * L_q).  lse: fp32 [Hq,total].  Telemetry as for mala_fwd / mala_bwd with N = max_seqlen (rows of blocks a sequence
 * does not have stay zero).  Workspace of the backward:
 * mala_workspace_bytes(MALA_OP_BWD, 1, Hq, Hkv, total + 128 * B, d, 0).  The tile that holds a sequence's last rows
 * also covers the first rows of the next one: those never reach a result, but they must be finite numbers. */
int mala_fwd_varlen(mala_tin q, mala_tin k, mala_tin v, const int32_t* cu_seqlens, mala_tout o, float* lse,
                    const mala_stats* st, int B, int Hq, int Hkv, int total, int max_seqlen, int d, int causal,
                    float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream);
int mala_bwd_varlen(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse,
                    const int32_t* cu_seqlens, mala_tout dq, mala_tout dk, mala_tout dv, const mala_stats* st, int B,
                    int Hq, int Hkv, int total, int max_seqlen, int d, int causal, float scale, float tau, void* ws,
                    size_t ws_bytes, void* cuda_stream);

/* Algorithm 1 on B packed sequences each of which has more keys than queries -- a batch of prefill chunks behind
 * cached prefixes.  q, o [1,total_q,Hq,d] with sequence b in rows cu_seqlens_q[b] .. cu_seqlens_q[b+1]-1; k, v
 * [1,total_k,Hkv,d] with its keys in rows cu_seqlens_k[b] .. cu_seqlens_k[b+1]-1 (both device int32 [B+1]).  Every
 * sequence is treated exactly as a mala_fwd_chunk call on its own rows: causal != 0 puts its queries at its last
 * positions (it must not have more queries than keys: such a sequence is left untouched), its query blocks follow its
 * key positions, L_q is the number of keys the row sees; causal == 0: every key of the sequence legal, L = its number
 * of keys.  max_seqlen_q / max_seqlen_k >= every length.  lse fp32 [Hq,total_q].  Telemetry as for mala_fwd_chunk
 * with Tq = ceil((max_seqlen_q + 127) / 128) and ceil(max_seqlen_k / 128) key blocks. */
int mala_fwd_varlen_prefix(mala_tin q, mala_tin k, mala_tin v, const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                           mala_tout o, float* lse, const mala_stats* st, int B, int Hq, int Hkv, int total_q,
                           int total_k, int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, float tau,
                           void* ws, size_t ws_bytes, void* cuda_stream);

/* Algorithm 2 for mala_fwd_varlen_prefix: every sequence is treated exactly as a mala_bwd_chunk call on its own
 * rows, with the query blocks following its key positions as in the forward call.  o, dout, dq like q; dk, dv like k;
 * lse fp32 [Hq,total_q] as the forward call wrote it.  A sequence without queries (or, causal != 0, with more queries
 * than keys) gets zero dk / dv rows (and zero dq rows).  Telemetry as for mala_bwd_chunk with ceil(max_seqlen_k / 128)
 * key blocks and Tq = ceil((max_seqlen_q + 127) / 128).  Workspace:
 * mala_workspace_bytes(MALA_OP_BWD, 1, Hq, Hkv, total_q + 384 * B, d, 0).  As for the other packed calls, the tiles at
 * a sequence's ends also cover rows of its neighbours, which must be finite numbers. */
int mala_bwd_varlen_prefix(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse,
                           const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, mala_tout dq, mala_tout dk,
                           mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int total_q, int total_k,
                           int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, float tau, void* ws,
                           size_t ws_bytes, void* cuda_stream);

/* mala_fwd_varlen_prefix with the keys and values held in pages: a batch of prefill chunks behind prefixes that
 * live in a paged cache (the chunks' own keys and values already written to their pages).  q, o [1,total_q,Hq,d]
 * packed by cu_seqlens_q (device int32 [B+1]); kpages, vpages [num_pages, page_size, Hkv, d] with page_size a multiple
 * of 128, or 8, 16, 32 or 64 (a tile is then put together from 128 / page_size pages, each with its own table
 * lookup, at reduced throughput); block_table device int32 [B, max_pages_per_seq] (keys page_size*x .. of sequence b in page
 * block_table[b][x]); seqlens_k device int32 [B], the keys sequence b holds, clamped to
 * max_pages_per_seq * page_size (what its block-table row can map), its queries being its last positions
 * (a sequence with no keys, or with fewer keys than queries when causal != 0, is left untouched).  Slots of a mapped
 * page beyond the sequence's length must hold finite numbers.  Everything else as mala_fwd_varlen_prefix with
 * max_seqlen_k = max_pages_per_seq * page_size. */
int mala_fwd_paged(mala_tin q, mala_tin kpages, mala_tin vpages, const int32_t* cu_seqlens_q, const int32_t* block_table,
                   const int32_t* seqlens_k, mala_tout o, float* lse, const mala_stats* st, int B, int Hq, int Hkv,
                   int total_q, int max_seqlen_q, int num_pages, int page_size, int max_pages_per_seq, int d, int causal,
                   float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream);

/* Split-KV decode of one new token per sequence ("Fused decoding execution").  q [B,1,Hq,d] (sn is
 * ignored); kcache, vcache [B,Nk,Hkv,d], the newest token's key/value included; o [B,1,Hq,d];
 * lse_opt fp32 [B,Hq] or NULL.  The Hq/Hkv query heads of one KV head are the rows of one tile; the
 * key range is cut into num_splits contiguous chunks of ceil(ceil(Nk/num_splits)/128)*128 keys,
 * each visited newest tile first with its own running state, L = Nk; partials are merged by the
 * normalizer-aware reduction.  Requires Hq/Hkv <= 16. */
int mala_decode(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, const mala_stats* st,
                int B, int Hq, int Hkv, int Nk, int d, float scale, float tau, int num_splits, void* ws,
                size_t ws_bytes, void* cuda_stream);

/* mala_decode over an 8-bit KV cache: the same operator ("Fused decoding execution"; the paper keeps the cache intact,
 * and so does this call -- only the storage type differs) on keys and values stored as e4m3 with one fp32 scale per
 * (sequence, KV head, 128-key tile):
 *     k[b, n, h, :] = kscale[b, h, n / 128] * e4m3(kcache8[b, n, h, :]),   v likewise with vscale.
 * The result is that of mala_decode on those dequantised values (the step streams half the bytes).
 * kcache8, vcache8: 8-bit [B,Nk,Hkv,d] views, strides in ELEMENTS (= bytes), multiples of 16; kscale, vscale: device
 * fp32 [B,Hkv,ceil(Nk/128)].  d a multiple of 16, at most 128; Hq/Hkv <= 8 (MALA_ERR_UNSUPPORTED otherwise).  q, o,
 * lse_opt, telemetry, splits and merge as in mala_decode.
 * Workspace: mala_workspace_bytes(MALA_OP_DECODE, B, Hq, Hkv, Nk, 128, num_splits). */
int mala_decode_fp8(mala_tin q, mala_tin kcache8, mala_tin vcache8, const float* kscale, const float* vscale,
                    mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq, int Hkv, int Nk, int d, float scale,
                    float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream);

/* mala_decode_fp8 with Sq new tokens per sequence: the rule and the layout of mala_decode_multi (q, o [B,Sq,Hq,d],
 * lse_opt [B,Sq,Hq], the new tokens' keys and values in the last Sq positions of the caches, token s at position
 * Nk - Sq + s with L = Nk - Sq + s + 1) on the storage of mala_decode_fp8.  Requires Sq * Hq/Hkv <= 8 and Sq <= Nk
 * (MALA_ERR_UNSUPPORTED otherwise); Sq = 1 is mala_decode_fp8.
 * Workspace: mala_workspace_bytes(MALA_OP_DECODE, B * Sq, Hq, Hkv, Nk, 128, num_splits). */
int mala_decode_fp8_multi(mala_tin q, mala_tin kcache8, mala_tin vcache8, const float* kscale, const float* vscale,
                          mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq, int Hkv, int Nk, int Sq, int d,
                          float scale, float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream);

/* mala_decode_fp8 over a paged 8-bit cache with one length per sequence: the layout of mala_decode_paged (one new token
 * per sequence) with the storage of mala_decode_fp8.  kpages8, vpages8: 8-bit [num_pages, page_size, Hkv, d] views
 * (strides in elements = bytes, multiples of 16), page_size a multiple of 128, or 16, 32 or 64 (MALA_ERR_UNSUPPORTED
 * otherwise); kscale, vscale: device fp32 [num_pages, Hkv, max(1, page_size/128)], the scale of tile y of page x at
 * [x][h][y] -- one scale per 128-key tile of a page, or one per page where a page is smaller than a tile (a tile is then
 * put together from 128 / page_size pages, each key scaled by its own page's scale; the skip rule's tile stays 128
 * keys).  block_table, seqlens, the split layout (Nk = max_pages_per_seq*page_size), the
 * clamping of seqlens, entries outside the pool (read as zeros) and telemetry as in mala_decode_paged; slots of a
 * mapped page beyond the sequence's length must hold codes other than e4m3's two NaN codes, 0x7f and 0xff (a
 * zero-initialised or recycled page does): their keys are masked out of the scores, but their values are multiplied by
 * zero probabilities.  (Where such slots share a scale with real keys -- the rest of the sequence's last page -- a
 * scale orders of magnitude above the real values' costs those values, and the step's 8-bit probabilities, precision:
 * quantise a page from the slots in use.)  d, Hq/Hkv and the workspace as in mala_decode_fp8. */
int mala_decode_fp8_paged(mala_tin q, mala_tin kpages8, mala_tin vpages8, const float* kscale, const float* vscale,
                          const int32_t* block_table, const int32_t* seqlens, mala_tout o, float* lse_opt,
                          const mala_stats* st, int B, int Hq, int Hkv, int num_pages, int page_size,
                          int max_pages_per_seq, int d, float scale, float tau, int num_splits, void* ws, size_t ws_bytes,
                          void* cuda_stream);

/* Split-KV decode of Sq new tokens per sequence at once (a verification step of speculative decoding, or a short
 * chunk).  q, o [B,Sq,Hq,d]; lse_opt fp32 [B,Sq,Hq] or NULL; kcache, vcache [B,Nk,Hkv,d] with the keys and values of
 * the Sq new tokens already in the last Sq positions.  Token s (0 = oldest) sits at position Nk - Sq + s, attends to
 * the keys before and at its own position and has L = Nk - Sq + s + 1, the number of keys it sees (Section 2.1).
 * The Sq * Hq/Hkv rows that share a KV head form one tile (one row that needs a key block retains it for all; a
 * row that sees no key of a block does not constrain it); requires Sq * Hq/Hkv <= 16 and Sq <= Nk.  Splits,
 * telemetry and merge as in mala_decode; Sq = 1 is mala_decode.
 * Workspace: mala_workspace_bytes(MALA_OP_DECODE, B * Sq, Hq, Hkv, Nk, d, num_splits). */
int mala_decode_multi(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, const mala_stats* st,
                      int B, int Hq, int Hkv, int Nk, int Sq, int d, float scale, float tau, int num_splits, void* ws,
                      size_t ws_bytes, void* cuda_stream);

/* Split-KV decode over a paged cache with one length per sequence (the serving-side layout of "Fused decoding
 * execution"; the rule itself is the one of mala_decode / mala_decode_multi with seqlens[b] in the place of Nk).
 * q, o [B,Sq,Hq,d], Sq >= 1 new tokens per sequence whose keys are the last Sq of the sequence's seqlens[b] keys
 * (Sq * Hq/Hkv <= 16; Sq = 1: sn of q and o is ignored); lse_opt fp32 [B,Sq,Hq] or NULL.
 * kpages, vpages [num_pages, page_size, Hkv, d] (sb = page stride, sn = key stride, sh = head stride);
 * page_size is a multiple of 128, or 8, 16, 32 or 64 (a 128-key tile is then fetched as several copies, which costs
 * throughput; MALA_ERR_UNSUPPORTED for any other size).  block_table: device int32
 * [B, max_pages_per_seq]; keys page_size*x .. page_size*(x+1)-1 of sequence b live in page block_table[b][x]
 * (entries beyond the sequence's length are never read; an entry outside [0, num_pages) reads zeros).
 * seqlens: device int32 [B], keys held by each sequence, clamped to [0, max_pages_per_seq*page_size], or NULL
 * if every sequence holds max_pages_per_seq*page_size keys; a token that sees no key (a sequence without keys, or
 * with fewer keys than new tokens) gets o = 0, lse = -inf.
 * The key positions 0 .. max_pages_per_seq*page_size-1 are cut into num_splits chunks as in mala_decode with
 * Nk = max_pages_per_seq*page_size; splits beyond a sequence's length are empty.  Telemetry shapes as for
 * mala_decode with that Nk.  The values stored in a mapped page beyond the sequence's length must be finite
 * bf16 numbers (a zero-initialised or recycled page is): they never reach the result, but the tile that holds
 * the newest key is multiplied as a whole.  Workspace: mala_workspace_bytes(MALA_OP_DECODE, B * Sq, Hq, Hkv,
 * max_pages_per_seq*page_size, d, num_splits).  The library reads block_table and seqlens on the device, on
 * cuda_stream, and keeps neither. */
int mala_decode_paged(mala_tin q, mala_tin kpages, mala_tin vpages, const int32_t* block_table,
                      const int32_t* seqlens, mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq,
                      int Hkv, int num_pages, int page_size, int max_pages_per_seq, int Sq, int d, float scale,
                      float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream);

/* Decode for callers that cannot allocate device memory.  (The paper has no counterpart: this entry point
 * exists for integration reasons only and computes exactly what mala_decode computes.)
 *
 * Some callers of this library have no way to obtain scratch memory at the point of the call: code
 * that runs inside a serving engine's pre-sized memory plan where every byte of the device pool is
 * already assigned, a plug-in that receives only its input and output buffers from the host framework,
 * or a latency-critical path that must not touch an allocator (cudaMalloc synchronises the device and
 * may fail under fragmentation).  For them this variant keeps the split partials -- the only scratch
 * the decode path needs -- in an array that is part of the library image: MALA_STATIC_SCRATCH_BYTES of
 * global memory on every GPU that loads the library, held until the process exits.  The caller still
 * passes all inputs and outputs; the call itself allocates nothing and frees nothing.
 *
 * Limits and rules
 *   - mala_workspace_bytes(MALA_OP_DECODE, ...) for the same arguments must not exceed
 *     MALA_STATIC_SCRATCH_BYTES; otherwise nothing is launched and
 *     MALA_ERR_STATIC_SCRATCH_EXCEEDED is returned (use fewer splits, or mala_decode with your own ws).
 *   - All calls on one device share the one array.  Two calls whose kernels can overlap on the GPU
 *     (different streams, or different host threads on different streams) race on it and give wrong
 *     results: keep calls on a device in one stream, or order them with events.  The array keeps the
 *     previous call's contents between calls; the kernels overwrite every entry they later read, so no
 *     clearing is needed.
 *   - The first call on each device looks up the array's device address (a one-time
 *     cudaGetSymbolAddress with that device current).  Make that first call outside any stream capture.
 *   - No telemetry (mala_stats) is available through this entry point.
 * Arguments, layouts, result and error codes otherwise as mala_decode. */
int mala_decode_static(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, int B, int Hq,
                       int Hkv, int Nk, int d, float scale, float tau, int num_splits, void* cuda_stream);

/* A split count for mala_decode and its variants (host only; nothing is launched).  The skip test of a split sees
 * only that split's partial normalizer ("Fused decoding execution"), so it passes more often the longer the split:
 * the best count is the SMALLEST one that still spreads the B * Hkv * num_splits work items evenly over the SMs.
 * Items differ in how many tiles they retain, so an SM needs several of them to even that out.
 * Returned: the smallest S with at least six items per SM and at least two tiles per split (without the first
 * condition where the two cannot both hold) whose longest per-SM queue, ceil(B*Hkv*S / sm_count) items of
 * ceil(ceil(Nk/128) / S) tiles each, is within 4 % of the shortest such queue any admissible S gives.
 * Nk: the (longest) cache length; sm_count <= 0: the current device's SM count is used.
 * Returns the count (>= 1) or a negative MALA_ERR_* code. */
int mala_decode_suggest_splits(int B, int Hkv, int Nk, int sm_count);

/* Scratch bytes needed by one call of `op` (MALA_OP_*); N is Nk for decode; num_splits is ignored
 * for fwd / bwd.  Returns 0 for unsupported arguments. */
size_t mala_workspace_bytes(int op, int B, int Hq, int Hkv, int N, int d, int num_splits);

/* Tile partition of `op` for head size d: Bq query rows x Bk keys.  For decode Bq is reported as 0
 * (the rows are the Hq/Hkv packed query heads).  Returns MALA_OK or MALA_ERR_UNSUPPORTED. */
int mala_tile_shape(int op, int d, int* Bq, int* Bk);

/* Reads the current device's status word into *code_out (MALA_OK or MALA_ERR_DEVICE_TIMEOUT) and, if
 * clear != 0, resets it.  Synchronises the device.  HOST pointer. */
int mala_device_status(int* code_out, int clear);

/* ---- Test support (not part of the operator) ------------------------------------------------------------------
 * Every wait inside the kernels is bounded (Conventions, last item).  This call makes one such wait run out on
 * purpose, in the only way that harms nothing: it launches a single small thread block whose one waiting thread
 * polls, with the kernels' own wait routine, a barrier that nobody ever arrives on, gives up after limit_cycles
 * clock cycles (1 .. 1e8; the kernels themselves use about 2 s), records MALA_ERR_DEVICE_TIMEOUT in the device's
 * status word and returns through the normal exit.  Nothing faults, traps or waits without a limit.  Afterwards
 * mala_device_status reports the code, and every later launch of this library on the device returns at once
 * without touching its outputs until the word is cleared (mala_device_status with clear != 0).
 * Asynchronous on cuda_stream; MALA_OK or a negative MALA_ERR_* code (MALA_ERR_INVALID_ARG for a limit out of range). */
int mala_test_expire_wait(long long limit_cycles, void* cuda_stream);

const char* mala_strerror(int code);
int mala_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MALA_H_ */
