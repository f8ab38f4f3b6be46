/*
 * hann.h -- C ABI of the B200 encrypted nearest-neighbour scoring library.
 *
 * The library implements the server-side hot path of hierarchical encrypted ANN search with RNS-CKKS:
 * one encrypted, rank-reduced query is scored against fetched batches of plaintext candidate rows at
 * each routing level (Sec. 2 "The round trip": coarse -> fine -> rerank; Sec. 3.2 "How": every level
 * is one call to the same stateless scorer), using the diagonal matrix-vector method with baby-step /
 * giant-step rotations (Sec. 3.1 "How" and Detail) and plaintext pre-rotation of the database diagonals
 * (Sec. 3.1 Detail).  The client half (key generation, query encryption, score decryption; Sec. 2,
 * steps 1, 3, 5, 7 of the round trip) is here too so that a user needs nothing else.
 *
 * Conventions
 *   - Every function returns HANN_OK (0) or a negative HANN_E* code; nothing throws or aborts across the
 *     boundary.  `hann_last_error` gives a one-line description of the last failure of a context.
 *     On error the outputs are unspecified but no buffer is freed or re-owned.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global memory on the context's
 *     device.  Device work is enqueued on the context's stream and is asynchronous; host-pointer
 *     functions synchronise that stream before they return.
 *   - The caller owns every buffer it passes.  The library owns the context, its tables and the keys
 *     uploaded with `hann_load_keys`; these live until `hann_ctx_destroy`.
 *   - Server-side calls (`hann_query_prepare`, `hann_encode_candidates`, `hann_score_level`,
 *     `hann_rotate_sum`, `hann_keyswitch`) allocate nothing: all temporaries live in the caller's
 *     workspace `ws` (256-byte aligned device memory, `ws_bytes` long; `hann_workspace_bytes` says how
 *     much is enough; HANN_EWORKSPACE if it is too short) -- the counterpart of the paper's single
 *     pre-allocated arena, Sec. 3.4.  One workspace serves one call at a time.  Two exceptions, both outside the
 *     steady state: while the per-launch profile (hann_kernel_profile) is on, every launch takes a CUDA event pair
 *     from a pool that grows on demand; and hann_score_level_host creates one event per block and per block group
 *     the first time it sees a level of that size (later calls of the same or a smaller size create nothing).
 *   - Canonical exchange layout (the only layout with a meaning outside the library): coefficient
 *     domain, natural coefficient order, residues in [0, q_i), uint64, index order [poly][limb][coeff];
 *     a ciphertext is 2 polynomials (c0, c1) of L limbs.  The internal device layout (transform domain,
 *     element order) is private; `hann_import` / `hann_export` convert.
 *   - Ring degree N = 2^logN, n = N/2 slots; L ciphertext primes q_0..q_{L-1} and one special prime p,
 *     each prime, below 2^62 and congruent to 1 mod 2N; R = padded vector dimension (R divides n);
 *     B = baby-step count (B divides R), G = R/B giant steps.
 *   - Row <-> slot mapping: row blk*n + i of a level's candidate list is slot i of score ciphertext blk;
 *     the last block is zero-padded.
 */
#ifndef HANN_H
#define HANN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HANN_OK 0
#define HANN_EINVAL (-1)     /* bad parameter value or null pointer                        */
#define HANN_ESHAPE (-2)     /* sizes inconsistent with the context (dim, counts, rotation) */
#define HANN_ENOKEY (-3)     /* a needed evaluation key has not been loaded                 */
#define HANN_EWORKSPACE (-4) /* workspace missing or misaligned                             */
#define HANN_ECUDA (-5)      /* a CUDA runtime call or kernel launch failed                 */
#define HANN_ENOMEM (-6)     /* host or device allocation failed (set-up calls only)        */

#define HANN_MAX_PRIMES 15

typedef struct hann_ctx hann_ctx; /* opaque */

typedef struct {
    int32_t logN;                /* 4..16                                                   */
    int32_t L;                   /* number of ciphertext primes, 1..HANN_MAX_PRIMES         */
    uint64_t q[HANN_MAX_PRIMES]; /* q_0..q_{L-1}                                            */
    uint64_t p;                  /* special prime of hybrid key switching                   */
    int32_t log_scale;           /* Delta = 2^log_scale for queries and candidates          */
    int32_t R;                   /* padded dimension                                        */
    int32_t B;                   /* baby-step count                                         */
    int32_t device;              /* CUDA device ordinal                                     */
    void *stream;                /* cudaStream_t the context enqueues on (NULL = default)   */
} hann_params;

/* what `hann_sizeof` can be asked */
enum {
    HANN_SIZE_POLY = 1,     /* one polynomial of L limbs: L*N*8                                          */
    HANN_SIZE_CT = 2,       /* one ciphertext: 2*L*N*8                                                    */
    HANN_SIZE_BABY = 3,     /* the B rotated query ciphertexts                                            */
    HANN_SIZE_PT_BLOCK = 4, /* encoded candidates of one block of n rows: R*L*(N/2)*8 (= 8*L*R bytes a row): the encoding
                             * of a real slot vector is fixed by X -> 1/X, so the second half of its transform is the
                             * mirror image of the first and is neither computed nor stored */
    HANN_SIZE_INNER = 5,    /* the G partial-sum ciphertexts of one block                                 */
    HANN_SIZE_EVK = 6,      /* one evaluation key in canonical layout: L*2*(L+1)*N*8                      */
    HANN_SIZE_ROWS_PER_BLOCK = 7, /* n                                                                    */
    HANN_SIZE_CTDB_BLOCK = 8 /* one ENCRYPTED block of candidates: R ciphertexts, [G][B][2][L][N] uint64      */
};

/* element kinds of `hann_import` / `hann_export` */
enum { HANN_KIND_POLY = 1, HANN_KIND_CT = 2, HANN_KIND_PT = 3 };

typedef struct {
    uint64_t launches;         /* kernels launched by this context since creation                      */
    float ms_query_prepare;    /* device time of the last call of each kind, milliseconds; valid after */
    float ms_encode;           /* hann_sync (0 if never called or timing disabled)                     */
    float ms_score_level;
    float ms_rotate_sum;
    float ms_keyswitch;
} hann_stats;

/* ---- context ------------------------------------------------------------------------------------------- */

/* Create a context: validates the parameters (HANN_EINVAL: not prime, not 1 mod 2N, out of range, B does not
 * divide R, R does not divide n), builds the transform and encode tables on the device.  *out is set only on
 * success and must be released with hann_ctx_destroy. */
int hann_ctx_create(const hann_params *params, hann_ctx **out);
void hann_ctx_destroy(hann_ctx *ctx);

/* Byte sizes of the private device layouts (see the enum); negative on a bad argument. */
int64_t hann_sizeof(const hann_ctx *ctx, int what);

/* Bytes of workspace the server-side calls need when at most `max_blocks` blocks are processed per call. */
int64_t hann_workspace_bytes(const hann_ctx *ctx, int64_t max_blocks);

/* Block until everything enqueued on the context's stream has finished; reports asynchronous CUDA errors and a
 * kernel that gave up a bounded wait (HANN_ECUDA, once: the report clears the condition).  Every host-pointer call
 * (hann_import, hann_export, hann_export_limbs, hann_expand_uniform, hann_score_level_host, the client half) ends
 * with the same check, so HANN_OK from any of them means that no kernel of the call was abandoned. */
int hann_sync(hann_ctx *ctx);
const char *hann_last_error(const hann_ctx *ctx);

/* ---- test, profiling and measurement hooks (not part of the scoring product; nothing on the hot path calls them) ----
 * hann_selftest_bounded_wait, hann_set_timing / hann_get_stats, hann_kernel_profile / hann_kernel_times,
 * hann_probe_rates, hann_debug_build / hann_debug_canaries / hann_debug_verify.  (The Python binding's HANN_LIB environment variable, which makes it load
 * another build of this library for A/B comparisons, is a hook of the same kind.) */

/* Self-test of the failure path of the bulk-copy kernels: launches one warp that waits, for limit_ms (1..1000), on a
 * completion barrier that nothing completes.  The wait runs out, the kernel raises the context's flag and returns; the
 * NEXT hann_sync therefore reports HANN_ECUDA ("a kernel gave up a bounded wait") and clears the flag, after which the
 * context works as before.  waited_ms (optional) receives the device time the warp spent waiting. */
int hann_selftest_bounded_wait(hann_ctx *ctx, int limit_ms, double *waited_ms);
/* Enable (1) or disable (0) per-call CUDA-event timing; disabled by default. */
int hann_set_timing(hann_ctx *ctx, int enable);
int hann_get_stats(hann_ctx *ctx, hann_stats *out);

/* Performance knobs (results never depend on them).  HANN_TUNE_ENCODE_GROUP: plaintexts encoded and transformed per
 * launch group in hann_encode_candidates (default: all R plaintexts of a block at once); ask hann_workspace_bytes again after changing it.
 * HANN_TUNE_HOST_LIMBS (this one DOES change a result's layout): hann_score_level_host downloads only the first `value`
 * limbs of every score polynomial, score_ct_host [blocks][2][value][N] -- the exact form of hann_compact_scores; decrypt
 * with hann_decrypt_compact(limbs = value, rescaled = 0).  Default L.
 * HANN_TUNE_ENCODE_SYMMETRY: 1 (default) lets hann_encode_candidates use the fact that the encoding of a REAL slot vector
 * is fixed by X -> 1/X, so that its number-theoretic transform takes each value twice (at psi^(2t+1) and at the inverse
 * of that root): only half of every transform is computed and the other half is written as a mirror image; 0 computes
 * every transform in full.  Same bits either way.
 * HANN_TUNE_HOST_GROUPS: number of block groups hann_score_level_host cuts a level into (a group is scored and its scores
 * are downloaded while the rows of the following groups still travel); 0 (default) chooses from the level's size.  Values
 * above 1 also make hann_query_level cut its level into that many groups (it keeps the plain order otherwise).  Ask
 * hann_level_host_bytes / hann_workspace_bytes again after changing it.
 * HANN_TUNE_GIANT_LAZY (this one changes the result's BITS, not its meaning): 1 makes hann_rotate_sum, and with it
 * hann_query_level and hann_score_level_host, evaluate the giant steps in the order of hann_rotate_sum_lazy (the keys of
 * rotations 2B .. (G-1)B must then be loaded as well); 0 (default) is Horner with the single key of rotation B.
 * HANN_TUNE_LAZY_LANES: block ranges (1..4, default 2) hann_rotate_sum_lazy runs side by side on helper streams.
 * HANN_TUNE_MAC_F64: 1 (default) lets the single-query multiply-accumulate of chains of primes below 2^50 sum its products
 * exactly in pairs of binary64 words on the FP64 pipe, 0 on the integer multiplier; same residues either way.
 * HANN_TUNE_PAIR_B32: 1 lets hann_score_level_batch serve two queries per pass over the stored plaintexts at B = 32 as well
 * (it does at B <= 16); 0 (default) gives every query its own pass there. */
enum { HANN_TUNE_ENCODE_GROUP = 1, HANN_TUNE_HOST_LIMBS = 2, HANN_TUNE_ENCODE_SYMMETRY = 3, HANN_TUNE_HOST_GROUPS = 4, HANN_TUNE_GIANT_LAZY = 5,
       HANN_TUNE_LAZY_LANES = 6, HANN_TUNE_MAC_F64 = 7, HANN_TUNE_PAIR_B32 = 8 };
int hann_set_tuning(hann_ctx *ctx, int what, int value);

/* Per-launch profile: while enabled every kernel launch of the context is bracketed by a CUDA event pair (this
 * serialises nothing but adds two event records per launch).  hann_kernel_times synchronises, writes the summed
 * device milliseconds and launch counts per kernel class (arrays of hann_kernel_classes() entries, class names from
 * hann_kernel_name) accumulated since the previous call, and clears them. */
int hann_kernel_classes(void);
const char *hann_kernel_name(int cls);
int hann_kernel_profile(hann_ctx *ctx, int enable);
int hann_kernel_times(hann_ctx *ctx, double *ms, uint64_t *launches);

/* Checks that stand in for a memory checker (never a trap, never an abort):
 *   - hann_debug_build() is 1 for a library compiled with -DHANN_DEBUG.  Such a build checks the computed indices of its
 *     gathers (automorphism sources, mirror positions, row gathers) against their ranges; a failing check SKIPS the access
 *     and records the source line in the context's error word, which the next synchronising call reports as HANN_ECUDA
 *     ("index range check failed ... source line N").  A release build has no such code.
 *   - hann_debug_canaries(ctx, 1) (any build) makes every server-side call put a 256-byte guard behind each sub-buffer it
 *     carves from the caller's workspace (the slack in hann_workspace_bytes covers them), filled with a pattern on the
 *     spot; hann_debug_verify(ctx, &checked, &damaged) checks all guards carved since the last verify, reports how many
 *     there were and how many a kernel overwrote (HANN_ECUDA if any, naming the first one), and forgets them.  Call it
 *     while the workspaces of those calls are still allocated.  A later call that carves the same workspace retires the
 *     guards its own sub-buffers cover (they are overwritten legitimately), so verify after the call you want checked. */
int hann_debug_build(void);
int hann_debug_canaries(hann_ctx *ctx, int enable);
int hann_debug_verify(hann_ctx *ctx, int64_t *guards_checked, int64_t *guards_damaged);

/* Measured arithmetic ceilings of the device (a set-up class call: allocates and frees a small buffer, synchronises):
 * binary64 modular butterflies per second of the register-resident round the transform kernels run (no memory traffic:
 * the rate no transform can exceed) and 32-bit integer multiply-adds per second (the multiply-accumulate spends three per
 * residue product).  bench.py reports the transform and multiply-accumulate kernels against these. */
int hann_probe_rates(hann_ctx *ctx, double *f64_butterflies_per_s, double *int32_madds_per_s);

/* ---- client side (host memory in and out; Sec. 2, The round trip, client steps) -------------------------- */

/* Evaluation keys for the left slot rotations rot[0..n_rot) from caller-drawn randomness (hybrid key switching,
 * one special prime, one digit per ciphertext prime).  For rotation r (Galois element k = 5^r mod 2N,
 * s' = s(X^k)) and digit j: b_j = -a_j*s + e_j + F_j*s' over the L+1 moduli, F_j = p mod q_j on limb j and
 * 0 elsewhere.
 *   s   [N]                      ternary secret, int8 in {-1,0,1}
 *   a   [n_rot][L][L+1][N]       uniform residues (limb order q_0..q_{L-1}, p), canonical
 *   e   [n_rot][L][N]            small errors, int8
 *   evk_out [n_rot][L][2][L+1][N]  canonical; [..][j][0] = b_j, [..][j][1] = a_j */
int hann_keygen_from_samples(hann_ctx *ctx, const int8_t *s, int n_rot, const int32_t *rot, const uint64_t *a,
                             const int8_t *e, uint64_t *evk_out);

/* The same keys from a 64-bit seed (Sec. 2, The round trip, client step 1: the client owns the secret key and hands the
 * server the evaluation keys): the ternary secret, the uniform halves and the rounded-Gaussian errors (sigma = 3.2) are
 * all drawn from the counter hash of hann_expand_uniform (streams 16..19; the uniform halves on the device) -- a
 * benchmark generator, NOT a cryptographic one.  A rotation's key depends on (seed, rotation) only, not on the list it
 * is generated with.  s_out [N] int8 receives the secret; evk_out as in hann_keygen_from_samples. */
int hann_keygen_seeded(hann_ctx *ctx, uint64_t seed, int n_rot, const int32_t *rot, int8_t *s_out, uint64_t *evk_out);

/* Relinearisation key (Sec. 2, encrypted database): the evaluation key for s' = s*s in the layout of
 * hann_keygen_from_samples for ONE key; a [L][L+1][N], e [L][N], evk_out [L][2][L+1][N].  hann_load_keys takes it under
 * rotation number 0. */
int hann_keygen_relin_from_samples(hann_ctx *ctx, const int8_t *s, const uint64_t *a, const int8_t *e, uint64_t *evk_out);

/* Enrolment of an encrypted block (Sec. 2: in deployment the candidate diagonals are ciphertexts): symmetric
 * encryption of the R encoded plaintexts of one block, ctdb[g][b] = (pt[g][b] - a*s + e, a).
 *   pt_dev one block as written by hann_encode_candidates (device, internal layout); a [R][L][N] uniform residues
 *   (canonical, host or device); e [R][N] int8 (host); ctdb_dev HANN_SIZE_CTDB_BLOCK bytes (device, internal). */
int hann_encrypt_block(hann_ctx *ctx, const int8_t *s, const void *pt_dev, const uint64_t *a, const int8_t *e, void *ctdb_dev);

/* Symmetric encryption of a query: the slot vector holds q[i mod R] (q zero-padded from `dim` to R and tiled
 * n/R times), encoded at scale Delta by the canonical encoder, then ct = (-a*s + e + m, a).
 *   q [dim] float32, dim <= R;  a [L][N] uniform residues;  e [N] int8;  ct_out [2][L][N] canonical. */
int hann_encrypt_query(hann_ctx *ctx, const int8_t *s, const float *q, int dim, const uint64_t *a, const int8_t *e,
                       uint64_t *ct_out);

/* Decrypt `count` score ciphertexts ct [count][2][L][N] (canonical) whose plaintext scale is 2^log_scale_out
 * (2*log_scale straight after scoring) into real parts scores [count][n]; imag_or_null, if given, receives the
 * imaginary parts [count][n] (pure noise for a correct computation). */
int hann_decrypt_scores(hann_ctx *ctx, const int8_t *s, const uint64_t *ct, int64_t count, int log_scale_out,
                        double *scores, double *imag_or_null);

/* Decrypt compacted score ciphertexts (hann_compact_scores, exported with hann_export_limbs): ct [count][2][limbs][N]
 * canonical, over the first `limbs` ciphertext primes; `log_scale_in` is the scale before compaction (2*log_scale after
 * scoring), `rescaled` says whether the compaction divided by the last prime. */
int hann_decrypt_compact(hann_ctx *ctx, const int8_t *s, const uint64_t *ct, int64_t count, int limbs, int rescaled,
                         int log_scale_in, double *scores, double *imag_or_null);

/* ---- server side ------------------------------------------------------------------------------------------ */

/* Upload evaluation keys (canonical layout as produced by hann_keygen_from_samples; `evk` may be a host or a
 * device pointer) into the context, replacing keys with the same rotation.  Allocates device memory owned by the
 * context.  Needed later: rotations 1..B-1 for hann_query_prepare, rotation B for hann_rotate_sum. */
int hann_load_keys(hann_ctx *ctx, const uint64_t *evk, int n_rot, const int32_t *rot);

/* Once per query (Sec. 3.1 Detail: the baby steps of the diagonal method; Sec. 3.4: the rotated query is computed
 * once and reused by every block and level): the B rotated copies rot_r(ct), r = 0..B-1, each taken directly from
 * the input ciphertext (key switch of the automorphed c1; the digit decomposition is shared by all rotations).
 *   ct_dev   one ciphertext, internal layout (device)
 *   baby_dev HANN_SIZE_BABY bytes (device), internal layout [B][2][L][N] */
int hann_query_prepare(hann_ctx *ctx, const void *ct_dev, void *baby_dev, void *ws, size_t ws_bytes);

/* Encode candidate rows into plaintext blocks (Sec. 2, storage paragraph: a block of n rows is held as R diagonals;
 * Sec. 3.1 Detail: each diagonal is shifted by the giant-step amount in plaintext, so the server needs no database
 * rotation keys).  rows_dev [n_rows][dim] float32 row-major (device), dim <= R
 * (rows are zero-padded to R).  Block blk holds rows blk*n .. blk*n+n-1 (missing rows are zero).  For g < G,
 * b < B plaintext (g,b) of a block encodes the slot vector z[i] = M[(i - g*B) mod n][(i + b) mod R] at scale
 * Delta, reduced into every ciphertext prime and transformed.
 *   pt_dev  ceil(n_rows/n) * HANN_SIZE_PT_BLOCK bytes (device), internal layout [blk][G][B][L][N/2] */
int hann_encode_candidates(hann_ctx *ctx, const float *rows_dev, int64_t n_rows, int dim, void *pt_dev, void *ws, size_t ws_bytes);

/* Multiply-accumulate of one level (Sec. 3.1 "How": the diagonal matrix-vector product; Sec. 3.2 "How": every level
 * is one call to the same stateless scorer): inner[blk][g] = sum_b pt[blk][g][b] * baby[b] (both ciphertext components,
 * every limb).   inner_dev n_blocks * HANN_SIZE_INNER bytes (device), internal layout [blk][G][2][L][N]. */
int hann_score_level(hann_ctx *ctx, const void *baby_dev, const void *pt_dev, int64_t n_blocks, void *inner_dev,
                     void *ws, size_t ws_bytes);

/* Cross-query batching (Sec. 7: score a whole batch of queries against each loaded region before it is evicted): the
 * same multiply-accumulate for n_queries prepared queries against the same encoded blocks, the plaintexts streamed from
 * HBM once per pair of queries instead of once per query.
 *   baby_dev  n_queries * HANN_SIZE_BABY bytes: the baby sets of the queries, one after the other;
 *   inner_dev n_queries * n_blocks * HANN_SIZE_INNER bytes: query-major, [query][blk][g]; hann_rotate_sum over
 *             n_queries * n_blocks "blocks" then yields score ciphertexts [query][blk].
 * Each query's result is bit-identical to hann_score_level on its own. */
int hann_score_level_batch(hann_ctx *ctx, const void *baby_dev, int n_queries, const void *pt_dev, int64_t n_blocks,
                           void *inner_dev, void *ws, size_t ws_bytes);

/* The multiply-accumulate against an ENCRYPTED block (Sec. 2, deployment setting): for every (blk, g) the degree-2
 * ciphertext sum_b ctdb[blk][g][b] (x) baby[b] = (x0 y0, x0 y1 + x1 y0, x1 y1) accumulated over the baby steps, then ONE
 * relinearisation per (blk, g): (d0 + ks0, d1 + ks1) with (ks0, ks1) the key switch of d2 under the relinearisation key
 * (loaded as rotation 0).  inner_dev as for hann_score_level (n_blocks * HANN_SIZE_INNER bytes); hann_rotate_sum follows
 * unchanged.  Ciphertext primes below 2^60, B <= 128.  ctdb_dev n_blocks * HANN_SIZE_CTDB_BLOCK bytes. */
int hann_score_level_ctdb(hann_ctx *ctx, const void *baby_dev, const void *ctdb_dev, int64_t n_blocks, void *inner_dev,
                          void *ws, size_t ws_bytes);

/* Ciphertext x ciphertext product of `count` independent pairs with relinearisation (the multiplication of a CKKS circuit;
 * Sec. 2: the encrypted database and the membership path need it): out[i] = (d0 + ks0, d1 + ks1), (d0, d1, d2) =
 * (a0 b0, a0 b1 + a1 b0, a1 b1) of pair i, (ks0, ks1) the key switch of d2 under the relinearisation key (rotation 0).
 * The scale of out is the product of the scales; hann_rescale follows in a circuit.  a_dev, b_dev, out_dev: count
 * ciphertexts each (internal layout, device memory, caller-owned); a and b may be the same buffer, out may not alias either.
 * Workspace: hann_workspace_bytes(ctx, 1) serves any count (the pairs then go through one at a time); with room for k
 * products (hann_workspace_bytes(ctx, k), k <= 8) k key switches run side by side.  Errors: HANN_EINVAL (null pointer,
 * negative count; count = 0 is a no-op), HANN_ESHAPE (a ciphertext prime of 2^62 or more), HANN_ENOKEY (no relinearisation
 * key loaded as rotation 0), HANN_EWORKSPACE. */
int hann_multiply(hann_ctx *ctx, const void *a_dev, const void *b_dev, int64_t count, void *out_dev, void *ws, size_t ws_bytes);

/* Rotate-and-sum (Sec. 3.1 Detail: the giant steps of the diagonal method): score_ct[blk] = sum_g rot_{g*B}(inner[blk][g]), evaluated by Horner with the single key of
 * rotation B: acc = inner[G-1]; for g = G-2..0: acc = rot_B(acc) + inner[g].
 *   score_ct_dev n_blocks * HANN_SIZE_CT bytes (device), internal layout. */
int hann_rotate_sum(hann_ctx *ctx, const void *inner_dev, int64_t n_blocks, void *score_ct_dev, void *ws, size_t ws_bytes);

/* The same sum, evaluated in the second order this library supports (the paper fixes the sum, not the order): every
 * term is rotated by its own amount with the key of that rotation, the key products of a block are added up over the
 * L+1 moduli and brought down by ONE ModDown:
 *     (U0, U1) = sum_{g>=1} KeyProduct_{gB}(phi_g(inner[g].c1)),   phi_g: X -> X^(5^(gB)),
 *     score = (inner[0].c0 + sum_{g>=1} phi_g(inner[g].c0) + ModDown(U0),  inner[0].c1 + ModDown(U1)).
 * One key-switch round of depth one instead of a chain of G-1, one rounding instead of G-1 (so slightly LESS noise),
 * at the price of G-1 resident keys (rotations B, 2B, .., (G-1)B: HANN_ENOKEY if one is missing) instead of one.  The
 * ciphertext bits differ from hann_rotate_sum's (both orders are reproduced bit for bit by the reference evaluation of
 * the same order); the decrypted scores agree within the key-switch noise.  Workspace: hann_workspace_bytes(ctx, blocks)
 * is enough; with more, more blocks go through one round. */
int hann_rotate_sum_lazy(hann_ctx *ctx, const void *inner_dev, int64_t n_blocks, void *score_ct_dev, void *ws, size_t ws_bytes);

/* One routing level for one query, device buffers in and out (Sec. 2 "Reproducing this": level + candidates +
 * encrypted query in, encrypted score vector out): hann_query_prepare, hann_encode_candidates,
 * hann_score_level and hann_rotate_sum, the same operations on the same data as the four calls in sequence (hence the same
 * bits) but not one after the other: the query preparation runs on a helper stream beside the candidate encoding, and with
 * HANN_TUNE_HOST_GROUPS above 1 the level is cut into groups of blocks, each scored (multiply-accumulate, rotate-and-sum)
 * on one of two scoring streams as soon as it is encoded, beside the encoding of the next group.  All buffers as in the four
 * calls; `ws` must hold hann_workspace_bytes(ctx, blocks) (with less, but enough for the four calls, the groups are given
 * up and the level is scored after its encoding).  On return everything is enqueued on the context's stream again (the
 * helper streams are joined). */
int hann_query_level(hann_ctx *ctx, const void *ct_dev, const float *rows_dev, int64_t n_rows, int dim, void *baby_dev,
                     void *pt_dev, void *inner_dev, void *score_ct_dev, void *ws, size_t ws_bytes);

/* Hybrid key switch (the operation behind every rotation of Sec. 3.1 and the relinearisation of Sec. 2's encrypted
 * database; the paper takes it from its CKKS library, the conventions are stated above) of one polynomial d (internal
 * layout, L limbs) with the loaded key of rotation `rot`, WITHOUT
 * applying the automorphism to d: outputs (ks0, ks1), L limbs each, with ks0 + ks1*s ~ d*s(X^k).
 * Steps: digits [d]_{q_j} (inverse transform), centred lift into all L+1 moduli, transform, inner product with
 * the key, ModDown: out_i = (u_i - centred([u]_p)) * p^{-1} mod q_i. */
int hann_keyswitch(hann_ctx *ctx, int rot, const void *poly_dev, void *ks0_dev, void *ks1_dev, void *ws, size_t ws_bytes);
/* Bytes of (256-byte aligned) workspace one hann_keyswitch call carves; never more than hann_workspace_bytes(ctx, 1). */
int64_t hann_keyswitch_bytes(const hann_ctx *ctx);

/* (No counterpart in the paper.)  hann_keyswitch for callers that can neither allocate device memory nor lend a
 * workspace -- for instance a request handler that must avoid the device-wide synchronisation of cudaMalloc/cudaFree,
 * or a process whose device memory was fully partitioned by its own pool at start-up.  Same inputs, outputs and result
 * bits as hann_keyswitch; the scratch is a fixed hann_static_scratch_bytes() (4 MiB) array inside the library image,
 * which every GPU that loads the library holds until the process exits.
 *   - Rings whose key switch needs more than that (e.g. N >= 2^15 with L = 4) are refused with HANN_ESHAPE and a message
 *     naming both sizes; use hann_keyswitch there.
 *   - The call performs no cudaMalloc/cudaFree and calls no allocating routine; it returns HANN_EINVAL while the
 *     per-launch profile (hann_kernel_profile) is on, because that profile creates events on demand.
 *   - The array's device address is looked up once per device, by hann_ctx_create (with the context's device
 *     current), so that this call only reads a cached address; if that look-up did not happen, the first call on the
 *     device does it -- so create the context (or make a first call) before starting any stream capture.
 *   - All calls on one device share the one array, which keeps whatever the last call left in it (nothing needs
 *     clearing: every part is written before it is read).  Two calls whose kernels overlap on the GPU -- different
 *     streams, different contexts, different threads -- race on it; serialise them. */
int64_t hann_static_scratch_bytes(void);
int hann_keyswitch_static(hann_ctx *ctx, int rot, const void *poly_dev, void *ks0_dev, void *ks1_dev);

/* ---- rank reduction under encryption, projection matrix packed by windows (Sec. 3.1 "How" and Detail) -----------------
 * Enc(q_R) = W^T Enc(q) for W of shape D x R, D = c R, c a power of two, D dividing n.  Reading taken (the paper gives no
 * index formulas): the n slots are viewed with period D, window k of a period is positions kR .. kR+R-1, and the query
 * ciphertext holds q[i mod D].  Chunk k of W is the R x R matrix W_k^T[r][col] = W[kR + col][r].
 *   - Packing: ONE stored plaintext per diagonal gB + b holds that diagonal of ALL c chunks, chunk k in window k, shifted
 *     inside its window by the giant-step amount: slot kR + j holds W[kR + (j + b) mod R][(j - gB) mod R].  R objects
 *     instead of D (the paper's factor c = 512 / R).
 *   - Baby steps: every chunk of the query must rotate INSIDE its window, which a slot rotation does not do; it is put
 *     together from two slot rotations and 0/1 plaintext masks -- a ciphertext x plaintext multiply, no key switch:
 *     cyc_b = lo_b * rot_b(ct) + hi_b * rot_{b-R}(ct), lo_b[i] = [(i mod R) + b < R], hi_b = 1 - lo_b.  One rescale follows.
 *   - Matrix product and giant steps: inner[g] = sum_b packed[g][b] * cyc_b, then sum_g rot_{gB}(inner[g]) with plain slot
 *     rotations.  These mix adjacent windows; the single final fold acc += rot_{R 2^t}(acc), t < log2 c, adds all windows
 *     up, and a fixed permutation of the windows is invisible to that sum.  Every slot i then holds q_R[i mod R]: the
 *     projected query, already tiled for the scoring levels.  A second rescale brings the scale back to about Delta.
 * Three contexts of the same ring, R, B and special prime carry this: `top` (L primes: baby rotations, masks), `mid` (the
 * first L - 1 primes: matrix product, giant steps, fold) and the scoring context (the first L - 2 primes).  Evaluation
 * keys of a shorter chain are the longer chain's keys restricted to its digits and limbs (one-prime digits), so the
 * client generates them once.  Keys needed: top: rotations b and n - R + b, b = 1 .. B-1; mid: B (Horner; or B .. (G-1)B
 * with HANN_TUNE_GIANT_LAZY) and R 2^t, t < log2 c. */

/* Hoisted slot rotations of one ciphertext: out[i] = rot_{rot0 + i}(ct), i < count -- one digit decomposition of c1, count
 * keys, one ModDown round (what hann_query_prepare does for rotations 1 .. B-1).  out_dev count * HANN_SIZE_CT bytes. */
int hann_rotate_hoisted(hann_ctx *ctx, const void *ct_dev, int rot0, int count, void *out_dev, void *ws, size_t ws_bytes);

/* Encode `count` real slot vectors z_dev [count][n] (device, binary64) at scale 2^log_scale into stored plaintexts
 * pt_dev [count][L][N/2] (the layout of one (g, b) plaintext of hann_encode_candidates).  Enrolment-time call. */
int hann_encode_slots(hann_ctx *ctx, const double *z_dev, int64_t count, int log_scale, void *pt_dev, void *ws, size_t ws_bytes);

/* Enrolment of the projection matrix: W_dev [D][R] float32 row-major (device) -> the R packed diagonals, pt_dev
 * [G][B][L][N/2] (HANN_SIZE_PT_BLOCK bytes: "one block" for hann_score_level) at scale 2^log_scale_w.  Call it on `mid`.
 * ws: hann_workspace_bytes(ctx, 1) is enough. */
int hann_project_enrol(hann_ctx *ctx, const float *W_dev, int D, int log_scale_w, void *pt_dev, void *ws, size_t ws_bytes);

/* The window masks lo_b, hi_b, b < B, as stored plaintexts [B][L][N/2] each at scale 2^log_scale_m.  Call it on `top`. */
int hann_project_masks(hann_ctx *ctx, int log_scale_m, void *lo_dev, void *hi_dev, void *ws, size_t ws_bytes);

/* The baby steps inside the windows: cyc_dev [B] ciphertexts (HANN_SIZE_BABY bytes, scale Delta * mask scale), from two
 * hoisted batches of slot rotations and the mask combine.  ws: hann_project_bytes is enough. */
int hann_project_baby(hann_ctx *ctx, const void *ct_dev, const void *lo_dev, const void *hi_dev, void *cyc_dev, void *ws,
                      size_t ws_bytes);

/* Rescale (the step between two multiplications of a CKKS circuit): every polynomial of `count` ciphertexts is divided
 * by the last prime with rounding, c' = (c - [c]_{q_{L-1}}) / q_{L-1}, which divides message and scale by q_{L-1}.
 * out_dev [count][2][L-1][N]: ciphertexts of the context whose chain is the first L - 1 primes.  (hann_compact_scores
 * with keep = L - 1 under the name the operation has in a circuit.) */
int hann_rescale(hann_ctx *ctx, const void *ct_dev, int64_t count, void *out_dev, void *ws, size_t ws_bytes);

/* Fold: ct += rot_{stride * 2^t}(ct) for t = 0 .. steps-1, in place (keys of those rotations must be loaded).  With
 * stride = R and steps = log2(D / R) this is the projection's final sum over the windows. */
int hann_fold(hann_ctx *ctx, void *ct_dev, int stride, int steps, void *ws, size_t ws_bytes);

/* The whole projection: hann_project_baby and hann_rescale on `top`, then hann_score_level (against the packed matrix as
 * its one block), hann_rotate_sum, hann_fold and hann_rescale on `mid`.  ct_dev: the query on `top`; out_dev: the projected
 * query, one ciphertext of the scoring context ([2][L-2][N]) at scale Delta * 2^log_scale_m / q_{L-1} * 2^log_scale_w /
 * q_{L-2}.  Both contexts must use the same device and stream.  ws: hann_project_bytes(top, mid) bytes. */
int64_t hann_project_bytes(const hann_ctx *top, const hann_ctx *mid);
int hann_project_query(hann_ctx *top, hann_ctx *mid, const void *ct_dev, const void *lo_dev, const void *hi_dev,
                       const void *wpt_dev, int D, void *out_dev, void *ws, size_t ws_bytes);

/* ---- membership (threshold) circuit of the face task (Sec. 3.1 "The norm problem", membership bullet; Sec. 2 "Security
 * parameters": depth 11) ---------------------------------------------------------------------------------------------
 * The server returns, per candidate, a ciphertext slot whose SIGN says whether <x, q_R> >= tau |q_R|: the threshold is
 * scaled into the query's units by r = kappa tau sqrt(|q_R|^2), the root taken by a low-degree Chebyshev polynomial of the
 * encrypted squared norm, and sign(s - r) is amplified by `sign_iters` iterations of f(x) = x (3 - x^2) / 2 (kappa = 1/2
 * keeps everything in [-1, 1]).  Depth: 1 (norm) + ceil(log2 deg) (Chebyshev basis by the product identity T_{m+n} =
 * 2 T_m T_n - T_{m-n}) + 1 (combination) + 2 per sign iteration: 11 at deg = 7, sign_iters = 3, on a chain of 12 primes.
 *   - Chain: prime i of the chain is consumed by the i-th rescale counted from the END; the primes consumed by the second
 *     product of a sign iteration must be about TWICE the scale (that rescale is the division by two), all other scaling
 *     primes about the scale, the first prime large enough for a value of magnitude 1 at that scale.
 *   - Contexts: arith[l-1], l = 1..L, the first l primes with R = B = 1 (relinearisation key loaded as rotation 0 where a
 *     product happens, the keys of rotations 1, 2, .., R/2 on arith[L-2] for the fold); `scorer`: the first
 *     L - depth(threshold) + 1 primes with the rank R and its own B (baby-step keys and the key of rotation B loaded).
 *     All keys are restrictions of the longest chain's keys.  All contexts on one device and stream.
 *   - The client sends lam q_R tiled with period R at scale 2^log_scale, lam^2 = a q_{L-1} / 2^log_scale, a = 2 / (t_hi -
 *     t_lo) ([t_lo, t_hi] must contain |q_R|^2); the candidates are enrolled (hann_encode_candidates on `scorer`) times
 *     kappa / lam.  coef[0..deg]: Chebyshev coefficients of kappa tau sqrt(t) on [t_lo, t_hi], computed by the caller (they
 *     decide integer constants of the circuit, so every party must use the same doubles).
 *   - out_dev [n_blocks][2][1][N] (ciphertexts on the first prime, *out_scale their scale); thr_dev (optional): the
 *     threshold ciphertext [2][*thr_level][N] at *thr_scale.  ws: hann_membership_bytes. */
typedef struct {
    int32_t R, deg, sign_iters, log_scale;
    double tau, t_lo, t_hi;
    const double *coef; /* deg + 1 values */
} hann_membership_params;
int hann_membership_levels(int deg, int sign_iters, int *chain_primes, int *score_level);
int64_t hann_membership_bytes(hann_ctx *const *arith, int L, const hann_ctx *scorer, const hann_membership_params *prm, int64_t n_blocks);
int hann_membership_decide(hann_ctx *const *arith, int L, hann_ctx *scorer, const hann_membership_params *prm, const void *ct_dev,
                           const void *pt_dev, int64_t n_blocks, void *out_dev, double *out_scale, void *thr_dev, int *thr_level,
                           double *thr_scale, void *ws, size_t ws_bytes);

/* Convert `count` elements between the canonical layout (host or device pointer) and the internal device layout.
 * kind POLY / PT: one polynomial of L limbs per element; CT: two.  The canonical form of every kind is [L][N] words per
 * polynomial; the internal form of POLY and CT has the same size, that of PT half of it (HANN_SIZE_PT_BLOCK / R per
 * plaintext), and hann_import of kind PT expects the encoding of a real slot vector (it keeps the first half of the
 * transform). */
int hann_import(hann_ctx *ctx, int kind, const uint64_t *canonical, int64_t count, void *internal_dev);
int hann_export(hann_ctx *ctx, int kind, const void *internal_dev, int64_t count, uint64_t *canonical_out);

/* Seed-compressed fresh ciphertexts (Sec. 7: the public-random half is regenerated from a short seed).  The uniform
 * polynomial is a pure function of (seed, stream): a[l][x] = h(seed, stream, l*N + x) mod q_l with the 64-bit counter
 * hash h = mix(mix(mix(seed + M1) ^ (stream * M2)) + ctr * M1), mix(x): x ^= x >> 32; x *= M1; x ^= x >> 29; x *= M2;
 * x ^= x >> 32, M1 = 0x9E3779B97F4A7C15, M2 = 0xBB67AE8584CAA73B (a benchmark generator, not a cryptographic one).
 * hann_expand_uniform writes a [L][N] (canonical; host or device pointer) -- the client passes it to hann_encrypt_query
 * and uploads only c0 and the seed; hann_import_seeded_ct builds the internal ciphertext (HANN_SIZE_CT bytes, device)
 * from c0 [L][N] (canonical, host or device) and the seed, enqueued on the context's stream. */
int hann_expand_uniform(hann_ctx *ctx, uint64_t seed, uint64_t stream, uint64_t *a_out);
int hann_import_seeded_ct(hann_ctx *ctx, const uint64_t *c0, uint64_t seed, uint64_t stream, void *ct_dev);
/* The same for npoly polynomials stored with `limbs` limbs each (compacted ciphertexts): internal [npoly][limbs][N] ->
 * canonical [npoly][limbs][N]. */
int hann_export_limbs(hann_ctx *ctx, const void *internal_dev, int64_t npoly, int limbs, uint64_t *canonical_out);

/* Output compaction (Sec. 7, storage and upload footprint: switch a ciphertext down to the minimal modulus the rest of
 * its life needs -- for a score ciphertext that is decryption only).  Each score ciphertext [2][L][N] becomes
 * [2][keep][N] (internal layout, transform domain):
 *   rescale = 0: limbs 0..keep-1 are kept as they are.  Exact: c0 + c1*s is the same integer modulo the smaller
 *       product, so this is valid while |scores * scale| stays below q_0..q_{keep-1} / 2 (scale 2^80, two ~50-bit
 *       limbs: scores up to 2^19);
 *   rescale = 1: every polynomial is first divided by the last prime with rounding, c' = (c - [c]_{q_{L-1}}) / q_{L-1}
 *       (centred residue), which divides message and scale by q_{L-1} and adds a rounding error of standard deviation
 *       ~ N / 6 per slot (real part, heavy-tailed: a product of two near-Gaussian values) -- at N = 2^16 and scale
 *       2^80 / q_3 ~ 2^30 that is 2^-16.6 per score, above the scoring path's own error; keep <= L-1.
 * out_dev: hann_compact_bytes(ctx, n_blocks, keep) bytes (device).  `ws` as for the other server calls (only used
 * with rescale = 1).  Nothing is allocated. */
int64_t hann_compact_bytes(const hann_ctx *ctx, int64_t n_blocks, int keep);
int hann_compact_scores(hann_ctx *ctx, const void *score_ct_dev, int64_t n_blocks, int keep, int rescale, void *out_dev,
                        void *ws, size_t ws_bytes);

/* One level end to end from HOST buffers, copies included (Sec. 2 "Reproducing this": one request of the persistent
 * scoring server): the query ciphertext goes up first and its baby set is
 * prepared on a helper stream; the rows follow block by block on an upload stream and every block is encoded as soon as
 * its rows have arrived; the level is cut into groups of blocks (HANN_TUNE_HOST_GROUPS), and a group's multiply-
 * accumulate, rotate-and-sum and export run on scoring streams while later groups are still uploaded and encoded, its
 * score ciphertexts travelling to the host (canonical layout) on a download stream.  Page-locked host buffers are needed
 * for the copies to overlap the kernels (pageable memory works but serialises).  Device buffers for the intermediates
 * are carved from `ws_dev`, which must hold
 * hann_level_host_bytes(ctx, n_rows) bytes.  Returns after everything has finished.
 *   ct_host [2][L][N];  rows_host [n_rows][dim] float32;  score_ct_host [ceil(n_rows/n)][2][L][N] (fewer limbs with
 *   HANN_TUNE_HOST_LIMBS). */
int64_t hann_level_host_bytes(const hann_ctx *ctx, int64_t n_rows);
int hann_score_level_host(hann_ctx *ctx, const uint64_t *ct_host, const float *rows_host, int64_t n_rows, int dim,
                          uint64_t *score_ct_host, void *ws_dev, size_t ws_bytes);

#ifdef __cplusplus
}
#endif
#endif /* HANN_H */
