/* libecospa -- coupled-sparsity hot path of EcoSpa for NVIDIA B200 (sm_100a).
 *
 * Plain C ABI.  Every pointer is tagged HOST or DEVICE below.  The library owns no
 * caller memory, allocates no device memory, and never synchronises the device: each
 * call validates its arguments on the host, enqueues its kernels on `stream`
 * (a cudaStream_t passed as void*) and returns.  Outputs never alias inputs.
 * All calls return an ecospa_status_t; nothing throws, aborts or traps.
 *
 * Vocabulary (paper, Sec. 3): a coupled pair is (W_1, W_2) whose product W_1 W_2 is
 * what the model uses; they share a dimension of size D.  "Shared index" j names
 * column j of W_1 and row j of W_2.  A stored tensor can hold several pairs side by
 * side (the h heads of W^Q): D = n_seg * seg_len, segment s = shared indices
 * [s*seg_len, (s+1)*seg_len) = one coupled pair (one head, Eq. 5).
 */
#ifndef ECOSPA_H_
#define ECOSPA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ECOSPA_OK = 0,
    ECOSPA_ERR_INVALID = 1,      /* null pointer, bad size, k out of range, aliasing              */
    ECOSPA_ERR_ALIGNMENT = 2,    /* pointer / leading dimension not aligned as documented         */
    ECOSPA_ERR_UNSUPPORTED = 3,  /* valid request outside what the kernels cover                  */
    ECOSPA_ERR_CUDA = 4,         /* a CUDA runtime/driver call failed (see ecospa_last_cuda_error) */
    ECOSPA_ERR_TIMEOUT = 5,      /* a bounded device-side wait expired (see ecospa_device_status)  */
    ECOSPA_ERR_WORKSPACE = 6     /* workspace missing or smaller than the matching *_workspace_bytes */
} ecospa_status_t;

typedef enum { ECOSPA_F32 = 0, ECOSPA_BF16 = 1 } ecospa_dtype_t;

/* Where the shared index sits in a row-major tensor. */
typedef enum {
    ECOSPA_SHARED_COLS = 0, /* other_dim x D : shared index j = column j (W_1 as written in Eq. 3: d_m x d) */
    ECOSPA_SHARED_ROWS = 1  /* D x other_dim : shared index j = row j    (W_2 as written in Eq. 3: d x d_m) */
} ecospa_layout_t;

typedef enum {
    ECOSPA_PAIR_PLAIN = 0, /* (W_1, W_2): W^Q/W^K, W^V/W^O per head, W_in/W_out                       */
    ECOSPA_PAIR_SWIGLU = 1 /* W_1 = W_gate (.) W_up (element-wise), W_2 = W_down (footnote to Eq. 8) */
} ecospa_pair_kind_t;

typedef enum {
    ECOSPA_ACT_NONE = 0,
    ECOSPA_ACT_GELU_ERF = 1,  /* x Phi(x), Eq. 3 */
    ECOSPA_ACT_GELU_TANH = 2, /* tanh approximation of the same */
    ECOSPA_ACT_SWIGLU = 3     /* silu(x W_gate) (.) (x W_up) */
} ecospa_act_t;

/* A row-major DEVICE tensor with a shared axis.  `ld` is the row pitch in elements.
 * A vector over the shared axis (a bias) is other_dim = 1, layout SHARED_COLS. */
typedef struct {
    void* ptr;         /* DEVICE; NULL = absent */
    int32_t dtype;     /* ecospa_dtype_t */
    int32_t layout;    /* ecospa_layout_t */
    int64_t other_dim; /* extent of the non-shared axis */
    int64_t ld;        /* elements; >= D (SHARED_COLS) or >= other_dim (SHARED_ROWS) */
} ecospa_mat_t;

/* Rotary position embedding (Eq. "self-attention-rope"): W_Q P_t and W_K P_s rotate the shared index in 2 x 2
 * blocks.  The footnote to Eq. "l2norm" removes on W_Q / W_K and has the position matrices shrink to the new
 * width, so the unit that can be removed is a rotation pair of shared indices; the rotations leave the Frobenius
 * norm of a pair's two columns unchanged at every position.  Which two indices of a segment form pair b: */
typedef enum {
    ECOSPA_ROPE_NONE = 0,        /* no rotation: every shared index is scored and removed on its own */
    ECOSPA_ROPE_INTERLEAVED = 1, /* (2b, 2b+1), the blocks as the paper prints them */
    ECOSPA_ROPE_HALF = 2         /* (b, b + seg_len/2), the "rotate half" storage of the same blocks */
} ecospa_rope_t;

/* One stored group of coupled pairs.  w1b/g1b only for ECOSPA_PAIR_SWIGLU (w1 = gate, w1b = up).
 * g1/g1b/g2 are dL/dW of w1/w1b/w2 in the same shape and layout; ptr == NULL skips Fisher. */
typedef struct {
    int32_t kind;    /* ecospa_pair_kind_t */
    int32_t n_seg;   /* pairs stored side by side (heads); 1 for an FFN */
    int32_t seg_len; /* shared indices per pair (d_h, or the FFN hidden width) */
    int32_t rope;    /* ecospa_rope_t: rotary position embedding acts on this pair group's shared index (Q/K pairs) */
    ecospa_mat_t w1, w1b, w2;
    ecospa_mat_t g1, g1b, g2;
    /* Grouped-query attention ("Extension to GQA": pairs W_i^Q W_g(i)^KT and W_g(i)^V W_i^O).  w1_rep > 1: w1 (and g1)
     * hold w1_rep heads per segment, the heads of a group side by side -- shared extent w1_rep * n_seg * seg_len, head
     * (s, r) in shared indices [(s*w1_rep + r)*seg_len, +seg_len) -- and the segment is scored as ONE pair whose W_1 is
     * the stack of those heads: the norm of index j on that side is taken over all of them (removing index j removes
     * it from every head of the group).  w2_rep likewise for w2 / g2 (the W^O row blocks of a V group).  0 and 1 both
     * mean an ordinary pair.  Plain pairs without rotation pairs only. */
    int32_t w1_rep, w2_rep;
} ecospa_pair_t;

/* One gather job of the compaction step: out = in restricted to the kept shared indices. */
typedef struct {
    ecospa_mat_t in;
    ecospa_mat_t out;    /* same dtype/layout/other_dim; SHARED_COLS: ld >= n_kept, columns [n_kept, ld) are zeroed */
    const int32_t* kept; /* DEVICE: n_kept ascending shared indices of `in` */
    int32_t n_kept;
    int32_t shared_dim;  /* D of `in`: indices are clamped to [0, D) on the device */
} ecospa_gather_t;

const char* ecospa_status_string(ecospa_status_t s);
/* Text of the last CUDA error this thread's calls ran into ("" if none). */
const char* ecospa_last_cuda_error(void);
/* Number of kernels this process has launched through the library so far (all threads). */
uint64_t ecospa_launch_count(void);

/* ---------------------------------------------------------------------------------------------
 * Step 1: coupled importance scores.   Eq. "l2norm" (per-index score upsilon) and
 * Eq. "importance" (pair-level empirical Fisher I_hat), Sec. 3.1-3.2.
 *
 *   raw[j]     = ||W_1[:, j]||_2 * ||W_2[j, :]||_2            (SwiGLU: W_1 = gate (.) up)
 *   upsilon[j] = raw[j] / ||raw[segment of j]||_2             (0 if the segment is all zero)
 *   fisher[s]  = 1/2 * ( SS(G_1, s)/|W_1,s| + SS(G_2, s)/|W_2,s| ) / n_samples
 *                (SwiGLU: the W_1 term is the mean of the gate and up terms)
 *   pair.rope != ECOSPA_ROPE_NONE (plain pairs with an even seg_len only): the scored unit is a rotation pair
 *   {j, j'} of shared indices,
 *                raw[j] = raw[j'] = ||W_1[:, {j, j'}]||_F * ||W_2[{j, j'}, :]||_F,
 *                upsilon[j] = upsilon[j'] = raw[j] / sqrt(sum over the segment's pairs of raw^2)
 *                (both members carry the pair's value; select with ecospa_select_rotation_pairs)
 *
 * pairs      HOST  array of n_pairs descriptors (device tensors inside)
 * n_samples        |D| of Eq. "importance"; > 0
 * upsilon    DEVICE out, fp32, concatenated over pairs: pair p starts at sum_{q<p} D_q
 * raw        DEVICE out, same shape, may be NULL
 * fisher     DEVICE out, fp32, concatenated: sum_p n_seg_p values; may be NULL (gradients ignored);
 *            if not NULL every pair must carry its gradients
 * workspace  DEVICE scratch of at least ecospa_score_workspace_bytes(pairs, n_pairs) bytes, 16-byte aligned;
 *            contents are overwritten; concurrent calls need distinct workspaces
 * Results are bit-identical from run to run (no floating-point atomics).
 * NaN/Inf inputs: unspecified.  Tensors with 16-byte aligned base and ld*sizeof(elem) % 16 == 0
 * take the vector path; others are read element-wise (slower, same results).
 * D = n_seg * seg_len up to 2^22 per pair group (ECOSPA_ERR_UNSUPPORTED beyond).
 */
size_t ecospa_score_workspace_bytes(const ecospa_pair_t* pairs, int32_t n_pairs);
ecospa_status_t ecospa_score_pairs(const ecospa_pair_t* pairs, int32_t n_pairs, double n_samples, float* upsilon,
                                   float* raw, float* fisher, void* workspace, size_t workspace_bytes,
                                   void* stream);

/* Scores of ONE pair group without any workspace argument.  (The paper has no counterpart: this entry
 * point exists only for the sake of callers that cannot allocate.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unavailable -- a plug-in invoked
 * from inside another framework's memory-managed region, a real-time loop that must not touch the
 * allocator, a process whose memory pool is fixed up front -- and therefore has no way to obtain the
 * scratch buffer that ecospa_score_pairs asks for.  Here the scratch is a fixed 4 MiB array inside the
 * library's device image (ecospa_score_pair_static_max_bytes()); every GPU that loads the library holds
 * it until the process exits.  The call itself allocates nothing on the device.
 *
 * Same inputs, outputs and results as ecospa_score_pairs with n_pairs == 1.  Differences:
 *   - a pair group whose scratch need exceeds the array returns ECOSPA_ERR_UNSUPPORTED (the text from
 *     ecospa_last_cuda_error says so) and launches nothing; ecospa_score_workspace_bytes(pair, 1) tells
 *     the need in advance;
 *   - the first call on each device looks up the array's device address (with that device current); make
 *     that first call before starting any stream capture;
 *   - every call on a device shares the one array and finds the previous call's data in it.  Nothing in
 *     it has to start at zero (each value is written before it is read), but two calls that overlap on
 *     the GPU (different streams, or several host threads) race on it: serialise them.
 */
size_t ecospa_score_pair_static_max_bytes(void);
ecospa_status_t ecospa_score_pair_static(const ecospa_pair_t* pair, double n_samples, float* upsilon, float* raw,
                                         float* fisher, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 2: aligned top-k per pair.   Definition 1 (coupled sparsification), App. A.2, applied to the
 * seg_len - k lowest-scored indices of each segment; Alg. 1 "remove smallest upsilon_i".
 *
 * Keeps, in every segment, the k indices with the largest score; equal scores keep the lower index
 * (comparison on the fp32 values as stored; -0 == +0).  Kept indices are written ascending, as shared
 * indices of the pair group (segment offset included), segments one after another.
 *
 * upsilon      DEVICE fp32, concatenated as written by ecospa_score_pairs
 * n_seg        HOST [n_pairs]     seg_len HOST [n_pairs]
 * k_per_seg    HOST concatenated over pairs (sum n_seg entries), 0 <= k <= seg_len
 * kept         DEVICE out int32, concatenated over all segments of all pairs (sum of k entries)
 * seg_offsets  DEVICE out int32 [total segments + 1] prefix sums of k; may be NULL
 * seg_len up to 2^20.  No workspace.
 */
ecospa_status_t ecospa_select_aligned_topk(const float* upsilon, const int32_t* n_seg, const int32_t* seg_len,
                                           const int32_t* k_per_seg, int32_t n_pairs, int32_t* kept,
                                           int32_t* seg_offsets, void* stream);

/* Step 2 with rotary position embedding: as ecospa_select_aligned_topk, but pair groups with rope[p] !=
 * ECOSPA_ROPE_NONE keep whole rotation pairs (footnote to Eq. "l2norm": removal on W_Q / W_K, the position
 * matrices shrink with them).  For such a group k_per_seg counts shared indices and must be even, seg_len must be
 * even; the k/2 pairs with the largest score stay (the score is read at a pair's first member; equal scores: the
 * lower pair first).  Kept indices are ascending; for ECOSPA_ROPE_HALF that puts the first members of the kept
 * pairs before their second members, so the compacted matrix keeps the (u, u + k/2) pairing.
 * rope HOST [n_pairs] of ecospa_rope_t.  Everything else as in ecospa_select_aligned_topk. */
ecospa_status_t ecospa_select_rotation_pairs(const float* upsilon, const int32_t* n_seg, const int32_t* seg_len,
                                             const int32_t* k_per_seg, const int32_t* rope, int32_t n_pairs,
                                             int32_t* kept, int32_t* seg_offsets, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 2, variable counts: the stopping rule of Algorithm 1 ("while the sum of the scores exceeds theta:
 * remove the smallest score and its row/column") and its choice of pairs ("the top-K coupled matrices with
 * the smallest importance").
 *
 * ecospa_choose_pairs: chosen[i] = 1 for the m smallest of the n importance values (Eq. "importance", as
 *   written by ecospa_score_pairs), equal values: lower index first; 0 otherwise.  n <= 16384.
 *   fisher DEVICE fp32 [n], chosen DEVICE out int32 [n].
 *
 * ecospa_select_aligned_threshold: for every segment, removes the lowest-scored indices one after the other
 *   (equal scores: the higher index goes first) while the sum of the scores that are left exceeds
 *   theta * total and more than k_min indices are left; total = the sum of all scores of the segment when
 *   l1 != 0 (theta = share of the score mass that may stay), 1 when l1 == 0 (scores compared as stored).
 *   Sums are taken in fp64.  Scores must be >= 0 (they are products of norms).  Segments with chosen[s] == 0
 *   keep everything (chosen may be NULL: every segment is processed).
 *   upsilon  DEVICE fp32, concatenated as written by ecospa_score_pairs
 *   n_seg, seg_len HOST [n_pairs]
 *   rope     HOST [n_pairs] of ecospa_rope_t, may be NULL (no rotation pairs).  A group with rotation pairs is
 *            processed pair by pair: every pair's score counts once, pairs leave whole, k_out is even and at
 *            least k_min rounded up to whole pairs (scores as written by ecospa_score_pairs for such a group)
 *   chosen   DEVICE int32 per segment (all pairs concatenated), may be NULL
 *   kept     DEVICE out int32 with one slot per shared index (sum of n_seg * seg_len entries): segment s of
 *            a pair writes its kept indices, ascending and relative to the pair group as in
 *            ecospa_select_aligned_topk, at the position of its first shared index; the first k_out[s]
 *            entries of the slot are valid, the rest is left untouched
 *   k_out    DEVICE out int32 per segment: how many indices stay.  The caller reads it back to size the
 *            compacted tensors (the counts are data dependent).
 * Errors: theta < 0 or NaN, k_min < 0 -> ECOSPA_ERR_INVALID; seg_len > 2^20 -> ECOSPA_ERR_UNSUPPORTED.
 */
ecospa_status_t ecospa_choose_pairs(const float* fisher, int32_t n, int32_t m, int32_t* chosen, void* stream);
ecospa_status_t ecospa_select_aligned_threshold(const float* upsilon, const int32_t* n_seg, const int32_t* seg_len,
                                                const int32_t* rope, int32_t n_pairs, double theta, int32_t l1,
                                                int32_t k_min, const int32_t* chosen, int32_t* kept, int32_t* k_out,
                                                void* stream);

/* Turns the slots that ecospa_select_aligned_threshold wrote into the kept list of a whole tensor (the input of
 * step 3): out[dst[s] + i] = slots[src[s] + i] + add[s] for i < k[s], segment by segment.  src, dst, k, add: HOST
 * [n_segs] (k as read back from k_out; add = what turns a slot's indices into shared indices of the tensor being
 * compacted, e.g. the column offset of a head that was scored as a group of its own).  slots, out: DEVICE.
 * Index bookkeeping only; no counterpart in the paper beyond "remove the i-th row/column" of Algorithm 1. */
ecospa_status_t ecospa_pack_kept(const int32_t* slots, const int32_t* src, const int32_t* dst, const int32_t* k,
                                 const int32_t* add, int32_t n_segs, int32_t* out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * One pass of the body of Algorithm 1 over whole groups of pairs (everything between "if Param(W_t) > c" and the
 * end of the loop body): importance of every pair, the n_choose pairs with the smallest importance, their scores,
 * removal of the lowest-scored aligned indices while the remaining score mass exceeds theta, and the removal of the
 * same rows / columns from every tensor of the group (gradients, optimizer moments, biases).
 *
 * A group = the tensors that live on one shared axis: the six tensors of ecospa_pair_t plus n_aux further ones (HOST
 * array `aux`; a 1-D bias is other_dim = 1, SHARED_COLS), and the widths of its pairs (HOST, n_pairs entries; the pairs sit
 * side by side on the shared axis, sum of widths = its extent; after a pass the widths differ from pair to pair; width 0
 * = a pair that has lost every index and takes no part).
 * ecospa_alg1_plan     enqueues scoring, pair choice and threshold selection, waits for the stream (the one
 *                      synchronisation: the counts size what follows) and writes the new width of every pair to
 *                      k_host (HOST, one entry per pair of every group, in order).  Gradients are required.
 * ecospa_alg1_apply    enqueues the removal: into the tensors of out[g] (same structure, caller-allocated for the
 *                      widths in k_host, padded pitches as in step 3), or, with in_place != 0, inside the tensors
 *                      themselves (out may be NULL; see ecospa_compact_tensors_inplace).  Must follow a plan call on the same
 *                      groups with the same workspace.
 * workspace: DEVICE, ecospa_alg1_workspace_bytes, 16-byte aligned; between the two calls it holds the scores,
 * importance values, choice flags and kept lists; ecospa_alg1_offsets gives their byte offsets
 * (offsets[0..3] = upsilon, importance, choice flags, kept lists; offsets[4..5] = total shared indices and pairs described),
 * in the order of the described pairs (groups in order, pairs of width 0 left out).  theta, l1, k_min as in
 * ecospa_select_aligned_threshold.  */
typedef struct {
    ecospa_mat_t w1, w1b, w2;   /* w1b: SwiGLU up matrix or absent */
    ecospa_mat_t g1, g1b, g2;
    const ecospa_mat_t* aux;    /* HOST [n_aux] */
    int32_t n_aux;
    int32_t n_pairs;
    const int32_t* widths;      /* HOST [n_pairs] */
    int32_t rope;               /* ecospa_rope_t of the group's pairs */
    int32_t reserved_;
} ecospa_group_t;

size_t ecospa_alg1_workspace_bytes(const ecospa_group_t* groups, int32_t n_groups);
ecospa_status_t ecospa_alg1_offsets(const ecospa_group_t* groups, int32_t n_groups, int64_t* offsets);
ecospa_status_t ecospa_alg1_plan(const ecospa_group_t* groups, int32_t n_groups, double n_samples, int32_t n_choose,
                                 double theta, int32_t l1, int32_t k_min, void* workspace, size_t workspace_bytes,
                                 int32_t* k_host, void* stream);
ecospa_status_t ecospa_alg1_apply(const ecospa_group_t* groups, int32_t n_groups, const int32_t* k_host,
                                  const ecospa_group_t* out, int32_t in_place, void* workspace, size_t workspace_bytes,
                                  void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 3: physical removal.   Definition 1: drop column j of W_1 and row j of W_2 for every removed j
 * "keeping the original pairings"; Alg. 1 also drops the same rows/columns of the optimizer moments.
 *
 * ecospa_compact_tensors: n_jobs independent gathers in one launch sequence (HOST array of jobs).
 * ecospa_compact_pair:    the three (two) weight tensors of one pair group plus n_aux auxiliary tensors
 *                         (bias over the shared axis, gradients, optimizer moments) with one kept list.
 * Byte-exact copies; pad elements up to the next 16-byte boundary of each output row (columns
 * [n_kept, round_up(n_kept, 16 bytes)) for SHARED_COLS, [other_dim, round_up(other_dim, 16 bytes)) for
 * SHARED_ROWS, never beyond ld) are zero-filled.  out must not overlap in.
 * kept indices must be ascending and < D (not checked on the device beyond a clamp that keeps every
 * access inside `in`).  An entry of -1 stands for "no index": the output gets a zero column (row) at that position
 * (used to pad every head's block of a compacted tensor to the width the attention kernels need).
 */
ecospa_status_t ecospa_compact_tensors(const ecospa_gather_t* jobs, int32_t n_jobs, void* stream);
/* In-place variant of the same removal (Algorithm 1 shrinks the matrices and the optimizer moments it holds; a caller
 * that cannot afford a second copy of them uses this form): every job must have out.ptr == in.ptr and out.ld == in.ld.
 * The kept part moves to the front of the shared axis (columns [0, n_kept) of a SHARED_COLS tensor, zero pad up to the
 * next 16-byte boundary as above; rows [0, n_kept) of a SHARED_ROWS tensor); what lies behind it afterwards is
 * unspecified.  Every kept index must be at least its position in the list, kept[c] >= c (true of any ascending list,
 * and of lists whose blocks are padded with -1 entries to no more than the blocks' original width): that is what makes
 * a front-to-back walk safe; -1 entries give zeros.
 * Same bytes as ecospa_compact_tensors on the kept part; slower (one warp walks a row or a 512-byte column stripe). */
ecospa_status_t ecospa_compact_tensors_inplace(const ecospa_gather_t* jobs, int32_t n_jobs, void* stream);
ecospa_status_t ecospa_compact_pair(const ecospa_pair_t* pair, const int32_t* kept, int32_t n_kept,
                                    const ecospa_mat_t* aux_in, const ecospa_mat_t* aux_out, int32_t n_aux,
                                    const ecospa_mat_t* w1_out, const ecospa_mat_t* w1b_out,
                                    const ecospa_mat_t* w2_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Step 4: forward / backward of the compacted coupled pairs.
 *
 * The dense layer math of Eq. 2 (Q, K, V projections), Eq. 5 (output projection with W^O as a stack of
 * per-head row blocks) and Eq. 3 (FFN; SwiGLU variant per the footnote to Eq. 8) evaluated on the
 * matrices that aligned removal leaves, and the reverse-mode derivatives of the same expressions.
 * bf16 operands on the tensor cores with fp32 accumulation; the FFN activation (and, in the backward
 * pass, its derivative) is fused into the epilogue of the W_1 (resp. dY W_2^T) product.
 *
 * Common conventions
 *   T, d_m        tokens (batch*seq) and model width; n / k = real number of kept shared indices.
 *   dtype         taken from the first weight descriptor.  ECOSPA_BF16: every activation, gradient and
 *                 output below is bf16.  ECOSPA_F32: X, upstream gradients, biases, Y/Q/K/V/Out, dX and all
 *                 weight/bias gradients are fp32; operands are rounded to bf16 in the workspace first.
 *                 The saved FFN tensors H, Hb, A are bf16 in both cases.
 *   weights       compacted matrices as written by step 3, each in either orientation (the descriptor's
 *                 layout says which): ECOSPA_SHARED_COLS = d_m x n, ECOSPA_SHARED_ROWS = n x d_m, pitch ld.
 *                 The equations' orientation is SHARED_COLS for W_Q^c, W_K^c, W_V^c, W_1^c (W_gate^c, W_up^c)
 *                 and SHARED_ROWS for W_O^c, W_2^c; the transposed storage of each (what a framework's
 *                 linear layer keeps) is consumed as it is, nothing is transposed in memory.  other_dim
 *                 must equal d_m.  A weight gradient is written in the orientation of its weight
 *                 (d_m x n with pitch >= n, or n x d_m with pitch >= d_m).
 *   pitches       all ld* in elements.  Every base pointer must be 16-byte aligned and every pitch a
 *                 multiple of 16 bytes (ECOSPA_ERR_ALIGNMENT otherwise); gradient outputs use the pitch
 *                 of a compacted weight (padded).  Only the real extent of an output is written (tile stores
 *                 clipped at n, k, d_m and T); pad columns keep what the buffer held.
 *   workspace     DEVICE scratch, 16-byte aligned, at least ecospa_proj_workspace_bytes /
 *                 ecospa_ffn_workspace_bytes; may be NULL when that function returns 0.
 *   1/sqrt(d_h)   is not applied: Q^c and K^c are the plain projections.
 * All DEVICE pointers; results are deterministic (fixed summation order).  A device-side wait that
 * expires records a code readable with ecospa_device_status.
 */
size_t ecospa_proj_workspace_bytes(int64_t T, int64_t d_m, int64_t n, int32_t dtype);
size_t ecospa_ffn_workspace_bytes(int64_t T, int64_t d_m, int64_t k, int32_t act, int32_t dtype);

/* Q^c = X W_Q^c + b_Q^c, K^c = X W_K^c + b_K^c (Eq. 2 on the compacted pair).  X: T x d_m (pitch ldx);
 * Qc, Kc: T x n (pitch ld_out).  bq_c / bk_c may be NULL.  wk_c == NULL computes Q^c only. */
ecospa_status_t ecospa_coupled_qk_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wq_c,
                                      const ecospa_mat_t* wk_c, int64_t n, const void* bq_c, const void* bk_c,
                                      void* Qc, void* Kc, int64_t ld_out, void* workspace, size_t workspace_bytes,
                                      void* stream);
/* Given dQc, dKc (T x n, pitch ld_dqk): dX = dQc W_Q^cT + dKc W_K^cT (added to dX if accumulate_dX),
 * dW_Q^c = X^T dQc, dW_K^c = X^T dKc (d_m x n, pitch ld_dw), db = column sums (may be NULL).
 * accumulate_dX, here and in the calls below: the product is rounded to the type of dX and then added to
 * the stored dX by one reducing tile store per element (bf16 models: two roundings; fp32 models: exact
 * fp32 addition); each element is added exactly once, so the result does not depend on timing. */
ecospa_status_t ecospa_coupled_qk_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wq_c,
                                      const ecospa_mat_t* wk_c, int64_t n, const void* dQc, const void* dKc,
                                      int64_t ld_dqk, void* dX, int64_t ld_dx, int32_t accumulate_dX, void* dWq_c,
                                      void* dWk_c, int64_t ld_dw, void* dbq_c, void* dbk_c, void* workspace,
                                      size_t workspace_bytes, void* stream);

/* V^c = X W_V^c + b_V^c;  Out = Ctx W_O^c + b_O, where Ctx (T x n) is the attention-mixed values of the
 * compacted heads supplied by the caller (Eq. 5).  */
ecospa_status_t ecospa_coupled_vo_fwd_v(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wv_c,
                                        int64_t n, const void* bv_c, void* Vc, int64_t ld_out, void* workspace,
                                        size_t workspace_bytes, void* stream);
ecospa_status_t ecospa_coupled_vo_fwd_o(const void* Ctx, int64_t ld_ctx, int64_t T, int64_t d_m,
                                        const ecospa_mat_t* wo_c, int64_t n, const void* bo, void* Out, int64_t ld_out,
                                        void* workspace, size_t workspace_bytes, void* stream);
/* dCtx = dOut W_O^cT, dW_O^c = Ctx^T dOut (n x d_m), dbo = colsum(dOut); dW_V^c = X^T dVc, dX (+)= dVc W_V^cT,
 * dbv = colsum(dVc). */
ecospa_status_t ecospa_coupled_vo_bwd(const void* X, int64_t ldx, const void* Ctx, int64_t ld_ctx, int64_t T,
                                      int64_t d_m, const ecospa_mat_t* wv_c, const ecospa_mat_t* wo_c, int64_t n,
                                      const void* dVc, int64_t ld_dv, const void* dOut, int64_t ld_dout, void* dX,
                                      int64_t ld_dx, int32_t accumulate_dX, void* dCtx, int64_t ld_dctx, void* dWv_c,
                                      int64_t ld_dwv, void* dWo_c, int64_t ld_dwo, void* dbv_c, void* dbo,
                                      void* workspace, size_t workspace_bytes, void* stream);

/* The same products grouped the way a training step meets them (one launch each):
 *   ecospa_coupled_qkv_fwd   Q^c, K^c (n_qk columns) and V^c (n_vo columns) from one X; the QK and VO pairs of
 *                            a block may keep different numbers of columns.
 *   ecospa_coupled_vo_bwd_o  what follows from dOut alone: dCtx = dOut W_O^cT (input of the caller's attention
 *                            backward), dW_O^c = Ctx^T dOut, dbo.
 *   ecospa_coupled_qkv_bwd   what follows once dQ^c, dK^c, dV^c are known: dW_Q^c, dW_K^c, dW_V^c, the three bias
 *                            gradients and dX = dQ^c W_Q^cT + dK^c W_K^cT + dV^c W_V^cT (added to dX if accumulate_dX).
 *   ecospa_coupled_vo_bwd_v  the V part of the above on its own.
 * Arguments as in the calls above (ld_dwqk / ld_dwv: pitches of the weight-gradient outputs). */
ecospa_status_t ecospa_coupled_qkv_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wq_c,
                                       const ecospa_mat_t* wk_c, const ecospa_mat_t* wv_c, int64_t n_qk, int64_t n_vo,
                                       const void* bq_c, const void* bk_c, const void* bv_c, void* Qc, void* Kc, void* Vc,
                                       int64_t ld_qk, int64_t ld_v, void* workspace, size_t workspace_bytes, void* stream);
ecospa_status_t ecospa_coupled_qkv_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wq_c,
                                       const ecospa_mat_t* wk_c, const ecospa_mat_t* wv_c, int64_t n_qk, int64_t n_vo,
                                       const void* dQc, const void* dKc, const void* dVc, int64_t ld_dqk, int64_t ld_dv,
                                       void* dX, int64_t ld_dx, int32_t accumulate_dX, void* dWq_c, void* dWk_c,
                                       void* dWv_c, int64_t ld_dwqk, int64_t ld_dwv, void* dbq_c, void* dbk_c,
                                       void* dbv_c, void* workspace, size_t workspace_bytes, void* stream);
ecospa_status_t ecospa_coupled_vo_bwd_o(const void* Ctx, int64_t ld_ctx, int64_t T, int64_t d_m,
                                        const ecospa_mat_t* wo_c, int64_t n, const void* dOut, int64_t ld_dout,
                                        void* dCtx, int64_t ld_dctx, void* dWo_c, int64_t ld_dwo, void* dbo,
                                        void* workspace, size_t workspace_bytes, void* stream);
ecospa_status_t ecospa_coupled_vo_bwd_v(const void* X, int64_t ldx, int64_t T, int64_t d_m, const ecospa_mat_t* wv_c,
                                        int64_t n, const void* dVc, int64_t ld_dv, void* dX, int64_t ld_dx,
                                        int32_t accumulate_dX, void* dWv_c, int64_t ld_dwv, void* dbv_c, void* workspace,
                                        size_t workspace_bytes, void* stream);

/* FFN on a compacted pair with k hidden units (Eq. 3):
 *   GELU   : H = X W_1^c + b_1^c, A = GELU(H), Y = A W_2^c + b_2
 *   SwiGLU : H = X W_gate^c, Hb = X W_up^c, A = silu(H) (.) Hb, Y = A W_2^c        (w1_c = gate, w1b_c = up)
 * H, Hb, A: bf16 T x k (pitch ld_h), written for the backward pass; Y: T x d_m (pitch ld_y). */
ecospa_status_t ecospa_coupled_ffn_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, int32_t act,
                                       const ecospa_mat_t* w1_c, const ecospa_mat_t* w1b_c, const ecospa_mat_t* w2_c,
                                       int64_t k, const void* b1_c, const void* b2, void* Y, int64_t ld_y, void* H,
                                       void* Hb, void* A, int64_t ld_h, void* workspace, size_t workspace_bytes,
                                       void* stream);
/* Given dY (T x d_m): dH = (dY W_2^cT) (.) act'(H)  [SwiGLU: dH = dA (.) Hb (.) silu'(H), dHb = dA (.) silu(H)],
 * dW_2^c = A^T dY (k x d_m, pitch ld_dw2), dW_1^c = X^T dH (d_m x k, pitch ld_dw1; dW1b_c = X^T dHb),
 * dX = dH W_1^cT (+ dHb W_up^cT), db1 = colsum(dH) (GELU only), db2 = colsum(dY); db* may be NULL. */
ecospa_status_t ecospa_coupled_ffn_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, int32_t act,
                                       const ecospa_mat_t* w1_c, const ecospa_mat_t* w1b_c, const ecospa_mat_t* w2_c,
                                       int64_t k, const void* H, const void* Hb, const void* A, int64_t ld_h,
                                       const void* dY, int64_t ld_dy, void* dX, int64_t ld_dx, void* dW1_c,
                                       void* dW1b_c, int64_t ld_dw1, void* dW2_c, int64_t ld_dw2, void* db1_c,
                                       void* db2, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Attention core on the compacted heads: the head of Eq. 2,
 *     head_i = phi( Q_i K_i^T / sqrt(d_h) ) V_i ,
 * evaluated on the matrices that aligned removal leaves (Sec. 3.1, "Coupled Weight Matrix in MHA": the pair
 * W_i^Q W_i^KT restricted to the kept indices of the QK pair, W_i^V W_i^O to those of the VO pair), so the Q/K width
 * and the V width differ from each other and from head to head.  It sits between ecospa_coupled_qkv_fwd and
 * ecospa_coupled_vo_fwd_o (and, in the backward pass, between ecospa_coupled_vo_bwd_o and ecospa_coupled_qkv_bwd).
 *
 * Layout: Qc, Kc (T x n_qk, pitch ld_qk) hold head h in columns [qk_off[h], qk_off[h] + qk_w[h]); Vc, Ctx and dCtx
 * hold it in columns [vo_off[h], vo_off[h] + vo_w[h]).  T = batch * seq, sequence b = rows [b*seq, (b+1)*seq).
 * Every width must be a multiple of 16 (at most 128) and every offset a multiple of 8: give the compaction step a
 * kept list in which every head's block is padded with -1 entries (ecospa_pad_kept) -- a zero column of Q^c / K^c adds
 * nothing to Q K^T and a zero column of V^c yields a zero column of Ctx, so results on the real columns do not
 * change.  bf16 tensors only; at most 128 heads.
 *   scale   the caller's 1/sqrt(d_h) with the architectural d_h of Eq. 2 (removal does not change it); > 0
 *   causal  != 0: query i attends to keys j <= i of its sequence (Eq. 2 prints no mask: causal == 0 is the equation
 *           as printed; decoder models mask)
 *   lse     DEVICE fp32 [n_heads * T]: lse[h*T + t] = log sum_j exp(scale * q_t . k_j), written by the forward call
 *           and read by the backward call
 * Forward: Ctx (T x n_vo, pitch ld_ctx); only the heads' columns of rows < T are written.
 * Backward (reverse mode of the same expression): given dCtx, writes dQc, dKc (pitch ld_dqk) and dVc (pitch ld_dv) in
 * the layout of Qc, Kc, Vc.  workspace: DEVICE, at least ecospa_attn_workspace_bytes, 16-byte aligned.
 * Results are deterministic (no atomics: dK and dV are accumulated by the CTA that owns the key block, dQ by the CTA
 * that owns the query block).  A device-side wait that expires records codes 11-13 (forward), 14-19 (backward).
 */
typedef struct {
    int32_t n_heads;       /* query heads */
    const int32_t* qk_off; /* HOST [n_heads] first column of head h in Qc (and in Kc, unless K/V heads are shared) */
    const int32_t* qk_w;   /* HOST [n_heads] its (padded) width */
    const int32_t* vo_off; /* HOST [n_heads] first column of head h in Ctx / dCtx (and in Vc, unless K/V heads are shared) */
    const int32_t* vo_w;   /* HOST [n_heads] its (padded) width */
    /* Grouped-query models (Sec. 3.1, "Extension to GQA"): n_kv_heads > 0 says that n_heads / n_kv_heads consecutive
     * query heads read the K and V columns of one K/V head, head h those of head g = h / (n_heads / n_kv_heads).  Kc,
     * dKc then hold one block per K/V head at k_off[g] (width qk_w of its query heads, which share the group's kept
     * indices and hence its widths: anything else is ECOSPA_ERR_INVALID), Vc, dVc one at v_off[g] (width vo_w); dKc and
     * dVc receive the sum over the group's query heads.  Pitches stay as documented (Kc shares ld_qk with Qc).
     * n_kv_heads == 0 (a zeroed tail of the struct): every query head has its own K/V head, k_off / v_off are not read. */
    int32_t n_kv_heads;
    const int32_t* k_off;  /* HOST [n_kv_heads] */
    const int32_t* v_off;  /* HOST [n_kv_heads] */
} ecospa_heads_t;

size_t ecospa_attn_workspace_bytes(int64_t batch, int64_t seq, int32_t n_heads);
ecospa_status_t ecospa_coupled_attn_fwd(const void* Qc, const void* Kc, int64_t ld_qk, const void* Vc, int64_t ld_v,
                                        int64_t batch, int64_t seq, const ecospa_heads_t* heads, float scale,
                                        int32_t causal, void* Ctx, int64_t ld_ctx, float* lse, void* stream);
ecospa_status_t ecospa_coupled_attn_bwd(const void* Qc, const void* Kc, int64_t ld_qk, const void* Vc, int64_t ld_v,
                                        const void* Ctx, int64_t ld_ctx, const void* dCtx, int64_t ld_dctx,
                                        const float* lse, int64_t batch, int64_t seq, const ecospa_heads_t* heads,
                                        float scale, int32_t causal, void* dQc, void* dKc, int64_t ld_dqk, void* dVc,
                                        int64_t ld_dv, void* workspace, size_t workspace_bytes, void* stream);

/* Kept list with padded segments: for every segment s (HOST arrays of n_segs entries), out[dst[s] + i] =
 * kept[src[s] + i] for i < k[s] and -1 for k[s] <= i < k_padded[s].  A -1 entry makes the compaction step write a
 * zero column (row) at that position.  kept, out: DEVICE int32.  Index bookkeeping only (no counterpart in the paper). */
ecospa_status_t ecospa_pad_kept(const int32_t* kept, const int32_t* src, const int32_t* dst, const int32_t* k,
                                const int32_t* k_padded, int32_t n_segs, int32_t* out, void* stream);

/* How many CTA pairs (2-SM clusters) of the GEMM engine are resident at once on the current device; 0 when
 * pair mode is off (environment ECOSPA_GEMM_PAIR=0), -1 on a CUDA error.  Informational. */
int32_t ecospa_gemm_resident_pairs(void);

/* Synchronises `stream` and reports the status word of the current device: ECOSPA_OK and *code = 0, or
 * ECOSPA_ERR_TIMEOUT and *code = which bounded wait expired (1 producer, 2 accumulator-free,
 * 3 operands-ready, 4 accumulator-ready; 11-19: the attention kernels); the word is cleared.  This is the one call
 * that blocks.
 * Every device the library is used on has its own status word. */
ecospa_status_t ecospa_device_status(void* stream, int32_t* code);

/* How long a device-side wait of the step-4 kernels (on an operand copy, a free pipeline stage or an
 * accumulator) may last before the kernel gives up, records its code and returns; nanoseconds, default
 * 2 s, process-wide, read when a call enqueues its launches.  ns == 0 -> ECOSPA_ERR_INVALID.  (No counterpart in
 * the paper: failure reporting of this library.) */
ecospa_status_t ecospa_set_device_wait_limit_ns(uint64_t ns);

#ifdef __cplusplus
}
#endif
#endif /* ECOSPA_H_ */
