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

/* One stored group of coupled pairs.  w1b/g1b only for ECOSPA_PAIR_SWIGLU (w1 = gate, w1b = up).
 * g1/g1b/g2 are dL/dW of w1/w1b/w2 in the same shape and layout; ptr == NULL skips Fisher. */
typedef struct {
    int32_t kind;    /* ecospa_pair_kind_t */
    int32_t n_seg;   /* pairs stored side by side (heads); 1 for an FFN */
    int32_t seg_len; /* shared indices per pair (d_h, or the FFN hidden width) */
    int32_t reserved;
    ecospa_mat_t w1, w1b, w2;
    ecospa_mat_t g1, g1b, g2;
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

/* ---------------------------------------------------------------------------------------------
 * Step 1: coupled importance scores.   Eq. "l2norm" (per-index score upsilon) and
 * Eq. "importance" (pair-level empirical Fisher I_hat), Sec. 3.1-3.2.
 *
 *   raw[j]     = ||W_1[:, j]||_2 * ||W_2[j, :]||_2            (SwiGLU: W_1 = gate (.) up)
 *   upsilon[j] = raw[j] / ||raw[segment of j]||_2             (0 if the segment is all zero)
 *   fisher[s]  = 1/2 * ( SS(G_1, s)/|W_1,s| + SS(G_2, s)/|W_2,s| ) / n_samples
 *                (SwiGLU: the W_1 term is the mean of the gate and up terms)
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
 */
size_t ecospa_score_workspace_bytes(const ecospa_pair_t* pairs, int32_t n_pairs);
ecospa_status_t ecospa_score_pairs(const ecospa_pair_t* pairs, int32_t n_pairs, double n_samples, float* upsilon,
                                   float* raw, float* fisher, void* workspace, size_t workspace_bytes,
                                   void* stream);

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
 * access inside `in`).
 */
ecospa_status_t ecospa_compact_tensors(const ecospa_gather_t* jobs, int32_t n_jobs, void* stream);
ecospa_status_t ecospa_compact_pair(const ecospa_pair_t* pair, const int32_t* kept, int32_t n_kept,
                                    const ecospa_mat_t* aux_in, const ecospa_mat_t* aux_out, int32_t n_aux,
                                    const ecospa_mat_t* w1_out, const ecospa_mat_t* w1b_out,
                                    const ecospa_mat_t* w2_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ECOSPA_H_ */
