/*
 * gpd.h — C ABI of the Generalized PolyDot coded matrix-multiplication library (sm_100a).
 *
 * Method: Dutta, Bai, Jeong, Low, Grover, "A Unified Coded Deep Neural Network Training
 * Strategy Based on Generalized PolyDot Codes for Matrix Multiplication" (arXiv 1811.10751).
 * The P "nodes" of the paper are P slices of batched kernels on one GPU.
 *
 * Conventions for every call
 *   - Orientation is the paper's (Section II-B): W is N1 x N0, X is N0 x B (a column is one
 *     sample), Delta^T is B x N1; every matrix is dense row-major.
 *   - W is split into m x n blocks, X into n x d1 blocks, Delta^T into d2 x m blocks
 *     (Section IV, Section VIII).  Substitution u = v^n, w = v^(mn) (Theorem 2).
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; pointers named *_host
 *     are HOST pointers read during the call.  The library keeps no reference to either
 *     after the call returns (device pointers: after the enqueued work completes).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Compute
 *     calls only enqueue work and never synchronise; the return value reports host-detectable
 *     errors only.  Data-dependent outcomes (no error / corrected / decoding failure) are
 *     written to a gpd_locate_result in device memory.  With the plan uploaded beforehand
 *     (gpd_plan_upload) the compute calls below, gpd_locate_errors_static excepted, may be issued
 *     on a stream that is being captured into a CUDA graph; the graph's kernels read the plan's
 *     device tables, so the plan must outlive every replay.
 *   - The library allocates device memory only for the plan's small coefficient tables and, on
 *     FP32 plans, a scratch area of 64 KB per SM behind them (one allocation, made by
 *     gpd_plan_upload or on the plan's first compute call, freed by gpd_plan_destroy).
 *   - Storage type of shares and worker outputs: float (GPD_PREC_FP32) or double
 *     (GPD_PREC_FP64); inputs W, X, Delta and decoded results are always float.
 *   - A plan is immutable after creation; concurrent calls on different streams need distinct
 *     workspaces and result structs.
 */
#ifndef GPD_H_
#define GPD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GPD_MAX_NODES 64        /* P <= 64 */
#define GPD_MAX_THRESHOLD 32    /* every recovery threshold of the plan <= 32 */
#define GPD_MAX_PARITY 32       /* P - Q <= 32 for every product of the plan */
#define GPD_STATIC_MAX_PARITY 16 /* P - Q <= 16 for gpd_locate_errors_static (built-in scratch) */

typedef struct gpd_plan_s* gpd_plan_t;

typedef enum {
    GPD_OK = 0,
    GPD_ERR_ARG = 1,            /* NULL pointer, bad enum value */
    GPD_ERR_SHAPE = 2,          /* m does not divide N1, n not N0, d1 or d2 not B, sizes <= 0 */
    GPD_ERR_POINTS = 3,         /* repeated or non-finite evaluation points */
    GPD_ERR_P_TOO_SMALL = 4,    /* P below a recovery threshold of the plan */
    GPD_ERR_Q_TOO_LARGE = 5,    /* threshold > GPD_MAX_THRESHOLD, P > GPD_MAX_NODES, P-Q > GPD_MAX_PARITY */
    GPD_ERR_WORKSPACE = 6,      /* NULL workspace */
    GPD_ERR_CUDA = 7,           /* a CUDA runtime call failed (no device, launch failure) */
    GPD_ERR_TIMEOUT = 8,        /* a bounded device-side wait expired (reported through status words) */
    GPD_ERR_UNSUPPORTED = 9,    /* combination not implemented */
    GPD_ERR_STATIC_LIMIT = 10   /* problem exceeds the built-in scratch of a no-allocation entry point */
} gpd_status;

/* The three exits of Algorithm 1 (Section V-A). */
typedef enum { GPD_NO_ERROR = 0, GPD_CORRECTED = 1, GPD_DECODE_FAILURE = 2 } gpd_outcome;

/* Which coded product a call works on. */
typedef enum {
    GPD_FWD = 0,                /* S = W X            (step O1; Theorem 2)                       */
    GPD_BWD = 1,                /* C^T = Delta^T W    (step O2; backpropagation stage, Sec. VIII) */
    GPD_UPD = 2,                /* W~_p += eta Delta^_p X^_p^T (step O3; Eq. 10)                  */
    GPD_AUDIT = 3               /* W itself read back from its shares (degree mn-1 polynomial;
                                   footnote on regeneration, Section VI)                         */
} gpd_product;

/* Which matrix gpd_encode_B encodes. */
typedef enum {
    GPD_OPERAND_X_FWD = 0,      /* X (N0 x B)  -> [P][N0/n][B/d1],  X_jk at v^(n-1-j + mn k)      */
    GPD_OPERAND_DELTAT_BWD = 1, /* Delta^T (B x N1) -> [P][B/d2][N1/m], block (k,i) at v^(mn k + n(m-1-i)) */
    GPD_OPERAND_DELTA_UPD = 2,  /* Delta (N1 x B) -> [P][N1/m][B],  Delta_i at v^(n i)  (ascending) */
    GPD_OPERAND_X_UPD = 3       /* X (N0 x B)  -> [P][N0/n][B],     X_j at v^j          (ascending) */
} gpd_operand;

typedef enum {
    GPD_PREC_AUTO = 0,          /* FP32 if every threshold of the plan is <= 9, else FP64 */
    GPD_PREC_FP32 = 1,          /* shares/outputs float; products in 3xTF32 (tensor cores) or FP32 FMA */
    GPD_PREC_FP64 = 2,          /* shares/outputs double; products in FP64 */
    GPD_PREC_FP64_SLICED = 3,   /* forward product only (gpd_encode_A, gpd_encode_B with GPD_OPERAND_X_FWD,
                                   gpd_worker_gemm with GPD_FWD, then inject / locate / decode as for
                                   GPD_PREC_FP64).  The shares W~_p (Eq. 1), X~_p (Theorem 2) are evaluated in
                                   FP64 and stored as six signed 8-bit digit planes plus one power-of-two
                                   scale per row of W~_p / column of X~_p (48 bits below the scale), in buffers
                                   of the same byte size as the FP64 shares (opaque to the caller); the worker
                                   products are exact int8 x int8 -> int32 tensor-core contractions of digit
                                   planes, recombined in FP64 (plane pairs below 2^-50 of row scale x column
                                   scale are not formed); worker outputs are double.  Needs N0/n divisible
                                   by 16 and at most 16384, 16-byte aligned W, X and share buffers
                                   (GPD_ERR_ARG otherwise), and finite inputs (a non-finite entry makes its
                                   share row meaningless without being flagged).  Every other call that takes
                                   shares returns GPD_ERR_UNSUPPORTED; gpd_plan returns it when the shapes do
                                   not fit.  An implementation choice of this library: the paper prescribes
                                   no arithmetic for the nodes' products. */
    GPD_PREC_FP64_SLICED40 = 4, /* the same with five digit planes (40 bits below the scale, 15 plane pairs
                                   instead of 21): worker outputs accurate to about 1e-10 of their scale,
                                   enough for recovery thresholds up to about 20 */
    GPD_PREC_FP64_SLICED_TRAIN = 5 /* digit-plane products (six planes) for every stage of the coded training
                                   step (Sections VI, VIII): forward and backward products and the update of
                                   Eq. 10 run as int8 tensor-core contractions; audit, regeneration and
                                   share-error injection work on FP64 shares.  The share buffer of W
                                   (GPD_Q_W_SHARE_ELEMS doubles, opaque, 16-byte aligned) holds the FP64
                                   shares [P][N1/m][N0/n] first, then two sliced copies (rows of W~_p for the
                                   forward product, columns for the backward product), re-cut by every call
                                   that changes the FP64 shares; the other operands' buffers keep the sizes
                                   of FP64 shares.  Needs N0/n, N1/m, B/d1, B/d2 and B divisible by 16 and at
                                   most 16384, finite inputs. */
} gpd_precision;

typedef enum {
    GPD_INJECT_BITFLIP = 0,     /* `count` distinct nodes, one entry each, one bit each */
    GPD_INJECT_ADDITIVE = 1,    /* selected nodes: additive errors on a random subset of entries */
    GPD_INJECT_GAUSS = 2        /* selected nodes: scale * N(0,1) added to every entry (Error Model 2) */
} gpd_inject_mode;

/* Garbage-alignment substitution (Section VI; Tables I, III; proofs of Theorems 4 and 6). */
typedef enum {
    GPD_SUBST_U_EQ_VN = 0,      /* u = v^n, w = v^(mn): Q_f = mn d1 + n - 1,      Q_b = mn d2 + mn - n  */
    GPD_SUBST_V_EQ_UM = 1       /* v = u^m, w = u^(mn): Q_f = mn d1 + mn - m,     Q_b = mn d2 + m - 1   */
} gpd_substitution;

typedef enum { GPD_ACT_IDENTITY = 0, GPD_ACT_RELU = 1, GPD_ACT_SIGMOID = 2 } gpd_activation_kind;

typedef enum {
    GPD_PHASE_FWD = 1, GPD_PHASE_BWD = 2, GPD_PHASE_UPD = 4,
    GPD_PHASE_REGEN = 8,          /* with FWD: regenerate the stored shares of the nodes the forward product flagged */
    GPD_PHASE_INJECT_SHARES = 16  /* with UPD: soft errors of the update stage, written into the updated shares */
} gpd_phase;

typedef struct { int64_t N1, N0, B; } gpd_shape;
typedef struct { int32_t m, n, d1, d2; } gpd_split;

/* Result of error detection / location; lives in device memory, copied back by the caller. */
typedef struct {
    int32_t outcome;            /* gpd_outcome */
    int32_t n_flagged;          /* number of nodes whose output must not be used */
    int32_t rank;               /* numerical rank of the syndrome Gram matrix */
    int32_t device_status;      /* 0, or a gpd_status raised on the device (GPD_ERR_TIMEOUT) */
    int64_t n_active;           /* codewords (output positions) that failed the zero-syndrome test */
    double  residual;           /* syndrome energy left outside span(H_A), per active codeword */
    double  max_inside;         /* largest subspace distance among nodes judged erroneous */
    double  min_outside;        /* smallest subspace distance among nodes judged clean */
    uint8_t flagged[GPD_MAX_NODES];   /* 1 = erroneous (the paper's length-P flag vector) */
    uint8_t forced[GPD_MAX_NODES];    /* 1 = erased by the caller or holding a non-finite value */
} gpd_locate_result;

/* Result of gpd_correct_positions; lives in device memory, copied back by the caller. */
typedef struct {
    int32_t outcome;            /* gpd_outcome: GPD_CORRECTED only if every failing position was repaired */
    int32_t max_errors;         /* largest number of errors corrected in one position */
    int32_t device_status;      /* 0 */
    int32_t reserved;
    int64_t n_active;           /* positions whose syndrome failed the zero test (non-finite ones included) */
    int64_t n_corrected;        /* of those, repaired in place */
    int64_t n_failed;           /* of those, left untouched: no support of size <= floor((P-Q)/2) explains the
                                   syndrome, or the position holds a non-finite value */
    int64_t n_entries;          /* worker-output entries changed */
    uint8_t touched[GPD_MAX_NODES];   /* 1 = at least one entry of this node was changed */
} gpd_position_result;

/* What gpd_plan_query returns. */
typedef enum {
    GPD_Q_THRESHOLD_FWD = 0,    /* mn d1 + n - 1   (Theorem 2)          or, alternate substitution, mn d1 + mn - m */
    GPD_Q_THRESHOLD_BWD = 1,    /* mn (d2 + 1) - n (proof of Theorem 6) or, alternate substitution, mn d2 + m - 1  */
    GPD_Q_THRESHOLD_AUDIT = 2,  /* mn                                               */
    GPD_Q_ELEMENT_SIZE = 3,     /* bytes per share / worker-output element (4 or 8) */
    GPD_Q_W_SHARE_ELEMS = 4,    /* P * (N1/m) * (N0/n); GPD_PREC_FP64_SLICED_TRAIN: that plus the two sliced copies */
    GPD_Q_X_SHARE_ELEMS = 5,    /* P * (N0/n) * (B/d1)                              */
    GPD_Q_DT_SHARE_ELEMS = 6,   /* P * (B/d2) * (N1/m)                              */
    GPD_Q_DHAT_ELEMS = 7,       /* P * (N1/m) * B                                   */
    GPD_Q_XHAT_ELEMS = 8,       /* P * (N0/n) * B                                   */
    GPD_Q_OUT_ELEMS_FWD = 9,    /* P * (N1/m) * (B/d1)                              */
    GPD_Q_OUT_ELEMS_BWD = 10,   /* P * (B/d2) * (N0/n)                              */
    GPD_Q_WORKSPACE_BYTES = 11, /* bytes of workspace for gpd_locate_errors / gpd_decode */
    GPD_Q_STEP_WORKSPACE_BYTES = 12, /* bytes of workspace for coded_layer_step       */
    GPD_Q_PRECISION = 13,       /* resolved gpd_precision                            */
    GPD_Q_NODES = 14,
    GPD_Q_POSITION_WORKSPACE_BYTES = 15, /* bytes of workspace for gpd_correct_positions (any product) */
    GPD_Q_TABLES_ON_DEVICE = 16 /* 1 once the plan's tables have been uploaded (device memory allocated), else 0 */
} gpd_query;

/* Host tables a test may read back with gpd_plan_table. */
typedef enum {
    GPD_TABLE_POINTS = 0,       /* P doubles: b_p                                                  */
    GPD_TABLE_PARITY_FWD = 1,   /* (P-Q_f) x P doubles, row-major, orthonormal rows, H V = 0       */
    GPD_TABLE_PARITY_BWD = 2,
    GPD_TABLE_PARITY_AUDIT = 3,
    GPD_TABLE_COEF_W = 4,       /* P x (m n): b_p^(n i + j)                                        */
    GPD_TABLE_COEF_X = 5,       /* P x (n d1): b_p^(n-1-j + mn k)                                  */
    GPD_TABLE_COEF_DT = 6       /* P x (d2 m): b_p^(mn k + n(m-1-i))                               */
} gpd_table;

const char* gpd_status_string(gpd_status s);

/*
 * gpd_plan — code construction (Section IV: block partition, encoding polynomials, evaluation
 * points; Section V-A: parity-check matrix H with H G^T = 0 for the Vandermonde generator).
 * points_host: P distinct finite doubles, or NULL for the roots of the first-kind Chebyshev
 * polynomial T_P on [-1,1].  Host only: needs no GPU.  Errors: GPD_ERR_SHAPE, GPD_ERR_POINTS,
 * GPD_ERR_P_TOO_SMALL (P below the forward threshold Q_f), GPD_ERR_Q_TOO_LARGE.
 * A plan with Q_f <= P < Q_b (or a backward threshold above GPD_MAX_THRESHOLD) is a forward-only
 * plan: every call on its backward product returns GPD_ERR_P_TOO_SMALL, and coded_layer_step
 * checks that before it enqueues anything.  GPD_Q_THRESHOLD_BWD still reports Q_b.
 */
gpd_status gpd_plan(const gpd_shape* shape, const gpd_split* split, int32_t P,
                    const double* points_host, gpd_precision precision, gpd_plan_t* out);
/* Same with the substitution chosen by the caller (gpd_plan uses GPD_SUBST_U_EQ_VN).  The alternate
 * substitution moves error tolerance from the forward to the backward product (proofs of Theorems
 * 4 and 6); exponent maps: W_ij at u^(i + m j), X_jk at u^(m(n-1-j) + mn k), Delta^T_ki at
 * u^(mn k + m-1-i), update operands Delta_i at u^i and X_j at u^(m j). */
gpd_status gpd_plan_subst(const gpd_shape* shape, const gpd_split* split, gpd_substitution subst, int32_t P,
                          const double* points_host, gpd_precision precision, gpd_plan_t* out);
/* Uploads the plan's coefficient tables to the current device now (one cudaMalloc - tables, plus the
 * scratch area of FP32 plans -, one synchronous copy of a few KB, and three one-block kernels that
 * precompute the decoding matrices of the error-free case, waited for) instead of at the plan's first compute call; a second call does nothing.  Lets a
 * caller keep allocation and synchronisation out of its timed or captured region. */
gpd_status gpd_plan_upload(gpd_plan_t plan);
gpd_status gpd_plan_destroy(gpd_plan_t plan);
gpd_status gpd_plan_query(gpd_plan_t plan, gpd_query what, int64_t* value);
/* Copies a host table into host_out (capacity in doubles); *count receives its length. */
gpd_status gpd_plan_table(gpd_plan_t plan, gpd_table which, double* host_out, int64_t capacity,
                          int64_t* count);

/*
 * gpd_encode_A — initial encoding of W (Eq. 1 / Eq. 3): W~_p = sum_ij W_ij b_p^(n i + j).
 * W_dev: N1 x N0 float.  W_shares_dev: [P][N1/m][N0/n] in the plan's storage type.
 */
gpd_status gpd_encode_A(gpd_plan_t plan, const float* W_dev, void* W_shares_dev, void* stream);

/*
 * gpd_encode_B — encoding of the other operand: X (Theorem 2), Delta^T (backpropagation stage)
 * or the two ascending-power operands of the update stage.  Layouts: see gpd_operand.
 */
gpd_status gpd_encode_B(gpd_plan_t plan, gpd_operand operand, const float* src_dev,
                        void* shares_dev, void* stream);

/*
 * gpd_worker_gemm — the P node products as one batched contraction (steps O1 / O2):
 *   GPD_FWD: out[p] = W~_p X~_p        ([N1/m x N0/n] [N0/n x B/d1])
 *   GPD_BWD: out[p] = Delta~^T_p W~_p  ([B/d2 x N1/m] [N1/m x N0/n])
 * outputs_dev: [P][rows][cols] in the plan's storage type.
 * FP32 plans: the tensor-core products keep partial sums in scratch memory that belongs to the plan
 * (allocated with its tables, see gpd_plan_upload), so two such calls on one plan must not run at the
 * same time on different streams; calls ordered on one stream, or on one plan per stream, are fine.
 */
gpd_status gpd_worker_gemm(gpd_plan_t plan, gpd_product which, const void* W_shares_dev,
                           const void* other_shares_dev, void* outputs_dev, void* stream);

/*
 * gpd_device_status — kernels that wait on hardware barriers (the tensor-core product path) bound
 * every wait; a wait that expires raises a device-side status word instead of hanging.  This call
 * synchronises the device, returns that word in *status_host (0, or GPD_ERR_TIMEOUT) and clears it.
 */
gpd_status gpd_device_status(int32_t* status_host);

/*
 * gpd_selftest_bounded_wait - exercises the bounded-wait mechanism of the tensor-core kernels without
 * touching them: one small CTA waits on a hardware barrier that nothing ever arrives at, gives up
 * after `limit_cycles` clock cycles (clamped to [1e3, 1e8]), raises the same status word and
 * returns.  Afterwards gpd_device_status reports GPD_ERR_TIMEOUT once, and the context stays usable.
 * (No counterpart in the paper: a check of this library's failure reporting.)
 */
gpd_status gpd_selftest_bounded_wait(int64_t limit_cycles, void* stream);

/*
 * gpd_update_shares — coded update (step O3, Eq. 10 and its weight-decay form):
 *   W~_p <- (1 - eta*lambda) W~_p + eta * Delta^_p X^_p^T   for all p, in place.
 * If gate_dev is non-NULL and gate_dev->outcome == GPD_DECODE_FAILURE the shares are left
 * untouched (the step that produced Delta is to be repeated from a checkpoint).
 */
gpd_status gpd_update_shares(gpd_plan_t plan, void* W_shares_dev, const void* Dhat_dev,
                             const void* Xhat_dev, float eta, float lambda,
                             const gpd_locate_result* gate_dev, void* stream);

/*
 * gpd_inject — seeded soft errors written into worker outputs (Error Model 2, Section V-B, and
 * the bit-flip / sparse-additive variants of the workloads).  Counter-based SplitMix64 draws.
 * which: GPD_FWD / GPD_BWD / GPD_AUDIT selects the buffer geometry ([P][L]).
 * Nodes are chosen with probability `prob` each, or, if prob < 0, by the bits of node_mask;
 * GPD_INJECT_BITFLIP uses `count` instead.  hit_mask_dev (optional) receives the chosen nodes.
 */
gpd_status gpd_inject(gpd_plan_t plan, gpd_product which, void* outputs_dev, uint64_t seed,
                      gpd_inject_mode mode, double prob, uint64_t node_mask, int32_t count,
                      double scale, uint64_t* hit_mask_dev, void* stream);

/*
 * gpd_locate_errors — Algorithm 1 at node level (Section V-A, Theorem 3; polynomial-time form
 * of the decoding appendix): zero-syndrome test of every codeword, Gram matrix of the failing
 * ones, support = nodes whose parity-check column lies in its range, residual verification.
 * erased_host: optional P bytes (1 = ignore this node; counts against the P-Q-1 budget).
 * result_dev: device gpd_locate_result.  workspace_dev: GPD_Q_WORKSPACE_BYTES bytes.
 */
gpd_status gpd_locate_errors(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                             const uint8_t* erased_host, gpd_locate_result* result_dev,
                             void* workspace_dev, void* stream);

/*
 * gpd_correct_positions — error correction of every output position on its own under the
 * adversarial model (lemma on real-number error correction under the adversarial model; section on
 * decoding methods): a position is one codeword of P node values; when its syndrome H z is not
 * zero, the solution of H e = H z with the fewest non-zeros, at most floor((P-Q)/2), is looked for
 * (power-sum syndromes, error-locator polynomial, least-squares error values, acceptance by the
 * zero test on what is left of the syndrome) and subtracted from outputs_dev IN PLACE.  Different
 * positions may blame different nodes, so more than P-Q-1 nodes may be hit overall - the case
 * gpd_locate_errors must give up on.  Afterwards gpd_decode with a use-mask of all nodes (or any
 * Q of them) reads the repaired outputs.  Positions that cannot be repaired are left as they are
 * and counted; the outcome is then GPD_DECODE_FAILURE.  Meant for small floor((P-Q)/2) (the
 * locator is found in the monomial basis).
 * result_dev: device gpd_position_result.  workspace_dev: GPD_Q_POSITION_WORKSPACE_BYTES bytes
 * (counters, a 4-byte index per position, and the syndromes of up to one position in 32 (at least 4096);
 * when more positions than that fail, the codewords of the others are read a second time).
 */
gpd_status gpd_correct_positions(gpd_plan_t plan, gpd_product which, void* outputs_dev,
                                 gpd_position_result* result_dev, void* workspace_dev, void* stream);

/*
 * gpd_locate_errors_static — gpd_locate_errors for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the call above, same arithmetic,
 * same result.)
 *
 * Who needs it: a fault-detection hook that runs inside a job whose framework has already handed
 * all of HBM to its own memory pool, so that a cudaMalloc made on the library's behalf fails or
 * eats into someone else's budget; and latency-critical loops that cannot afford the device-wide
 * synchronisation an allocation implies.  gpd_locate_errors itself asks the caller for a workspace
 * and, on a plan's first use, uploads the plan's tables into memory it allocates.  This variant
 * does neither: its scratch (Gram matrix, counters and the parity-check matrix, about 10 KB) is a
 * fixed array compiled into the library, present once on every GPU that loads the library until
 * the process exits, and the parity-check matrix is copied into it from the plan's host tables on
 * every call.  No cudaMalloc, cudaFree or allocating library routine is called on its path.
 *
 * Limit: products with P - Q <= GPD_STATIC_MAX_PARITY (16); beyond that the call returns
 * GPD_ERR_STATIC_LIMIT and does nothing.
 * Set-up: the first call on a device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.  The address is kept for the life of
 * the process's context on that device (a cudaDeviceReset invalidates it).
 * Lifetime: every call enqueues an asynchronous copy of the parity-check matrix out of the plan's
 * host tables, so the plan must stay alive until the enqueued work has completed.
 * Sharing: every call on a GPU uses the same array.  It is cleared by the call itself, but two
 * calls whose work overlaps on the GPU (different streams, different threads) race on it: keep
 * calls to this entry point ordered on one stream per GPU.
 * Arguments as for gpd_locate_errors, without the workspace.
 */
gpd_status gpd_locate_errors_static(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                                    const uint8_t* erased_host, gpd_locate_result* result_dev,
                                    void* stream);

/*
 * gpd_decode — interpolation of the wanted coefficients from the clean evaluations
 * (Theorem 2's proof; Vandermonde system of the decoding appendix), least squares over all
 * nodes in use.  use_mask_host: optional P bytes (1 = use); if NULL the nodes not flagged in
 * result_dev are used and nothing is written when result_dev->outcome is a decoding failure.
 * out_dev: S (N1 x B), C^T (B x N0) or W (N1 x N0), float.  activation is applied to what is
 * stored in act_out_dev (optional, same shape; step C1).
 */
gpd_status gpd_decode(gpd_plan_t plan, gpd_product which, const void* outputs_dev,
                      const uint8_t* use_mask_host, const gpd_locate_result* result_dev,
                      float* out_dev, float* act_out_dev, gpd_activation_kind activation,
                      void* workspace_dev, void* stream);

/*
 * gpd_regenerate_shares — regeneration of erroneous nodes (Section VI, "Regeneration"): the share
 * W~_p is the evaluation at b_p of a polynomial of degree mn-1 whose coefficients are the blocks
 * W_ij, so the share of every node flagged in result_dev is recomputed from the shares of the
 * clean nodes (interpolation over all of them, least squares, then evaluation at b_p), in place.
 * Needs at least mn clean nodes; does nothing when result_dev reports no flagged node or a
 * decoding failure.  workspace_dev: GPD_Q_WORKSPACE_BYTES bytes.
 */
gpd_status gpd_regenerate_shares(gpd_plan_t plan, void* W_shares_dev, const gpd_locate_result* result_dev,
                                 void* workspace_dev, void* stream);

/* Element-wise steps C1 / C2 and the last-layer transitions (Section II-B; Section IX). */
gpd_status gpd_activation(gpd_activation_kind kind, const float* S_dev, float* X_next_dev,
                          int64_t count, void* stream);
/* Delta = (Y_onehot - softmax_columns(S)) / B for S (C x B); writes Delta (C x B), Delta^T (B x C)
 * and the mean cross-entropy (one float).  Any output pointer may be NULL. */
gpd_status gpd_softmax_xent_delta(const float* S_dev, const int32_t* labels_dev, float* Delta_dev,
                                  float* DeltaT_dev, float* loss_dev, int64_t C, int64_t B,
                                  void* stream);
/* Delta_prev = C o g(X) with g(f(u)) = f'(u); CT is B x N, X is N x B (the layer's input, i.e. the
 * previous layer's activation output); writes Delta_prev (N x B) and Delta_prev^T (B x N). */
gpd_status gpd_backprop_hadamard(gpd_activation_kind kind, const float* CT_dev, const float* X_dev,
                                 float* Delta_dev, float* DeltaT_dev, int64_t N, int64_t B,
                                 void* stream);
/* Sparse autoencoder (Section IX): Delta2 = (2/B)(X - S2) (N x B), its transpose, and the
 * reconstruction loss (1/B) sum ||S2 - X||^2. */
gpd_status gpd_sae_output_delta(const float* S2_dev, const float* X_dev, float* Delta2_dev,
                                float* Delta2T_dev, float* loss_dev, int64_t N, int64_t B,
                                void* stream);
/* Delta1 = (C2 - (beta/B) Q(rho_hat) 1^T) o Y1 o (1 - Y1) with rho_hat_i = mean_b Y1[i,b] and
 * Q(r) = -rho/r + (1-rho)/(1-r); C2T is B x N, Y1 is N x B; also the KL term beta * sum_i KL. */
gpd_status gpd_sae_hidden_delta(const float* C2T_dev, const float* Y1_dev, float rho, float beta,
                                float* Delta1_dev, float* Delta1T_dev, float* kl_loss_dev,
                                int64_t N, int64_t B, void* stream);

/*
 * coded_layer_step — one layer of the coded training step (Sections VI and VIII), composed from
 * the calls above on one stream with no host synchronisation:
 *   GPD_PHASE_FWD: encode X -> P products -> inject -> locate -> decode S (-> activation)
 *                  (+ GPD_PHASE_REGEN: then regenerate the shares of the nodes just flagged, which is
 *                  how errors left in the shares by an earlier update are repaired, Section VI)
 *   GPD_PHASE_BWD: encode Delta^T -> P products -> inject -> locate -> decode C^T
 *   GPD_PHASE_UPD: encode Delta, X ascending -> W~_p += eta Delta^_p X^_p^T;
 *                  skipped on the device if this call's backward product declared a decoding failure.
 *                  (+ GPD_PHASE_INJECT_SHARES: Gaussian node errors written into the updated shares,
 *                  seed inject_seed + 2; they surface at the next forward product of the layer.)
 * X_dev: N0 x B.  Delta_dev: N1 x B and DeltaT_dev: B x N1 (needed for BWD / UPD).
 * S_out_dev, Xnext_out_dev: N1 x B (FWD; Xnext optional).  CT_out_dev: B x N0 (BWD).
 * inject_prob <= 0 disables injection; product k of the call uses seed inject_seed + k
 * (k = 0 forward, 1 backward) and Gaussian whole-node errors of the given scale.
 * results_dev: three gpd_locate_result (forward, backward, unused).
 * workspace_dev: GPD_Q_STEP_WORKSPACE_BYTES bytes.
 */
gpd_status coded_layer_step(gpd_plan_t plan, int32_t phases, void* W_shares_dev,
                            const float* X_dev, const float* Delta_dev, const float* DeltaT_dev,
                            gpd_activation_kind activation, float eta, float lambda,
                            uint64_t inject_seed, double inject_prob, double inject_scale,
                            float* S_out_dev, float* Xnext_out_dev, float* CT_out_dev,
                            gpd_locate_result* results_dev, void* workspace_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GPD_H_ */
