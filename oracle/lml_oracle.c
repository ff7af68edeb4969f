/*
 * fp64 CPU oracle for the mixed-adapter LoRA linear layer.  TEST INFRASTRUCTURE ONLY:
 * the product (the CUDA library) never links, imports or calls this file; only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg do.
 *
 * What it computes is the plain definition of the layer.  Several agents' tokens share one
 * frozen base weight and each token is bound to one resident (adapter, version) entry —
 * the paper's Section 2 ("LoRA adapters": small low-rank modules on a shared frozen base,
 * requests routed to the correct adapter), Section 4.2 (inference binds the last committed
 * version while newer state stays private) and Section 5.1 (the adapter identifies the
 * LoRA slot, the adapter version the committed state).  For a token row x bound to entry s
 *
 *     y[n] = sum_k x[k] * W0[n][k]  +  scale_s * sum_j ( sum_k x[k] * A_s[j][k] ) * B_s[n][j]
 *
 * and a token bound to no adapter (entry -1) gets the first sum only.  Storage is row-major:
 * x[T][K], W0[N][K], A_s[r_s][K], B_s[N][r_s], all bf16 bit patterns (uint16), widened
 * exactly to double here; every sum runs in ascending index order in fp64; the result is
 * returned unrounded.  No blocking, no reordering, no fast-math.  Rows are independent, so
 * the optional OpenMP loop over rows changes no arithmetic.
 *
 * Parity pins (tests/test_oracle_pins.py): exact base-only result when B = 0 or entry = -1,
 * agreement with the merged weight W0 + s*A*B formed by numpy in float64, exact row
 * permutation under segment permutation, closed forms for constant inputs, one-hot inputs,
 * a hand-worked 2x2 example, an integer-lattice case, and the brute-force twin below.
 * The backward pass (lml_oracle_backward, the gradients of the training task) is pinned in
 * tests/test_oracle_backward_pins.py: central differences of the forward oracle in every
 * coordinate of x, A and B, a hand-worked rank-one example, the matrix identities formed by
 * numpy in float64, and structural cases (unbound rows, unused and repeated entries).
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* status flags reported through *flags_out (bit set = condition seen) */
#define ORC_FLAG_BAD_SLOT 1u    /* a segment named an entry >= num_entries or a dead entry  */
#define ORC_FLAG_BAD_OFFSETS 2u /* seg_offsets not 0-based, monotone and ending at T        */

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* entry of position p, or -1; also validates the entry id */
static int entry_of_position(int p, int G, const int32_t *seg_offsets, const int32_t *seg_entry,
                             int num_entries, const int32_t *live, uint32_t *flags)
{
    for (int g = 0; g < G; ++g) {
        if (p >= seg_offsets[g] && p < seg_offsets[g + 1]) {
            int e = seg_entry[g];
            if (e < 0) return -1;
            if (e >= num_entries || !live[e]) {
                *flags |= ORC_FLAG_BAD_SLOT;
                return -1; /* affected tokens get the base output only */
            }
            return e;
        }
    }
    return -1;
}

static int offsets_ok(int T, int G, const int32_t *seg_offsets)
{
    if (G == 0) return 1;
    if (seg_offsets[0] != 0 || seg_offsets[G] != T) return 0;
    for (int g = 0; g < G; ++g)
        if (seg_offsets[g + 1] < seg_offsets[g]) return 0;
    return 1;
}

/*
 * Forward pass on the positions listed in `positions` (npos of them), or on every position
 * 0..T-1 when positions == NULL.  Position p addresses row perm[p] (row p when perm == NULL)
 * of x and of the output.  y64 is [T][N] doubles and only the addressed rows are written.
 * A[e], B[e] point at entry e's matrices; rank[e], scale[e], live[e] describe it.
 * Malformed seg_offsets: flag set and every row gets the base output only.
 * Returns 0, or -1 on a null / negative argument.
 */
int lml_oracle_forward(const uint16_t *x, const uint16_t *W0, int T, int K, int N,
                       int num_entries, const uint16_t *const *A, const uint16_t *const *B,
                       const int32_t *rank, const float *scale, const int32_t *live,
                       int G, const int32_t *seg_offsets, const int32_t *seg_entry,
                       const int32_t *perm, const int32_t *positions, int npos,
                       double *y64, uint32_t *flags_out, int nthreads)
{
    if (T < 0 || K < 0 || N < 0 || G < 0 || num_entries < 0) return -1;
    if (T > 0 && (!x || !W0 || !y64)) return -1;
    uint32_t flags = 0;
    int use_lora = 1;
    if (!offsets_ok(T, G, seg_offsets)) {
        flags |= ORC_FLAG_BAD_OFFSETS;
        use_lora = 0;
    }
    int count = positions ? npos : T;
    int nt = 1;
#ifdef _OPENMP
    nt = nthreads > 0 ? nthreads : omp_get_max_threads();
#else
    (void)nthreads;
#endif
    uint32_t flag_acc = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : flag_acc) num_threads(nt)
    for (int i = 0; i < count; ++i) {
        int p = positions ? positions[i] : i;
        int t = perm ? perm[p] : p;
        const uint16_t *xr = x + (size_t)t * K;
        double *yr = y64 + (size_t)t * N;
        uint32_t f = 0;
        int e = use_lora ? entry_of_position(p, G, seg_offsets, seg_entry, num_entries, live, &f) : -1;
        flag_acc |= f;

        /* base term: acc[n] = sum_k x[k] * W0[n][k], k ascending */
        for (int n = 0; n < N; ++n) {
            const uint16_t *wr = W0 + (size_t)n * K;
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += bf16_to_f64(xr[k]) * bf16_to_f64(wr[k]);
            yr[n] = acc;
        }
        if (e < 0) continue;

        /* shrink: u[j] = sum_k x[k] * A_e[j][k] */
        int r = rank[e];
        double u[256];
        if (r > 256) r = 256;
        for (int j = 0; j < r; ++j) {
            const uint16_t *ar = A[e] + (size_t)j * K;
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += bf16_to_f64(xr[k]) * bf16_to_f64(ar[k]);
            u[j] = acc;
        }
        /* expand, scale, add: y[n] += scale_e * sum_j u[j] * B_e[n][j] */
        double s = (double)scale[e];
        for (int n = 0; n < N; ++n) {
            const uint16_t *br = B[e] + (size_t)n * rank[e];
            double d = 0.0;
            for (int j = 0; j < r; ++j) d += u[j] * bf16_to_f64(br[j]);
            yr[n] += s * d;
        }
    }
    if (flags_out) *flags_out = flags | flag_acc;
    return 0;
}

/*
 * Brute-force twin: a different loop nest (output column outermost, no intermediate u, the
 * LoRA term as a double sum over j and k).  Agrees with lml_oracle_forward to rounding
 * (~1e-13 relative); a wrong index, a dropped term or a transposed operand in either shows up
 * as a disagreement.  Meant for tiny inputs: cost is T*N*K*(1 + r).
 */
int lml_oracle_forward_brute(const uint16_t *x, const uint16_t *W0, int T, int K, int N,
                             int num_entries, const uint16_t *const *A, const uint16_t *const *B,
                             const int32_t *rank, const float *scale,
                             int G, const int32_t *seg_offsets, const int32_t *seg_entry,
                             const int32_t *perm, double *y64)
{
    (void)num_entries;
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            int e = seg_entry[g];
            for (int p = seg_offsets[g]; p < seg_offsets[g + 1]; ++p) {
                int t = perm ? perm[p] : p;
                double base = 0.0;
                for (int k = 0; k < K; ++k)
                    base += bf16_to_f64(x[(size_t)t * K + k]) * bf16_to_f64(W0[(size_t)n * K + k]);
                double delta = 0.0;
                if (e >= 0) {
                    for (int j = 0; j < rank[e]; ++j)
                        for (int k = 0; k < K; ++k)
                            delta += bf16_to_f64(x[(size_t)t * K + k]) *
                                     bf16_to_f64(A[e][(size_t)j * K + k]) *
                                     bf16_to_f64(B[e][(size_t)n * rank[e] + j]);
                    delta *= (double)scale[e];
                }
                y64[(size_t)t * N + n] = base + delta;
            }
        }
    }
    return 0;
}

/*
 * Token segmentation: group T tokens by entry id.  Stable (tokens keep their relative order
 * inside a group), groups in ascending entry id, tokens tagged -1 (no adapter) last.  Written
 * as an insertion-style stable ordering straight from that rule: O(T * groups), no counting
 * tricks.  Outputs: perm[T] (position -> row), seg_offsets[num_segs+1], seg_entry[num_segs];
 * only groups with at least one token produce a segment.  Ids outside [-1, num_entries) are
 * treated as -1 and reported with ORC_FLAG_BAD_SLOT.
 */
int lml_oracle_segment(const int32_t *token_entry, int T, int num_entries, int32_t *perm,
                       int32_t *seg_offsets, int32_t *seg_entry, int32_t *num_segs,
                       uint32_t *flags_out)
{
    uint32_t flags = 0;
    int pos = 0, segs = 0;
    seg_offsets[0] = 0;
    for (int key = 0; key <= num_entries; ++key) { /* key == num_entries stands for -1 */
        int before = pos;
        for (int t = 0; t < T; ++t) {
            int e = token_entry[t];
            if (e < -1 || e >= num_entries) {
                if (key == 0) flags |= ORC_FLAG_BAD_SLOT;
                e = -1;
            }
            int k = e < 0 ? num_entries : e;
            if (k == key) perm[pos++] = t;
        }
        if (pos > before) {
            seg_entry[segs] = key < num_entries ? key : -1;
            seg_offsets[++segs] = pos;
        }
    }
    *num_segs = segs;
    if (flags_out) *flags_out = flags;
    return 0;
}

/*
 * Backward pass of the layer for the training task (Section 2.2, online RL: adapters are updated
 * in the background; Section 4.1, task model: the training step is one of the tasks that share
 * the GPU).  With
 *     y[t] = x[t].W0^T + s_e (x[t].A_e^T).B_e^T          (e = entry of the position of row t)
 * and an upstream gradient dy [T][N] (bf16 like every activation), the definitions are
 *     dx[t]     = dy[t].W0 + s_e (dy[t].B_e).A_e
 *     dA_e[j][k] = s_e sum_{t bound to e} (dy[t].B_e)[j] x[t][k]
 *     dB_e[n][j] = s_e sum_{t bound to e} dy[t][n] (x[t].A_e^T)[j]
 * written out as plain loops in double precision.  dx64 is [T][K]; dA64[e] is [rank_e][K] and
 * dB64[e] is [N][rank_e], both overwritten (zero for entries no token is bound to).  Any of the
 * three output arguments may be NULL.  Rows are addressed as in the forward pass (perm).
 * Positions bound to a dead or out-of-range entry count as unbound (flag); malformed offsets:
 * flag set, every row unbound.  Returns 0, or -1 on a null / negative argument.
 */
int lml_oracle_backward(const uint16_t *x, const uint16_t *dy, const uint16_t *W0, int T, int K, int N,
                        int num_entries, const uint16_t *const *A, const uint16_t *const *B,
                        const int32_t *rank, const float *scale, const int32_t *live,
                        int G, const int32_t *seg_offsets, const int32_t *seg_entry,
                        const int32_t *perm, double *dx64, double *const *dA64, double *const *dB64,
                        uint32_t *flags_out)
{
    if (T < 0 || K < 0 || N < 0 || G < 0 || num_entries < 0) return -1;
    if (T > 0 && (!x || !dy || !W0)) return -1;
    uint32_t flags = 0;
    int use_lora = 1;
    if (!offsets_ok(T, G, seg_offsets)) {
        flags |= ORC_FLAG_BAD_OFFSETS;
        use_lora = 0;
    }
    for (int e = 0; e < num_entries; ++e) {
        if (dA64 && dA64[e]) for (size_t i = 0; i < (size_t)rank[e] * K; ++i) dA64[e][i] = 0.0;
        if (dB64 && dB64[e]) for (size_t i = 0; i < (size_t)N * rank[e]; ++i) dB64[e][i] = 0.0;
    }
    for (int p = 0; p < T; ++p) {
        int t = perm ? perm[p] : p;
        const uint16_t *xr = x + (size_t)t * K;
        const uint16_t *gr = dy + (size_t)t * N;
        int e = use_lora ? entry_of_position(p, G, seg_offsets, seg_entry, num_entries, live, &flags) : -1;
        if (dx64) {
            double *dxr = dx64 + (size_t)t * K;
            for (int k = 0; k < K; ++k) {
                double acc = 0.0;
                for (int n = 0; n < N; ++n) acc += bf16_to_f64(gr[n]) * bf16_to_f64(W0[(size_t)n * K + k]);
                dxr[k] = acc;
            }
        }
        if (e < 0) continue;
        int r = rank[e];
        if (r > 256) r = 256;
        double s = (double)scale[e];
        double g[256], h[256];
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int n = 0; n < N; ++n) acc += bf16_to_f64(gr[n]) * bf16_to_f64(B[e][(size_t)n * rank[e] + j]);
            g[j] = acc;                       /* (dy.B)[j] */
            acc = 0.0;
            for (int k = 0; k < K; ++k) acc += bf16_to_f64(xr[k]) * bf16_to_f64(A[e][(size_t)j * K + k]);
            h[j] = acc;                       /* (x.A^T)[j] */
        }
        if (dx64) {
            double *dxr = dx64 + (size_t)t * K;
            for (int k = 0; k < K; ++k) {
                double acc = 0.0;
                for (int j = 0; j < r; ++j) acc += g[j] * bf16_to_f64(A[e][(size_t)j * K + k]);
                dxr[k] += s * acc;
            }
        }
        if (dA64 && dA64[e])
            for (int j = 0; j < r; ++j)
                for (int k = 0; k < K; ++k) dA64[e][(size_t)j * K + k] += s * g[j] * bf16_to_f64(xr[k]);
        if (dB64 && dB64[e])
            for (int n = 0; n < N; ++n)
                for (int j = 0; j < r; ++j) dB64[e][(size_t)n * rank[e] + j] += s * bf16_to_f64(gr[n]) * h[j];
    }
    if (flags_out) *flags_out = flags;
    return 0;
}

int lml_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
