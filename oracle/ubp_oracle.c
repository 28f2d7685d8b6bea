/*
 * CPU oracle for unaligned block-wise pruned (UBP) layers.
 *
 * TEST INFRASTRUCTURE ONLY. Nothing in the product path may call into this
 * file; it exists so that the CUDA kernels and the library's packer can be
 * compared against a plain, slow, independent statement of what the method
 * computes. It shares no code, header, table or helper with the library.
 *
 * What is here, and the passage each function follows:
 *   orc_block_budget      m = floor(b*(1-p)/N), b = c_out*c_in      (Section 3.1)
 *   orc_decode_mask       re-cut runs of ones into N-row blocks      (Algorithm 2,
 *                         with the no-overlap / in-bounds rules of Eq. 1, Eq. 2)
 *   orc_pack / orc_unpack indptr / indices / rotated values          (Section 4.2,
 *                         "weights for output channel i move to slot i mod N")
 *   orc_masked_matmul     Y = act(Wm X + bias), Wm = W where mask    (Section 3.1:
 *                         weights outside the kept blocks are pruned) -- the
 *                         plain definition, double accumulation, zeros included
 *   orc_masked_conv3x3    same for a 3x3 / stride 1 / pad 1 cross-correlation
 *   orc_wros_spmm         the weight-rotating output-stationary walk (Section 4.2):
 *                         tile i = start row i, N stationary accumulators, store
 *                         slot (i mod N) after tile i, flush N-1 rows at the end
 *   orc_*_samples         single output elements of the two definitions
 *
 * Arithmetic: inputs are fp32, every product and sum is done in double.
 * All pins for these functions live in the CPU test-suite (worked example of
 * Section 3.3 / 4.2, brute force on tiny inputs, library matmul / conv / CSR
 * special cases, invariants); no function here is "parity unpinned".
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_E_ARG (-1)
#define ORC_E_RAGGED (-2)   /* a run of ones cannot be cut into whole blocks */
#define ORC_E_SPACE (-3)
#define ORC_E_FORMAT (-4)

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 3.1: m_l = floor(b_l (1 - p_l) / N), p given in whole percent. */
int64_t orc_block_budget(int64_t M, int64_t C, int sparsity_pct, int Nb)
{
    return (M * C * (int64_t)(100 - sparsity_pct)) / (100 * (int64_t)Nb);
}

/*
 * Algorithm 2 (block division) applied to a mask: visit the linear block
 * index k = i + M*j in ascending order; a one that lies at or after next_idx
 * opens a new block there and moves next_idx N rows down; ones before
 * next_idx belong to the block just opened. A block has to stay inside its
 * column (Eq. 1: i + N - 1 < c_out) and consist of ones only, otherwise the
 * run it came from was not a whole number of blocks.
 * bi/bj receive start row / input channel of each block in visiting order.
 */
int orc_decode_mask(const uint8_t *mask, int M, int C, int Nb,
                    int32_t *bi, int32_t *bj, int64_t cap, int64_t *nblocks)
{
    if (!mask || !nblocks || M <= 0 || C <= 0 || Nb <= 0 || Nb > M) return ORC_E_ARG;
    int64_t nb = 0;
    for (int j = 0; j < C; ++j) {
        int next_idx = 0;
        for (int i = 0; i < M; ++i) {
            uint8_t v = mask[(size_t)i * C + j];
            if (v > 1) return ORC_E_ARG;
            if (!v) {
                if (i < next_idx) return ORC_E_RAGGED; /* hole inside a block */
                continue;
            }
            if (i < next_idx) continue;               /* inside the open block */
            if (i + Nb - 1 >= M) return ORC_E_RAGGED;  /* Eq. 1 */
            if (bi && bj) {
                if (nb >= cap) return ORC_E_SPACE;
                bi[nb] = i;
                bj[nb] = j;
            }
            ++nb;
            next_idx = i + Nb;
        }
    }
    *nblocks = nb;
    return ORC_OK;
}

/* ---- canonical packed format ------------------------------------------- */
/* header (64 bytes, little endian):
 *   char magic[4] = "UBP1"; u32 version = 1; i32 M, C, R, Nb, m; u32 flags (bit0: rotated)
 * then indptr i32[M+1], indices i32[m], values f32[m][Nb][R], each section
 * starting on a 64-byte boundary, padding bytes zero.
 */
static size_t up64(size_t x) { return (x + 63u) & ~(size_t)63u; }

static void put_u32(uint8_t *p, uint32_t v)
{
    p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); p[2] = (uint8_t)(v >> 16); p[3] = (uint8_t)(v >> 24);
}
static uint32_t get_u32(const uint8_t *p)
{
    return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

size_t orc_blob_size(int M, int R, int Nb, int64_t m)
{
    return 64 + up64(4 * (size_t)(M + 1)) + up64(4 * (size_t)m) + up64(4 * (size_t)m * Nb * R);
}

/*
 * Section 4.2 storage: blocks grouped by the output row they start at
 * (indptr over start rows, indices = input channel), ascending input channel
 * inside a start row, and inside a block the weight of output row rho is
 * placed in slot rho mod N. Values are copied as bits.
 */
int orc_pack(const float *W, const uint8_t *mask, int M, int C, int R, int Nb,
             uint8_t *blob, size_t cap, size_t *len)
{
    if (!W || !mask || !len || R <= 0) return ORC_E_ARG;
    int64_t m = 0;
    int rc = orc_decode_mask(mask, M, C, Nb, NULL, NULL, 0, &m);
    if (rc) return rc;
    size_t need = orc_blob_size(M, R, Nb, m);
    *len = need;
    if (!blob) return ORC_OK;
    if (cap < need) return ORC_E_SPACE;

    int32_t *bi = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m + 1));
    int32_t *bj = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m + 1));
    int32_t *cursor = (int32_t *)calloc((size_t)M + 1, sizeof(int32_t));
    if (!bi || !bj || !cursor) { free(bi); free(bj); free(cursor); return ORC_E_SPACE; }
    orc_decode_mask(mask, M, C, Nb, bi, bj, m, &m);

    memset(blob, 0, need);
    memcpy(blob, "UBP1", 4);
    put_u32(blob + 4, 1u);
    put_u32(blob + 8, (uint32_t)M);
    put_u32(blob + 12, (uint32_t)C);
    put_u32(blob + 16, (uint32_t)R);
    put_u32(blob + 20, (uint32_t)Nb);
    put_u32(blob + 24, (uint32_t)m);
    put_u32(blob + 28, 1u);
    uint8_t *p_indptr = blob + 64;
    uint8_t *p_indices = p_indptr + up64(4 * (size_t)(M + 1));
    uint8_t *p_values = p_indices + up64(4 * (size_t)m);

    /* count blocks per start row, prefix-sum into indptr */
    for (int64_t b = 0; b < m; ++b) cursor[bi[b] + 1]++;
    for (int i = 0; i < M; ++i) cursor[i + 1] += cursor[i];
    for (int i = 0; i <= M; ++i) put_u32(p_indptr + 4 * (size_t)i, (uint32_t)cursor[i]);
    /* the decode order is column-major (j ascending), so filling each start
       row's slots in that order leaves j ascending inside a start row */
    for (int64_t b = 0; b < m; ++b) {
        int i = bi[b], j = bj[b];
        int32_t slot = cursor[i]++;
        put_u32(p_indices + 4 * (size_t)slot, (uint32_t)j);
        for (int t = 0; t < Nb; ++t) {
            int rho = i + t;
            int p = rho % Nb;
            for (int r = 0; r < R; ++r) {
                float w = W[((size_t)rho * C + j) * R + r];
                memcpy(p_values + 4 * (((size_t)slot * Nb + p) * R + r), &w, 4);
            }
        }
    }
    free(bi); free(bj); free(cursor);
    return ORC_OK;
}

typedef struct {
    int M, C, R, Nb; int64_t m;
    const uint8_t *indptr, *indices, *values;
} orc_view;

static int view_blob(const uint8_t *blob, size_t len, orc_view *v)
{
    if (!blob || len < 64 || memcmp(blob, "UBP1", 4) != 0 || get_u32(blob + 4) != 1u) return ORC_E_FORMAT;
    v->M = (int)get_u32(blob + 8); v->C = (int)get_u32(blob + 12);
    v->R = (int)get_u32(blob + 16); v->Nb = (int)get_u32(blob + 20);
    v->m = (int64_t)get_u32(blob + 24);
    if (v->M <= 0 || v->C <= 0 || v->R <= 0 || v->Nb <= 0 || v->Nb > v->M) return ORC_E_FORMAT;
    if (len < orc_blob_size(v->M, v->R, v->Nb, v->m)) return ORC_E_FORMAT;
    v->indptr = blob + 64;
    v->indices = v->indptr + up64(4 * (size_t)(v->M + 1));
    v->values = v->indices + up64(4 * (size_t)v->m);
    return ORC_OK;
}

int orc_blob_dims(const uint8_t *blob, size_t len, int32_t *dims /* M,C,R,Nb,m */)
{
    orc_view v; int rc = view_blob(blob, len, &v);
    if (rc) return rc;
    dims[0] = v.M; dims[1] = v.C; dims[2] = v.R; dims[3] = v.Nb; dims[4] = (int32_t)v.m;
    return ORC_OK;
}

/* Inverse of orc_pack: W_out [M][C][R] zero-filled, mask_out [M][C]. */
int orc_unpack(const uint8_t *blob, size_t len, float *W_out, uint8_t *mask_out)
{
    orc_view v; int rc = view_blob(blob, len, &v);
    if (rc) return rc;
    if (W_out) memset(W_out, 0, sizeof(float) * (size_t)v.M * v.C * v.R);
    if (mask_out) memset(mask_out, 0, (size_t)v.M * v.C);
    for (int i = 0; i < v.M; ++i) {
        uint32_t b0 = get_u32(v.indptr + 4 * (size_t)i), b1 = get_u32(v.indptr + 4 * (size_t)(i + 1));
        if (b1 < b0 || (int64_t)b1 > v.m) return ORC_E_FORMAT;
        if (b1 > b0 && i + v.Nb > v.M) return ORC_E_FORMAT;
        for (uint32_t b = b0; b < b1; ++b) {
            int j = (int)get_u32(v.indices + 4 * (size_t)b);
            if (j < 0 || j >= v.C) return ORC_E_FORMAT;
            for (int t = 0; t < v.Nb; ++t) {
                int rho = i + t, p = rho % v.Nb;
                if (mask_out) mask_out[(size_t)rho * v.C + j] = 1;
                if (W_out)
                    memcpy(&W_out[((size_t)rho * v.C + j) * v.R],
                           v.values + 4 * (((size_t)b * v.Nb + p) * v.R), 4 * (size_t)v.R);
            }
        }
    }
    return ORC_OK;
}

/* ---- the definition: dense product of the masked weight ----------------- */
/*
 * Z[o][n] = sum_{c=0}^{C-1} Wm[o][c] * X[c][n], c ascending, pruned weights
 * enter as exact zeros; Y = act(Z + bias[o]); A[o][n] = sum |Wm||X| + |bias|.
 * W: [M][C] fp32, mask: [M][C], X: [C][ldx] fp32 (Nc columns used),
 * Y, A: [M][Nc] double (A may be NULL).
 */
int orc_masked_matmul(const float *W, const uint8_t *mask, int M, int C,
                      const float *X, int64_t ldx, int64_t Nc,
                      const float *bias, int relu, double *Y, double *A)
{
    if (!W || !mask || !X || !Y || M <= 0 || C <= 0 || Nc < 0 || ldx < Nc) return ORC_E_ARG;
    int err = 0;
#pragma omp parallel
    {
        double *z = (double *)malloc(sizeof(double) * (size_t)(Nc > 0 ? Nc : 1));
        double *a = (double *)malloc(sizeof(double) * (size_t)(Nc > 0 ? Nc : 1));
        if (!z || !a) {
#pragma omp atomic write
            err = 1;
        } else {
#pragma omp for schedule(static)
            for (int o = 0; o < M; ++o) {
                for (int64_t n = 0; n < Nc; ++n) { z[n] = 0.0; a[n] = 0.0; }
                for (int c = 0; c < C; ++c) {
                    double w = mask[(size_t)o * C + c] ? (double)W[(size_t)o * C + c] : 0.0;
                    double aw = fabs(w);
                    const float *x = X + (size_t)c * (size_t)ldx;
                    for (int64_t n = 0; n < Nc; ++n) {
                        z[n] += w * (double)x[n];
                        a[n] += aw * fabs((double)x[n]);
                    }
                }
                double b = bias ? (double)bias[o] : 0.0;
                for (int64_t n = 0; n < Nc; ++n) {
                    double y = z[n] + b;
                    if (relu && y < 0.0) y = 0.0;
                    Y[(size_t)o * (size_t)Nc + (size_t)n] = y;
                    if (A) A[(size_t)o * (size_t)Nc + (size_t)n] = a[n] + fabs(b);
                }
            }
        }
        free(z); free(a);
    }
    return err ? ORC_E_SPACE : ORC_OK;
}

/* single elements of orc_masked_matmul: outputs (so[s], sn[s]) */
int orc_masked_matmul_samples(const float *W, const uint8_t *mask, int M, int C,
                              const float *X, int64_t ldx, int64_t Nc,
                              const float *bias, int relu,
                              const int32_t *so, const int64_t *sn, int64_t ns,
                              double *Y, double *A)
{
    if (!W || !mask || !X || !Y || !so || !sn) return ORC_E_ARG;
    for (int64_t s = 0; s < ns; ++s)
        if (so[s] < 0 || so[s] >= M || sn[s] < 0 || sn[s] >= Nc) return ORC_E_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < ns; ++s) {
        int o = so[s]; int64_t n = sn[s];
        double z = 0.0, a = 0.0;
        for (int c = 0; c < C; ++c) {
            double w = mask[(size_t)o * C + c] ? (double)W[(size_t)o * C + c] : 0.0;
            double x = (double)X[(size_t)c * (size_t)ldx + (size_t)n];
            z += w * x; a += fabs(w) * fabs(x);
        }
        double b = bias ? (double)bias[o] : 0.0;
        double y = z + b;
        if (relu && y < 0.0) y = 0.0;
        Y[s] = y;
        if (A) A[s] = a + fabs(b);
    }
    return ORC_OK;
}

/*
 * 3x3 cross-correlation, stride 1, zero padding 1, on the masked weight:
 * Z[b][o][y][x] = sum_c sum_r sum_s Wm[o][c][3r+s] * In[b][c][y+r-1][x+s-1].
 * A block keeps or drops all nine taps of (o, c) together (Section 3.1: the
 * block spans the whole h x w kernel), so mask is [M][C].
 * In / Y are addressed through element strides (batch, channel); rows of an
 * image are contiguous (row stride Wd). Y, A double with their own strides.
 */
int orc_masked_conv3x3(const float *W, const uint8_t *mask, int M, int C,
                       const float *In, int B, int H, int Wd,
                       int64_t in_sb, int64_t in_sc,
                       const float *bias, int relu,
                       double *Y, double *A, int64_t out_sb, int64_t out_sc)
{
    if (!W || !mask || !In || !Y || M <= 0 || C <= 0 || B < 0 || H <= 0 || Wd <= 0) return ORC_E_ARG;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int o = 0; o < M; ++o) {
            double bo = bias ? (double)bias[o] : 0.0;
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < Wd; ++x) {
                    double z = 0.0, a = 0.0;
                    for (int c = 0; c < C; ++c) {
                        if (!mask[(size_t)o * C + c]) continue; /* nine exact zeros */
                        const float *w = W + ((size_t)o * C + c) * 9;
                        const float *in = In + (size_t)b * (size_t)in_sb + (size_t)c * (size_t)in_sc;
                        for (int r = 0; r < 3; ++r) {
                            int yy = y + r - 1;
                            if (yy < 0 || yy >= H) continue;
                            for (int s = 0; s < 3; ++s) {
                                int xx = x + s - 1;
                                if (xx < 0 || xx >= Wd) continue;
                                double wv = (double)w[3 * r + s];
                                double xv = (double)in[(size_t)yy * Wd + xx];
                                z += wv * xv; a += fabs(wv) * fabs(xv);
                            }
                        }
                    }
                    double v = z + bo;
                    if (relu && v < 0.0) v = 0.0;
                    size_t off = (size_t)b * (size_t)out_sb + (size_t)o * (size_t)out_sc + (size_t)y * Wd + x;
                    Y[off] = v;
                    if (A) A[off] = a + fabs(bo);
                }
        }
    return ORC_OK;
}

/* single elements of orc_masked_conv3x3: (sb, so, sy, sx) per sample */
int orc_masked_conv3x3_samples(const float *W, const uint8_t *mask, int M, int C,
                               const float *In, int B, int H, int Wd,
                               int64_t in_sb, int64_t in_sc, const float *bias, int relu,
                               const int32_t *sb, const int32_t *so, const int32_t *sy, const int32_t *sx,
                               int64_t ns, double *Y, double *A)
{
    if (!W || !mask || !In || !Y) return ORC_E_ARG;
    for (int64_t s = 0; s < ns; ++s)
        if (sb[s] < 0 || sb[s] >= B || so[s] < 0 || so[s] >= M || sy[s] < 0 || sy[s] >= H ||
            sx[s] < 0 || sx[s] >= Wd) return ORC_E_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < ns; ++q) {
        int b = sb[q], o = so[q], y = sy[q], x = sx[q];
        double z = 0.0, a = 0.0;
        for (int c = 0; c < C; ++c) {
            if (!mask[(size_t)o * C + c]) continue;
            const float *w = W + ((size_t)o * C + c) * 9;
            const float *in = In + (size_t)b * (size_t)in_sb + (size_t)c * (size_t)in_sc;
            for (int r = 0; r < 3; ++r)
                for (int s = 0; s < 3; ++s) {
                    int yy = y + r - 1, xx = x + s - 1;
                    if (yy < 0 || yy >= H || xx < 0 || xx >= Wd) continue;
                    double wv = (double)w[3 * r + s], xv = (double)in[(size_t)yy * Wd + xx];
                    z += wv * xv; a += fabs(wv) * fabs(xv);
                }
        }
        double bo = bias ? (double)bias[o] : 0.0;
        double v = z + bo;
        if (relu && v < 0.0) v = 0.0;
        Y[q] = v;
        if (A) A[q] = a + fabs(bo);
    }
    return ORC_OK;
}

/* ---- the paper's dataflow on the packed format -------------------------- */
/*
 * Weight-rotating, output-stationary walk (Section 4.2) for a 1x1 layer
 * (R == 1). Output columns are handled in tiles of `tile_w` columns. For one
 * column tile keep N accumulator vectors R_0..R_{N-1}. Tile i (i = 0..M-N)
 * holds the blocks that start at output row i: for each of them load the
 * input vector of channel indices[b] and add values[b][p] * x into R_p for
 * every slot p -- no slot arithmetic at run time, the rotation was done when
 * packing. After tile i only R_{i mod N} is complete (row i); store it and
 * clear it. After the last tile the N-1 rows still in the register file are
 * stored by the epilogue. Y: [M][Nc] double.
 */
int orc_wros_spmm(const uint8_t *blob, size_t len, const float *X, int64_t ldx, int64_t Nc,
                  const float *bias, int relu, int tile_w, double *Y)
{
    orc_view v; int rc = view_blob(blob, len, &v);
    if (rc) return rc;
    if (v.R != 1 || !X || !Y || tile_w <= 0 || ldx < Nc) return ORC_E_ARG;
    const int N = v.Nb, M = v.M;
    double *Rf = (double *)malloc(sizeof(double) * (size_t)N * (size_t)tile_w);
    if (!Rf) return ORC_E_SPACE;
    for (int64_t n0 = 0; n0 < Nc; n0 += tile_w) {
        int tw = (int)((Nc - n0 < tile_w) ? (Nc - n0) : tile_w);
        for (int q = 0; q < N * tile_w; ++q) Rf[q] = 0.0;
        for (int i = 0; i + N <= M; ++i) {
            uint32_t b0 = get_u32(v.indptr + 4 * (size_t)i), b1 = get_u32(v.indptr + 4 * (size_t)(i + 1));
            for (uint32_t b = b0; b < b1; ++b) {
                int j = (int)get_u32(v.indices + 4 * (size_t)b);
                const float *x = X + (size_t)j * (size_t)ldx + (size_t)n0;
                for (int p = 0; p < N; ++p) {
                    float w; memcpy(&w, v.values + 4 * ((size_t)b * N + p), 4);
                    for (int t = 0; t < tw; ++t) Rf[p * tile_w + t] += (double)w * (double)x[t];
                }
            }
            int p = i % N;                                  /* the finished row */
            double bo = bias ? (double)bias[i] : 0.0;
            for (int t = 0; t < tw; ++t) {
                double y = Rf[p * tile_w + t] + bo;
                if (relu && y < 0.0) y = 0.0;
                Y[(size_t)i * (size_t)Nc + (size_t)(n0 + t)] = y;
                Rf[p * tile_w + t] = 0.0;
            }
        }
        for (int rho = M - N + 1; rho < M; ++rho) {         /* epilogue: N-1 rows */
            int p = rho % N;
            double bo = bias ? (double)bias[rho] : 0.0;
            for (int t = 0; t < tw; ++t) {
                double y = Rf[p * tile_w + t] + bo;
                if (relu && y < 0.0) y = 0.0;
                Y[(size_t)rho * (size_t)Nc + (size_t)(n0 + t)] = y;
            }
        }
    }
    free(Rf);
    return ORC_OK;
}
