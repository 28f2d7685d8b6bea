// Host-side canonical format of a UBP weight: mask -> blocks -> indptr /
// indices / rotated values (Section 4.2 of the paper; mask decoding is the
// block-division step, Algorithm 2), and back. Pure CPU code, no CUDA.
#include "ubp_internal.h"

#include <cstring>
#include <new>
#include <vector>

namespace ubp {

static inline size_t align64(size_t x) { return (x + 63) / 64 * 64; }

struct BlobLayout {
    size_t off_indptr, off_indices, off_values, total;
};

static BlobLayout layout_of(int M, int R, int Nb, int64_t m)
{
    BlobLayout l;
    l.off_indptr = 64;
    l.off_indices = l.off_indptr + align64(sizeof(int32_t) * (size_t)(M + 1));
    l.off_values = l.off_indices + align64(sizeof(int32_t) * (size_t)m);
    l.total = l.off_values + align64(sizeof(float) * (size_t)m * (size_t)Nb * (size_t)R);
    return l;
}

struct Header {           // 32 meaningful bytes, little endian (x86 / aarch64 hosts)
    char magic[4];
    uint32_t version;
    int32_t M, C, R, Nb, m;
    uint32_t flags;
};
static_assert(sizeof(Header) == 32, "header layout");

// Count the blocks starting at each row: per column, every maximal run of
// ones [a, b) must have (b - a) % Nb == 0 and is cut at a, a+Nb, ...
// starts_per_row has M entries. Returns status.
static int count_starts(const uint8_t *mask, int M, int C, int Nb, std::vector<int32_t> &starts_per_row)
{
    starts_per_row.assign((size_t)M, 0);
    for (int j = 0; j < C; ++j) {
        int a = -1;                           // first row of the open run, -1 = none
        for (int i = 0; i <= M; ++i) {
            int v = 0;
            if (i < M) {
                v = mask[(size_t)i * C + j];
                if (v > 1) return UBP_E_ARG;
            }
            if (v) {
                if (a < 0) a = i;
            } else if (a >= 0) {
                if ((i - a) % Nb != 0) return UBP_E_RAGGED;
                for (int s = a; s < i; s += Nb) starts_per_row[(size_t)s]++;
                a = -1;
            }
        }
    }
    return UBP_OK;
}

int pack(const float *W, const uint8_t *mask, int M, int C, int R, int Nb,
         void *blob, size_t blob_cap, size_t *blob_len)
{
    if (!W || !mask || !blob_len || M <= 0 || C <= 0 || R <= 0 || Nb <= 0 || Nb > M) return UBP_E_ARG;
    std::vector<int32_t> cnt;
    int rc = count_starts(mask, M, C, Nb, cnt);
    if (rc) return rc;
    int64_t m = 0;
    for (int i = 0; i < M; ++i) m += cnt[(size_t)i];
    if (m > INT32_MAX) return UBP_E_UNSUPPORTED;
    BlobLayout l = layout_of(M, R, Nb, m);
    *blob_len = l.total;
    if (!blob) return UBP_OK;
    if (blob_cap < l.total) return UBP_E_SPACE;

    uint8_t *base = static_cast<uint8_t *>(blob);
    std::memset(base, 0, l.total);
    Header h;
    std::memcpy(h.magic, "UBP1", 4);
    h.version = 1; h.M = M; h.C = C; h.R = R; h.Nb = Nb; h.m = (int32_t)m; h.flags = 1u;
    std::memcpy(base, &h, sizeof h);
    int32_t *indptr = reinterpret_cast<int32_t *>(base + l.off_indptr);
    int32_t *indices = reinterpret_cast<int32_t *>(base + l.off_indices);
    float *values = reinterpret_cast<float *>(base + l.off_values);

    indptr[0] = 0;
    for (int i = 0; i < M; ++i) indptr[i + 1] = indptr[i] + cnt[(size_t)i];
    // Row-major sweep: for start row i, columns in ascending order. A block
    // starts at (i, j) iff mask[i][j] is one and the number of ones directly
    // above it in the column is a multiple of Nb. `above` carries that count.
    std::vector<int32_t> above((size_t)C, 0);
    int32_t b = 0;
    for (int i = 0; i < M; ++i) {
        const uint8_t *mrow = mask + (size_t)i * C;
        for (int j = 0; j < C; ++j) {
            if (!mrow[j]) { above[(size_t)j] = 0; continue; }
            if (above[(size_t)j] % Nb == 0) {
                indices[b] = j;
                float *dst = values + (size_t)b * Nb * R;
                for (int t = 0; t < Nb; ++t) {
                    const int rho = i + t;
                    std::memcpy(dst + (size_t)(rho % Nb) * R, W + ((size_t)rho * C + j) * R,
                                sizeof(float) * (size_t)R);
                }
                ++b;
            }
            above[(size_t)j]++;
        }
    }
    return (b == (int32_t)m) ? UBP_OK : UBP_E_FORMAT;
}

int blob_view(const void *blob, size_t len, ubp_view_t *v)
{
    if (!blob || !v) return UBP_E_ARG;
    if (len < 64) return UBP_E_FORMAT;
    Header h;
    std::memcpy(&h, blob, sizeof h);
    if (std::memcmp(h.magic, "UBP1", 4) != 0 || h.version != 1 || !(h.flags & 1u)) return UBP_E_FORMAT;
    if (h.M <= 0 || h.C <= 0 || h.R <= 0 || h.Nb <= 0 || h.Nb > h.M || h.m < 0) return UBP_E_FORMAT;
    BlobLayout l = layout_of(h.M, h.R, h.Nb, h.m);
    if (len < l.total) return UBP_E_FORMAT;
    const uint8_t *base = static_cast<const uint8_t *>(blob);
    v->M = h.M; v->C = h.C; v->R = h.R; v->Nb = h.Nb; v->m = h.m;
    v->indptr = reinterpret_cast<const int32_t *>(base + l.off_indptr);
    v->indices = reinterpret_cast<const int32_t *>(base + l.off_indices);
    v->values = reinterpret_cast<const float *>(base + l.off_values);
    // structural checks: monotone indptr ending at m, no start below M - Nb,
    // channels in range and ascending inside a start row, and no two blocks of
    // one input channel overlapping (Eq. 2): walking the start rows upwards,
    // next_free[j] is the first row of channel j not covered by a block so far
    if (v->indptr[0] != 0 || v->indptr[h.M] != h.m) return UBP_E_FORMAT;
    std::vector<int32_t> next_free;
    try { next_free.assign((size_t)h.C, 0); } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
    for (int i = 0; i < h.M; ++i) {
        const int32_t b0 = v->indptr[i], b1 = v->indptr[i + 1];
        if (b1 < b0 || b1 > h.m) return UBP_E_FORMAT;
        if (b1 > b0 && i + h.Nb > h.M) return UBP_E_FORMAT;
        for (int32_t b = b0; b < b1; ++b) {
            const int32_t j = v->indices[b];
            if (j < 0 || j >= h.C) return UBP_E_FORMAT;
            if (b > b0 && v->indices[b - 1] >= j) return UBP_E_FORMAT;
            if (next_free[(size_t)j] > i) return UBP_E_FORMAT;
            next_free[(size_t)j] = i + h.Nb;
        }
    }
    return UBP_OK;
}

int unpack(const void *blob, size_t len, float *W_out, uint8_t *mask_out)
{
    ubp_view_t v;
    int rc = blob_view(blob, len, &v);
    if (rc) return rc;
    const size_t MC = (size_t)v.M * v.C;
    if (W_out) std::memset(W_out, 0, sizeof(float) * MC * v.R);
    if (mask_out) std::memset(mask_out, 0, MC);
    for (int i = 0; i < v.M; ++i)
        for (int32_t b = v.indptr[i]; b < v.indptr[i + 1]; ++b) {
            const int j = v.indices[b];
            const float *src = v.values + (size_t)b * v.Nb * v.R;
            for (int t = 0; t < v.Nb; ++t) {
                const int rho = i + t;
                if (mask_out) {
                    if (mask_out[(size_t)rho * v.C + j]) return UBP_E_FORMAT;   // overlapping blocks
                    mask_out[(size_t)rho * v.C + j] = 1;
                }
                if (W_out)
                    std::memcpy(W_out + ((size_t)rho * v.C + j) * v.R, src + (size_t)(rho % v.Nb) * v.R,
                                sizeof(float) * (size_t)v.R);
            }
        }
    return UBP_OK;
}

}  // namespace ubp
