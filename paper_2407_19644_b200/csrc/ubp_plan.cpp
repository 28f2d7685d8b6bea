// Plan builder: re-buckets the canonical blocks (start row, input channel,
// rotated values; Section 4.2) for the GPU kernels. Host code only.
//
// Each canonical block is un-rotated, cut into entries of `nbk` rows and
// filed under (input-channel tile, row panel, start offset inside the panel).
// An entry whose rows cross a panel boundary is filed in both panels (with a
// negative start offset in the lower one); each panel's kernel code touches
// only its own rows, so every output element has exactly one writer and a
// fixed summation order -- the GPU counterpart of the paper's fix for
// overlapping output tiles (Section 3.3).
#include "ubp_internal.h"

#include <algorithm>
#include <cstdio>
#include <cstring>

namespace ubp {

const std::vector<KernelCfg> &kernel_cfgs()
{
    static const std::vector<KernelCfg> cfgs = {
#define UBP_CFG(ID, KIND, NBK, P_, V_, WR_, WC_, KT_, DUP) {ID, KIND, NBK, P_, V_, WR_, WC_, KT_, DUP},
#include "ubp_cfgs.inc"
#undef UBP_CFG
    };
    return cfgs;
}

const KernelCfg *find_cfg(int id)
{
    for (const auto &c : kernel_cfgs())
        if (c.id == id) return &c;
    return nullptr;
}

static int largest_pow2_divisor_le16(int Nb)
{
    int k = 1;
    while (k < 16 && Nb % (k * 2) == 0) k *= 2;
    return k;
}

const KernelCfg *auto_cfg(int M, int C, int R, int Nb, int64_t m)
{
    (void)M; (void)C; (void)m;
    const int nbk = largest_pow2_divisor_le16(Nb);
    const double dens = (double)m * Nb / ((double)M * C);
    // The tensor-core variants run on CTA pairs, and there the bf16-product form (ids + 4: half the tensor-core and
    // shared-memory time, error <= 3 * 2^-16 |w||x|, inside the 1e-4 gate) is the default; the TF32-product ids stay
    // selectable (with at most 128 rows they run the one-CTA kernel).
    const int fast = 4;
    if (R == 9 && tensor_core_pays(M, C, dens) && M >= 128 && C >= 16) {    // implicit GEMM on tensor cores, taps as operand shifts
        switch (nbk) {
            case 16: case 8: return find_cfg(64);
            case 4: return find_cfg(65);
            case 2: return find_cfg(66);
            default: return find_cfg(67);
        }
    }
    if (R == 9) {
        switch (nbk) {
            case 16: case 8: return find_cfg(20);
            case 4: return find_cfg(21);
            case 2: return find_cfg(22);
            default: return find_cfg(23);
        }
    }
    if (R != 1) return nullptr;
    // Dense tensor-core variant when enough of the weight survives (tensor_core_pays) and the layer is large enough
    // to amortise its per-tile set-up: it pays from 128 rows and 64 input channels on (measured on the
    // MobileNet-shaped layers, launches back to back: 128 -> 128 channels 42 us against 60 us; 64 -> 128 channels 35
    // against 39; 32 -> 64 channels 95 against 54, so below that the sparse kernel stays).
    if (tensor_core_pays(M, C, dens) && M >= 128 && C >= 64) {
        switch (nbk) {
            case 16: case 8: return find_cfg(33 + fast);
            case 4: return find_cfg(32 + fast);
            case 2: return find_cfg(31 + fast);
            default: return find_cfg(30 + fast);
        }
    }
    // Sparse kernel (measured sweep): 8-row panels, 256 columns per warp; 16 warps per CTA, or 8 when the layer has
    // no more than 64 output rows; 64-channel tiles, or 32 when the layer has no more than 32 input channels.
    // 16-row blocks run as two 8-row entries.
    const bool few_rows = M <= 64, few_ch = C <= 32;
    int id;
    switch (nbk) {
        case 16: case 8: id = few_rows ? (few_ch ? 54 : 55) : 16; break;
        case 4: id = few_rows ? (few_ch ? 50 : 51) : 14; break;
        case 2: id = few_rows ? (few_ch ? 52 : 53) : 15; break;
        default: id = few_rows ? (few_ch ? 56 : 57) : 17; break;
    }
    return find_cfg(id);
}

static inline size_t pad16(size_t x) { return (x + 15) & ~(size_t)15; }

int build_plan_image(const ubp_view_t &v, const KernelCfg &cfg, bool count_only, PlanImage &img, size_t *bytes)
{
    const int M = v.M, C = v.C, R = v.R, Nb = v.Nb;
    if (cfg.kind == 4) {
        // the canonical arrays as they are, behind the 256-byte header with the status word
        if (R != 1 || (Nb != 1 && Nb != 2 && Nb != 4 && Nb != 8 && Nb != 16)) return UBP_E_UNSUPPORTED;
        const size_t o0 = 256, o1 = pad16(o0 + sizeof(int32_t) * ((size_t)M + 1));
        const size_t o2 = pad16(o1 + sizeof(int32_t) * (size_t)v.m);
        const size_t total = (o2 + sizeof(float) * (size_t)v.m * Nb + 255) & ~(size_t)255;
        img = PlanImage();
        img.wros_off[0] = o0; img.wros_off[1] = o1; img.wros_off[2] = o2;
        img.entries = v.m;
        if (bytes) *bytes = total;
        if (count_only) return UBP_OK;
        img.bytes.assign(total, 0);
        std::memcpy(img.bytes.data() + o0, v.indptr, sizeof(int32_t) * ((size_t)M + 1));
        std::memcpy(img.bytes.data() + o1, v.indices, sizeof(int32_t) * (size_t)v.m);
        std::memcpy(img.bytes.data() + o2, v.values, sizeof(float) * (size_t)v.m * Nb);
        return UBP_OK;
    }
    const int nbk = cfg.nbk, P = cfg.P, KT = cfg.KT, WR = cfg.WR;
    // kind 5: the blob is that of the TRANSPOSED layer (ubp_pack_kmajor): its "rows" are the layer's input channels,
    // its "channels" the layer's output rows, and a block is Nb consecutive input channels of one output row. An
    // entry = one such run (or the part of it inside one channel tile): nbk = Nb weights in channel order, filed
    // under (channel tile, row panel, row inside the panel).
    const bool krun = cfg.kind == 5;
    if (krun ? (Nb != nbk || nbk > 16 || R != 1 || KT < nbk) : (Nb % nbk != 0)) return UBP_E_UNSUPPORTED;
    const bool conv = (cfg.kind == 1 || cfg.kind == 3);
    if ((!conv && R != 1) || (conv && R != 9)) return UBP_E_UNSUPPORTED;
    const int rowsL = krun ? C : M, chanL = krun ? M : C;            // the layer's output rows / input channels
    const int nkt = (chanL + KT - 1) / KT;
    const int NP = (rowsL + P - 1) / P;
    const int NG = (NP + WR - 1) / WR;
    const int F = krun ? P : P + nbk - 1;
    const int sub = krun ? 1 : Nb / nbk;
    const size_t wfloats = (size_t)nbk * R * (cfg.dupw ? 2 : 1);   // floats per entry
    // Every entry of the plan, in filing order: fn(channel tile, panel, fragment, channel inside the tile, weights).
    std::vector<float> wblk((size_t)Nb * R);
    auto for_each_entry = [&](auto &&fn) {
        for (int i = 0; i < M; ++i)
            for (int32_t b = v.indptr[i]; b < v.indptr[i + 1]; ++b) {
                const int j = v.indices[b];
                const float *val = v.values + (size_t)b * Nb * R;
                for (int t = 0; t < Nb; ++t)       // undo the rotation: row i+t lives in slot (i+t) mod Nb
                    std::memcpy(&wblk[(size_t)t * R], val + (size_t)((i + t) % Nb) * R, sizeof(float) * (size_t)R);
                if (krun) {
                    // run of channels i .. i+Nb-1 of output row j; cut at channel-tile boundaries. A piece is stored as
                    // a full-length entry that lies wholly inside its tile: its start is moved into the tile and the
                    // places of channels that do not belong to the piece hold zero weights (the activations read there
                    // are real, finite values of the same tile).
                    float wpart[16];
                    for (int kt = i / KT; kt <= (i + Nb - 1) / KT; ++kt) {
                        const int T0 = kt * KT;
                        int ks = i - T0;
                        if (ks < 0) ks = 0;
                        if (ks > KT - Nb) ks = KT - Nb;
                        for (int u = 0; u < Nb; ++u) {
                            const int c = T0 + ks + u;
                            wpart[u] = (c >= i && c < i + Nb) ? wblk[(size_t)(c - i)] : 0.0f;
                        }
                        fn(kt, j / P, j % P, ks, wpart);
                    }
                    continue;
                }
                const int kt = j / KT, jl = j % KT;
                for (int u = 0; u < sub; ++u) {
                    const int r0 = i + u * nbk;
                    const int p = r0 / P, s = r0 % P;
                    fn(kt, p, s + nbk - 1, jl, &wblk[(size_t)u * nbk * R]);
                    if (s + nbk > P) fn(kt, p + 1, s - P + nbk - 1, jl, &wblk[(size_t)u * nbk * R]);   // crosses into the next panel
                }
            }
    };

    // pass 1: entries per (kt, panel, fragment)
    std::vector<uint32_t> cnt((size_t)nkt * NP * F, 0);
    auto bucket = [&](int kt, int p, int f) -> size_t { return ((size_t)kt * NP + p) * F + f; };
    int64_t entries = 0;
    for_each_entry([&](int kt, int p, int f, int, const float *) { cnt[bucket(kt, p, f)]++; ++entries; });

    // layout
    const size_t tab_off = 256;
    const size_t tab_bytes = pad16(sizeof(uint32_t) * ((size_t)nkt * NG + 1));
    const size_t poff_bytes = pad16(sizeof(uint32_t) * (size_t)(WR + 1));
    const size_t fo_bytes = pad16(sizeof(uint16_t) * (size_t)(F + 1));
    std::vector<size_t> seg_off((size_t)nkt * NP, 0);        // absolute offset of each panel sub-segment
    std::vector<size_t> grp_off((size_t)nkt * NG + 1, 0);
    size_t cur = pad16(tab_off + tab_bytes);
    uint32_t max_group = 0;
    for (int kt = 0; kt < nkt; ++kt)
        for (int g = 0; g < NG; ++g) {
            grp_off[(size_t)kt * NG + g] = cur;
            const size_t g0 = cur;
            cur += poff_bytes;
            for (int p = g * WR; p < std::min(NP, (g + 1) * WR); ++p) {
                size_t n = 0;
                for (int f = 0; f < F; ++f) n += cnt[bucket(kt, p, f)];
                if (n > 65535) return UBP_E_UNSUPPORTED;
                seg_off[(size_t)kt * NP + p] = cur;
                cur += fo_bytes + pad16(2 * (n + 4)) + pad16(4 * (n + 2) * wfloats);
            }
            if (cur - g0 > max_group) max_group = (uint32_t)(cur - g0);
        }
    grp_off[(size_t)nkt * NG] = cur;
    size_t total = (cur + 255) & ~(size_t)255;
    if (total / 16 > 0xffffffffull) return UBP_E_UNSUPPORTED;
    img.tc_off = 0; img.tc_kp = 0; img.tc16_off = 0; img.tc16_kp = 0;
    if (cfg.kind == 2 || cfg.kind == 3) {   // dense part for the tensor-core kernel: Wh, Wl as [M][Kp] floats,
        img.tc_kp = (C * R + 3) & ~3;       // reduction index k = tap * C + channel (tap-major)
        img.tc_off = total;
        total += ((size_t)2 * M * img.tc_kp * sizeof(float) + 255) & ~(size_t)255;
        // The same matrix as two bf16 pieces, tiled for the CTA-pair kernel: one 8 KB block per (128-row tile,
        // 16-channel chunk) = [piece W1, W2][128 rows][16 channels] exactly as the kernel wants it in shared memory
        // (rows of 32 bytes whose two 16-byte halves are swapped on rows with bit 2 set: the 32-byte swizzle of a
        // K-major operand), so that a chunk is ONE contiguous bulk copy instead of 256 row pieces. A layer of at most
        // 128 rows puts half of them into each of the pair's two tiles (the rest of a tile stays zero).
        img.tc16_kp = (C * R + 15) & ~15;   // padded reduction length: whole chunks
        img.tc16_off = total;
        img.tc16_pieces = cfg_pieces(cfg);  // 2 pieces: 8 KB blocks; 3 pieces (W3 = what W1 + W2 leave): 12 KB blocks
        total += (size_t)((M + 255) / 256) * 2 * (img.tc16_kp / 16) * 4096 * img.tc16_pieces;   // whole pairs of row tiles
    }
    if (bytes) *bytes = total;
    img.nkt = nkt; img.NP = NP; img.NG = NG; img.F = F; img.entries = entries; img.max_group_bytes = max_group;
    if (count_only) return UBP_OK;

    img.bytes.assign(total, 0);
    uint8_t *base = img.bytes.data();
    uint32_t *tab = reinterpret_cast<uint32_t *>(base + tab_off);
    for (size_t q = 0; q < grp_off.size(); ++q) tab[q] = (uint32_t)(grp_off[q] / 16);
    // group headers, fragment offsets; cursors start at the fragment offsets
    std::vector<uint32_t> cursor(cnt.size(), 0);
    for (int kt = 0; kt < nkt; ++kt)
        for (int g = 0; g < NG; ++g) {
            const size_t g0 = grp_off[(size_t)kt * NG + g];
            uint32_t *poff = reinterpret_cast<uint32_t *>(base + g0);
            size_t end = g0 + poff_bytes;
            for (int w = 0; w <= WR; ++w) {
                const int p = g * WR + w;
                if (w < WR && p < NP) {
                    const size_t so = seg_off[(size_t)kt * NP + p];
                    poff[w] = (uint32_t)(so - g0);
                    uint16_t *fo = reinterpret_cast<uint16_t *>(base + so);
                    uint32_t acc = 0;
                    for (int f = 0; f < F; ++f) {
                        fo[f] = (uint16_t)acc;
                        cursor[bucket(kt, p, f)] = acc;
                        acc += cnt[bucket(kt, p, f)];
                    }
                    fo[F] = (uint16_t)acc;
                    end = so + fo_bytes + pad16(2 * ((size_t)acc + 4)) + pad16(4 * ((size_t)acc + 2) * wfloats);
                } else {
                    poff[w] = (uint32_t)(end - g0);
                }
            }
        }
    // pass 2: file the entries (start rows ascending, then input channel ascending)
    auto put = [&](int kt, int p, int f, int jl, const float *wsrc /* [nbk][R] */) {
        const size_t so = seg_off[(size_t)kt * NP + p];
        const uint16_t *fo = reinterpret_cast<const uint16_t *>(base + so);
        const size_t n = fo[F];
        const uint32_t e = cursor[bucket(kt, p, f)]++;
        uint16_t *jl_arr = reinterpret_cast<uint16_t *>(base + so + fo_bytes);
        float *w_arr = reinterpret_cast<float *>(base + so + fo_bytes + pad16(2 * (n + 4)));
        jl_arr[e] = (uint16_t)jl;
        float *dst = w_arr + (size_t)e * wfloats;
        if (cfg.dupw) {
            for (size_t q = 0; q < (size_t)nbk * R; ++q) { dst[2 * q] = wsrc[q]; dst[2 * q + 1] = wsrc[q]; }
        } else {
            std::memcpy(dst, wsrc, sizeof(float) * (size_t)nbk * R);
        }
    };
    for_each_entry(put);
    if (cfg.kind == 2 || cfg.kind == 3) {
        // Densify and split every kept weight into the part a TF32 operand holds exactly (sign, exponent,
        // top 10 mantissa bits) and the remainder, itself cut to TF32; pruned positions stay zero.
        float *Wh = reinterpret_cast<float *>(base + img.tc_off);
        float *Wl = Wh + (size_t)M * img.tc_kp;
        // and into two bf16 pieces: the weight rounded to nearest-even bf16, and the (exact) remainder rounded
        uint8_t *W16 = base + img.tc16_off;
        const size_t nchunk16 = (size_t)img.tc16_kp / 16;
        auto w16_at = [&](int row, size_t k, int piece) -> uint16_t * {
            const size_t blk = (size_t)(row / 128) * nchunk16 + k / 16;
            const int i = row % 128;           // position in the 128-row tile = tensor-memory lane of the output row
            const int kk = (int)(k % 16);
            return reinterpret_cast<uint16_t *>(W16 + blk * (4096 * (size_t)img.tc16_pieces) + (size_t)piece * 4096 + (size_t)i * 32 +
                                                (size_t)(((kk >> 3) ^ ((i >> 2) & 1)) * 16) + (size_t)(kk & 7) * 2);
        };
        auto bf16_rn = [](float f) -> uint16_t {
            uint32_t b;
            std::memcpy(&b, &f, 4);
            if ((b & 0x7f800000u) == 0x7f800000u) return (uint16_t)((b >> 16) | ((b & 0xffffu) ? 0x40u : 0u));   // inf / nan
            b += 0x7fffu + ((b >> 16) & 1u);
            return (uint16_t)(b >> 16);
        };
        auto bf16_f = [](uint16_t h) -> float {
            const uint32_t b = (uint32_t)h << 16;
            float f;
            std::memcpy(&f, &b, 4);
            return f;
        };
        for (int i = 0; i < M; ++i)
            for (int32_t b = v.indptr[i]; b < v.indptr[i + 1]; ++b) {
                const int j = v.indices[b];
                const float *val = v.values + (size_t)b * Nb * R;
                for (int t = 0; t < Nb; ++t)
                  for (int r = 0; r < R; ++r) {
                    const float w = val[(size_t)((i + t) % Nb) * R + r];
                    uint32_t bits;
                    std::memcpy(&bits, &w, 4);
                    bits &= 0xffffe000u;
                    float hi;
                    std::memcpy(&hi, &bits, 4);
                    float lo = w - hi;
                    std::memcpy(&bits, &lo, 4);
                    bits &= 0xffffe000u;
                    std::memcpy(&lo, &bits, 4);
                    Wh[(size_t)(i + t) * img.tc_kp + (size_t)r * C + j] = hi;
                    Wl[(size_t)(i + t) * img.tc_kp + (size_t)r * C + j] = lo;
                    const uint16_t w1 = bf16_rn(w);
                    const uint16_t w2 = bf16_rn(w - bf16_f(w1));
                    *w16_at(i + t, (size_t)r * C + j, 0) = w1;
                    *w16_at(i + t, (size_t)r * C + j, 1) = w2;
                    if (img.tc16_pieces == 3) *w16_at(i + t, (size_t)r * C + j, 2) = bf16_rn((w - bf16_f(w1)) - bf16_f(w2));
                  }
            }
    }
    return UBP_OK;
}

}  // namespace ubp
