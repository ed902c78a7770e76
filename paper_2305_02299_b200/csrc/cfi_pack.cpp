// Host side of the library that needs no CUDA: cfi_pack and the status names.
#include "cfi.h"

#include <cstddef>
#include <algorithm>
#include <vector>

extern "C" const char* cfi_status_string(cfi_status_t s) {
    switch (s) {
        case CFI_OK: return "CFI_OK";
        case CFI_ERR_NULL: return "CFI_ERR_NULL: a required pointer is NULL";
        case CFI_ERR_SHAPE: return "CFI_ERR_SHAPE: a size is negative, inconsistent or unsupported";
        case CFI_ERR_NOT_CONSTANT_FAN_IN: return "CFI_ERR_NOT_CONSTANT_FAN_IN: non-empty rows keep different numbers of weights";
        case CFI_ERR_INDEX_RANGE: return "CFI_ERR_INDEX_RANGE: a column index or row number is out of range or repeated";
        case CFI_ERR_BUFFER_TOO_SMALL: return "CFI_ERR_BUFFER_TOO_SMALL: batch exceeds the size the buffers were created for";
        case CFI_ERR_DTYPE: return "CFI_ERR_DTYPE: unknown or mismatched dtype, activation or variant";
        case CFI_ERR_ALLOC: return "CFI_ERR_ALLOC: allocation failed";
        case CFI_ERR_CUDA: return "CFI_ERR_CUDA: a CUDA call or kernel launch failed";
        case CFI_ERR_DEVICE_FLAG: return "CFI_ERR_DEVICE_FLAG: a kernel recorded an error in the device status word";
        case CFI_ERR_ALIGNMENT: return "CFI_ERR_ALIGNMENT: x or y is not 16-byte aligned";
    }
    return "unknown cfi_status_t";
}

namespace {
// Structure test for one dense entry: the mask decides when there is one; otherwise any
// value that compares unequal to zero is kept (so -0.0 is pruned and NaN is kept).
inline bool kept(const float* w, const uint8_t* mask, size_t p) { return mask ? mask[p] != 0 : w[p] != 0.0f; }
}  // namespace

extern "C" cfi_status_t cfi_pack(const float* w_dense, const uint8_t* mask, int32_t out_features, int32_t in_features,
                                 int32_t* k, int32_t* n_active, float* values, int32_t* indices,
                                 int32_t* active_rows) {
    if (!w_dense || !k || !n_active) return CFI_ERR_NULL;
    if (out_features < 0 || in_features < 0) return CFI_ERR_SHAPE;
    const bool fill = values || indices || active_rows;
    if (fill && !(values && indices && active_rows)) return CFI_ERR_NULL;

    // One pass over the rows: count, check the constant-fan-in property, and, when filling, emit
    // the row as soon as its count is known to be right (the first non-empty row fixes k).
    int32_t fan_in = 0, rows = 0;
    for (int32_t o = 0; o < out_features; ++o) {
        const size_t base = (size_t)o * (size_t)in_features;
        int32_t cnt = 0;
        for (int32_t c = 0; c < in_features; ++c) cnt += kept(w_dense, mask, base + c) ? 1 : 0;
        if (cnt == 0) continue;
        if (fan_in == 0) fan_in = cnt;
        else if (cnt != fan_in) return CFI_ERR_NOT_CONSTANT_FAN_IN;
        if (fill) {
            float* vrow = values + (size_t)rows * fan_in;
            int32_t* irow = indices + (size_t)rows * fan_in;
            int32_t j = 0;
            for (int32_t c = 0; c < in_features; ++c)
                if (kept(w_dense, mask, base + c)) { vrow[j] = w_dense[base + c]; irow[j] = c; ++j; }
            active_rows[rows] = o;
        }
        ++rows;
    }
    *k = fan_in;
    *n_active = rows;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_compact_producer(const float* bias, const int32_t* active_rows, int32_t n_active,
                                             int32_t out_features, float* bias_compact, int32_t* rows_compact) {
    if ((n_active > 0 && (!active_rows || !bias_compact || !rows_compact))) return CFI_ERR_NULL;
    if (n_active < 0 || out_features < 0 || n_active > out_features) return CFI_ERR_SHAPE;
    std::vector<char> seen((size_t)out_features, 0);
    for (int32_t r = 0; r < n_active; ++r) {
        const int32_t o = active_rows[r];
        if (o < 0 || o >= out_features || seen[o]) return CFI_ERR_INDEX_RANGE;
        seen[o] = 1;
    }
    for (int32_t r = 0; r < n_active; ++r) {
        bias_compact[r] = bias ? bias[active_rows[r]] : 0.0f;
        rows_compact[r] = r;
    }
    return CFI_OK;
}

extern "C" cfi_status_t cfi_compact_consumer(const int32_t* prod_active_rows, int32_t prod_n_active, int32_t prod_out,
                                             const float* prod_const, float* values, int32_t* indices,
                                             const int32_t* active_rows, int32_t n_active, int32_t k, float* bias,
                                             int32_t out_features) {
    if (prod_n_active < 0 || prod_out < 0 || prod_n_active > prod_out || n_active < 0 || k < 0 || out_features < 0 ||
        n_active > out_features)
        return CFI_ERR_SHAPE;
    if ((prod_n_active > 0 && !prod_active_rows) || (n_active > 0 && (!active_rows || !bias)) ||
        ((size_t)n_active * k > 0 && (!values || !indices)))
        return CFI_ERR_NULL;
    if (k > prod_n_active && n_active > 0) return CFI_ERR_SHAPE;
    // rank[c] = compact column of the producer's column c, or -1 if c is ablated.
    std::vector<int32_t> rank((size_t)prod_out, -1);
    for (int32_t r = 0; r < prod_n_active; ++r) {
        const int32_t o = prod_active_rows[r];
        if (o < 0 || o >= prod_out || rank[o] >= 0) return CFI_ERR_INDEX_RANGE;
        rank[o] = r;
    }
    for (int32_t r = 0; r < n_active; ++r) {
        if (active_rows[r] < 0 || active_rows[r] >= out_features) return CFI_ERR_INDEX_RANGE;
        for (int32_t j = 0; j < k; ++j) {
            const int32_t c = indices[(size_t)r * k + j];
            if (c < 0 || c >= prod_out) return CFI_ERR_INDEX_RANGE;
        }
    }
    std::vector<char> used((size_t)prod_n_active, 0);
    for (int32_t r = 0; r < n_active; ++r) {
        float* v = values + (size_t)r * k;
        int32_t* ix = indices + (size_t)r * k;
        std::fill(used.begin(), used.end(), 0);
        for (int32_t j = 0; j < k; ++j)
            if (rank[ix[j]] >= 0) used[rank[ix[j]]] = 1;
        int32_t spare = 0;  // next candidate for an unused compact column
        for (int32_t j = 0; j < k; ++j) {
            const int32_t c = ix[j];
            if (rank[c] >= 0) {
                ix[j] = rank[c];
                continue;
            }
            bias[active_rows[r]] += v[j] * (prod_const ? prod_const[c] : 0.0f);
            v[j] = 0.0f;
            while (spare < prod_n_active && used[spare]) ++spare;
            if (spare >= prod_n_active) return CFI_ERR_SHAPE;  // cannot happen when k <= prod_n_active and columns are distinct
            used[spare] = 1;
            ix[j] = spare;
        }
    }
    return CFI_OK;
}
