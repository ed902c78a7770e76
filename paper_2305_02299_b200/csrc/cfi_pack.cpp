// Host side of the library that needs no CUDA: cfi_pack and the status names.
#include "cfi.h"

#include <cstddef>

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
