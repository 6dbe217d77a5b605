// Host partitioner: tensor descriptors -> flat block table.
//
// Paper, Algorithm 3 ("Partition for Transformers"): embedding/output tensors
// are cut per token row, query/key per head, value / attention projection /
// MLP per output neuron, everything else is one block (which is also
// Algorithm 2, "Partition for non-Transformers").  With [out, in] row-major
// weights every block is a contiguous run, so a tensor is n_blocks runs of one
// length and the table needs one row per tensor.
#include "adammini_internal.h"

#include <cstring>
#include <limits>
#include <new>

namespace {

// Block length of one tensor, or 0 if the descriptor is inconsistent.
int64_t block_length(const am_tensor_desc &d, int64_t numel) {
    switch (d.kind) {
    case AM_WHOLE:
        return numel;
    case AM_ROWS:
    case AM_TOKENS:
        return d.cols;
    case AM_HEADS:
        if (d.n_heads <= 0 || d.rows % d.n_heads != 0) return 0;
        return (d.rows / d.n_heads) * d.cols;
    case AM_FIXED:
        if (d.fixed_block_len <= 0 || numel % d.fixed_block_len != 0) return 0;
        return d.fixed_block_len;
    case AM_PART:               // the local part of one longer block is this tensor's single "block"
        if (d.rows != 1 || d.fixed_block_len < numel) return 0;
        return numel;
    default:
        return 0;
    }
}

bool contains(const char *hay, const char *needle) { return std::strstr(hay, needle) != nullptr; }

}  // namespace

extern "C" {

int adammini_partition_build(const am_tensor_desc *descs, int32_t n_tensors, am_partition **out) {
    if (!out) return AM_ERR_INVALID_ARGUMENT;
    *out = nullptr;
    if (n_tensors < 0 || (n_tensors > 0 && !descs)) return AM_ERR_INVALID_ARGUMENT;
    am_partition *part = new (std::nothrow) am_partition();
    if (!part) return AM_ERR_ALLOC;
    try {
        part->rows.reserve(n_tensors);
        int64_t v_offset = 0, total_elems = 0;
        for (int32_t i = 0; i < n_tensors; ++i) {
            const am_tensor_desc &d = descs[i];
            if (d.rows <= 0 || d.cols <= 0 || d.rows > std::numeric_limits<int64_t>::max() / d.cols) {
                delete part;
                return AM_ERR_SHAPE;
            }
            if ((d.grad_dtype != AM_F32 && d.grad_dtype != AM_BF16) || d.kind < AM_WHOLE || d.kind > AM_PART) {
                delete part;
                return AM_ERR_INVALID_ARGUMENT;
            }
            const int64_t numel = d.rows * d.cols;
            const int64_t L = block_length(d, numel);
            if (L <= 0) {
                delete part;
                return AM_ERR_SHAPE;
            }
            if (numel > std::numeric_limits<int64_t>::max() - total_elems) {     // the table's totals stay in int64
                delete part;
                return AM_ERR_TOO_LARGE;
            }
            total_elems += numel;               // bounds the block count too: n_blocks <= numel
            am_table_row r;
            r.numel = numel;
            r.block_len = L;
            r.n_blocks = numel / L;
            r.v_offset = v_offset;
            r.kind = d.kind;
            r.grad_dtype = d.grad_dtype;
            r.wd = d.apply_weight_decay ? 1 : 0;
            r.pad = 0;
            r.mean_len = d.kind == AM_PART ? d.fixed_block_len : L;
            part->rows.push_back(r);
            v_offset += r.n_blocks;
        }
        part->total_blocks = v_offset;
    } catch (...) {
        delete part;
        return AM_ERR_ALLOC;
    }
    *out = part;
    return AM_OK;
}

int32_t adammini_partition_num_tensors(const am_partition *part) {
    return part ? static_cast<int32_t>(part->rows.size()) : 0;
}

int adammini_partition_export(const am_partition *part, am_table_row *rows, int64_t *total_blocks) {
    if (!part) return AM_ERR_INVALID_ARGUMENT;
    if (rows && !part->rows.empty())
        std::memcpy(rows, part->rows.data(), part->rows.size() * sizeof(am_table_row));
    if (total_blocks) *total_blocks = part->total_blocks;
    return AM_OK;
}

void adammini_partition_free(am_partition *part) { delete part; }

int32_t adammini_kind_from_name(const char *name) {
    if (!name) return AM_WHOLE;
    if (contains(name, "embed") || contains(name, "output")) return AM_TOKENS;
    if (contains(name, "query") || contains(name, "key")) return AM_HEADS;
    if (contains(name, "value") || contains(name, "attn.proj") || contains(name, "mlp")) return AM_ROWS;
    return AM_WHOLE;
}

const char *adammini_status_string(int status) {
    switch (status) {
    case AM_OK: return "ok";
    case AM_ERR_INVALID_ARGUMENT: return "invalid argument";
    case AM_ERR_SHAPE: return "shape does not divide into blocks";
    case AM_ERR_MISALIGNED: return "device pointer not 16-byte aligned";
    case AM_ERR_CUDA: return "CUDA error";
    case AM_ERR_TIMEOUT: return "device-side bounded wait timed out";
    case AM_ERR_ALLOC: return "allocation failed";
    case AM_ERR_TOO_LARGE: return "size exceeds the entry point's limit";
    default: return "unknown status";
    }
}

}  // extern "C"
