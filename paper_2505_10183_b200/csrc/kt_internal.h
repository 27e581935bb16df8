// kt_internal.h -- what the translation units of the library share with each other; not part
// of the ABI (that is include/kaitian.h).
#pragma once

#include <cstdint>
#include <vector>

#include "../../include/kaitian.h"

namespace ktd {

// Stores the message kt_last_error() returns to the calling thread; returns `code`.
int fail(int code, const char *fmt, ...);

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Bucket plan (DDP-style bucketing, Section III): tensors in reverse list order, greedy fill up to cap elements, tensors never
// split, every tensor at a multiple of 8 elements, every bucket at a multiple of 64.
struct BucketPlan {
    std::vector<int64_t> offset;      // [T] list order
    std::vector<int32_t> bucket_of;   // [T] list order
    std::vector<int64_t> start;       // [n_buckets]
    std::vector<int> u_lo, u_hi;      // transport-order tensor range of each bucket
    int64_t total = 0;
};

void plan_buckets(const int64_t *numel, int T, int64_t bucket_cap_bytes, BucketPlan *bp);

// Member m of M owns units [floor(m U / M), floor((m + 1) U / M)) of a range of U work units.
void member_units(int64_t U, int member, int M, int64_t *first, int64_t *past);

// KT_OK, or KT_ERR_INVALID with a message when a share is missing or below one.
int check_shares(const int32_t *shares, int K);

}  // namespace ktd

#define KT_CUDA(call)                                                                       \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess)                                                              \
            return ::ktd::fail(KT_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_));       \
    } while (0)
