/*
 * kt_oracle.c -- plain CPU oracle for KAITIAN's hierarchical, load-weighted
 * gradient synchronisation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the hot path computes.  It is written from the paper's description
 * (Section III-A hierarchical communication, Section III-C load-adaptive
 * scheduling) and shares no code, header, table or helper with the CUDA library.
 * Only tests, the smoke check and the bench's CPU-baseline leg may call it.
 *
 * Everything is single threaded and element by element, in a fixed summation
 * order: ascending rank inside a group, ascending group across groups.  Compile
 * with -O2 -ffp-contract=off so that the only fused multiply-adds are the explicit
 * fmaf() calls below.
 *
 * Pins (see tests/test_oracle_*.py): every function in this file is pinned to
 * something other than itself -- exact rational arithmetic, closed forms, a library
 * cast routine, numpy means, brute-force re-derivation.  No function here is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define KTO_OK 0
#define KTO_ERR_INVALID (-1)

/* ------------------------------------------------------------------------- */
/* Section III-C, "Initial Benchmarking" and "Dynamic Data Allocation".         */
/*                                                                           */
/* score_i = time_fastest / time_i (fastest device scores 1.0);               */
/* quota_i = score_i / sum_j score_j * B_global;                               */
/* shares are the quotas rounded to integers such that they still add up to     */
/* B_global.  The paper does not say how the sum is repaired; the               */
/* reading used is the largest-remainder rule (floor every quota, hand the      */
/* missing units to the largest fractional parts, ties to the lower index),    */
/* which equals nearest rounding whenever nearest rounding already sums to B.   */
/* A rank never gets zero samples: a zero share is raised to one, taken from    */
/* the currently largest share (tie: the slowest of them, then higher index).   */
/* ------------------------------------------------------------------------- */
/* The scores alone: score_i = time_fastest / time_i (Section III-C). */
int kto_scores(const double *step_times, int K, double *scores)
{
    if (!step_times || !scores || K < 1)
        return KTO_ERR_INVALID;
    for (int i = 0; i < K; ++i)
        if (!(step_times[i] > 0.0) || !isfinite(step_times[i]))
            return KTO_ERR_INVALID;
    double t_min = step_times[0];
    for (int i = 1; i < K; ++i)
        if (step_times[i] < t_min)
            t_min = step_times[i];
    for (int i = 0; i < K; ++i)
        scores[i] = t_min / step_times[i];
    return KTO_OK;
}

int kto_schedule(const double *step_times, int K, int global_batch, int32_t *shares)
{
    if (!step_times || !shares || K < 1 || global_batch < K)
        return KTO_ERR_INVALID;
    for (int i = 0; i < K; ++i)
        if (!(step_times[i] > 0.0) || !isfinite(step_times[i]))
            return KTO_ERR_INVALID;

    double t_min = step_times[0];
    for (int i = 1; i < K; ++i)
        if (step_times[i] < t_min)
            t_min = step_times[i];

    double *score = (double *)malloc(sizeof(double) * (size_t)K);
    double *frac = (double *)malloc(sizeof(double) * (size_t)K);
    if (!score || !frac) {
        free(score);
        free(frac);
        return KTO_ERR_INVALID;
    }

    double sum = 0.0;
    for (int i = 0; i < K; ++i) {
        score[i] = t_min / step_times[i];
        sum = sum + score[i];
    }

    int64_t given = 0;
    for (int i = 0; i < K; ++i) {
        double q = score[i] / sum * (double)global_batch;
        double f = floor(q);
        shares[i] = (int32_t)f;
        frac[i] = q - f;
        given += shares[i];
    }

    int64_t missing = (int64_t)global_batch - given;
    while (missing > 0) {
        int best = -1;
        for (int i = 0; i < K; ++i)
            if (frac[i] >= 0.0 && (best < 0 || frac[i] > frac[best]))
                best = i;
        if (best < 0) { /* every rank already got one extra unit: start again */
            for (int i = 0; i < K; ++i)
                frac[i] = 0.0;
            continue;
        }
        shares[best] += 1;
        frac[best] = -1.0; /* at most one extra unit per round */
        --missing;
    }
    while (missing < 0) { /* only reachable through rounding of the quotas */
        int big = 0;
        for (int i = 1; i < K; ++i)
            if (shares[i] > shares[big])
                big = i;
        shares[big] -= 1;
        ++missing;
    }

    /* nobody idles: the donor is the largest share; among equal shares the slowest
     * device, among equally slow ones the higher index -- so that a faster device
     * never ends up with less than a slower one */
    for (int i = 0; i < K; ++i) {
        if (shares[i] >= 1)
            continue;
        int big = 0;
        for (int j = 1; j < K; ++j)
            if (shares[j] > shares[big] ||
                (shares[j] == shares[big] && step_times[j] >= step_times[big]))
                big = j;
        shares[big] -= 1;
        shares[i] += 1;
    }

    free(score);
    free(frac);
    return KTO_OK;
}

/* ------------------------------------------------------------------------- */
/* Online adaptation of the scores (Section III-C names it as future work:      */
/* "continuously monitor computation times per batch during training and        */
/* dynamically adjust scores").  The paper gives no rule; the reading used:     */
/*  - a rank's measured step time T_r was spent on b_r samples, so its speed    */
/*    shows in the per-sample time tau_r = T_r / b_r (the initial benchmark of   */
/*    Section III-C gives every device the same amount of data, where time and   */
/*    per-sample time are proportional);                                       */
/*  - tau_r is smoothed by an exponential moving average with factor alpha      */
/*    (the first observation initialises it);                                  */
/*  - every `period` observations the schedule of Section III-C is recomputed   */
/*    from the smoothed per-sample times; the new shares are adopted only if     */
/*    the step time they predict, max_r tau_r * b_r, is below (1 - hysteresis)   */
/*    times the one predicted for the shares in use, so that measurement noise   */
/*    does not make the shares flip back and forth.                            */
/* State is held by the caller: ema[K] (doubles), shares[K], *count.            */
/* Returns 1 if the shares changed, 0 if not, KTO_ERR_INVALID on bad input.      */
/* ------------------------------------------------------------------------- */
int kto_adapt_observe(double *ema, int32_t *shares, int64_t *count, int K, int global_batch,
                      double alpha, int period, double hysteresis, const double *step_times)
{
    if (!ema || !shares || !count || !step_times || K < 1 || period < 1 || !(alpha > 0.0) ||
        !(alpha <= 1.0) || !(hysteresis >= 0.0) || !(hysteresis < 1.0))
        return KTO_ERR_INVALID;
    for (int r = 0; r < K; ++r)
        if (!(step_times[r] > 0.0) || !isfinite(step_times[r]) || shares[r] < 1)
            return KTO_ERR_INVALID;
    for (int r = 0; r < K; ++r) {
        double tau = step_times[r] / (double)shares[r];
        if (*count == 0)
            ema[r] = tau;
        else
            ema[r] = (1.0 - alpha) * ema[r] + alpha * tau;
    }
    *count += 1;
    if (*count % period != 0)
        return 0;
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)K);
    if (!cand)
        return KTO_ERR_INVALID;
    if (kto_schedule(ema, K, global_batch, cand) != KTO_OK) {
        free(cand);
        return KTO_ERR_INVALID;
    }
    double now = 0.0, then = 0.0;
    int differs = 0;
    for (int r = 0; r < K; ++r) {
        double a = ema[r] * (double)shares[r], b = ema[r] * (double)cand[r];
        if (a > now)
            now = a;
        if (b > then)
            then = b;
        if (cand[r] != shares[r])
            differs = 1;
    }
    int adopt = differs && then < (1.0 - hysteresis) * now;
    if (adopt)
        for (int r = 0; r < K; ++r)
            shares[r] = cand[r];
    free(cand);
    return adopt;
}

/* ------------------------------------------------------------------------- */
/* Load-adaptive sampler (Section III-C "Dynamic Data Allocation", Section IV-A  */
/* "DistributedSampler Override": the sampler takes the per-device scores and   */
/* distributes dataset indices accordingly).  With the integer shares b_r of     */
/* the schedule, B = sum b_r and c_r = b_0 + ... + b_{r-1}:                       */
/*  - an epoch has S = floor(D / B) steps when the incomplete last batch is      */
/*    dropped, else S = ceil(D / B), the index list being continued from its     */
/*    own start (position p reads list entry p mod D);                         */
/*  - step s consumes positions [s B, (s+1) B) of the epoch's index list; rank r  */
/*    takes the b_r consecutive positions starting at s B + c_r;                */
/*  - rank r's epoch list is its slices of steps 0..S-1 one after the other:     */
/*      out_r[s b_r + j] = list[(s B + c_r + j) mod D],  0 <= j < b_r.            */
/* list is the epoch's permutation of 0..D-1 (NULL = identity, no shuffling);   */
/* how it is drawn is outside this function.                                   */
/* ------------------------------------------------------------------------- */
int64_t kto_sampler_steps(int64_t dataset_size, int64_t global_batch, int drop_last)
{
    if (dataset_size < 1 || global_batch < 1)
        return -1;
    if (drop_last)
        return dataset_size / global_batch;
    return (dataset_size + global_batch - 1) / global_batch;
}

int kto_sampler_indices(const int64_t *list, int64_t dataset_size, const int32_t *shares, int K,
                        int drop_last, int64_t *const *out)
{
    if (!shares || !out || K < 1 || dataset_size < 1)
        return KTO_ERR_INVALID;
    int64_t B = 0;
    for (int r = 0; r < K; ++r) {
        if (shares[r] < 1)
            return KTO_ERR_INVALID;
        B += shares[r];
    }
    const int64_t S = kto_sampler_steps(dataset_size, B, drop_last);
    int64_t c = 0; /* c_r */
    for (int r = 0; r < K; ++r) {
        for (int64_t s = 0; s < S; ++s)
            for (int64_t j = 0; j < shares[r]; ++j) {
                int64_t p = (s * B + c + j) % dataset_size;
                out[r][s * shares[r] + j] = list ? list[p] : p;
            }
        c += shares[r];
    }
    return KTO_OK;
}

/* ------------------------------------------------------------------------- */
/* Dispatch decision (Section III-B, steps 1-3): a collective whose              */
/* participating ranks all sit in one group of like accelerators is homogeneous  */
/* (returns 0: handled inside the group); one whose participants span groups is  */
/* heterogeneous (returns 1: needs the relay through host memory).              */
/* Returns KTO_ERR_INVALID for an empty list, a rank out of range or a repeat.    */
/* ------------------------------------------------------------------------- */
int kto_route(const int32_t *group_of, int K, const int32_t *participants, int n)
{
    if (!group_of || !participants || K < 1 || n < 1)
        return KTO_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        if (participants[i] < 0 || participants[i] >= K)
            return KTO_ERR_INVALID;
        for (int j = 0; j < i; ++j)
            if (participants[j] == participants[i])
                return KTO_ERR_INVALID;
    }
    for (int i = 1; i < n; ++i)
        if (group_of[participants[i]] != group_of[participants[0]])
            return 1;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Weights of the two-level mean (Section III-A groups, Section III-C shares).  */
/* B_g = sum of the shares of group g, B = sum of all shares.                  */
/* a_r = b_r / B_g  (weight of rank r inside its group),                       */
/* W_g = B_g / B    (weight of group g in the global result),                  */
/* w_r = b_r / B    (weight of rank r in the one-level, "flat" mean).          */
/* Each quotient is formed in double and rounded once to float.               */
/* ------------------------------------------------------------------------- */
int kto_coefficients(const int32_t *group_of, const int32_t *shares, int K, int G,
                     float *a, float *W, float *w_flat)
{
    if (!group_of || !shares || K < 1 || G < 1 || G > K)
        return KTO_ERR_INVALID;
    int64_t *Bg = (int64_t *)calloc((size_t)G, sizeof(int64_t));
    if (!Bg)
        return KTO_ERR_INVALID;
    int64_t B = 0;
    for (int r = 0; r < K; ++r) {
        if (group_of[r] < 0 || group_of[r] >= G || shares[r] < 1) {
            free(Bg);
            return KTO_ERR_INVALID;
        }
        Bg[group_of[r]] += shares[r];
        B += shares[r];
    }
    for (int g = 0; g < G; ++g)
        if (Bg[g] == 0) { /* empty group */
            free(Bg);
            return KTO_ERR_INVALID;
        }
    for (int r = 0; r < K; ++r) {
        if (a)
            a[r] = (float)((double)shares[r] / (double)Bg[group_of[r]]);
        if (w_flat)
            w_flat[r] = (float)((double)shares[r] / (double)B);
    }
    if (W)
        for (int g = 0; g < G; ++g)
            W[g] = (float)((double)Bg[g] / (double)B);
    free(Bg);
    return KTO_OK;
}

/* ------------------------------------------------------------------------- */
/* Bucket plan (gradient bucketing of the data-parallel reducer, Section III).  */
/* The paper only says gradients are all-reduced by DDP; the reading used:     */
/*  - tensors are visited in reverse list order (gradients of the last layers   */
/*    become ready first);                                                     */
/*  - a bucket holds at most cap = bucket_cap_bytes / 4 transport elements      */
/*    (the transport is fp32 whatever the gradient dtype); a tensor is never    */
/*    split and a tensor larger than the cap gets a bucket of its own;          */
/*  - inside the transport every tensor starts at a multiple of 8 elements and  */
/*    every bucket at a multiple of 64 elements; the gaps are zero padding.     */
/* Outputs: tensor_offset[t] (element offset in the transport), bucket_of[t],  */
/* bucket_start[b], bucket_numel[b] (start of bucket b to start of b+1, the     */
/* last one up to transport_numel), n_buckets, transport_numel (multiple of 64).*/
/* bucket_start/bucket_numel must have room for T entries.                     */
/* ------------------------------------------------------------------------- */
static int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

int kto_bucket_plan(const int64_t *numel, int T, int64_t bucket_cap_bytes,
                    int64_t *tensor_offset, int32_t *bucket_of, int64_t *bucket_start,
                    int64_t *bucket_numel, int32_t *n_buckets, int64_t *transport_numel)
{
    if (!numel || T < 1 || bucket_cap_bytes < 4)
        return KTO_ERR_INVALID;
    for (int t = 0; t < T; ++t)
        if (numel[t] < 0)
            return KTO_ERR_INVALID;
    const int64_t cap = bucket_cap_bytes / 4;

    int32_t nb = 0;
    int64_t cursor = 0;     /* next free transport element */
    int64_t start = 0;      /* start of the open bucket */
    int open_has_tensor = 0;
    for (int t = T - 1; t >= 0; --t) {
        int64_t off = round_up(cursor, 8);
        if (open_has_tensor && (off - start) + numel[t] > cap) {
            /* close the bucket, open the next one on a 64-element boundary */
            ++nb;
            start = round_up(cursor, 64);
            off = start;
            open_has_tensor = 0;
        }
        if (!open_has_tensor)
            bucket_start[nb] = start;
        tensor_offset[t] = off;
        bucket_of[t] = nb;
        cursor = off + numel[t];
        open_has_tensor = 1;
    }
    ++nb;
    const int64_t total = round_up(cursor, 64);
    for (int b = 0; b < nb; ++b)
        bucket_numel[b] = (b + 1 < nb ? bucket_start[b + 1] : total) - bucket_start[b];
    *n_buckets = nb;
    *transport_numel = total;
    return KTO_OK;
}

/* ------------------------------------------------------------------------- */
/* One rank per device: which part of a bucket each member of a group reduces.  */
/* The paper hands the intra-group collective to the vendor library (Section    */
/* III-A, first bullet) and says nothing of how the work is split among the     */
/* devices of a group.  Reading taken: the range of a collective (one bucket,   */
/* or the whole transport when bucket < 0) is cut into work units of `unit`     */
/* elements that never cross a tensor: tensor t, which occupies the transport   */
/* from its offset up to the next tensor's offset (padding included), holds     */
/* ceil(extent / unit) of them, the last one possibly short.  The units of the  */
/* range are numbered in transport order; with U units and M members, member m  */
/* owns units floor(m U / M) ... floor((m+1) U / M) - 1, a contiguous element    */
/* range [lo_out[m], lo_out[m] + n_out[m]).  A member that owns no unit gets      */
/* n_out = 0 (lo_out then marks where its empty range sits).                     */
/* ------------------------------------------------------------------------- */
int kto_shard_ranges(const int64_t *numel, int T, int64_t bucket_cap_bytes, int64_t unit,
                     int bucket, int n_members, int64_t *lo_out, int64_t *n_out)
{
    if (!numel || T < 1 || unit < 1 || n_members < 1 || !lo_out || !n_out)
        return KTO_ERR_INVALID;
    int64_t *offset = (int64_t *)malloc(sizeof(int64_t) * (size_t)T);
    int32_t *bucket_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    int64_t *bstart = (int64_t *)malloc(sizeof(int64_t) * (size_t)T);
    int64_t *bnumel = (int64_t *)malloc(sizeof(int64_t) * (size_t)T);
    int32_t nb = 0;
    int64_t total = 0;
    int rc = kto_bucket_plan(numel, T, bucket_cap_bytes, offset, bucket_of, bstart, bnumel, &nb, &total);
    if (rc == KTO_OK && (bucket < -1 || bucket >= nb))
        rc = KTO_ERR_INVALID;
    if (rc != KTO_OK) {
        free(offset); free(bucket_of); free(bstart); free(bnumel);
        return rc;
    }
    const int64_t range_hi = bucket < 0 ? total : bstart[bucket] + bnumel[bucket];

    /* pass 1 counts the units of the range, pass 2 hands them out */
    int64_t U = 0;
    for (int pass = 0; pass < 2; ++pass) {
        int64_t index = 0;
        if (pass == 1) {
            for (int m = 0; m < n_members; ++m) {
                n_out[m] = 0;
                /* an empty share sits where its first unit would be */
                lo_out[m] = range_hi;
            }
        }
        for (int t = T - 1; t >= 0; --t) {              /* transport order */
            if (bucket >= 0 && bucket_of[t] != bucket)
                continue;
            const int64_t end = t > 0 ? offset[t - 1] : total;   /* the next tensor in the transport is t-1 */
            const int64_t extent = end - offset[t];
            for (int64_t at = 0; at < extent; at += unit, ++index) {
                if (pass == 0)
                    continue;
                const int64_t len = extent - at < unit ? extent - at : unit;
                for (int m = 0; m < n_members; ++m) {
                    const int64_t first = (int64_t)m * U / n_members;
                    const int64_t past = (int64_t)(m + 1) * U / n_members;
                    if (index >= first && index < past) {
                        if (n_out[m] == 0)
                            lo_out[m] = offset[t] + at;
                        n_out[m] += len;
                    }
                }
            }
        }
        if (pass == 0)
            U = index;
    }
    /* empty shares: place them at the start of the next member's range */
    for (int m = n_members - 1; m >= 0; --m)
        if (n_out[m] == 0)
            lo_out[m] = m + 1 < n_members ? lo_out[m + 1] : range_hi;
    free(offset); free(bucket_of); free(bstart); free(bnumel);
    return KTO_OK;
}

/* ------------------------------------------------------------------------- */
/* Casts.  bf16 is the upper half of an IEEE-754 binary32 pattern.             */
/* Widening is exact.  Narrowing rounds to nearest, ties to even, on the bit    */
/* pattern; a NaN keeps its sign and upper payload and is made quiet.           */
/* ------------------------------------------------------------------------- */
static float bits_to_f32(uint32_t u)
{
    float f;
    memcpy(&f, &u, 4);
    return f;
}
static uint32_t f32_to_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}

float kto_bf16_to_f32_one(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

uint16_t kto_f32_to_bf16_one(float f)
{
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) /* NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

void kto_bf16_to_f32(const uint16_t *in, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = kto_bf16_to_f32_one(in[i]);
}

void kto_f32_to_bf16(const float *in, uint16_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = kto_f32_to_bf16_one(in[i]);
}

/* dtype codes used by the element accessors below */
#define KTO_F32 0
#define KTO_BF16 1

static float load_as_f32(const void *base, int dtype, int64_t i)
{
    if (dtype == KTO_BF16)
        return kto_bf16_to_f32_one(((const uint16_t *)base)[i]);
    return ((const float *)base)[i];
}

/* ------------------------------------------------------------------------- */
/* Standalone pack: the flat bucket copy of one rank's gradient list.          */
/* flat[tensor_offset[t] + j] = x^(t)[j] (bit copy, same dtype), padding = 0.   */
/* elem_size is 4 (fp32) or 2 (bf16).                                          */
/* ------------------------------------------------------------------------- */
void kto_pack(const void *const *tensors, const int64_t *numel, const int64_t *tensor_offset,
              int T, int elem_size, int64_t transport_numel, void *flat)
{
    memset(flat, 0, (size_t)transport_numel * (size_t)elem_size);
    for (int t = 0; t < T; ++t) {
        const unsigned char *src = (const unsigned char *)tensors[t];
        unsigned char *dst = (unsigned char *)flat + tensor_offset[t] * elem_size;
        for (int64_t j = 0; j < numel[t] * elem_size; ++j)
            dst[j] = src[j];
    }
}

/* ------------------------------------------------------------------------- */
/* Hierarchical broadcast (model synchronisation; Section III routes Broadcast  */
/* through the same hierarchy as AllReduce).  What it must produce is plain:    */
/* every rank ends up with the root's tensors, bit for bit.  The flat buffer    */
/* that crosses the host is the pack of the root's list; a receiving group      */
/* copies each tensor out of it again:                                         */
/*   out^(t)[j] = flat[tensor_offset[t] + j]  (bit copy, same dtype).           */
/* ------------------------------------------------------------------------- */
void kto_unpack_copy(const void *flat, const int64_t *numel, const int64_t *tensor_offset,
                     int T, int elem_size, void *const *out)
{
    for (int t = 0; t < T; ++t) {
        const unsigned char *src = (const unsigned char *)flat + tensor_offset[t] * elem_size;
        unsigned char *dst = (unsigned char *)out[t];
        for (int64_t j = 0; j < numel[t] * elem_size; ++j)
            dst[j] = src[j];
    }
}

/* ------------------------------------------------------------------------- */
/* Intra-group reduce (Section III-A, first bullet: the collective among the    */
/* homogeneous devices of one group), with the in-group batch-share weights:   */
/*   P_g[i] = sum over the ranks r of group g, ascending r, of a_r * x_r[i].     */
/* The first term is one rounded product, every later term one fmaf.           */
/* grads is rank-major: grads[r*T + t] is tensor t of rank r.  transport[g]     */
/* receives group g's fp32 partial at the bucket offsets; padding is zero.      */
/* ------------------------------------------------------------------------- */
void kto_intra_reduce(const void *const *grads, int in_dtype, const int64_t *numel,
                      const int64_t *tensor_offset, int T, int64_t transport_numel,
                      const int32_t *group_of, const float *a, int K, int G,
                      float *const *transport)
{
    for (int g = 0; g < G; ++g) {
        float *P = transport[g];
        for (int64_t i = 0; i < transport_numel; ++i)
            P[i] = 0.0f;
        for (int t = 0; t < T; ++t) {
            for (int64_t j = 0; j < numel[t]; ++j) {
                float acc = 0.0f;
                int first = 1;
                for (int r = 0; r < K; ++r) {
                    if (group_of[r] != g)
                        continue;
                    float x = load_as_f32(grads[(size_t)r * (size_t)T + (size_t)t], in_dtype, j);
                    if (first) {
                        acc = a[r] * x;
                        first = 0;
                    } else {
                        acc = fmaf(a[r], x, acc);
                    }
                }
                P[tensor_offset[t] + j] = acc;
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Inter-group combine (Section III-A, second bullet: the reduction between     */
/* groups, done on host-relayed fp32 partials), with the group weights:        */
/*   S[i] = sum over groups g, ascending g, of W_g * P_g[i].                     */
/* ------------------------------------------------------------------------- */
void kto_combine(const float *const *partials, const float *W, int G, int64_t n, float *S)
{
    for (int64_t i = 0; i < n; ++i) {
        float acc = W[0] * partials[0][i];
        for (int g = 1; g < G; ++g)
            acc = fmaf(W[g], partials[g][i], acc);
        S[i] = acc;
    }
}

/* ------------------------------------------------------------------------- */
/* Unpack + scale: the copy from the reduced bucket back into per-parameter     */
/* gradients.  out^(t)[j] = cast(scale * S[tensor_offset[t] + j]); the product  */
/* is one rounded fp32 multiply; cast is the identity for fp32 and the           */
/* round-to-nearest-even narrowing above for bf16.  Padding is ignored.         */
/* ------------------------------------------------------------------------- */
void kto_unpack_scale(const float *S, const int64_t *numel, const int64_t *tensor_offset,
                      int T, float scale, int out_dtype, void *const *out)
{
    for (int t = 0; t < T; ++t) {
        for (int64_t j = 0; j < numel[t]; ++j) {
            float y = S[tensor_offset[t] + j] * scale;
            if (out_dtype == KTO_BF16)
                ((uint16_t *)out[t])[j] = kto_f32_to_bf16_one(y);
            else
                ((float *)out[t])[j] = y;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* One-level ("flat") weighted mean over all ranks, for the invariant           */
/* "hierarchical equals flat within tolerance":                                */
/*   F[i] = sum_r w_r * x_r[i], ascending r, in fp32 (fmaf chain) and, with the  */
/* exact rational weights b_r / B, in fp64.  x is one flat buffer per rank.      */
/* ------------------------------------------------------------------------- */
void kto_flat_reduce_f32(const void *const *x, int in_dtype, const float *w_flat, int K,
                         int64_t n, float *F)
{
    for (int64_t i = 0; i < n; ++i) {
        float acc = w_flat[0] * load_as_f32(x[0], in_dtype, i);
        for (int r = 1; r < K; ++r)
            acc = fmaf(w_flat[r], load_as_f32(x[r], in_dtype, i), acc);
        F[i] = acc;
    }
}

void kto_flat_reduce_f64(const void *const *x, int in_dtype, const int32_t *shares, int K,
                         int64_t n, double *F, double *absF)
{
    int64_t B = 0;
    for (int r = 0; r < K; ++r)
        B += shares[r];
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0, mag = 0.0;
        for (int r = 0; r < K; ++r) {
            double v = (double)load_as_f32(x[r], in_dtype, i);
            acc += (double)shares[r] * v;
            mag += (double)shares[r] * fabs(v);
        }
        F[i] = acc / (double)B;
        if (absF)
            absF[i] = mag / (double)B; /* sum_r w_r |x_r[i]|: forward-error scale */
    }
}
