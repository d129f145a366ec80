// Host-side cut of the look-up-table kernel's task space into one contiguous share per CTA (plain C++, no CUDA).
//
// A launch covers n linears; linear k contributes nslices[k] slices of nrg[k] tasks each (a task: 16 rows x 512
// columns), slices and linears laid end to end.  A CTA that visits a slice pays a fixed set-up (tables, drain,
// hand-over) worth `segment_cost` tasks, so the cost of a share is its tasks plus segment_cost per slice it touches.
// The cut minimises the most expensive share: for a given bound every CTA in turn takes as many tasks as fit under
// it, and the smallest bound for which `grid` CTAs cover everything is found by bisection.
#pragma once

namespace bpdq {

constexpr int kPartitionMinSegment = 8;   // a share is closed rather than opened into a slice for fewer tasks than this

// Fills t_begin[0..grid] (CTA b takes the tasks [t_begin[b], t_begin[b+1])) and returns the cost of the dearest share.
// grid >= 1; nrg[k], nslices[k] >= 1; the total number of tasks must fit an int.
inline double cut_task_space(const int* nrg, const int* nslices, int n, int grid, int segment_cost, int* t_begin) {
    long long total = 0;
    for (int k = 0; k < n; ++k) total += (long long)nslices[k] * nrg[k];
    // fills t_begin for the bound; true when `grid` shares cover the task space
    auto sweep = [&](const double bound, double* dearest) {
        long long t = 0, lin_begin = 0;
        int k = 0, b = 0;
        double worst = 0.0;
        t_begin[0] = 0;
        while (t < total && b < grid) {
            double budget = bound;
            const long long start = t;
            while (t < total) {
                while (k + 1 < n && t >= lin_begin + (long long)nslices[k] * nrg[k]) { lin_begin += (long long)nslices[k] * nrg[k]; ++k; }
                const long long in_slice = nrg[k] - (t - lin_begin) % nrg[k];      // tasks left in the current slice
                const double room = budget - segment_cost;
                if (t > start && room < (double)(in_slice < kPartitionMinSegment ? in_slice : kPartitionMinSegment)) break;
                long long take = room >= 1.0 ? (long long)room : 1;
                if (take > in_slice) take = in_slice;
                t += take;
                budget -= (double)(segment_cost + take);
                if (take < in_slice) break;
            }
            if (bound - budget > worst) worst = bound - budget;
            t_begin[++b] = (int)t;
        }
        const bool covered = t >= total;
        for (int c = b + 1; c <= grid; ++c) t_begin[c] = (int)total;
        if (dearest) *dearest = worst;
        return covered;
    };
    double lo = (double)total / grid, hi = 2.0 * (double)total / grid + 16.0 * segment_cost + 16.0;
    while (!sweep(hi, nullptr)) hi *= 2.0;            // terminates: a bound above the whole cost covers everything
    for (int it = 0; it < 24 && hi - lo > 0.5; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (sweep(mid, nullptr)) hi = mid; else lo = mid;
    }
    double dearest = 0.0;
    sweep(hi, &dearest);
    return dearest;
}

}  // namespace bpdq
