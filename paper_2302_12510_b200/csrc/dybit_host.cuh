// Host-side logic: status strings, sizes, Eq. 1 enumeration, container choice.
#pragma once

#include <math.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <vector>

#include "dybit_common.cuh"

namespace dybit {

int sm_count() {
    static std::atomic<int> cached[64];     // filled on first use; every thread computes the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Value of an m-bit magnitude pattern (Eq. 1).  The field is read the way the
// decoder of Section III-B.2 does: find the highest zero bit; the ones above
// it are the unary exponent, the bits below it the fraction.
static float magnitude_value(int m, unsigned c) {
    const unsigned field = (1u << m) - 1u;
    c &= field;
    if (c == 0) return 0.0f;
    if (((c >> (m - 1)) & 1u) == 0) return ldexpf((float)c, -(m - 1));   // start bit 0: pure fraction
    unsigned zeros = (~c) & field;
    if (zeros == 0) return ldexpf(1.0f, m - 1);                          // all ones: largest value
    int p = 31 - __builtin_clz(zeros);       // position of the terminating zero = fraction width k
    int run = m - 1 - p;                     // leading ones, i
    unsigned frac = c & ((1u << p) - 1u);
    return ldexpf((float)((1u << p) + frac), run - 1 - p);               // 2^(i-1) * (1 + x / 2^k)
}

static float code_value(dybit_fmt f, unsigned code) {
    int m = mag_bits(f);
    float v = magnitude_value(m, code);
    if (f.is_signed && ((code >> m) & 1u) && v != 0.0f) v = -v;
    return v;
}

static void fill_table(dybit_fmt f, float *table) {
    for (unsigned c = 0; c < 256u; ++c) table[c] = (c < (1u << f.bits)) ? code_value(f, c) : 0.0f;
}

// Facts about one format's value set, found by enumeration.
struct TableFacts {
    int int_exp;        // smallest e >= 0 with value * 2^e integral for every code
    int max_int;        // max |value * 2^int_exp|
    bool fits_e4m3;     // every value exactly representable in fp8 e4m3
    bool fits_bf16;     // every value exactly representable in bf16
    float max_abs;
};

static bool exact_in_float_format(float v, int sig_bits, int min_exp_of_lsb, float max_finite) {
    if (v == 0.0f) return true;
    float a = fabsf(v);
    if (a > max_finite) return false;
    int e;
    float fr = frexpf(a, &e);                 // a = fr * 2^e, fr in [0.5, 1)
    // significand with sig_bits bits: fr * 2^sig_bits must be an integer
    float scaled = ldexpf(fr, sig_bits);
    if (scaled != floorf(scaled)) {
        return false;
    }
    // lowest set bit must not fall below the format's smallest subnormal step
    int lsb_exp = e - sig_bits;
    float m = scaled;
    while (m != 0.0f && fmodf(m, 2.0f) == 0.0f) { m *= 0.5f; ++lsb_exp; }
    return lsb_exp >= min_exp_of_lsb;
}

static TableFacts enumerate_facts(dybit_fmt f) {
    float tab[256];
    fill_table(f, tab);
    TableFacts t;
    t.int_exp = 0;
    t.max_abs = 0.0f;
    t.fits_e4m3 = true;
    t.fits_bf16 = true;
    for (unsigned c = 0; c < (1u << f.bits); ++c) {
        float v = tab[c];
        t.max_abs = fmaxf(t.max_abs, fabsf(v));
        int e = 0;
        while (e < 30 && ldexpf(v, e) != rintf(ldexpf(v, e))) ++e;
        if (e > t.int_exp) t.int_exp = e;
        // e4m3: 4 significant bits, smallest subnormal 2^-9, largest finite 448
        if (!exact_in_float_format(v, 4, -9, 448.0f)) t.fits_e4m3 = false;
        // bf16: 8 significant bits, fp32 exponent range
        if (!exact_in_float_format(v, 8, -133, 3.38e38f)) t.fits_bf16 = false;
    }
    t.max_int = (int)lrintf(ldexpf(t.max_abs, t.int_exp));
    return t;
}

struct ContainerPlan {
    dybit_container container;
    int exp_a, exp_b;       // power-of-two rescale applied before conversion (int8 only)
    int64_t max_product;    // int8: max |ia * ib|
};

static dybit_status plan_container_uncached(dybit_fmt fa, dybit_fmt fb, ContainerPlan *plan) {
    if (!fmt_ok(fa) || !fmt_ok(fb)) return DYBIT_ERR_INVALID_ARG;
    TableFacts a = enumerate_facts(fa), b = enumerate_facts(fb);
    plan->exp_a = plan->exp_b = 0;
    plan->max_product = 0;
    if (a.max_int <= 127 && b.max_int <= 127) {
        plan->container = DYBIT_CONTAINER_I8;
        plan->exp_a = a.int_exp;
        plan->exp_b = b.int_exp;
        plan->max_product = (int64_t)a.max_int * b.max_int;
    } else if (a.fits_e4m3 && b.fits_e4m3) {
        plan->container = DYBIT_CONTAINER_E4M3;
    } else if (a.fits_bf16 && b.fits_bf16) {
        plan->container = DYBIT_CONTAINER_BF16;
    } else {
        return DYBIT_ERR_UNSUPPORTED;
    }
    return DYBIT_OK;
}

// There are only 14 formats: every pair is enumerated once per process (the enumeration walks up to 256
// codes with several libm calls each, far too slow to repeat on every GEMM call).
static int fmt_index(dybit_fmt f) { return (f.bits - 2) * 2 + (f.is_signed ? 1 : 0); }

static dybit_status plan_container(dybit_fmt fa, dybit_fmt fb, ContainerPlan *plan) {
    if (!fmt_ok(fa) || !fmt_ok(fb)) return DYBIT_ERR_INVALID_ARG;
    struct Entry {
        std::atomic<int> state{0};      // 0 empty, 1 being filled, 2 ready
        ContainerPlan plan;
        dybit_status status;
    };
    static Entry cache[14][14];
    Entry &e = cache[fmt_index(fa)][fmt_index(fb)];
    if (e.state.load(std::memory_order_acquire) != 2) {
        int expected = 0;
        if (e.state.compare_exchange_strong(expected, 1)) {
            e.status = plan_container_uncached(fa, fb, &e.plan);
            e.state.store(2, std::memory_order_release);
        } else {
            // another thread is filling the entry: compute privately rather than wait
            return plan_container_uncached(fa, fb, plan);
        }
    }
    *plan = e.plan;
    return e.status;
}

static inline int container_elem_bytes(dybit_container c) { return c == DYBIT_CONTAINER_BF16 ? 2 : 1; }

}  // namespace dybit

extern "C" {

const char *dybit_status_string(dybit_status st) {
    switch (st) {
        case DYBIT_OK: return "ok";
        case DYBIT_ERR_INVALID_ARG: return "invalid argument";
        case DYBIT_ERR_UNSUPPORTED: return "unsupported configuration";
        case DYBIT_ERR_ALIGNMENT: return "misaligned pointer or stride";
        case DYBIT_ERR_WORKSPACE: return "workspace missing or too small";
        case DYBIT_ERR_CUDA: return "CUDA call failed";
        case DYBIT_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
        case DYBIT_ERR_DEVICE_BOUNDS: return "range check of the debug build failed (access skipped)";
    }
    return "unknown status";
}

size_t dybit_packed_bytes(int64_t n, int bits) {
    if (n < 0 || bits < 2 || bits > 8) return 0;
    int64_t bytes = (n * bits + 7) / 8;
    return (size_t)dybit::round_up(bytes, 16);
}

size_t dybit_row_stride_bytes(int64_t k, int bits) {
    if (k <= 0 || bits < 2 || bits > 8) return 0;
    return (size_t)(dybit::round_up(k, 128) * bits / 8);
}

dybit_status dybit_decode_table(dybit_fmt fmt, float *table) {
    if (!dybit::fmt_ok(fmt) || table == nullptr) return DYBIT_ERR_INVALID_ARG;
    dybit::fill_table(fmt, table);
    return DYBIT_OK;
}

dybit_status dybit_choose_container(dybit_fmt fa, dybit_fmt fb, dybit_container *container,
                                    int *exp_a, int *exp_b) {
    dybit::ContainerPlan plan;
    dybit_status st = dybit::plan_container(fa, fb, &plan);
    if (st != DYBIT_OK) return st;
    if (container) *container = plan.container;
    if (exp_a) *exp_a = plan.exp_a;
    if (exp_b) *exp_b = plan.exp_b;
    return DYBIT_OK;
}

dybit_status dybit_conv2d_out_hw(const dybit_conv_desc *d, int *oh, int *ow) {
    if (d == nullptr) return DYBIT_ERR_INVALID_ARG;
    if (d->n <= 0 || d->h <= 0 || d->w <= 0 || d->c <= 0 || d->k <= 0 || d->r <= 0 || d->s <= 0 ||
        d->stride <= 0 || d->pad < 0 || d->dilation <= 0)
        return DYBIT_ERR_INVALID_ARG;
    int eh = d->h + 2 * d->pad - d->dilation * (d->r - 1) - 1;
    int ew = d->w + 2 * d->pad - d->dilation * (d->s - 1) - 1;
    if (eh < 0 || ew < 0) return DYBIT_ERR_INVALID_ARG;
    if (oh) *oh = eh / d->stride + 1;
    if (ow) *ow = ew / d->stride + 1;
    return DYBIT_OK;
}

// Algorithm 1.  Tables are [layer][a][w] with index 0, 1, 2 <-> 8, 4, 2 bits.
dybit_status dybit_search_bitwidths(int num_layers, const double *lat, const double *rmse, int strategy,
                                    double constraint, int top_k, int *w_bits, int *a_bits) {
    if (num_layers <= 0 || !lat || !rmse || !w_bits || !a_bits || top_k <= 0 || (strategy != 0 && strategy != 1) ||
        !(constraint > 0.0))
        return DYBIT_ERR_INVALID_ARG;
    const int n = num_layers;
    std::vector<int> wl(n, 0), al(n, 0);                       // level index: 0 -> 8 bits, 1 -> 4, 2 -> 2
    auto at = [&](const double *t, int i) { return t[(i * 3 + al[i]) * 3 + wl[i]]; };
    auto total = [&](const double *t) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += at(t, i);
        return s;
    };
    const double *budget = strategy == 0 ? lat : rmse;
    const double base = total(budget);
    auto meets = [&]() {
        const double cur = total(budget);
        return strategy == 0 ? constraint * cur <= base       // Eq. 3
                             : cur > constraint * base;       // Eq. 4 budget exhausted
    };
    // one pass of Degrade_level over `order`; returns {changed, stop}
    auto degrade = [&](const std::vector<int> &order, std::vector<int> &level, bool &changed) {
        for (int i : order) {
            if (level[i] == 2) continue;
            level[i] += 1;
            changed = true;
            if (strategy == 1 && total(rmse) > constraint * base) {
                level[i] -= 1;                                 // the step that breaks the Eq. 4 budget is taken back
                return true;
            }
            if (meets()) return true;
        }
        return false;
    };
    if (!(strategy == 0 && meets())) {
        for (;;) {
            std::vector<int> live;
            for (int i = 0; i < n; ++i)
                if (wl[i] < 2 || al[i] < 2) live.push_back(i);
            if (live.empty()) break;
            std::vector<double> lnow(n), rnow(n);
            for (int i = 0; i < n; ++i) {
                lnow[i] = at(lat, i);
                rnow[i] = at(rmse, i);
            }
            std::vector<int> order = live;
            if (strategy == 0) {
                std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return lnow[a] > lnow[b]; });
                if ((int)order.size() > top_k) order.resize(top_k);
                std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
                    return rnow[a] < rnow[b] || (rnow[a] == rnow[b] && a < b);
                });
            } else {
                std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return rnow[a] < rnow[b]; });
                if ((int)order.size() > top_k) order.resize(top_k);
                std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
                    return lnow[a] > lnow[b] || (lnow[a] == lnow[b] && a < b);
                });
            }
            bool changed = false;
            if (degrade(order, wl, changed)) break;
            if (degrade(order, al, changed)) break;
            if (!changed) break;
        }
    }
    static const int kBits[3] = {8, 4, 2};
    for (int i = 0; i < n; ++i) {
        w_bits[i] = kBits[wl[i]];
        a_bits[i] = kBits[al[i]];
    }
    return DYBIT_OK;
}

uint64_t dybit_launch_count(void) { return dybit::launch_counter().load(std::memory_order_relaxed); }

dybit_status dybit_profile_next_gemm(void *ev_start, void *ev_stop) {
    if ((ev_start == nullptr) != (ev_stop == nullptr)) return DYBIT_ERR_INVALID_ARG;
    dybit::profile_events().start = static_cast<cudaEvent_t>(ev_start);
    dybit::profile_events().stop = static_cast<cudaEvent_t>(ev_stop);
    return DYBIT_OK;
}

dybit_status dybit_profile_next_gemm_clock(unsigned long long *t2) {
    if (!dybit::aligned(t2, 8)) return DYBIT_ERR_ALIGNMENT;
    dybit::profile_events().clock = t2;
    return DYBIT_OK;
}

dybit_status dybit_last_device_status(void *stream, uint32_t *detail) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int word = 0, zero = 0;
    DYBIT_CUDA_TRY(cudaMemcpyFromSymbolAsync(&word, dybit::g_device_status, sizeof(word), 0,
                                             cudaMemcpyDeviceToHost, s));
    DYBIT_CUDA_TRY(cudaStreamSynchronize(s));
    if (word != 0) {
        DYBIT_CUDA_TRY(cudaMemcpyToSymbolAsync(dybit::g_device_status, &zero, sizeof(zero), 0,
                                               cudaMemcpyHostToDevice, s));
        DYBIT_CUDA_TRY(cudaStreamSynchronize(s));
    }
    if (detail) *detail = word;
    if (word == 0) return DYBIT_OK;
    return (word & 1u) ? DYBIT_ERR_DEVICE_TIMEOUT : DYBIT_ERR_DEVICE_BOUNDS;
}

}  // extern "C"
