// Host-side check of FastDiv (the multiply-and-shift division the persistent kernels use to turn
// a work item's index into batch, head and tile): every divisor up to 4096 and a spread of larger
// ones, against the C++ operators, on dividends around every multiple boundary and at the top of
// the supported range.  Built and run by tests/test_host_logic.py; needs no GPU.
#include <cstdio>
#include <cstdint>
#include <initializer_list>
#include "../../paper_2410_16663_b200/csrc/prefill_simple.cuh"

static long long g_checked = 0;

static bool check(const fa::FastDiv& f, int d, int n) {
    int q, r;
    f.divmod(n, q, r);
    ++g_checked;
    if (q != n / d || r != n % d || f.div(n) != n / d) {
        std::printf("MISMATCH d=%d n=%d: got q=%d r=%d, want q=%d r=%d\n", d, n, q, r, n / d, n % d);
        return false;
    }
    return true;
}

int main() {
    const int kMax = 0x7fffffff;
    bool ok = true;
    auto run = [&](int d) {
        fa::FastDiv f;
        f.set(d);
        const long long first = 3ll * d + 3 < 20000 ? 3ll * d + 3 : 20000;
        for (long long n = 0; n < first && n <= kMax && ok; ++n) ok = check(f, d, (int)n);
        // around multiples of d spread over the whole range, and the very top
        for (int k = 1; k <= 64 && ok; ++k) {
            const long long m = (long long)(kMax / d) * k / 64 * d;
            for (long long n = m - 2; n <= m + 2 && ok; ++n)
                if (n >= 0 && n <= kMax) ok = check(f, d, (int)n);
        }
        for (int n = kMax - 3; ok && n < kMax; ++n) ok = check(f, d, n);
        if (ok) ok = check(f, d, kMax);
    };
    for (int d = 1; d <= 4096 && ok; ++d) run(d);
    for (int d : {4097, 5000, 65535, 65536, 65537, 1000003, 16777216, 16777217, 1 << 30, kMax - 1, kMax})
        if (ok) run(d);
    std::printf("%s %lld checks\n", ok ? "OK" : "FAILED", g_checked);
    return ok ? 0 : 1;
}
