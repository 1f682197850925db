// Host-logic check of csrc/mxfp8_host.h (no GPU is touched): a value per device, filled once per device, with the
// device index given explicitly; tensor maps keyed by their arguments; division by a precomputed multiplier.
#include <cstdio>
#include <cstring>

#include "mxfp8_host.h"

struct FakeMap { unsigned char bytes[128]; };

int main()
{
    using namespace mxfp8;
    int fails = 0;
    auto check = [&](bool ok, const char* what) { if (!ok) { std::printf("FAIL: %s\n", what); ++fails; } };

    // ---- one value per device
    PerDeviceCache<int*> cache;
    int words[3] = {0, 0, 0};
    int fills[3] = {0, 0, 0};
    auto fill = [&](int dev, int*& out) { ++fills[dev]; out = &words[dev]; return true; };
    int* got = nullptr;
    check(cache.get(got, fill, 0) && got == &words[0], "device 0 gets its own word");
    check(cache.get(got, fill, 1) && got == &words[1], "device 1 gets its own word, not device 0's");
    check(cache.get(got, fill, 0) && got == &words[0], "device 0 again");
    check(cache.get(got, fill, 2) && got == &words[2], "device 2");
    check(cache.get(got, fill, 1) && got == &words[1], "device 1 again");
    check(fills[0] == 1 && fills[1] == 1 && fills[2] == 1, "each device looked up exactly once");
    check(!cache.get(got, fill, 64) && !cache.get(got, fill, 1000), "device index out of range is refused");

    // a failed lookup is not remembered
    PerDeviceCache<int> flaky;
    int calls = 0, v = 0;
    auto fail_once = [&](int, int& out) { out = 148; return ++calls > 1; };
    check(!flaky.get(v, fail_once, 5), "first lookup fails");
    check(flaky.get(v, fail_once, 5) && v == 148, "second lookup succeeds");
    check(flaky.get(v, fail_once, 5) && calls == 2, "then it is cached");

    // ---- tensor maps keyed by every encode argument
    TensorMapCache<FakeMap> maps;
    int encodes = 0;
    auto encode = [&](FakeMap* m) { std::memset(m, ++encodes, sizeof(*m)); return true; };
    const uint64_t d1[2] = {4096, 8192}, s1[1] = {4096};
    const uint32_t b1[2] = {128, 128};
    char buf_a[16], buf_b[16];
    FakeMap m{};
    check(maps.get(tensor_map_key(buf_a, 0, 2, d1, s1, b1, 3, 2), &m, encode) && m.bytes[0] == 1, "miss encodes");
    check(maps.get(tensor_map_key(buf_a, 0, 2, d1, s1, b1, 3, 2), &m, encode) && m.bytes[0] == 1 && encodes == 1, "same arguments hit");
    check(maps.get(tensor_map_key(buf_b, 0, 2, d1, s1, b1, 3, 2), &m, encode) && m.bytes[0] == 2, "another address misses");
    const uint32_t b2[2] = {128, 64};
    check(maps.get(tensor_map_key(buf_a, 0, 2, d1, s1, b2, 3, 2), &m, encode) && m.bytes[0] == 3, "another box misses");
    const uint64_t d2[2] = {4096, 4096};
    check(maps.get(tensor_map_key(buf_a, 0, 2, d2, s1, b1, 3, 2), &m, encode) && m.bytes[0] == 4, "another extent misses");
    check(maps.get(tensor_map_key(buf_a, 0, 2, d1, s1, b1, 3, 2), &m, encode) && m.bytes[0] == 1 && encodes == 4, "the first one is still there");
    auto refuse = [&](FakeMap*) { return false; };
    check(!maps.get(tensor_map_key(buf_a, 7, 2, d1, s1, b1, 3, 2), &m, refuse), "a failed encode is reported");
    check(maps.get(tensor_map_key(buf_a, 7, 2, d1, s1, b1, 3, 2), &m, encode) && encodes == 5, "and not cached");

    // ---- division by multiplication: every divisor a tile grid can have against tile indices around its multiples,
    // around powers of two and at the top of the range
    {
        long bad = 0;
        auto one = [&](uint32_t n, uint32_t d) {
            int q = -1, r = -1;
            divmod(n, d, div_magic(d), q, r);
            if ((uint32_t)q != n / d || (uint32_t)r != n % d) ++bad;
        };
        for (uint32_t d = 1; d <= 70000; d += (d < 3000 ? 1 : 37)) {
            for (uint32_t k = 0; k < 40; ++k) {
                const uint64_t m = (uint64_t)d * (k * 53ull + (k > 30 ? 1000003ull * k : 0ull));
                for (int off = -2; off <= 2; ++off) {
                    const int64_t n = (int64_t)m + off;
                    if (n >= 0 && n < 0x7FFFFFFFll) one((uint32_t)n, d);
                }
            }
            for (int sh = 0; sh < 31; ++sh) { one((1u << sh) - 1u, d); one(1u << sh, d); one((1u << sh) + 1u, d); }
            one(0x7FFEFFFFu, d); one(0x7FFFFFFEu, d);
        }
        check(bad == 0, "quotient and remainder by multiplication equal the division");
    }

    std::printf(fails ? "%d checks failed\n" : "all checks passed\n", fails);
    return fails ? 1 : 0;
}
