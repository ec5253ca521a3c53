"""The range arithmetic behind A2SGD_DEBUG_CHECKS, compiled for the host and exercised without a
GPU: the same header the checked kernels include decides whether an access lies inside the live
elements of one row of a buffer."""
import os
import subprocess
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER_DIR = os.path.join(ROOT, "paper_2006_07405_b200", "csrc")

PROGRAM = textwrap.dedent(r"""
    #include <cstdio>
    #include <cstdlib>
    #include "a2sgd_debug_check.h"
    using namespace a2sgd_check;
    static int failures = 0;
    #define EXPECT(cond) do { if (!(cond)) { std::printf("FAILED line %d: %s\n", __LINE__, #cond); ++failures; } } while (0)
    int main()
    {
        // 3 rows of 10 live floats, 16 floats apart, starting at address 1000
        const DebugRange r{1000, 64, 40, 3};
        EXPECT(debug_range_contains(r, 1000, 4));            // first element
        EXPECT(debug_range_contains(r, 1036, 4));            // last element of row 0
        EXPECT(!debug_range_contains(r, 1040, 4));           // padding between rows
        EXPECT(!debug_range_contains(r, 1032, 16));          // vector straddling the row end
        EXPECT(debug_range_contains(r, 1008, 32));           // 256-bit vector inside row 0
        EXPECT(debug_range_contains(r, 1064, 4));            // first element of row 1
        EXPECT(debug_range_contains(r, 1000 + 2 * 64 + 36, 4)); // last element of the last row
        EXPECT(!debug_range_contains(r, 1000 + 3 * 64, 4));  // a row that does not exist
        EXPECT(!debug_range_contains(r, 996, 4));            // before the buffer
        EXPECT(!debug_range_contains(r, 998, 4));            // straddling the start
        EXPECT(!debug_range_contains(r, 1036, 0xffffffffffffffffull)); // length that wraps around
        // one shared row (stride 0): anything past its live bytes is outside
        const DebugRange w{5000, 0, 400, 1};
        EXPECT(debug_range_contains(w, 5000, 400));
        EXPECT(debug_range_contains(w, 5396, 4));
        EXPECT(!debug_range_contains(w, 5400, 4));
        EXPECT(!debug_range_contains(w, 5398, 4));
        const DebugRange none{5000, 0, 400, 0};
        EXPECT(!debug_range_contains(none, 5000, 4));        // an unused slot matches nothing
        // a call's set of buffers
        const DebugRange set[3] = {r, w, none};
        EXPECT(debug_any_range_contains(set, 3, 1064, 4));
        EXPECT(debug_any_range_contains(set, 3, 5396, 4));
        EXPECT(!debug_any_range_contains(set, 3, 3000, 4));
        EXPECT(!debug_any_range_contains(set, 0, 1000, 4));
        // exhaustive sweep against a plain restatement: every 4-byte access at every address
        for (uint64_t a = 900; a < 1300; ++a) {
            bool inside = false;
            for (uint64_t row = 0; row < 3; ++row) {
                const uint64_t lo = 1000 + row * 64, hi = lo + 40;
                if (a >= lo && a + 4 <= hi) inside = true;
            }
            EXPECT(debug_range_contains(r, a, 4) == inside);
        }
        // index form (tensors of a segment list)
        EXPECT(debug_span_inside(0, 8, 8));
        EXPECT(!debug_span_inside(1, 8, 8));
        EXPECT(debug_span_inside(7, 1, 8));
        EXPECT(!debug_span_inside(8, 1, 8));
        EXPECT(!debug_span_inside(0xfffffffffffffff0ull, 0x20, 8));
        std::printf("%s\n", failures ? "FAILED" : "ok");
        return failures ? 1 : 0;
    }
""")


def test_debug_range_arithmetic_host_compiled(tmp_path):
    src = tmp_path / "check.cpp"
    exe = tmp_path / "check"
    src.write_text(PROGRAM)
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-Wall", "-I", HEADER_DIR, "-o", str(exe), str(src)])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip().endswith("ok"), out.stdout
