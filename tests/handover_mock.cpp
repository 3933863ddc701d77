// CPU-thread model of the decode kernels' hand-over protocol through the workspace, for the
// tests only: threads stand in for CTAs, std::atomic words for device-scope relaxed accesses.
//
// The protocol, as the kernels implement it:
//   * a partial-sum slot is a run of 32-bit words, each its own "empty" flag: 0xFFFFFFFF means
//     nothing there yet; a writer stores fp32 bits (a value whose bits equal the flag is stored
//     as a quiet NaN); the one reader of a slot polls until no word is empty, adds the words in
//     list order and writes the flag back, so that the workspace is ready for the next call;
//   * T entries are single 64-bit words {payload, call number}; the call number is
//     departures / n_ctas + 1, read at the start of a call; a fetcher polls an entry until its
//     call number is the current one, and nobody resets entries;
//   * every poll has a limit; when it runs out the poller sets the time-out bit (plus a bit
//     naming the kind of wait) in the status word, takes what it has and goes on; every CTA
//     still leaves and adds one to the departure counter.
//
// Usage: handover_mock <n_ctas> <n_units> <calls> <withhold_call> <poll_limit>
//   Every CTA writes one partial per unit (unit u's partial of CTA c is c + 1 + u / 1024), unit
//   u is reduced by CTA u % n_ctas, which publishes the sum as a T entry; every CTA then fetches
//   all entries and checks them.  In call number `withhold_call` (1-based, 0 = never) CTA 0
//   writes nothing.  Prints one line per call: status word, departures, wrong sums seen, slots
//   left non-empty; exit code 0 unless the model itself failed.
#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <thread>
#include <vector>

namespace {

constexpr uint32_t kEmpty = 0xFFFFFFFFu;
constexpr uint32_t kNanBits = 0x7FC00000u;
constexpr uint32_t kTimeoutBit = 1u << 7;          // SLIM_ERR_TIMEOUT
constexpr uint32_t kWaitPartials = 64u << 16;      // which wait expired: partials of T
constexpr uint32_t kWaitPublished = 128u << 16;    //                     published T

struct Workspace {
    std::atomic<uint64_t> departures{0};
    std::vector<std::atomic<uint64_t>> t_final;    // [n_units]
    std::vector<std::atomic<uint32_t>> parts;      // [n_units][n_ctas]
    Workspace(int n_units, int n_ctas) : t_final(n_units), parts((size_t)n_units * n_ctas) { reset(); }
    void reset() {
        departures.store(0);
        for (auto& e : t_final) e.store(~0ull);
        for (auto& s : parts) s.store(kEmpty);
    }
};

uint32_t slot_bits(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    return u == kEmpty ? kNanBits : u;
}
float as_float(uint32_t u) { float v; memcpy(&v, &u, 4); return v; }

struct CallResult { uint32_t status; uint64_t departures; int wrong; int left; };

void cta_body(Workspace& ws, int cta, int n_ctas, int n_units, bool withhold, uint32_t poll_limit,
              std::atomic<uint32_t>& status, std::atomic<int>& wrong)
{
    const auto relaxed = std::memory_order_relaxed;
    // the number of this call on this workspace, before any CTA of the call can have left
    const uint32_t call = (uint32_t)(ws.departures.load(relaxed) / (uint64_t)n_ctas) + 1u;
    // ---- writer: one partial per unit
    if (!withhold)
        for (int u = 0; u < n_units; ++u)
            ws.parts[(size_t)u * n_ctas + cta].store(slot_bits((float)(cta + 1) + (float)u / 1024.f), relaxed);
    // ---- reader of the units dealt to this CTA: poll, add in list order, empty the slots, publish
    for (int u = cta; u < n_units; u += n_ctas) {
        std::vector<uint32_t> v(n_ctas);
        for (int c = 0; c < n_ctas; ++c) v[c] = ws.parts[(size_t)u * n_ctas + c].load(relaxed);
        for (uint32_t spins = 0;; ++spins) {
            bool all = true;
            for (int c = 0; c < n_ctas; ++c)
                if (v[c] == kEmpty) { v[c] = ws.parts[(size_t)u * n_ctas + c].load(relaxed); all = false; }
            if (all) break;
            if (spins > poll_limit) { status.fetch_or(kTimeoutBit | kWaitPartials, relaxed); break; }
            std::this_thread::yield();
        }
        float sum = 0.f;
        for (int c = 0; c < n_ctas; ++c) {
            sum += as_float(v[c]);
            ws.parts[(size_t)u * n_ctas + c].store(kEmpty, relaxed);
        }
        uint32_t bits;
        memcpy(&bits, &sum, 4);
        ws.t_final[u].store(((uint64_t)call << 32) | bits, relaxed);         // one 64-bit word: never torn
    }
    // ---- every CTA fetches every entry of this call
    for (int u = 0; u < n_units; ++u) {
        uint64_t e = ws.t_final[u].load(relaxed);
        for (uint32_t spins = 0; (uint32_t)(e >> 32) != call; ++spins) {
            if (spins > poll_limit) { status.fetch_or(kTimeoutBit | kWaitPublished, relaxed); break; }
            std::this_thread::yield();
            e = ws.t_final[u].load(relaxed);
        }
        float expect = 0.f;
        for (int c = 0; c < n_ctas; ++c) expect += (float)(c + 1) + (float)u / 1024.f;
        if ((uint32_t)(e >> 32) != call || as_float((uint32_t)e) != expect) wrong.fetch_add(1, relaxed);
    }
    ws.departures.fetch_add(1, relaxed);                                     // leaves, whatever happened
}

CallResult run_call(Workspace& ws, int n_ctas, int n_units, bool withhold_cta0, uint32_t poll_limit) {
    std::atomic<uint32_t> status{0};
    std::atomic<int> wrong{0};
    std::vector<std::thread> th;
    for (int c = 0; c < n_ctas; ++c)
        th.emplace_back(cta_body, std::ref(ws), c, n_ctas, n_units, withhold_cta0 && c == 0, poll_limit,
                        std::ref(status), std::ref(wrong));
    for (auto& t : th) t.join();                                             // a call ends when every CTA has left
    int left = 0;
    for (auto& s : ws.parts) left += s.load() != kEmpty;
    return {status.load(), ws.departures.load(), wrong.load(), left};
}

}  // namespace

int main(int argc, char** argv) {
    if (argc != 6) { fprintf(stderr, "usage: %s n_ctas n_units calls withhold_call poll_limit\n", argv[0]); return 2; }
    const int n_ctas = atoi(argv[1]), n_units = atoi(argv[2]), calls = atoi(argv[3]), withhold = atoi(argv[4]);
    const uint32_t poll_limit = (uint32_t)strtoul(argv[5], nullptr, 10);
    if (n_ctas < 1 || n_units < 1 || calls < 1) return 2;
    Workspace ws(n_units, n_ctas);
    for (int k = 1; k <= calls; ++k) {
        const CallResult r = run_call(ws, n_ctas, n_units, k == withhold, poll_limit);
        printf("call %d status %u departures %llu wrong %d left %d\n", k, r.status, (unsigned long long)r.departures, r.wrong, r.left);
        if (r.status != 0) { ws.reset(); printf("reset\n"); }               // the caller's duty after a time-out
    }
    return 0;
}
