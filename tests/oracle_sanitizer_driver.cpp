// Test driver (not product): runs the CPU oracle under AddressSanitizer and UndefinedBehaviorSanitizer.
// Built and run by tests/test_oracle_pins.py::test_oracle_is_clean_under_address_and_ub_sanitizers as
//   g++ -O1 -g -std=c++17 -ffp-contract=off -fsanitize=address,undefined -fno-sanitize-recover=all
// Every array is a heap allocation of exactly the size the oracle may touch, so an index past either end
// of any of them aborts the program. Sizes cover empty, one element, one short of a block, a block, one
// past a block, and several blocks with a ragged tail; both parameter types, both gradient types, both
// kinds of state, the search and the brute-force quantizer, a clipped and a skipped (non-finite) step.
#include "../oracle/lt_oracle.cpp"

#include <cstdio>
#include <cstdlib>
#include <memory>

namespace {

uint32_t g_seed = 12345u;
float next_normalish() {   // cheap deterministic values in (-1, 1), then scaled by the caller
    g_seed = g_seed * 1664525u + 1013904223u;
    return ((float)(g_seed >> 8) / 8388608.0f) - 1.0f;
}

struct Arrays {
    std::unique_ptr<unsigned char[]> param, grad, m, v;
    std::unique_ptr<float[]> am, av;
    lto_tensor t;
};

Arrays make(int64_t n, int block, int pdt, int gdt, int sdt) {
    Arrays a;
    const int ps = pdt == 0 ? 4 : 2, gs = gdt == 0 ? 4 : 2, ss = sdt == 1 ? 4 : 1;
    const int64_t nb = (n + block - 1) / block;
    a.param.reset(new unsigned char[n * ps]);
    a.grad.reset(new unsigned char[n * gs]);
    a.m.reset(new unsigned char[n * ss]);
    a.v.reset(new unsigned char[n * ss]);
    a.am.reset(new float[nb]);
    a.av.reset(new float[nb]);
    for (int64_t i = 0; i < n; ++i) {
        const float p = 0.02f * next_normalish(), g = 1e-3f * next_normalish();
        uint32_t pb, gb;
        std::memcpy(&pb, &p, 4);
        std::memcpy(&gb, &g, 4);
        if (pdt == 0) std::memcpy(a.param.get() + 4 * i, &p, 4);
        else { const uint16_t h = (uint16_t)(pb >> 16); std::memcpy(a.param.get() + 2 * i, &h, 2); }
        if (gdt == 0) std::memcpy(a.grad.get() + 4 * i, &g, 4);
        else { const uint16_t h = (uint16_t)(gb >> 16); std::memcpy(a.grad.get() + 2 * i, &h, 2); }
    }
    a.t = lto_tensor{a.param.get(), a.grad.get(), a.m.get(), a.v.get(), sdt == 1 ? nullptr : a.am.get(),
                     sdt == 1 ? nullptr : a.av.get(), n, pdt, gdt, sdt, 0};
    return a;
}

}  // namespace

int main() {
    const int64_t sizes[] = {0, 1, 7, 255, 256, 257, 2047, 2048, 2049, 5000, 3 * 4096 + 17};
    long checks = 0;
    for (int block : {256, 2048, 4096}) {
        for (int pdt = 0; pdt < 2; ++pdt) for (int gdt = 0; gdt < 2; ++gdt) for (int sdt = 0; sdt < 2; ++sdt) {
            std::vector<Arrays> owned;
            std::vector<lto_tensor> list;
            for (int64_t n : sizes) { owned.push_back(make(n, block, pdt, gdt, sdt)); list.push_back(owned.back().t); }
            lto_state_init(list.data(), (int32_t)list.size(), block);
            lto_hparams hp{1e-5f, 0.9f, 0.999f, 1e-8f, 0.01f, 1e-4f, 1};   // a max_norm small enough to clip
            int32_t status = 0;
            for (int step = 1; step <= 3; ++step) {
                hp.step = step;
                const double S = lto_grad_sqnorm_multi(list.data(), (int32_t)list.size(), 0.0);
                if (!(S > 0.0)) { std::printf("unexpected norm\n"); return 2; }
                lto_hybrid8_step(list.data(), (int32_t)list.size(), block, &hp, S, &status, step == 2 ? 1 : 0);
                ++checks;
            }
            lto_hybrid8_step(list.data(), (int32_t)list.size(), block, &hp, std::nan(""), &status, 0);   // skipped
            if (status != 1) { std::printf("skip not reported\n"); return 3; }
        }
    }
    float tab[256];
    lto_code_table(1, tab);
    lto_code_table(0, tab);
    for (float x : {-2.0f, -1.0f, -0.0f, 0.0f, 1e-30f, 0.5f, 1.0f, 2.0f})
        if (lto_nearest(1, x) != lto_nearest_brute(1, x) || lto_nearest(0, std::fabs(x)) != lto_nearest_brute(0, std::fabs(x))) return 4;
    std::printf("sanitizer run clean: %ld steps\n", checks);
    return 0;
}
