// Host-side buffer planning for a fixed sequence of fused operators (Section 4.5: liveness analysis,
// Eq. 14, and linear-scan buffer allocation, Algorithm 2, with the buffer reduction ratio of Eq. 15).
// A "register" is an intermediate tensor of the sequence; registers whose live intervals do not overlap
// share one physical buffer.  Nothing here touches the GPU.
#include <algorithm>
#include <numeric>
#include <vector>

#include "forge_common.cuh"

extern "C" int forge_plan_liveness(int num_ops, const int* out_reg, const int* in_off, const int* in_regs,
                                   int num_regs, int* start, int* end) {
    if (num_ops < 0 || num_regs < 0 || (num_ops > 0 && (!out_reg || !in_off || !in_regs)) ||
        (num_regs > 0 && (!start || !end)))
        return FORGE_ERR_INVALID_ARG;
    for (int r = 0; r < num_regs; ++r) start[r] = end[r] = -1;
    for (int j = 0; j < num_ops; ++j) {
        if (in_off[j + 1] < in_off[j]) return FORGE_ERR_INVALID_ARG;
        for (int p = in_off[j]; p < in_off[j + 1]; ++p) {
            const int r = in_regs[p];
            if (r < 0 || r >= num_regs) return FORGE_ERR_INVALID_ARG;
            end[r] = std::max(end[r], j);  // Eq. 14: the last instruction that reads r
        }
        const int w = out_reg[j];
        if (w >= num_regs) return FORGE_ERR_INVALID_ARG;
        if (w >= 0) {
            if (start[w] >= 0) return FORGE_ERR_INVALID_ARG;  // every register has one writer
            start[w] = j;                                     // Eq. 14: the instruction that writes r
        }
    }
    for (int r = 0; r < num_regs; ++r) {
        if (end[r] < start[r]) end[r] = start[r];  // never read: dead right after its writer
        if (start[r] >= 0 && end[r] >= 0 && end[r] < start[r]) return FORGE_ERR_INVALID_ARG;
    }
    return FORGE_OK;
}

extern "C" int forge_plan_linear_scan(int n, const int* start, const int* end, const size_t* bytes,
                                      const unsigned char* pinned, int* buf_of, size_t* buf_bytes, int* num_bufs) {
    if (n < 0 || !num_bufs || (n > 0 && (!start || !end || !buf_of))) return FORGE_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (end[i] < start[i]) return FORGE_ERR_INVALID_ARG;
    // Algorithm 2, line 1: intervals in order of their start (ties: by register number)
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return start[a] < start[b]; });
    struct Live { int end, buf; };
    std::vector<Live> active;    // intervals still in flight, in the order they were opened
    std::vector<int> free_pool;  // released buffers, oldest release first
    std::vector<size_t> sizes;   // bytes of each buffer: the largest register it ever holds
    for (int r : order) {
        // expire what ended before this interval starts; the buffers go back to the pool
        std::vector<Live> alive;
        for (const Live& a : active) {
            if (a.end < start[r]) free_pool.push_back(a.buf);
            else alive.push_back(a);
        }
        active.swap(alive);
        const size_t need = bytes ? bytes[r] : 1;
        int b;
        if ((pinned && pinned[r]) || free_pool.empty()) {
            b = (int)sizes.size();  // a new buffer
            sizes.push_back(need);
        } else {
            b = free_pool.front();  // reuse the one released longest ago
            free_pool.erase(free_pool.begin());
            sizes[b] = std::max(sizes[b], need);
        }
        buf_of[r] = b;
        active.push_back({end[r], b});
    }
    *num_bufs = (int)sizes.size();
    if (buf_bytes) std::copy(sizes.begin(), sizes.end(), buf_bytes);
    return FORGE_OK;
}
