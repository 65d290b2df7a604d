// Host-side neuron reordering for locality of the gathered operand (set-up, untimed).
//
// The paper partitions the rows of every W^k over processors with a hypergraph model (Section 5): a vertex per row, a
// net per column, so that rows sharing x entries land in the same part; the rows within a part may then be reordered
// freely, and its experiments attribute a 1.9-2.7x faster local SpMV to the temporal locality this gives (Section 6).
// On one GPU the "part" is what one CTA stages in shared memory: a group of rows of W^k whose columns fit a window of
// at most `col_cap` neurons of layer k-1.  This file finds such groups by greedy column-net clustering (grow a group
// from a seed row through the nets it touches, breadth first, while the group's column set stays within the window),
// and renumbers the neurons of layer k-1 so that every group's columns are one contiguous range: the window can then
// be copied with plain strided loads.  The renumbering of layer k-1 is the coupling between consecutive layers that the
// paper expresses with fixed vertices: it decides where layer k-1 WRITES its outputs, so W^{k-1} keeps its own row
// groups but stores each output row at its neuron's new number.
//
// A layer whose rows share too few columns for this (a uniformly random pattern) is reported as unstructured and is
// left alone.
#pragma once
#include <algorithm>
#include <cstdint>
#include <vector>

namespace sdnn_reorder {

struct Grouping {
    bool structured = false;          // groups with contiguous, capped windows were found
    std::vector<int> row_order;       // [n] storage position -> row of W^k (groups are consecutive runs)
    std::vector<int> group_row0;      // [groups + 1] first storage position of each group
    std::vector<int> group_c0;        // [groups] first new column number of the group's window
    std::vector<int> group_wlen;      // [groups] window length
    std::vector<int> col_label;       // [n] column (neuron of layer k-1) -> new number
    int64_t window_cols_total = 0;    // sum of the groups' distinct columns (diagnostic)
};

// rp/col: CSR of one layer (n x n).  Returns true and fills `g` when the layer is structured.
inline bool cluster_rows(int n, const int32_t* rp, const int32_t* col, int col_cap, int row_cap, Grouping& g) {
    g = Grouping();
    const int64_t nnz = rp[n];
    // nets: rows of every column
    std::vector<int> cptr(n + 1, 0);
    for (int64_t p = 0; p < nnz; ++p) ++cptr[col[p] + 1];
    for (int j = 0; j < n; ++j) cptr[j + 1] += cptr[j];
    std::vector<int> pins((size_t)nnz);
    {
        std::vector<int> cur(cptr.begin(), cptr.end() - 1);
        for (int i = 0; i < n; ++i)
            for (int p = rp[i]; p < rp[i + 1]; ++p) pins[cur[col[p]]++] = i;
    }
    std::vector<int> group_of(n, -1), queued(n, -1), col_stamp(n, -1);
    std::vector<int> order, row0{0}, queue;
    std::vector<std::vector<int>> group_cols;
    order.reserve(n);
    int64_t rows_done = 0, cols_sum = 0;
    int gid = 0;
    for (int seed = 0; seed < n; ++seed) {
        if (group_of[seed] >= 0 || rp[seed + 1] == rp[seed]) continue;
        queue.clear();
        queue.push_back(seed);
        queued[seed] = gid;
        std::vector<int> mine;
        int nrows = 0;
        for (size_t head = 0; head < queue.size(); ++head) {
            const int r = queue[head];
            if (group_of[r] >= 0) continue;
            int fresh = 0;
            for (int p = rp[r]; p < rp[r + 1]; ++p) fresh += col_stamp[col[p]] != gid;
            if ((int)mine.size() + fresh > col_cap || nrows + 1 > row_cap) continue;      // stays free for a later group
            group_of[r] = gid;
            order.push_back(r);
            ++nrows;
            for (int p = rp[r]; p < rp[r + 1]; ++p) {
                const int c = col[p];
                if (col_stamp[c] == gid) continue;
                col_stamp[c] = gid;
                mine.push_back(c);
                for (int q = cptr[c]; q < cptr[c + 1]; ++q) {
                    const int r2 = pins[q];
                    if (group_of[r2] < 0 && queued[r2] != gid) { queued[r2] = gid; queue.push_back(r2); }
                }
            }
        }
        if (nrows == 0) {      // the seed alone does not fit the window: no grouping possible
            return false;
        }
        rows_done += nrows;
        cols_sum += (int64_t)mine.size();
        group_cols.push_back(std::move(mine));
        row0.push_back((int)order.size());
        ++gid;
        // rows that share columns need, on average, at most two window columns per row; a random pattern needs k per row
        if (rows_done >= std::min<int64_t>(n, 4096) / 2 && cols_sum > 2 * rows_done) return false;
    }
    if (cols_sum > 2 * std::max<int64_t>(rows_done, 1)) return false;
    // new numbers for the columns: group by group, first touch wins; untouched neurons last
    std::vector<int> label(n, -1);
    int next = 0;
    std::vector<int> c0(gid), wlen(gid);
    for (int q = 0; q < gid; ++q) {
        std::vector<int>& cs = group_cols[q];
        std::sort(cs.begin(), cs.end());
        int lo = n, hi = -1;
        const int first_new = next;
        for (int c : cs) if (label[c] < 0) label[c] = next++;
        (void)first_new;
        for (int c : cs) { lo = std::min(lo, label[c]); hi = std::max(hi, label[c]); }
        if (hi - lo + 1 > col_cap) return false;      // a column shared with an earlier group lies too far away
        c0[q] = lo; wlen[q] = hi - lo + 1;
    }
    for (int j = 0; j < n; ++j) if (label[j] < 0) label[j] = next++;
    // rows without entries: one last group with an empty window
    int empties = 0;
    for (int i = 0; i < n; ++i) if (group_of[i] < 0) { order.push_back(i); ++empties; }
    if (empties) { row0.push_back((int)order.size()); c0.push_back(0); wlen.push_back(0); }
    g.structured = true;
    g.row_order = std::move(order);
    g.group_row0 = std::move(row0);
    g.group_c0 = std::move(c0);
    g.group_wlen = std::move(wlen);
    g.col_label = std::move(label);
    g.window_cols_total = cols_sum;
    return true;
}

}  // namespace sdnn_reorder
