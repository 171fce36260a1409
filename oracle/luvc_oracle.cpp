// CPU oracle for the two LUVC token-compression operators (OIM, SPU).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
// statement of what the operators compute.  It shares no code with the CUDA
// library and must never be linked into, imported by, or called from the
// product path; only the tests, the smoke check and the CPU-baseline leg of
// the benchmark use it.
//
// OIM follows Section 3.2 of the paper (row merge giving H x (W-m), then
// column merge giving (H-m) x (W-m)), the size vector s of Eq. 3 and the
// iteration strategy of Appendix "Iterative Strategy and Pseudocode of OIM"
// (alternating axes, merge number 2).  SPU follows Eq. 4-8 and Algorithm 2.
// Where the paper is silent the reading taken is stated next to the code.
//
// Parity unpinned (no value in the paper to check against): the default
// low-pass cutoff, the two readings of "similarity calculations and binary
// matching" (adjacent neighbours; every even cell against every odd cell of
// its line), the rule mapping a target count to a final grid, and the axis
// order.  Everything else is pinned by the CPU tests.
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -pthread luvc_oracle.cpp -o libluvc_oracle.so

#include <algorithm>
#include <cmath>
#include <complex>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

using cd = std::complex<double>;
const double kPi = 3.14159265358979323846264338327950288;

// ----------------------------------------------------------------------------
// OIM
// ----------------------------------------------------------------------------

struct Cell {
    std::vector<double> v;     // mean vector of the cell
    long long s = 1;           // number of source tokens merged into it (Eq. 3's s)
    std::vector<int> src;      // indices of those source tokens in the H*W input
};

double dot(const std::vector<double>& a, const std::vector<double>& b) {
    double acc = 0.0;
    for (size_t i = 0; i < a.size(); ++i) acc += a[i] * b[i];
    return acc;
}

// Cosine similarity; defined as 0 when either vector has zero norm.
double cosine(const std::vector<double>& a, const std::vector<double>& b) {
    const double na = std::sqrt(dot(a, a)), nb = std::sqrt(dot(b, b));
    if (na == 0.0 || nb == 0.0) return 0.0;
    return dot(a, b) / (na * nb);
}

// Number of cells merged away from a line of length `len` in one step:
// the paper's merge number r, never more than what is left to remove and never
// more than the number of even-position cells (each of which has a neighbour
// as soon as len >= 2).
int merges_this_step(int len, int len_final, int r) {
    int m = std::min(r, len - len_final);
    m = std::min(m, (len + 1) / 2);
    if (len < 2) m = 0;
    return m;
}

struct Candidate {
    int pos;        // even position in the line
    double cl, cr;  // cosine to the left / right neighbour (NaN if absent)
    double score;   // the larger of the two
    int dir;        // 0 = left (pos-1), 1 = right (pos+1); ties go left
};

struct OimStats {
    double min_sel_margin = std::numeric_limits<double>::infinity();
    double min_dir_margin = std::numeric_limits<double>::infinity();
    long long violations = 0;  // replay: decisions outside the tolerance (or malformed)
    long long deviations = 0;  // replay: decisions that differ from the oracle's own
};

// One merge step along one axis, applied to every line of the grid from the
// pre-step state.  axis 0: lines are rows (width shrinks); axis 1: lines are
// columns (height shrinks).  `trace_in` (replay) supplies m entries per line,
// each (pos*2 + dir); `trace_out` receives the decisions that were applied.
void oim_step(std::vector<Cell>& grid, int& h, int& w, int axis, int m,
              const int32_t* trace_in, double tol, int32_t* trace_out, OimStats& st) {
    const int nlines = axis == 0 ? h : w;
    const int len = axis == 0 ? w : h;
    auto at = [&](int line, int pos) -> Cell& {
        return axis == 0 ? grid[(size_t)line * w + pos] : grid[(size_t)pos * w + line];
    };
    const int nh = axis == 0 ? h : h - m, nw = axis == 0 ? w - m : w;
    std::vector<Cell> next((size_t)nh * nw);

    for (int line = 0; line < nlines; ++line) {
        // similarity of every even-position cell to its (at most two) odd neighbours
        std::vector<Candidate> cand;
        for (int j = 0; j < len; j += 2) {
            Candidate c;
            c.pos = j;
            c.cl = j >= 1 ? cosine(at(line, j).v, at(line, j - 1).v) : std::nan("");
            c.cr = j + 1 < len ? cosine(at(line, j).v, at(line, j + 1).v) : std::nan("");
            if (std::isnan(c.cl)) { c.dir = 1; c.score = c.cr; }
            else if (std::isnan(c.cr)) { c.dir = 0; c.score = c.cl; }
            else if (c.cr > c.cl) { c.dir = 1; c.score = c.cr; }
            else { c.dir = 0; c.score = c.cl; }
            cand.push_back(c);
        }
        // order: score descending, position ascending; the first m are merged
        std::vector<int> order(cand.size());
        for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
        std::stable_sort(order.begin(), order.end(),
                         [&](int a, int b) { return cand[a].score > cand[b].score; });

        std::vector<int> chosen_pos(m), chosen_dir(m);
        if (!trace_in) {
            for (int k = 0; k < m; ++k) {
                chosen_pos[k] = cand[order[k]].pos;
                chosen_dir[k] = cand[order[k]].dir;
            }
        } else {
            const int32_t* t = trace_in + (size_t)line * m;
            std::vector<char> is_chosen(cand.size(), 0);
            bool ok = true;
            for (int k = 0; k < m; ++k) {
                const int pos = t[k] >> 1, dir = t[k] & 1;
                const bool valid = t[k] >= 0 && pos < len && pos % 2 == 0 &&
                                   !is_chosen[pos / 2] &&
                                   (dir == 0 ? pos >= 1 : pos + 1 < len);
                if (!valid) { ok = false; break; }
                is_chosen[pos / 2] = 1;
                chosen_pos[k] = pos;
                chosen_dir[k] = dir;
            }
            if (!ok) {
                // malformed decision: count it and fall back to the oracle's own choice
                st.violations++;
                for (int k = 0; k < m; ++k) {
                    chosen_pos[k] = cand[order[k]].pos;
                    chosen_dir[k] = cand[order[k]].dir;
                }
            } else {
                double min_chosen = std::numeric_limits<double>::infinity();
                double max_unchosen = -std::numeric_limits<double>::infinity();
                for (size_t i = 0; i < cand.size(); ++i) {
                    if (is_chosen[i]) min_chosen = std::min(min_chosen, cand[i].score);
                    else max_unchosen = std::max(max_unchosen, cand[i].score);
                }
                if (m > 0 && min_chosen < max_unchosen - tol) st.violations++;
                bool differs = false;
                for (int k = 0; k < m; ++k) {
                    const Candidate& c = cand[chosen_pos[k] / 2];
                    const double got = chosen_dir[k] == 0 ? c.cl : c.cr;
                    if (got < c.score - tol) st.violations++;
                    if (chosen_dir[k] != c.dir) differs = true;
                    bool in_top = false;
                    for (int q = 0; q < m; ++q) in_top |= cand[order[q]].pos == chosen_pos[k];
                    if (!in_top) differs = true;
                }
                if (differs) st.deviations++;
            }
        }

        // decision margins of the oracle's own ordering on this state
        if (m > 0 && (size_t)m < cand.size())
            st.min_sel_margin = std::min(st.min_sel_margin,
                                         cand[order[m - 1]].score - cand[order[m]].score);
        for (int k = 0; k < m; ++k) {
            const Candidate& c = cand[chosen_pos[k] / 2];
            if (!std::isnan(c.cl) && !std::isnan(c.cr))
                st.min_dir_margin = std::min(st.min_dir_margin, std::fabs(c.cl - c.cr));
        }
        if (trace_out)
            for (int k = 0; k < m; ++k)
                trace_out[(size_t)line * m + k] = chosen_pos[k] * 2 + chosen_dir[k];

        // size-weighted merge into the destination cells, from the pre-step state
        std::vector<char> removed(len, 0);
        std::vector<std::vector<int>> incoming(len);
        for (int k = 0; k < m; ++k) {
            const int a = chosen_pos[k], b = chosen_dir[k] == 0 ? a - 1 : a + 1;
            removed[a] = 1;
            incoming[b].push_back(a);
        }
        int out_pos = 0;
        for (int j = 0; j < len; ++j) {
            if (removed[j]) continue;
            Cell c = at(line, j);
            if (!incoming[j].empty()) {
                const size_t D = c.v.size();
                std::vector<double> wsum(D);
                long long stot = c.s;
                for (size_t i = 0; i < D; ++i) wsum[i] = (double)c.s * c.v[i];
                for (int a : incoming[j]) {
                    const Cell& ca = at(line, a);
                    for (size_t i = 0; i < D; ++i) wsum[i] += (double)ca.s * ca.v[i];
                    stot += ca.s;
                    c.src.insert(c.src.end(), ca.src.begin(), ca.src.end());
                }
                for (size_t i = 0; i < D; ++i) c.v[i] = wsum[i] / (double)stot;
                c.s = stot;
            }
            if (axis == 0) next[(size_t)line * nw + out_pos] = std::move(c);
            else next[(size_t)out_pos * nw + line] = std::move(c);
            ++out_pos;
        }
    }
    grid.swap(next);
    h = nh;
    w = nw;
}

// The full-line reading of "similarity calculations and binary matching" (Section 3.2;
// the O(n_v^1.5 k) cost the paper states for OIM corresponds to a similarity matrix per
// line): the cells of a line are split into set A (even positions) and set B (odd
// positions), every A cell is compared with EVERY B cell of its line and proposes the
// most similar one (ties: the lowest position), and the m proposals with the highest
// similarity (ties: the lowest A position) are merged, size-weighted, into the proposed
// B cells; several A cells may end in the same B cell.  The line closes up in order.
// Trace entries are (A position << 16) | B position.
void oim_step_bipartite(std::vector<Cell>& grid, int& h, int& w, int axis, int m,
                        const int32_t* trace_in, double tol, int32_t* trace_out, OimStats& st) {
    const int nlines = axis == 0 ? h : w;
    const int len = axis == 0 ? w : h;
    auto at = [&](int line, int pos) -> Cell& {
        return axis == 0 ? grid[(size_t)line * w + pos] : grid[(size_t)pos * w + line];
    };
    const int nh = axis == 0 ? h : h - m, nw = axis == 0 ? w - m : w;
    std::vector<Cell> next((size_t)nh * nw);
    const int na = (len + 1) / 2, nb = len / 2;

    for (int line = 0; line < nlines; ++line) {
        // similarity matrix S[i][j] = cos(cell 2i, cell 2j+1)
        std::vector<double> S((size_t)na * nb);
        for (int i = 0; i < na; ++i)
            for (int j = 0; j < nb; ++j) S[(size_t)i * nb + j] = cosine(at(line, 2 * i).v, at(line, 2 * j + 1).v);
        // proposal of every A cell: first maximum of its row
        std::vector<int> prop(na, 0);
        std::vector<double> score(na, -std::numeric_limits<double>::infinity());
        for (int i = 0; i < na; ++i)
            for (int j = 0; j < nb; ++j)
                if (S[(size_t)i * nb + j] > score[i]) { score[i] = S[(size_t)i * nb + j]; prop[i] = j; }
        std::vector<int> order(na);
        for (int i = 0; i < na; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return score[a] > score[b]; });

        std::vector<int> src(m), dst(m);      // positions in the line
        auto own_choice = [&]() {
            for (int k = 0; k < m; ++k) { src[k] = 2 * order[k]; dst[k] = 2 * prop[order[k]] + 1; }
        };
        if (!trace_in) {
            own_choice();
        } else {
            const int32_t* t = trace_in + (size_t)line * m;
            std::vector<char> is_chosen(na, 0);
            bool ok = true;
            for (int k = 0; k < m; ++k) {
                const int a = t[k] >> 16, b = t[k] & 0xffff;
                const bool valid = t[k] >= 0 && a < len && a % 2 == 0 && b < len && b % 2 == 1 && !is_chosen[a / 2];
                if (!valid) { ok = false; break; }
                is_chosen[a / 2] = 1;
                src[k] = a;
                dst[k] = b;
            }
            if (!ok) {
                st.violations++;
                own_choice();
            } else {
                double min_chosen = std::numeric_limits<double>::infinity();
                double max_unchosen = -std::numeric_limits<double>::infinity();
                for (int i = 0; i < na; ++i) {
                    if (is_chosen[i]) min_chosen = std::min(min_chosen, score[i]);
                    else max_unchosen = std::max(max_unchosen, score[i]);
                }
                if (m > 0 && min_chosen < max_unchosen - tol) st.violations++;
                bool differs = false;
                for (int k = 0; k < m; ++k) {
                    const int i = src[k] / 2, j = dst[k] / 2;
                    if (S[(size_t)i * nb + j] < score[i] - tol) st.violations++;
                    if (j != prop[i]) differs = true;
                    bool in_top = false;
                    for (int q = 0; q < m; ++q) in_top |= order[q] == i;
                    if (!in_top) differs = true;
                }
                if (differs) st.deviations++;
            }
        }

        // margins of the oracle's own decisions on this state: between the last taken and the
        // first refused proposal, and between the best and second-best B cell of a merged A cell
        if (m > 0 && m < na)
            st.min_sel_margin = std::min(st.min_sel_margin, score[order[m - 1]] - score[order[m]]);
        for (int k = 0; k < m; ++k) {
            const int i = src[k] / 2;
            for (int j = 0; j < nb; ++j)
                if (j != prop[i]) st.min_dir_margin = std::min(st.min_dir_margin, score[i] - S[(size_t)i * nb + j]);
        }
        if (trace_out)
            for (int k = 0; k < m; ++k) trace_out[(size_t)line * m + k] = (src[k] << 16) | dst[k];

        std::vector<char> removed(len, 0);
        std::vector<std::vector<int>> incoming(len);
        for (int k = 0; k < m; ++k) {
            removed[src[k]] = 1;
            incoming[dst[k]].push_back(src[k]);
        }
        int out_pos = 0;
        for (int j = 0; j < len; ++j) {
            if (removed[j]) continue;
            Cell c = at(line, j);
            if (!incoming[j].empty()) {
                const size_t D = c.v.size();
                std::vector<double> wsum(D);
                long long stot = c.s;
                for (size_t i = 0; i < D; ++i) wsum[i] = (double)c.s * c.v[i];
                for (int a : incoming[j]) {
                    const Cell& ca = at(line, a);
                    for (size_t i = 0; i < D; ++i) wsum[i] += (double)ca.s * ca.v[i];
                    stot += ca.s;
                    c.src.insert(c.src.end(), ca.src.begin(), ca.src.end());
                }
                for (size_t i = 0; i < D; ++i) c.v[i] = wsum[i] / (double)stot;
                c.s = stot;
            }
            if (axis == 0) next[(size_t)line * nw + out_pos] = std::move(c);
            else next[(size_t)out_pos * nw + line] = std::move(c);
            ++out_pos;
        }
    }
    grid.swap(next);
    h = nh;
    w = nw;
}

// ----------------------------------------------------------------------------
// SPU
// ----------------------------------------------------------------------------

int smallest_factor(int n) {
    for (int p = 2; (long long)p * p <= n; ++p)
        if (n % p == 0) return p;
    return n;
}

// exp(sign * 2*pi*i * j / n) with the angle reduced exactly in integers
cd root_of_unity(long long j, long long n, int sign) {
    j %= n;
    const double ang = 2.0 * kPi * (double)j / (double)n;
    return cd(std::cos(ang), sign * std::sin(ang));
}

// Recursive mixed-radix Cooley-Tukey on a strided input.  `roots` holds the
// n_total-th roots of unity of the outermost call; a size-n level uses every
// (n_total/n)-th of them.  A prime length falls back to the plain sum.
void fft_rec(const cd* x, size_t stride, int n, cd* y, const std::vector<cd>& roots, int n_total) {
    if (n == 1) { y[0] = x[0]; return; }
    const int step = n_total / n;
    const int p = smallest_factor(n);
    if (p == n) {
        for (int k = 0; k < n; ++k) {
            cd acc = 0.0;
            for (int j = 0; j < n; ++j) acc += x[(size_t)j * stride] * roots[(size_t)((long long)j * k % n) * step];
            y[k] = acc;
        }
        return;
    }
    const int m = n / p;
    std::vector<cd> sub((size_t)n);
    for (int r = 0; r < p; ++r) fft_rec(x + (size_t)r * stride, stride * p, m, sub.data() + (size_t)r * m, roots, n_total);
    for (int q = 0; q < m; ++q)
        for (int s = 0; s < p; ++s) {
            const int k = q + m * s;
            cd acc = 0.0;
            for (int r = 0; r < p; ++r) acc += sub[(size_t)r * m + q] * roots[(size_t)((long long)r * k % n) * step];
            y[k] = acc;
        }
}

std::vector<cd> make_roots(int n, int sign) {
    std::vector<cd> roots((size_t)n);
    for (int j = 0; j < n; ++j) roots[j] = root_of_unity(j, n, sign);
    return roots;
}

// Eq. 5 as read here: a Hamming window centred on the zero frequency, over the
// signed frequency f(k) = k for k <= N/2, k - N otherwise; pass band |f| <= sigma.
void spu_mask(int N, int sigma, int hamming, double* M) {
    for (int k = 0; k < N; ++k) {
        const int f = k <= N / 2 ? k : k - N;
        if (std::abs(f) > sigma) { M[k] = 0.0; continue; }
        if (!hamming || N == 1) { M[k] = 1.0; continue; }
        M[k] = 0.54 + 0.46 * std::cos(2.0 * kPi * (double)f / (double)(N - 1));
    }
}

// Squared low-pass energy of every token, summed over the channels [d0, d1).
// method 0: Eq. 4 and Eq. 7 as plain O(N^2) sums; method 1: the oracle's FFT.
void spu_energy_channels(const float* x, int N, int D, const std::vector<double>& M, int method,
                         int d0, int d1, std::vector<double>& e2) {
    e2.assign((size_t)N, 0.0);
    std::vector<cd> col((size_t)N), spec((size_t)N), back((size_t)N);
    std::vector<cd> fwd_roots, inv_roots;
    if (method == 1) { fwd_roots = make_roots(N, -1); inv_roots = make_roots(N, +1); }
    for (int d = d0; d < d1; ++d) {
        for (int n = 0; n < N; ++n) col[n] = cd((double)x[(size_t)n * D + d], 0.0);
        if (method == 0) {
            for (int k = 0; k < N; ++k) {              // Eq. 4
                cd acc = 0.0;
                if (M[k] != 0.0)                        // bins the mask zeroes need no sum
                    for (int n = 0; n < N; ++n) acc += col[n] * root_of_unity((long long)k * n, N, -1);
                spec[k] = acc * M[k];                   // Eq. 6
            }
            for (int n = 0; n < N; ++n) {              // Eq. 7
                cd acc = 0.0;
                for (int k = 0; k < N; ++k)
                    if (M[k] != 0.0) acc += spec[k] * root_of_unity((long long)k * n, N, +1);
                back[n] = acc / (double)N;
            }
        } else {
            fft_rec(col.data(), 1, N, spec.data(), fwd_roots, N);
            for (int k = 0; k < N; ++k) spec[k] *= M[k];
            fft_rec(spec.data(), 1, N, back.data(), inv_roots, N);
            for (int n = 0; n < N; ++n) back[n] /= (double)N;
        }
        // Eq. 8: the filtered signal is real (the mask is even in f), its
        // imaginary part is rounding noise and is dropped.
        for (int n = 0; n < N; ++n) e2[n] += back[n].real() * back[n].real();
    }
}

}  // namespace

extern "C" {

int oracle_abi_version(void) { return 1; }

// Final grid for a target token count: the factor pair (Hf, Wf) of `target`
// with Hf <= H, Wf <= W whose aspect ratio is closest (in log) to H/W; a tie
// goes to the larger Hf.  Returns 0 on success, 1 if no pair exists.
int oracle_oim_final_dims(int H, int W, int target, int* Hf, int* Wf) {
    if (H < 1 || W < 1 || target < 1 || (long long)target > (long long)H * W) return 1;
    double best = std::numeric_limits<double>::infinity();
    int bh = 0, bw = 0;
    for (int hf = 1; hf <= H; ++hf) {
        if (target % hf) continue;
        const int wf = target / hf;
        if (wf > W) continue;
        const double cost = std::fabs(std::log((double)hf / wf) - std::log((double)H / W));
        if (cost < best - 1e-12 || (std::fabs(cost - best) <= 1e-12 && hf > bh)) {
            best = cost; bh = hf; bw = wf;
        }
    }
    if (!bh) return 1;
    *Hf = bh; *Wf = bw;
    return 0;
}

// Step list of the iteration: alternately one width step and one height step
// (the other order when height_first), each removing m cells per line, until
// the grid is Hf x Wf.  axes[i] is 0 (width) or 1 (height).  Returns the number
// of steps, or -1 if the target cannot be reached.
// r_w cells leave every row in a width step, r_h cells every column in a height step
// (the appendix uses 2 for both; its anyres variant lets the two differ with the image's shape).
int oracle_oim_schedule(int H, int W, int Hf, int Wf, int r_w, int r_h, int height_first,
                        int32_t* axes, int32_t* ms, int cap) {
    if (Hf < 1 || Wf < 1 || Hf > H || Wf > W || r_w < 1 || r_h < 1) return -1;
    int h = H, w = W, n = 0;
    while (h != Hf || w != Wf) {
        bool progressed = false;
        for (int turn = 0; turn < 2; ++turn) {
            const int axis = height_first ? 1 - turn : turn;
            const int len = axis == 0 ? w : h, lf = axis == 0 ? Wf : Hf;
            const int m = merges_this_step(len, lf, axis == 0 ? r_w : r_h);
            if (m <= 0) continue;
            if (axes && n < cap) { axes[n] = axis; ms[n] = m; }
            ++n;
            if (axis == 0) w -= m; else h -= m;
            progressed = true;
        }
        if (!progressed) return -1;
    }
    return n;
}

// Merge numbers for an image whose sides differ (appendix, the variant for encoders that keep the
// image's aspect ratio: "the merging operations along the spatial dimensions are dynamically
// adjusted based on the aspect ratio").  The reading taken: `ops` operations, each one width step
// and one height step; the shorter side loses r cells per step and the longer side
// round(r * long / short), so that both sides shrink by about the same fraction and the grid
// keeps its shape.  Returns 0 and the per-axis numbers and final grid, 1 if a side would vanish.
int oracle_oim_anyres_plan(int H, int W, int ops, int r, int* r_h, int* r_w, int* Hf, int* Wf) {
    if (H < 1 || W < 1 || ops < 0 || r < 1) return 1;
    int rh = r, rw = r;
    if (W > H) rw = (int)std::floor((double)r * (double)W / (double)H + 0.5);
    if (H > W) rh = (int)std::floor((double)r * (double)H / (double)W + 0.5);
    const long long hf = (long long)H - (long long)ops * rh, wf = (long long)W - (long long)ops * rw;
    if (hf < 1 || wf < 1) return 1;
    *r_h = rh; *r_w = rw; *Hf = (int)hf; *Wf = (int)wf;
    return 0;
}

// OIM on one image.  tokens: [H*W][D] (exact input values as float).
// out_tokens: [Hf*Wf][D] double; out_sizes: [Hf*Wf]; out_map: [H*W] (final
// row-major cell of every source token).  trace_in == NULL: the oracle decides.
// Otherwise the decisions in trace_in (one int per merge, ordered by step, line,
// rank; pos*2+dir for matching 0, (A position << 16) | B position for matching 1,
// the full-line bipartite reading) are checked against `tol` and applied.  trace_out (may be
// NULL) gets the applied decisions.  stats[0..3] = minimum selection margin,
// minimum direction margin, violations, deviations.
int oracle_oim_image(const float* tokens, int H, int W, int D, int Hf, int Wf, int r_w, int r_h, int height_first, int matching,
                     double* out_tokens, int32_t* out_sizes, int32_t* out_map,
                     const int32_t* trace_in, double tol, int32_t* trace_out, double* stats) {
    std::vector<int32_t> axes(2 * (size_t)(H + W) + 4), ms(axes.size());
    const int nsteps = oracle_oim_schedule(H, W, Hf, Wf, r_w, r_h, height_first, axes.data(), ms.data(), (int)axes.size());
    if (nsteps < 0) return 1;
    std::vector<Cell> grid((size_t)H * W);
    for (int i = 0; i < H * W; ++i) {
        grid[i].v.assign(tokens + (size_t)i * D, tokens + (size_t)(i + 1) * D);
        grid[i].s = 1;
        grid[i].src = {i};
    }
    int h = H, w = W;
    size_t off = 0;
    OimStats st;
    for (int s = 0; s < nsteps; ++s) {
        const int nlines = axes[s] == 0 ? h : w;
        (matching == 1 ? oim_step_bipartite : oim_step)(grid, h, w, axes[s], ms[s], trace_in ? trace_in + off : nullptr,
                                                        tol, trace_out ? trace_out + off : nullptr, st);
        off += (size_t)nlines * ms[s];
    }
    for (int c = 0; c < Hf * Wf; ++c) {
        for (int i = 0; i < D; ++i) out_tokens[(size_t)c * D + i] = grid[c].v[i];
        out_sizes[c] = (int32_t)grid[c].s;
        for (int i : grid[c].src) out_map[i] = c;
    }
    if (stats) {
        stats[0] = st.min_sel_margin; stats[1] = st.min_dir_margin;
        stats[2] = (double)st.violations; stats[3] = (double)st.deviations;
    }
    return 0;
}

// A batch of images on `nthreads` host threads (images are independent).
int oracle_oim_batch(const float* tokens, int B, int H, int W, int D, int Hf, int Wf, int r_w, int r_h, int height_first, int matching,
                     double* out_tokens, int32_t* out_sizes, int32_t* out_map,
                     const int32_t* trace_in, double tol, int32_t* trace_out, double* stats, int nthreads) {
    const size_t ntrace = (size_t)H * W - (size_t)Hf * Wf;
    std::vector<int> rc((size_t)B, 0);
    auto work = [&](int t) {
        for (int b = t; b < B; b += nthreads)
            rc[b] = oracle_oim_image(tokens + (size_t)b * H * W * D, H, W, D, Hf, Wf, r_w, r_h, height_first, matching,
                                     out_tokens + (size_t)b * Hf * Wf * D, out_sizes + (size_t)b * Hf * Wf,
                                     out_map + (size_t)b * H * W,
                                     trace_in ? trace_in + (size_t)b * ntrace : nullptr, tol,
                                     trace_out ? trace_out + (size_t)b * ntrace : nullptr,
                                     stats ? stats + (size_t)b * 4 : nullptr);
    };
    nthreads = std::max(1, std::min(nthreads, B));
    std::vector<std::thread> pool;
    for (int t = 0; t < nthreads; ++t) pool.emplace_back(work, t);
    for (auto& th : pool) th.join();
    for (int b = 0; b < B; ++b) if (rc[b]) return rc[b];
    return 0;
}

// Eq. 4 for one real channel, as the plain O(N^2) sum.
void oracle_dft_naive(const double* x, int N, double* Xre, double* Xim) {
    for (int k = 0; k < N; ++k) {
        cd acc = 0.0;
        for (int n = 0; n < N; ++n) acc += x[n] * root_of_unity((long long)k * n, N, -1);
        Xre[k] = acc.real(); Xim[k] = acc.imag();
    }
}

// The oracle's FFT (sign -1 forward, +1 inverse without the 1/N factor).
void oracle_fft(const double* re, const double* im, int N, int sign, double* out_re, double* out_im) {
    std::vector<cd> in((size_t)N), out((size_t)N);
    for (int n = 0; n < N; ++n) in[n] = cd(re[n], im ? im[n] : 0.0);
    const std::vector<cd> roots = make_roots(N, sign);
    fft_rec(in.data(), 1, N, out.data(), roots, N);
    for (int k = 0; k < N; ++k) { out_re[k] = out[k].real(); out_im[k] = out[k].imag(); }
}

// Cutoff (fraction of the band [0, floor(N/2)]) to the last passed bin.
int oracle_spu_sigma(int N, double cutoff) { return (int)std::floor(cutoff * (double)(N / 2)); }

void oracle_spu_mask(int N, int sigma, int hamming, double* M) { spu_mask(N, sigma, hamming, M); }

// Scores E[n] of Eq. 8 for one sequence x: [N][D].  Channels are split over
// `nthreads` host threads; partial sums are added in thread order.
int oracle_spu_scores(const float* x, int N, int D, int sigma, int hamming, int method, int nthreads, double* E) {
    if (N < 1 || D < 1 || sigma < 0) return 1;
    std::vector<double> M((size_t)N);
    spu_mask(N, sigma, hamming, M.data());
    nthreads = std::max(1, std::min(nthreads, D));
    std::vector<std::vector<double>> part((size_t)nthreads);
    std::vector<std::thread> pool;
    for (int t = 0; t < nthreads; ++t) {
        const int d0 = (int)((long long)D * t / nthreads), d1 = (int)((long long)D * (t + 1) / nthreads);
        pool.emplace_back([&, t, d0, d1] { spu_energy_channels(x, N, D, M, method, d0, d1, part[t]); });
    }
    for (auto& th : pool) th.join();
    for (int n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int t = 0; t < nthreads; ++t) acc += part[t][n];
        E[n] = std::sqrt(acc);
    }
    return 0;
}

// Scores at chosen tokens only, straight from the definition: the filter of
// Eq. 5-7 is a circular convolution with h[j] = (1/N) sum_k M[k] e^{+2 pi i k j / N}.
int oracle_spu_scores_at(const float* x, int N, int D, int sigma, int hamming,
                         const int32_t* tokens, int count, double* E) {
    std::vector<double> M((size_t)N), hker((size_t)N);
    spu_mask(N, sigma, hamming, M.data());
    for (int j = 0; j < N; ++j) {
        double acc = 0.0;
        for (int k = 0; k < N; ++k)
            if (M[k] != 0.0) acc += M[k] * root_of_unity((long long)k * j, N, +1).real();
        hker[j] = acc / (double)N;
    }
    std::vector<double> filt((size_t)D);
    for (int c = 0; c < count; ++c) {
        const int n = tokens[c];
        std::fill(filt.begin(), filt.end(), 0.0);
        for (int mm = 0; mm < N; ++mm) {
            const double hv = hker[(size_t)(((n - mm) % N + N) % N)];
            const float* row = x + (size_t)mm * D;
            for (int d = 0; d < D; ++d) filt[d] += hv * (double)row[d];
        }
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += filt[d] * filt[d];
        E[c] = std::sqrt(acc);
    }
    return 0;
}

// Algorithm 2's top-k: the `keep` largest scores, ties to the lowest index,
// returned in ascending index order (the kept tokens stay in sequence order).
int oracle_spu_select(const double* E, int N, int keep, int32_t* idx) {
    if (keep < 0 || keep > N) return 1;
    std::vector<int> order((size_t)N);
    for (int n = 0; n < N; ++n) order[n] = n;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return E[a] > E[b]; });
    std::vector<int> kept(order.begin(), order.begin() + keep);
    std::sort(kept.begin(), kept.end());
    for (int j = 0; j < keep; ++j) idx[j] = kept[j];
    return 0;
}

int oracle_hardware_threads(void) {
    const unsigned n = std::thread::hardware_concurrency();
    return n ? (int)n : 1;
}

}  // extern "C"
