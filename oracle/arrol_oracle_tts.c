/*
 * CPU oracle, test-time half: rank-weighted voting with quality-head scores (Section 4.4).
 * TEST INFRASTRUCTURE ONLY (see arrol_oracle.c).
 *
 * Per group of G candidates: sort the candidates by score; a candidate's weight is its rank rescaled linearly to
 * [0,1] (lowest score 0, highest 1; a single candidate gets 1).  Equal scores keep index order (the lower index
 * takes the lower rank).  The vote: every distinct answer collects the weights of its candidates, the answer with
 * the largest total wins; of equal totals the answer that appears first wins.  Answers < 0 mean "no answer" and
 * do not vote; a group without any answer has winner -1.  Totals are compared as integer rank sums.
 */
#include <stdint.h>

void oracle_rank_vote(const float* score, const int32_t* answer, int P, int G, double* weight, int32_t* winner,
                      double* winner_weight) {
    for (int p = 0; p < P; ++p) {
        const float* s = score + (int64_t)p * G;
        const int32_t* a = answer + (int64_t)p * G;
        int rank[1024];
        for (int i = 0; i < G; ++i) {
            int r = 0;
            for (int j = 0; j < G; ++j)
                if (s[j] < s[i] || (s[j] == s[i] && j < i)) r += 1;
            rank[i] = r;
            weight[(int64_t)p * G + i] = G > 1 ? (double)r / (double)(G - 1) : 1.0;
        }
        int best = -1;
        long best_total = -1;
        for (int i = 0; i < G; ++i) {
            if (a[i] < 0) continue;
            int first = 1;
            for (int j = 0; j < i; ++j) if (a[j] == a[i]) first = 0;
            if (!first) continue;
            long total = 0;
            for (int j = 0; j < G; ++j) if (a[j] == a[i]) total += (G > 1 ? rank[j] : 1);
            if (total > best_total) { best_total = total; best = i; }
        }
        winner[p] = best >= 0 ? a[best] : -1;
        winner_weight[p] = best >= 0 ? (G > 1 ? (double)best_total / (double)(G - 1) : (double)best_total) : 0.0;
    }
}
