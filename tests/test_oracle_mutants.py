"""Planted mistakes in the oracle must be caught by its pins (CPU only).

Each case edits one spot of oracle/ones_oracle.c (a swapped coefficient, a dropped term, a wrong
index, a flipped comparison, ...), builds that variant in a temporary directory and runs the named pin
tests against it: at least one of them has to fail.  This shows that the pins constrain the oracle
rather than restate it.
"""
import os
import subprocess

import pytest

import oracle

import test_oracle_model as M
import test_oracle_rng as R
import test_oracle_search as S
import test_oracle_truncation as T
import test_oracle_per_gpu as P
import test_oracle_refresh as RF

SRC = os.path.join(os.path.dirname(oracle.__file__), "ones_oracle.c")

# (name, text to replace, replacement, pins that must notice)
CASES = [
    ("philox multipliers swapped", "MUL_A = 0xD2511F53u, MUL_B = 0xCD9E8D57u", "MUL_A = 0xCD9E8D57u, MUL_B = 0xD2511F53u",
     [R.test_philox_matches_independent_implementation]),
    ("philox nine rounds", "round < 10; ++round", "round < 9; ++round", [R.test_philox_matches_independent_implementation]),
    ("philox key not bumped", "k1 += WEYL_B;", "k1 += WEYL_A;", [R.test_philox_matches_independent_implementation]),
    ("wrong output word", "return out[col & 3u];", "return out[(col + 1u) & 3u];", [R.test_word_layout]),
    ("row and column swapped in the counter", "uint32_t ctr[4] = {col >> 2, row,", "uint32_t ctr[4] = {row, col >> 2,",
     [R.test_word_layout]),
    ("c and d swapped in the model", "(job->a + job->c * local) + job->d * lg", "(job->a + job->d * local) + job->c * lg",
     [M.test_model_hand_values]),
    ("fixed cost dropped", "(job->a + job->c * local) + job->d * lg", "(job->c * local) + job->d * lg", [M.test_model_hand_values]),
    ("global instead of local batch", "double local = (double)b / (double)gpus;", "double local = (double)b;",
     [M.test_model_hand_values]),
    ("floor instead of ceiling", "int64_t gpus = (b + m - 1) / m;", "int64_t gpus = b / m > 0 ? b / m : 1;",
     [M.test_gpu_count_is_ceiling]),
    ("throughput inverted", "*X = (double)b / t;", "*X = t / (double)b;", [M.test_model_hand_values]),
    ("natural log", "double lg = log2((double)gpus);", "double lg = log((double)gpus);", [M.test_model_hand_values]),
    ("limit ignored", "if (k < 0 || k > job->kmax) return ORACLE_OK;", "if (k < 0) return ORACLE_OK;", [M.test_model_waiting_state]),
    ("penalty dropped", "*F = part[0] - penalty * (double)over;", "*F = part[0];", [M.test_fitness_hand_values]),
    ("penalty sign", "*F = part[0] - penalty * (double)over;", "*F = part[0] + penalty * (double)over;",
     [M.test_penalty_is_per_gpu_over_capacity]),
    ("penalty on demand, not on excess", "int32_t over = demand32 > capacity ? demand32 - capacity : 0;",
     "int32_t over = demand32;", [M.test_fitness_hand_values]),
    ("last job skipped in the sum", "for (int32_t j = 0; j < n_jobs; ++j) {\n        double term;",
     "for (int32_t j = 0; j + 1 < n_jobs; ++j) {\n        double term;", [M.test_fitness_hand_values]),
    ("other summation order", "part[(j >> 2) & 31] += term;", "part[j & 31] += term;",
     [M.test_summation_order_is_the_documented_one]),
    ("sruf term not negated", "-((job->weight * (double)*g) / X)", "((job->weight * (double)*g) / X)", [M.test_sruf_term]),
    ("ties to the higher index", "(F[x] == F[y] && x < y)", "(F[x] == F[y] && x > y)", [S.test_ties_go_to_the_lower_index]),
    ("tournament keeps the worst", "if (win < 0 || better(F, idx, win)) win = idx;", "if (win < 0 || better(F, win, idx)) win = idx;",
     [S.test_tournament_size_one_is_uniform_and_large_picks_best]),
    ("tournament ignores all but the first draw", "for (int32_t t = 0; t < tournament; ++t) {\n        uint32_t w = oracle_word(seed, gen_abs, q, (uint32_t)t, stream);",
     "for (int32_t t = 0; t < 1; ++t) {\n        uint32_t w = oracle_word(seed, gen_abs, q, (uint32_t)t, stream);",
     [S.test_tournament_size_one_is_uniform_and_large_picks_best]),
    ("threshold rounds down", "long t = lround(p_mut * 65536.0);", "long t = (long)(p_mut * 65536.0);", [S.test_thr16]),
    ("lower limit dropped from the draw", "return kmin + (int32_t)(((uint64_t)frac * range) >> 32);",
     "return (int32_t)(((uint64_t)frac * range) >> 32);", [S.test_lower_limits_are_respected]),
    ("draw can exceed the upper limit", "uint64_t range = (uint64_t)(kmax - kmin + 1);", "uint64_t range = (uint64_t)(kmax - kmin + 2);",
     [S.test_genes_stay_in_range_and_pinned_never_move]),
    ("children not complementary", "int32_t child1 = flip ? A[j] : B[j];", "int32_t child1 = flip ? B[j] : A[j];",
     [S.test_crossover_children_are_complementary_without_mutation]),
    ("crossover coin is biased", "int flip = (int)(W & 1u); /* which child inherits the first parent's gene */\n                int32_t child0",
     "int flip = (int)((W & 3u) == 3u);\n                int32_t child0", [S.test_crossover_children_are_complementary_without_mutation]),
    ("both children use the same field", "if ((W >> 16) < thr) child1 = draw_gene(odd_fraction(W)", "if ((W & 0xFFFFu) < thr) child1 = draw_gene(odd_fraction(W)",
     [S.test_sibling_children_mutate_independently]),
    ("value drawn from the child's own field", "static uint32_t even_fraction(uint32_t W) { return W * 0x9E360001u; }",
     "static uint32_t even_fraction(uint32_t W) { return W << 16; }", [S.test_mutation_rate_and_value_distribution]),
    ("elites in reverse order", "memcpy(&c->next[(size_t)r * J], &c->pop[(size_t)c->elites[r] * J]", "memcpy(&c->next[(size_t)(E - 1 - r) * J], &c->pop[(size_t)c->elites[r] * J]",
     [S.test_elitism_keeps_best_monotone_and_elites_verbatim]),
    ("generation counter not advanced", "c->gen_abs = gen + 1;\n        score_population(c);", "score_population(c);",
     [S.test_determinism_and_split_runs]),
    ("repair shrinks the smallest holder", "if (g_now > g_less && g_now > pick_g) { pick = j; pick_g = g_now; }",
     "if (g_now > g_less && (pick < 0 || g_now < pick_g)) { pick = j; pick_g = g_now; }", [S.test_repair]),
    ("repair parks the newest job", "if (g > 0) { park = j; break; }", "if (g > 0) { park = j; }", [S.test_repair]),
    ("remap without clamping", "if (k > jobs[j].kmax) k = jobs[j].kmax;", "", [S.test_update_jobs_remaps_columns]),
    ("new jobs start at their upper limit", "int32_t k = jobs[j].kmin;\n            if (remap[j] >= 0) {", "int32_t k = jobs[j].kmax;\n            if (remap[j] >= 0) {",
     [S.test_update_jobs_remaps_columns]),
    ("truncation keeps the worst", "for (int32_t r = 0; r < k; ++r) keep[order[r]] = 1;", "for (int32_t r = 0; r < k; ++r) keep[order[n - 1 - r]] = 1;",
     [T.test_keep_best_against_sorted]),
    ("per-GPU: the smallest batch that fits instead of the largest", "if (g <= count[j]) kbest = k;", "if (g <= count[j] && kbest < 0) kbest = k;",
     [P.test_fitness_counts_gpus_and_picks_the_largest_batch_that_fits]),
    ("per-GPU: a job may use more GPUs than it holds", "if (g <= count[j]) kbest = k;", "if (g <= count[j] + 1) kbest = k;",
     [P.test_fitness_counts_gpus_and_picks_the_largest_batch_that_fits]),
    ("per-GPU: lower limit ignored", "for (int32_t k = jobs[j].kmin; k <= jobs[j].kmax; ++k) {\n            double X; int32_t g;\n            oracle_model(&jobs[j], k, &X, &g);\n            if (g <= count[j]) kbest = k;",
     "for (int32_t k = 0; k <= jobs[j].kmax; ++k) {\n            double X; int32_t g;\n            oracle_model(&jobs[j], k, &X, &g);\n            if (g <= count[j]) kbest = k;",
     [P.test_fitness_counts_gpus_and_picks_the_largest_batch_that_fits]),
    ("reorder: idle GPUs first", "    int32_t at = 0;\n    for (int32_t i = 0; i < n_gpus; ++i) { /* jobs in the order of their first occurrence */",
     "    int32_t at = 0;\n    for (int32_t i = 0; i < n_gpus; ++i) if (slots[i] < 0 || slots[i] >= n_jobs) out[at++] = -1;\n    for (int32_t i = 0; i < n_gpus; ++i) { /* jobs in the order of their first occurrence */",
     [P.test_reorder_examples]),
    ("reorder: jobs by id, not by first occurrence", "for (int32_t i = 0; i < n_gpus; ++i) { /* jobs in the order of their first occurrence */\n        int32_t j = slots[i];",
     "for (int32_t i = 0; i < n_gpus; ++i) { /* jobs in the order of their first occurrence */\n        int32_t j = i < n_jobs ? i : -1;",
     [P.test_reorder_examples]),
    ("per-GPU search skips the reorder", "for (int32_t i = 0; i < N; ++i) oracle_reorder(&c->next[(size_t)i * J], J, c->J);", "(void)0;",
     [P.test_search_on_the_per_gpu_genome]),
    ("refresh: surplus GPUs freed from the front", "for (int32_t i = n_gpus - 1; i >= 0; --i) {\n        int32_t j = slots[i];\n        if (j >= 0 && count[j] > limit[j])",
     "for (int32_t i = 0; i < n_gpus; ++i) {\n        int32_t j = slots[i];\n        if (j >= 0 && count[j] > limit[j])",
     [RF.test_scale_down_frees_the_last_gpus_beyond_the_limit]),
    ("refresh: no scale-down", "if (j >= 0 && count[j] > limit[j]) { slots[i] = -1; count[j] -= 1; }", "(void)j;",
     [RF.test_scale_down_frees_the_last_gpus_beyond_the_limit]),
    ("refresh: GPUs taken from the newest job", "for (int32_t q = 0; q < n_jobs && v < 0; ++q) if (!is_new[q] && count[q] > 0) v = q;",
     "for (int32_t q = n_jobs - 1; q >= 0 && v < 0; --q) if (!is_new[q] && count[q] > 0) v = q;",
     [RF.test_new_job_takes_the_last_gpu_of_the_longest_present_job_when_nothing_is_idle]),
    ("refresh: the victim's first GPU instead of its last", "for (int32_t i = n_gpus - 1; i >= 0 && at < 0; --i) if (slots[i] == v) at = i;",
     "for (int32_t i = 0; i < n_gpus && at < 0; ++i) if (slots[i] == v) at = i;",
     [RF.test_new_job_takes_the_last_gpu_of_the_longest_present_job_when_nothing_is_idle]),
    ("refresh: one GPU per new job whatever its smallest batch needs", "oracle_model(&jobs[j], jobs[j].kmin, &X, &want);",
     "oracle_model(&jobs[j], jobs[j].kmin, &X, &want); want = 1;",
     [RF.test_new_job_takes_the_last_gpu_of_the_longest_present_job_when_nothing_is_idle]),
    ("refresh: the smallest gain goes first", "if (pick < 0 || gain > best) { pick = j; best = gain; }",
     "if (pick < 0 || gain < best) { pick = j; best = gain; }", [RF.test_fig5_like_example_finished_job_new_job_and_refill]),
    ("refresh: ties to the higher index", "if (pick < 0 || gain > best) { pick = j; best = gain; }",
     "if (pick < 0 || gain >= best) { pick = j; best = gain; }", [RF.test_fig5_like_example_finished_job_new_job_and_refill]),
    ("refresh: the gain ignores what the job runs at now", "double gain = top - now;", "double gain = top;",
     [RF.test_refresh_against_the_python_restatement_and_invariants]),
    ("refresh: new jobs wait behind the refill", "if (!is_new[j]) continue;", "if (1) continue;",
     [RF.test_fig5_like_example_finished_job_new_job_and_refill]),
    ("a job-set change skips the refresh", "oracle_refresh(jobs, n_jobs, c->prm.flags, inv, c->J, is_new, row, c->W);", "(void)0;",
     [RF.test_search_refreshes_every_candidate_at_a_job_set_change]),
    ("mutants take the parents' stream", "(uint32_t)m, (uint32_t)j, ORACLE_STREAM_MUTANT);", "(uint32_t)m, (uint32_t)j, ORACLE_STREAM_MUT);",
     [T.test_generation_is_best_k_of_originals_children_and_mutants]),
]


@pytest.mark.parametrize("name,old,new,pins", CASES, ids=[c[0] for c in CASES])
def test_planted_mistake_is_caught(tmp_path, name, old, new, pins):
    text = open(SRC).read()
    assert text.count(old) == 1, f"the spot to edit must be unique: {old!r}"
    src = tmp_path / "ones_oracle.c"
    src.write_text(text.replace(old, new))
    (tmp_path / "ones_oracle.h").write_text(open(SRC[:-2] + ".h").read())
    so = tmp_path / "liboracle_mutant.so"
    subprocess.run(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-w", "-o", str(so), str(src), "-lm"],
                   check=True, capture_output=True)
    caught = False
    with oracle.use_library(str(so)):
        for pin in pins:
            try:
                pin()
            except pytest.skip.Exception:
                pytest.skip("pin not runnable here")
            except Exception:
                caught = True
    assert caught, f"no pin noticed: {name}"


def test_the_unedited_oracle_passes_those_pins():
    for pin in {p for c in CASES for p in c[3] if getattr(p, "__name__", "") != "<lambda>"}:
        pin()
