"""Are the oracle's pins sharp?  Each case plants ONE plausible mistake in a copy of the
oracle's source (on the CPU; the real oracle is untouched), builds it, and runs the pin tests
against the broken copy in a subprocess: they must fail.  A mistake that survives would mean a
part of the oracle is not pinned."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "gsd_oracle.c")

# (name, text to replace, replacement, pin files that must catch it)
MUTATIONS = [
    ("gqa_mapping", "const int c = h / G;", "const int c = h % Hkv;", "test_oracle_attn.py"),
    ("mask_bit_order", "(mrow[j / 32] >> (j % 32))", "(mrow[j / 32] >> (31 - j % 32))", "test_oracle_attn.py"),
    ("mask_word_order", "(mrow[j / 32] >> (j % 32))", "(mrow[W - 1 - j / 32] >> (j % 32))", "test_oracle_attn.py"),
    ("softmax_scale", "1.0 / sqrt((double)D)", "1.0 / (double)D", "test_oracle_attn.py"),
    ("prefix_length_off_by_one", "const int L = seq_lens[b];", "const int L = seq_lens[b] + (seq_lens[b] < Lmax);",
     "test_oracle_attn.py"),
    ("no_max_subtraction", "s[i] = exp(s[i] - smax);", "s[i] = exp(s[i]);", "test_oracle_attn.py"),
    ("draft_value_index", "const uint16_t *vrow = draft_v + (((size_t)b * N + j)",
     "const uint16_t *vrow = draft_v + (((size_t)b * N + (N - 1 - j))", "test_oracle_attn.py"),
    ("tie_read_forwards", "for (int i = len - 1; i >= 0; --i) {", "for (int i = 0; i < len; ++i) {",
     "test_oracle_accept.py"),
    ("longest_ge", "edges > w->best_edges ||", "edges >= w->best_edges ||", "test_oracle_accept.py"),
    ("argmax_last_of_ties", "row[i] > row[best]) best = i;", "row[i] >= row[best]) best = i;", "test_oracle_accept.py"),
    ("bonus_token_node", "= amax[best[m]];", "= amax[best[m > 0 ? m - 1 : 0]];", "test_oracle_accept.py"),
    ("edge_rule", "w->tok[w->stack[i]] != w->amax[w->stack[i - 1]]", "w->tok[w->stack[i]] != w->amax[w->stack[i]]",
     "test_oracle_accept.py"),
    ("commit_position", "k_cache + ((size_t)b * Lmax + pos) * row, draft_k",
     "k_cache + ((size_t)b * Lmax + pos + 1 - (pos + 1 >= Lmax)) * row, draft_k", "test_oracle_commit.py"),
    ("sampled_le", "(double)draft_q[(size_t)b * N + v] < prob);", "(double)draft_q[(size_t)b * N + v] <= prob);",
     "test_oracle_accept_sampled.py"),
    ("sampled_without_q", "(double)u_accept[(size_t)b * N + v] * (double)draft_q[(size_t)b * N + v] < prob",
     "(double)u_accept[(size_t)b * N + v] < prob", "test_oracle_accept_sampled.py"),
    ("sampled_child_logits", "exp((double)lg[(size_t)p * V + tok[v]] - mx[p]) / sm[p]",
     "exp((double)lg[(size_t)v * V + tok[v]] - mx[v]) / sm[v]", "test_oracle_accept_sampled.py"),
    ("sampled_cdf_ge", "if (cum > target) { pick = j; break; }", "if (cum >= target) { pick = j; break; }",
     "test_oracle_accept_sampled.py"),
    ("sampled_regenerates_at_parent", "const int end = best[m];", "const int end = best[m > 0 ? m - 1 : 0];",
     "test_oracle_accept_sampled.py"),
    ("sampled_regenerates_from_target", "if (mass > 1e-6) memcpy(wgt, res, sizeof(double) * (size_t)V);", "(void)mass;",
     "test_oracle_accept_sampled.py"),
    ("sampled_residual_sign", "const double r = wgt[j] - exp((double)y[j] - mq) / sq;",
     "const double r = exp((double)y[j] - mq) / sq - wgt[j];", "test_oracle_accept_sampled.py"),
    ("sampled_residual_at_a_leaf", "if (draft_logits && rejected_children > 0) {", "if (draft_logits) {",
     "test_oracle_accept_sampled.py"),
    ("sampled_residual_of_the_root", "const float *y = draft_logits + ((size_t)b * N + end) * V;",
     "const float *y = draft_logits + ((size_t)b * N) * V;", "test_oracle_accept_sampled.py"),
    ("sampled_residual_unclamped", "res[j] = r > 0.0 ? r : 0.0;", "res[j] = r > 0.0 ? r : -r;",
     "test_oracle_accept_sampled.py"),
    ("draft_tie_highest", "if (!taken[j] && (best < 0 || P[j] > P[best])) best = j;",
     "if (!taken[j] && (best < 0 || P[j] >= P[best])) best = j;", "test_oracle_draft.py"),
    ("draft_prob_le", "lf[c] = (P[best] < theta_prob) ||", "lf[c] = (P[best] <= theta_prob) ||", "test_oracle_draft.py"),
    ("draft_sibling_vs_previous", "if (i == 0) qmax = P[best];", "qmax = (i == 0) ? P[best] : P[best] * 2.0;",
     "test_oracle_draft.py"),
    ("draft_gram_ignores_ancestors", "if (tok[a] != tok[b]) return 0;\n        a = par[a];",
     "if (tok[a] != tok[b]) return 0;\n        if (i == 0) return 1;\n        a = par[a];", "test_oracle_draft.py"),
    ("draft_last_occurrence", "for (int e = 0; e < c; ++e)\n                if (same_gram(tok, par, c, e, tau))",
     "for (int e = c - 1; e >= 0; --e)\n                if (same_gram(tok, par, c, e, tau))", "test_oracle_draft.py"),
    ("draft_short_paths_count", "if (a < 0 || b < 0) return 0;          /* a path shorter than tau */",
     "if (a < 0 || b < 0) return a < 0 && b < 0;", "test_oracle_draft.py"),
    ("unmerge_children_descending", "for (int v = 0; v < N; ++v) {          /* children of the copied node, ascending id */",
     "for (int v = N - 1; v >= 0; --v) {", "test_oracle_unmerge.py"),
    ("unmerge_parent_is_the_source", "tp[count] = u;", "tp[count] = ts[u];", "test_oracle_unmerge.py"),
    ("unmerge_depth_off_by_one", "if (depth[u] >= max_depth) continue;", "if (depth[u] > max_depth) continue;",
     "test_oracle_unmerge.py"),
    ("unmerge_token_of_the_parent", "tt[count] = tok[v]; tp[count] = u;", "tt[count] = tok[ts[u]]; tp[count] = u;",
     "test_oracle_unmerge.py"),
    ("mask_without_self", "row[v / 32] |= 1u << (v % 32);", "if (v != n) row[v / 32] |= 1u << (v % 32);",
     "test_oracle_mask.py"),
    ("mask_parents_only", "seen[p] = 1;\n                    todo[top++] = p;", "seen[p] = 1;\n                    if (v == n) todo[top++] = p;",
     "test_oracle_mask.py"),
]


@pytest.mark.parametrize("name,old,new,pins", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(tmp_path, name, old, new, pins):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation {name} no longer applies"
    src = tmp_path / "gsd_oracle_mutated.c"
    src.write_text(text.replace(old, new))
    env = dict(os.environ, GSD_ORACLE_SRC=str(src), GSD_ORACLE_LIB=str(tmp_path / "mutated.so"))
    # the quick pins only (the config-sized cross-checks are not needed to notice these)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", pins), "-k", "not configs and not matrix_closure"]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, cwd=ROOT, timeout=300)
    assert r.returncode != 0, f"the pins did not notice the planted mistake '{name}'"
    assert "failed" in r.stdout or "error" in r.stdout.lower()
