"""Plausible mistakes planted in copies of the Python partition rules must each
trip one of the checks that hold those rules to the paper's counts."""
import sys
import types

import pytest

import test_partition_ref as checks
from oracle import partition_ref as pr

SOURCE = pr.__file__

MUTANTS = {
    "head_block_is_one_row": ("return (d.rows // d.n_heads) * d.cols", "return d.cols"),
    "head_block_forgets_columns": ("return (d.rows // d.n_heads) * d.cols", "return d.rows // d.n_heads"),
    "heads_times_columns": ("return (d.rows // d.n_heads) * d.cols", "return d.n_heads * d.cols"),
    "token_block_is_a_column": ("if d.kind in (ROWS, TOKENS):             # one block per output neuron / token\n        return d.cols",
                                "if d.kind in (ROWS, TOKENS):             # one block per output neuron / token\n        return d.rows"),
    "rows_treated_as_whole": ("if d.kind == WHOLE:", "if d.kind in (WHOLE, ROWS):"),
    "offsets_not_accumulated": ("        v_offset += nb\n", "        v_offset = nb\n"),
    "offset_counts_elements": ("        v_offset += nb\n", "        v_offset += numel\n"),
    "block_count_off_by_one": ("nb = numel // L", "nb = numel // L + 1"),
    "indivisible_heads_accepted": ("if d.n_heads <= 0 or d.rows % d.n_heads:", "if d.n_heads <= 0:"),
    "indivisible_fixed_accepted": ("if d.fixed_block_len <= 0 or numel % d.fixed_block_len:", "if d.fixed_block_len <= 0:"),
    "query_before_embed": ('    if "embed" in name or "output" in name:\n        return TOKENS\n    if "query" in name or "key" in name:\n        return HEADS\n',
                           '    if "query" in name or "key" in name:\n        return HEADS\n    if "embed" in name or "output" in name:\n        return TOKENS\n'),
    "value_by_head": ('if "query" in name or "key" in name:', 'if "query" in name or "key" in name or "value" in name:'),
    "mlp_whole": ('if "value" in name or "attn.proj" in name or "mlp" in name:', 'if "value" in name or "attn.proj" in name:'),
    "output_not_by_token": ('if "embed" in name or "output" in name:', 'if "embed" in name:'),
}

CHECKS = [
    lambda: checks.test_parameter_counts_match_table1("Llama-2-7B", checks.W.llama2_7b),
    lambda: checks.test_parameter_counts_match_table1("Llama-3-8B", checks.W.llama3_8b),
    checks.test_block_counts_follow_algorithm3,
    checks.test_workload_kinds_agree_with_name_rule,
    checks.test_totals_of_the_five_workloads,
    checks.test_rejects_indivisible_shapes,
    checks.test_name_rule_precedence,
]


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_partition_mutant_is_caught(monkeypatch, name):
    old, new = MUTANTS[name]
    src = open(SOURCE).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique"
    mutant = types.ModuleType("partition_mutant")
    monkeypatch.setitem(sys.modules, "partition_mutant", mutant)      # dataclasses look their module up
    exec(compile(src.replace(old, new), "partition_mutant.py", "exec"), mutant.__dict__)
    for attr in ("block_len_of", "build_table", "kind_from_name"):
        monkeypatch.setattr(pr, attr, getattr(mutant, attr))
    caught = []
    for check in CHECKS:
        try:
            check()
        except (AssertionError, ValueError, ZeroDivisionError, pytest.fail.Exception):
            caught.append(check)
    assert caught, f"no check noticed the mutant '{name}'"
