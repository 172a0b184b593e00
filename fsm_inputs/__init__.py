"""Seeded synthetic inputs (automata, vocabularies, logits) shared by the CPU
oracle's tests and the CUDA library's tests and benchmark.  Nothing in this
package computes any part of the vocabulary index or of the masked decode step."""
from .configs import (BASE_SEED, JSON_OBJECT_REGEX, Workload, f32_to_bf16_bits, make_config,
                      start_states, step_logits_numpy)
from .dfa import paper_float_example_dfa, paper_name_dfa, random_class_dfa, signed_decimal_dfa
from .regex_dfa import DFA, compile_regex, dfa_run
from .vocab import bpe_like_vocab, numeric_mix_vocab, token_bytes, vocab_from_strings
