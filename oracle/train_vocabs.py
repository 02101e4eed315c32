"""Writes the stored vocabularies under workloads/vocabs/ (test/bench inputs).

Each benchmark configuration names a merge count and a corpus size; this script draws the seeded
corpus from the workload generator, runs the oracle's BPE trainer on it with the configuration's
pattern, and stores the merge list (pairs int32[n,2]; result id = 256 + rank; identity byte map).
It calls only the oracle and the input generator.  Usage:  python -m oracle.train_vocabs [C1 C2 ...]
"""
import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import oracle            # noqa: E402
import workloads as wl   # noqa: E402


def main(names):
    done = set()
    for name in names:
        cfg = wl.CONFIGS[name]
        if cfg.vocab_file in done:
            continue
        done.add(cfg.vocab_file)
        t0 = time.time()
        corpus = wl.corpus(cfg)
        pairs, n_distinct = oracle.train(corpus, cfg.pattern_id, cfg.n_merges)
        if pairs.shape[0] != cfg.n_merges:
            raise SystemExit(f"{name}: corpus yields only {pairs.shape[0]} of {cfg.n_merges} merges "
                             f"({n_distinct} distinct pieces); raise the corpus diversity")
        os.makedirs(os.path.dirname(cfg.vocab_file), exist_ok=True)
        np.savez_compressed(cfg.vocab_file, pairs=pairs.astype(np.int32),
                            meta=np.array([cfg.pattern_id, cfg.n_merges, cfg.corpus_chars, wl.corpus_seed(cfg)], dtype=np.int64))
        print(f"{name}: {cfg.n_merges} merges from {corpus.size} corpus bytes, {n_distinct} distinct pieces, "
              f"{time.time() - t0:.1f}s -> {cfg.vocab_file} ({os.path.getsize(cfg.vocab_file)} bytes)", flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["C1", "C2", "C3", "C4"])
