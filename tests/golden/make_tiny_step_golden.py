"""Writes tests/golden/tiny_step.txt: the oracle's outputs for the `tiny` configuration.

Calls only oracle/ and the seeded input generators.  The file is a regression anchor for the oracle
itself (a later change of its arithmetic must be deliberate); it comes from no other implementation.
Run from the repository root:  python tests/golden/make_tiny_step_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import specs_oracle as O                       # noqa: E402
from paper_2506_15733_b200 import inputs as I              # noqa: E402


def main():
    x = I.make_step_inputs(I.CONFIGS["tiny"])
    r = O.beam_step(x.hidden, x.w_vocab, x.token_ids, x.block_offsets, x.cand_offsets, x.draft_tok_logprob,
                    x.reward, 1.0, x.uniforms, 0.7)
    path = os.path.join(ROOT, "tests", "golden", "tiny_step.txt")
    with open(path, "w") as f:
        f.write("# oracle outputs for inputs.CONFIGS['tiny'], beta = 1, tau = 0.7 (Eq. 1, Algorithm 2, Algorithm 1 Step III)\n")
        f.write("# written by tests/golden/make_tiny_step_golden.py; hexadecimal floats are exact\n")
        f.write("tok_logprob " + " ".join(float(v).hex() for v in r["tok_logprob"]) + "\n")
        f.write("blk_logprob " + " ".join(float(v).hex() for v in r["blk_logprob"]) + "\n")
        f.write("weights " + " ".join(float(v).hex() for v in r["weights"]) + "\n")
        f.write("chosen " + " ".join(str(int(v)) for v in r["chosen"]) + "\n")
        f.write("accept " + " ".join(str(int(v)) for v in r["accept"]) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
