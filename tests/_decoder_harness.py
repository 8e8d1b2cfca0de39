"""The random-initialised decoder used by the generation-loop tests lives in the package
(paper_2605_12825_b200/decoder_harness.py), where the benchmark can reach it too."""
from paper_2605_12825_b200.decoder_harness import Decoder  # noqa: F401
