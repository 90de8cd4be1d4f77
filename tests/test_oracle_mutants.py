"""A sample of the mutation check (tests/oracle_mutants.py runs all of it): the pins must fail for an oracle with a
planted mistake.  Three mutants keep the CPU suite short."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def test_pins_kill_a_sample_of_planted_mistakes():
    import oracle_mutants as om
    names = [m[0] for m in om.MUTANTS]
    sample = [names.index("race: tie goes to the device"), names.index("buffer test: > becomes >="),
              names.index("cost: exchange rate dropped")]
    assert om.run(sample, verbose=False) == []
