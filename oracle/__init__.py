"""CPU oracle of the tree-verify step.  Test infrastructure: never imported by the product package."""
